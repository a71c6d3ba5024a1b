"""The paper's analytical model: the oracle restatement (oracle/queue_model.py) is pinned to the values the
paper prints (tests/golden/*.txt), then the library's implementation (C-ABI, host-only) is compared with the
oracle on those tables and on random mixes.  Printed values are matched to half a unit of their last digit."""
import json
import math
import random
from pathlib import Path

import pytest

from oracle import queue_model as qm

GOLDEN = Path(__file__).resolve().parent / "golden"


def rows(name):
    out = []
    for line in (GOLDEN / name).read_text().splitlines():
        line = line.strip()
        if line and not line.startswith("#"):
            out.append(line.split())
    return out


def printed_close(value, printed: str):
    digits = len(printed.split(".")[1]) if "." in printed else 0
    return abs(value - float(printed)) <= 0.5 * 10 ** (-digits) + 1e-12


# ---- the oracle against the paper -----------------------------------------------------------------

def test_oracle_little_law_worked_example():
    r = rows("little_law_example.txt")
    pipes = [x for x in r if x[0] != "result"]
    lam = qm.outer_product_throughput([float(x[1]) for x in pipes], [float(x[2]) for x in pipes])
    assert lam == float([x for x in r if x[0] == "result"][0][1]) == 0.25


def test_oracle_xeon_phi_table():
    for perm, bcast, l_mem, l_p0, lam_p, fpc_p, gf_p in rows("xeon_phi_8x30_mixes.txt"):
        perm, bcast = int(perm), int(bcast)
        assert perm * 4 + bcast == 30  # the mixes tile the 30 columns
        mem, p0 = 1 + perm + bcast + 4, 1 + 5 * perm + bcast
        assert (mem, p0) == (int(l_mem), int(l_p0))
        lam = qm.outer_product_throughput([1.0, 1.0], [mem, p0])
        assert printed_close(lam, lam_p)
        fpc = qm.flop_per_cycle(lam, 8, 30)
        assert printed_close(fpc, fpc_p)
        gf = qm.gflops(1.053, fpc)
        if perm == 4:  # printed 14.41 is a misprint: same lambda as the first row, which prints 14.44
            assert printed_close(gf, "14.44") and not printed_close(gf, gf_p)
        else:
            assert printed_close(gf, gf_p)
    best = max(rows("xeon_phi_8x30_mixes.txt"), key=lambda r: float(r[4]))
    assert (best[0], best[1]) == ("1", "26")  # the mix the paper finds fastest


def test_oracle_sandy_bridge_table():
    for mr, nr, bcast, shuf, l_mem, l_fma, l_shuf, lam_p, fpc_p, gf_p in rows("sandy_bridge_mixes.txt"):
        mr, nr = int(mr), int(nr)
        assert int(l_fma) == mr * nr // 4  # one multiply+add pair per vector of 4
        lam = qm.outer_product_throughput([2.0, 1.0, 1.0], [int(l_mem), int(l_fma), int(l_shuf)])
        assert printed_close(lam, lam_p)
        fpc = qm.flop_per_cycle(lam, mr, nr)
        assert abs(fpc - 8.0) < 1e-12 and fpc_p == "4"  # printed 4 is read as 8 (26.4 / 3.3 = 8)
        assert printed_close(qm.gflops(3.3, fpc), gf_p)


def test_oracle_register_formula_instances():
    for name, r_total, v, mr, nr, r_a, r_r, n_p, ms, ns, holds in rows("register_blocking.txt"):
        r_total, v, mr, nr, r_a, r_r, ms, ns = map(int, (r_total, v, mr, nr, r_a, r_r, ms, ns))
        n = qm.n_updates(r_total, mr, nr, v, r_a, r_r)
        assert n == int(n_p), name
        assert qm.sub_block_fits(ms, ns, n, v) == bool(int(holds)), name


def test_oracle_stall_correction():
    # no dependent instructions: back to 1/L; n dependent instructions of latency k add n*k cycles
    assert qm.stalled_throughput(8, 0, 5) == 1 / 8
    assert qm.stalled_throughput(8, 2, 5) == 1 / 18
    assert qm.stalled_throughput(8, 2, 5) < qm.outer_product_throughput([1.0], [8])


# ---- the library against the oracle and the paper -------------------------------------------------

def test_library_matches_paper_tables(b2):
    assert b2.b2_model_throughput([2, 1, 1, 1], [5, 4, 4, 4]) == 0.25
    for perm, bcast, l_mem, l_p0, lam_p, *_ in rows("xeon_phi_8x30_mixes.txt"):
        assert printed_close(b2.b2_model_throughput([1.0, 1.0], [float(l_mem), float(l_p0)]), lam_p)
    for mr, nr, bcast, shuf, l_mem, l_fma, l_shuf, lam_p, *_ in rows("sandy_bridge_mixes.txt"):
        assert printed_close(b2.b2_model_throughput([2.0, 1.0, 1.0], [float(l_mem), float(l_fma), float(l_shuf)]), lam_p)
    for name, r_total, v, mr, nr, r_a, r_r, n_p, *_ in rows("register_blocking.txt"):
        assert b2.b2_model_register_updates(*map(int, (r_total, mr, nr, v, r_a, r_r))) == int(n_p), name


def test_library_matches_oracle_on_random_mixes(b2):
    rnd = random.Random(5)
    for _ in range(300):
        n = rnd.randint(1, 6)
        rates = [rnd.choice([0.25, 0.5, 1.0, 2.0]) for _ in range(n)]
        jobs = [rnd.choice([0, 1, 3, 8, 30, 2.5]) for _ in range(n)]
        want = qm.outer_product_throughput(rates, jobs)
        got = b2.b2_model_throughput(rates, jobs)
        assert got == want or (math.isinf(got) and math.isinf(want))
        l, nd, k = rnd.randint(1, 40), rnd.randint(0, 5), rnd.choice([1, 4, 5, 8])
        assert b2.b2_model_stalled_throughput(l, nd, k) == qm.stalled_throughput(l, nd, k)
        args = (rnd.choice([16, 32, 255]), rnd.randint(1, 12), rnd.randint(1, 12), rnd.choice([1, 2, 4, 8]),
                rnd.randint(0, 4), rnd.choice([1, 2]))
        assert b2.b2_model_register_updates(*args) == qm.n_updates(*args)


def test_library_rejects_bad_input(b2):
    assert b2.b2_model_throughput([], []) == -1
    assert b2.b2_model_throughput([0.0], [1.0]) == -1
    assert b2.b2_model_throughput([1.0], [-1.0]) == -1
    assert b2.b2_model_stalled_throughput(0, 1, 1) == -1
    with pytest.raises(b2.B2Error):
        b2.b2_model_register_updates(16, 4, 4, 0, 2, 2)
    with pytest.raises(b2.B2Error):
        b2.b2_model_predict_variant(0, 99)


def test_sm_predictions(b2):
    """The model re-targeted at an SM sub-partition: the tensor-core and FP64-FMA kernels are predicted
    pipe-bound (the model, like the paper's Sandy Bridge table, cannot separate them), the scalar FFMA kernel is
    predicted issue-bound below the packed-pair kernel -- the order the measurements show."""
    pred = {}
    for dtype in (0, 1):
        for v in range(b2.b2_variant_count(dtype)):
            frac, js = b2.b2_model_predict_variant(dtype, v)
            d = json.loads(js)
            assert 0 < frac <= 1 and abs(d["predicted_fraction"] - frac) < 1e-4
            pred[d["variant"]] = (frac, d)
    f64 = {k: v for k, v in pred.items() if k.startswith("d")}
    assert all(abs(v[0] - 1.0) < 1e-9 for v in f64.values())
    for name, (frac, d) in f64.items():
        bound = max(d["clocks_per_k"], key=d["clocks_per_k"].get)
        assert bound == ("tensor64" if name.startswith("dmma") else "fp64")
    assert abs(pred["dmma_tma_64x64x16_s3"][1]["measured_fraction"] - 0.97) < 1e-9
    ffma = pred["ffma_128x64x16_s4"]
    ffma2 = pred["ffma2_128x64x16_s4"]
    assert max(ffma[1]["clocks_per_k"], key=ffma[1]["clocks_per_k"].get) == "issue"
    assert ffma[0] < ffma2[0] and ffma[1]["measured_fraction"] < ffma2[1]["measured_fraction"]
    # shared-memory share of the DMMA 64x64 kernel: a quarter of the LSU rate, as the profiler counter shows
    d = pred["dmma_64x64x16_s3"][1]
    assert abs(d["clocks_per_k"]["lsu"] / d["clocks_per_k"]["tensor64"] - 0.25) < 1e-9
