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


def _predictions(b2):
    pred = {}
    for dtype in (0, 1):
        for v in range(b2.b2_variant_count(dtype)):
            frac, js = b2.b2_model_predict_variant(dtype, v)
            d = json.loads(js)
            assert 0 < frac <= 1 and abs(d["predicted_fraction"] - frac) < 1e-4
            assert abs(min(d["pipe_fraction"], d["feed_fraction"]) * d["coverage"] * d["stall"] - frac) < 1e-3
            pred[d["variant"]] = (frac, d)
    return pred


def test_sm_predictions(b2):
    """The model re-targeted at an SM sub-partition, factor by factor.  Pipelines: the tensor-core kernels are bound
    by the FP64 tensor pipe, the scalar FFMA kernel and the packed-pair kernels by issue slots: a pair instruction and a
    16-byte shared-memory load hold the dispatch port for two clocks each, so the 8 x 8 block's 64 + 8 slots per
    rank-1 update leave 0.87 of the FP32 pipe at best and the 16 x 8 block's 128 + 12 leave 0.91, which is what the
    instruction-mix probes measure (0.87, 0.92).  Stall
    term: only kernels with a CTA-wide barrier per slab carry it, and more resident CTAs cover more of it.  Coverage
    grows with the independent tensor instructions per scheduler."""
    pred = _predictions(b2)
    for name, (frac, d) in pred.items():
        bound = max(d["clocks_per_k"], key=d["clocks_per_k"].get)
        if name.startswith("dmma"):
            assert bound == "tensor64" and d["pipe_fraction"] == 1.0
        staged_by_tma = "tma" in name or "_ws_" in name
        assert (d["stall"] == 1.0) == staged_by_tma, name
    d = pred["ffma2_128x64x16_s4"][1]
    assert d["jobs_per_k"]["fp32"] == 64.0 and max(d["clocks_per_k"], key=d["clocks_per_k"].get) == "issue"
    assert 64 / (72 + 4) < d["pipe_fraction"] < 64 / 72  # slots of the loop itself, plus a few for staging
    wide = pred["ffma2_t16x8_128x128x16_s3"][1]
    assert 128 / (140 + 5) < wide["pipe_fraction"] < 128 / 140 and wide["pipe_fraction"] > d["pipe_fraction"]
    assert max(pred["ffma_128x64x16_s4"][1]["clocks_per_k"], key=pred["ffma_128x64x16_s4"][1]["clocks_per_k"].get) == "issue"
    # shared-memory share of the DMMA 64x64 kernel: a quarter of the LSU rate, as the profiler counter shows
    d = pred["dmma_64x64x16_s3"][1]
    assert abs(d["clocks_per_k"]["lsu"] / d["clocks_per_k"]["tensor64"] - 0.25) < 1e-9
    # W = L + n*k: one CTA on the SM pays the whole barrier stall, two CTAs half of it
    one, two = pred["dmma_128x128x16_s4"][1], pred["dmma_128x64x16_s3"][1]
    assert abs(one["stall"] - 2048 / (2048 + 250)) < 1e-3 and abs(two["stall"] - 2048 / (2048 + 125)) < 1e-3
    assert pred["dmma_tma_32x32x16_s3"][1]["coverage"] < pred["dmma_tma_64x64x16_s3"][1]["coverage"]
    # Section 5 restated for a thread: N_updates = floor((255 - accumulators - R_A) / R_R) >= 2 for every built kernel,
    # and the register estimate is close to what the compiler uses (120-128 and 200-218 for the two DMMA warp tiles)
    assert all(d["n_updates"] >= 2 for _, d in pred.values())
    assert pred["dmma_64x64x16_s3"][1]["registers"] == 120 and pred["dmma_128x64x16_s3"][1]["registers"] == 200
    assert abs(pred["dmma_tma_64x64x16_s3"][1]["measured_fraction"] - 0.97) < 1e-9


def test_predicted_order_of_built_variants_matches_measured_order(b2):
    """The paper validates its model by the ORDER it predicts for the candidate kernels against the measured order
    (Section 6.1, Xeon Phi: preserved but for one mix).  The same check for the variants built here, per data type:
    no pair whose predicted and measured fractions both differ by more than 0.05 may be ordered the other way round,
    and every variant the selector may choose is predicted within 0.08 of its measured fraction or is on the
    short list of known misses (fp32 tiles measured with a k-contiguous B, whose element-wise transposing copy the
    model does not price)."""
    pred = _predictions(b2)
    known_misses = {"ffma2_64x64x16_s4", "ffma2_t4_32x32x16_s4", "ffma2_t16x8_128x128x16_s3"}
    for prefix in ("d", "f"):
        items = [(n, f, d["measured_fraction"]) for n, (f, d) in pred.items() if n.startswith(prefix)]
        for n1, p1, m1 in items:
            for n2, p2, m2 in items:
                if n1 in known_misses or n2 in known_misses:
                    continue
                if p1 - p2 > 0.05 and m2 - m1 > 0.05:
                    raise AssertionError(f"{n1} predicted above {n2} ({p1:.3f} > {p2:.3f}) but measured below "
                                         f"({m1:.3f} < {m2:.3f})")
        for n, p, m in items:
            comparison_only = n.startswith(("dfma", "ffma_", "dmma_w8", "dmma_ws", "ffma2_tma"))
            if n not in known_misses and not comparison_only:
                assert abs(p - m) <= 0.08, (n, p, m)
    for n in known_misses:
        assert pred[n][0] - pred[n][1]["measured_fraction"] > 0.08  # still a miss: take it off the list when fixed


def test_enumeration_ranks_candidates_under_the_register_and_shared_memory_limits(b2):
    """Section 5.1's work flow: every candidate in the list fits the limits, the list is sorted by prediction, every
    built variant appears with its rank, and the best fp64 candidates are tensor-core kernels fed by the tensor
    memory accelerator -- the family the library's headline kernel belongs to."""
    for dtype in (0, 1):
        e = json.loads(b2.b2_model_enumerate(dtype, 12))
        ranked = e["ranked"]
        assert e["candidates"] > 100 and len(ranked) >= 12
        top = [r for r in ranked if r["rank"] <= 12]
        assert [r["rank"] for r in top] == list(range(1, 13))
        assert all(a["predicted_fraction"] >= b["predicted_fraction"] - 1e-9 for a, b in zip(ranked, ranked[1:]))
        for r in ranked:
            assert r["registers"] <= 255 and r["n_updates"] >= 2 and r["ctas_per_sm"] >= 1
            assert r["smem_bytes"] * r["ctas_per_sm"] <= 233472
            assert r["cta_tile"] == [r["warp_tile"][0] * r["warps"][0], r["warp_tile"][1] * r["warps"][1]]
        built = {r["built_as"] for r in ranked if r["built_as"]}
        names = {b2.b2_variant_name(dtype, v) for v in range(b2.b2_variant_count(dtype))}
        assert built <= names and len(built) >= (5 if dtype == 1 else 8)
        if dtype == 0:
            assert all(r["kind"] == "dmma" and r["tma"] for r in top)
            best_built = min((r for r in ranked if r["built_as"]), key=lambda r: r["rank"])
            assert "tma" in best_built["built_as"]
    with pytest.raises(b2.B2Error):
        b2.b2_model_enumerate(2, 4)
    with pytest.raises(b2.B2Error):
        b2.b2_model_enumerate(0, 0)
