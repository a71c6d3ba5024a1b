"""GPU parity tests: the CUDA path, called through the C-ABI, against the CPU oracle on identical seeded inputs.

Tolerances (written here on purpose): integer-valued problems must be bit-exact; otherwise every element must
satisfy |C - C_ref| <= 2*k*u*(|alpha||A||B| + |beta||C|)_ij with u = 2^-53 (fp64) or 2^-24 (fp32); the 4M complex
entry uses 2*(2k+4)*u per component (each component is a 2k-term sum of products of a once-rounded alpha*A).
"""
import itertools

import numpy as np
import pytest
import torch

from gpu_util import declines_transposes, run_and_check, sample_columns, staged_by_tma
from paper_1611_08035_b200 import synth

pytestmark = pytest.mark.gpu
TRANS = list(itertools.product("NT", "NT"))


def nvariants(b2, kind):
    return b2.b2_variant_count(0 if kind == "d" else 1)


# ---- the five benchmark configurations -------------------------------------------------------------

def test_config1_dgemm_256(b2, oracle):
    r = run_and_check(b2, oracle, "d", "N", "N", 256, 256, 256, 1.0, 0.0, dist="uniform", seed=0, c_dist="zero")
    assert r <= 1.0


@pytest.mark.parametrize("kind", ["d", "s"])
@pytest.mark.parametrize("size", [512, 1024])
def test_config2_square_small_full(b2, oracle, kind, size):
    seed = (2000 if kind == "d" else 2100) + int(np.log2(size))
    run_and_check(b2, oracle, kind, "N", "N", size, size, size, 1.5, 0.5, dist="uniform", seed=seed)
    run_and_check(b2, oracle, kind, "N", "N", size, size, size, 1.5, 0.5, dist="int9", seed=seed, expect_exact=True)


@pytest.mark.parametrize("kind", ["d", "s"])
@pytest.mark.parametrize("size", [2048, 4096, 8192])
def test_config2_square_large_sampled(b2, oracle, kind, size):
    """Full benchmark sizes in the launch configuration the benchmark times (automatic variant, aligned
    operands); the oracle evaluates a column sample (first, last, tile boundaries, random)."""
    seed = (2000 if kind == "d" else 2100) + int(np.log2(size))
    cols = sample_columns(size, tile=64, extra=16 if size == 8192 else 24, seed=seed)
    run_and_check(b2, oracle, kind, "N", "N", size, size, size, 1.5, 0.5, dist="uniform", seed=seed, cols=cols)
    if size <= 4096:
        run_and_check(b2, oracle, kind, "N", "N", size, size, size, 1.5, 0.5, dist="int9", seed=seed, cols=cols,
                      expect_exact=True)


def test_config2_integer_8192_fp64_sampled(b2, oracle):
    cols = sample_columns(8192, tile=64, extra=8, seed=1)
    run_and_check(b2, oracle, "d", "N", "N", 8192, 8192, 8192, 1.5, 0.5, dist="int9", seed=2013, cols=cols,
                  expect_exact=True)


@pytest.mark.parametrize("k", [64, 128, 256])
def test_config3_rank_k_update_sampled(b2, oracle, k):
    cols = sample_columns(16384, tile=64, extra=40, seed=k)
    run_and_check(b2, oracle, "d", "N", "N", 16384, 16384, k, -1.0, 1.0, dist="normal", seed=3000 + k, cols=cols)


@pytest.mark.parametrize("k", [64, 128])
def test_rank_k_update_whole_matrix_every_staging(b2, oracle, k):
    """The short-k shape launches 65536 short-lived CTAs, where a slot of the staging ring is recycled right
    after the CTA starts: the place a producer/consumer hand-off error shows.  Integer data make the exact
    result independent of the summation order, so every fp64 tensor-core variant must produce the same bits
    over the WHOLE matrix, launch after launch; the oracle then checks a column sample of that result."""
    m = n = 16384
    A, lda, B, ldb, C, ldc = synth.gemm_inputs("N", "N", m, n, k, "int9", 3100 + k, torch.float64, device="cuda")
    names = [b2.b2_variant_name(0, v) for v in range(nvariants(b2, "d"))]
    first = None
    for v, name in enumerate(names):
        if "dmma" not in name:
            continue
        for rep in range(3 if staged_by_tma(name) else 1):
            Cd = C.clone()
            b2.b2_dgemm("N", "N", m, n, k, -1.0, A, lda, B, ldb, 1.0, Cd, ldc, variant=v)
            assert b2.b2_device_status() == 0
            if first is None:
                first = Cd
            else:
                differing = int((Cd != first).sum())
                assert differing == 0, f"{name}, launch {rep}: {differing} elements differ from {names[0]}"
    cols = sample_columns(n, tile=64, extra=24, seed=k)
    want = C.cpu().numpy()
    oracle.ref_gemm("N", "N", m, n, k, -1.0, A.cpu().numpy(), lda, B.cpu().numpy(), ldb, 1.0, want, ldc, cols=cols)
    got = first.cpu().numpy().reshape(n, ldc)[cols]
    assert got.tobytes() == want.reshape(n, ldc)[cols].tobytes()


@pytest.mark.parametrize("kind", ["d", "s"])
@pytest.mark.parametrize("ta,tb", TRANS)
def test_config4_fringe_and_transposes(b2, oracle, kind, ta, tb):
    seed = 4000 + 2 * (ta == "T") + (tb == "T")
    run_and_check(b2, oracle, kind, ta, tb, 1001, 999, 1003, 0.7, -0.3, dist="uniform", seed=seed, pad=True)
    run_and_check(b2, oracle, kind, ta, tb, 1001, 999, 1003, 1.5, 0.5, dist="int9", seed=seed, pad=True,
                  expect_exact=True)


def test_config5_complex_4m_4096_sampled(b2, oracle):
    cols = sample_columns(4096, tile=64, extra=8, seed=5)
    run_and_check(b2, oracle, "z", "N", "N", 4096, 4096, 4096, 1 + 0.5j, 0j, dist="uniform", seed=5000, cols=cols)


# ---- every variant, every transpose, shapes around every tile edge ---------------------------------

EDGE = [1, 2, 3, 7, 8, 9, 15, 16, 17, 31, 33, 63, 64, 65, 127, 128, 129, 191, 257]


@pytest.mark.parametrize("kind", ["d", "s"])
def test_all_variants_edge_shapes(b2, oracle, kind):
    rng = np.random.default_rng(42)
    for v in range(nvariants(b2, kind)):
        for ta, tb in TRANS:
            for trial in range(10):
                m, n, k = (int(rng.choice(EDGE)) for _ in range(3))
                pad = bool(trial % 2)
                run_and_check(b2, oracle, kind, ta, tb, m, n, k, 0.7, -0.3, seed=trial, pad=pad, variant=v)
                run_and_check(b2, oracle, kind, ta, tb, m, n, k, 1.5, 0.5, dist="int9", seed=trial, pad=pad,
                              variant=v, expect_exact=True)


@pytest.mark.parametrize("kind", ["d", "s"])
def test_all_variants_multi_tile_ragged(b2, oracle, kind):
    """Several tiles in both directions with ragged tails in m, n and k, aligned and padded leading dimensions,
    beta == 0 and beta != 0."""
    for v in range(nvariants(b2, kind)):
        for ta, tb in TRANS:
            run_and_check(b2, oracle, kind, ta, tb, 333, 270, 145, 0.7, -0.3, seed=v, pad=True, variant=v)
            run_and_check(b2, oracle, kind, ta, tb, 300, 260, 136, 1.0, 0.0, seed=v, pad=False, variant=v)
            run_and_check(b2, oracle, kind, ta, tb, 300, 260, 136, 1.5, 0.5, dist="int9", seed=v, variant=v,
                          expect_exact=True)
            # beta == 1 with 16-byte aligned columns of C: interior tiles may be added to C in memory by bulk
            # reductions (fp32 kernels, TMA-staged fp64 kernels), edge tiles take the ordinary epilogue
            run_and_check(b2, oracle, kind, ta, tb, 300, 260, 136, -1.0, 1.0, seed=v + 1, variant=v)
            run_and_check(b2, oracle, kind, ta, tb, 300, 260, 136, -1.0, 1.0, dist="int9", seed=v + 1, variant=v,
                          expect_exact=True)


@pytest.mark.parametrize("kind", ["d", "s"])
def test_tma_variants_aligned_ragged_shapes(b2, oracle, kind):
    """The TMA-staged variants on shapes with ragged m, n and k (edge tiles and the partial last slab are
    zero-filled by the hardware), leading dimensions of A and B that are whole 16-byte units, an odd one for C.
    fp32: the boxes of k-contiguous operands are swizzled, and each transpose pair runs its own inner loop."""
    dt = 0 if kind == "d" else 1
    vec = 2 if kind == "d" else 4
    tma = [v for v in range(nvariants(b2, kind)) if staged_by_tma(b2.b2_variant_name(dt, v))]
    assert len(tma) >= (3 if kind == "d" else 1)
    for v in tma:
        for ta, tb in TRANS:
            if declines_transposes(b2.b2_variant_name(dt, v), ta, tb):
                continue
            for (m, n, k) in [(200, 136, 75), (129, 65, 17), (1, 1, 1), (7, 300, 33), (333, 270, 145), (64, 64, 1030)]:
                (ra, _), (rb, _) = synth.operand_shapes(ta, tb, m, n, k)
                lds = ((ra + vec - 1) // vec * vec + vec, (rb + vec - 1) // vec * vec, m | 1)
                r = run_and_check(b2, oracle, kind, ta, tb, m, n, k, 0.7, -0.3, seed=m + k, variant=v, lds=lds)
                assert r is not None
                r = run_and_check(b2, oracle, kind, ta, tb, m, n, k, 1.5, 0.5, dist="int9", seed=m + k, variant=v,
                                  lds=lds, expect_exact=True)
                assert r is not None
            # beta == 1: interior tiles of the fp64 kernels leave by bulk reductions that add to C in memory, edge
            # tiles and a C with an odd leading dimension by the ordinary epilogue -- both in one launch here
            for (m, n, k) in [(200, 136, 75), (333, 270, 145)]:
                (ra, _), (rb, _) = synth.operand_shapes(ta, tb, m, n, k)
                for ldc in (m + (m & 1) + 2, m | 1):
                    lds = ((ra + vec - 1) // vec * vec + vec, (rb + vec - 1) // vec * vec, ldc)
                    assert run_and_check(b2, oracle, kind, ta, tb, m, n, k, -1.0, 1.0, seed=m + k + 1, variant=v,
                                         lds=lds) is not None
                    assert run_and_check(b2, oracle, kind, ta, tb, m, n, k, -1.0, 1.0, dist="int9", seed=m + k + 1,
                                         variant=v, lds=lds, expect_exact=True) is not None


def test_bounded_wait_reports_timeout(b2):
    """A device-side wait that nothing completes gives up after its bound and reports B2_ERR_TIMEOUT through the
    status word; the context stays usable and the word is cleared by the read."""
    assert b2.b2_device_status() == 0
    assert b2.b2_selftest_wait_timeout() == 0
    assert b2.b2_device_status() == 1001
    assert b2.b2_device_status() == 0
    x = torch.ones(8, device="cuda")
    assert float(x.sum()) == 8.0


@pytest.mark.parametrize("kind", ["d", "s"])
def test_misaligned_base_pointers(b2, oracle, kind):
    """Base pointers shifted by one element (8- or 4-byte aligned only) with otherwise aligned leading dimensions."""
    for ta, tb in TRANS:
        run_and_check(b2, oracle, kind, ta, tb, 200, 136, 75, 0.7, -0.3, seed=3, offset=1)
        run_and_check(b2, oracle, kind, ta, tb, 200, 136, 75, 1.5, 0.5, dist="int9", seed=3, offset=1, expect_exact=True)


def test_skinny_and_degenerate_shapes(b2, oracle):
    for kind in "ds":
        for (m, n, k) in [(1, 1, 1), (1, 1000, 1), (1000, 1, 1), (1, 1, 1000), (5, 3, 0), (0, 7, 9), (7, 0, 9),
                          (2049, 3, 5), (3, 2049, 5), (64, 64, 4097)]:
            for ta, tb in TRANS:
                run_and_check(b2, oracle, kind, ta, tb, m, n, k, 0.7, -0.3, seed=m + n + k, pad=True)


# ---- BLAS conventions ------------------------------------------------------------------------------

@pytest.mark.parametrize("kind", ["d", "s"])
def test_quick_returns_and_nan_poison(b2, oracle, kind):
    tdt = torch.float64 if kind == "d" else torch.float32
    fn = b2.b2_dgemm if kind == "d" else b2.b2_sgemm
    m, n, k = 70, 50, 40
    A, lda, B, ldb, C, ldc = synth.gemm_inputs("N", "N", m, n, k, "uniform", 9, tdt, m + 3, k + 3, m + 3)
    nanA, nanB = torch.full_like(A, float("nan")).cuda(), torch.full_like(B, float("nan")).cuda()
    Cv = C.view(n, ldc)
    # beta == 0: NaN in the old C must not propagate
    Cd = torch.full_like(C, float("nan")).cuda()
    fn("N", "N", m, n, k, 1.0, A.cuda(), lda, B.cuda(), ldb, 0.0, Cd, ldc)
    out = Cd.cpu().view(n, ldc)
    assert torch.isfinite(out[:, :m]).all() and torch.isnan(out[:, m:]).all()
    # alpha == 0: A, B not referenced (NaN-filled); C = beta*C exactly
    Cd = C.cuda()
    fn("N", "N", m, n, k, 0.0, nanA, lda, nanB, ldb, 0.5, Cd, ldc)
    out = Cd.cpu().view(n, ldc)
    assert torch.equal(out[:, :m], 0.5 * Cv[:, :m]) and torch.equal(out[:, m:], Cv[:, m:])
    # alpha == 0 and beta == 0: zeros
    Cd = torch.full_like(C, float("nan")).cuda()
    fn("N", "N", m, n, k, 0.0, nanA, lda, nanB, ldb, 0.0, Cd, ldc)
    assert (Cd.cpu().view(n, ldc)[:, :m] == 0).all()
    # k == 0 with null A and B: C = beta*C
    Cd = C.cuda()
    fn("N", "N", m, n, 0, 1.0, None, max(1, m), None, 1, -1.0, Cd, ldc)
    assert torch.equal(Cd.cpu().view(n, ldc)[:, :m], -Cv[:, :m])
    # alpha == 0, beta == 1 / empty problems: untouched
    Cd = C.cuda()
    fn("N", "N", m, n, k, 0.0, nanA, lda, nanB, ldb, 1.0, Cd, ldc)
    fn("N", "N", 0, n, k, 1.0, None, 1, B.cuda(), ldb, 0.0, Cd, ldc)
    fn("N", "N", m, 0, k, 1.0, A.cuda(), lda, None, ldb, 0.0, Cd, ldc)
    torch.cuda.synchronize()
    assert torch.equal(Cd.cpu().view(torch.uint8), C.view(torch.uint8))
    # NaN in A propagates to its row of C even when B is zero (no shortcuts on zeros)
    A2 = A.clone()
    A2.view(k, lda)[1, 2] = float("nan")
    Cd = torch.zeros_like(C).cuda()
    fn("N", "N", m, n, k, 1.0, A2.cuda(), lda, torch.zeros_like(B).cuda(), ldb, 0.0, Cd, ldc)
    out = Cd.cpu().view(n, ldc)
    assert torch.isnan(out[:, 2]).all() and (out[:, [0, 1, 3]] == 0).all()


def test_lowercase_and_c_transposes(b2, oracle):
    for kind in "ds":
        run_and_check(b2, oracle, kind, "n", "t", 65, 33, 17, 0.7, -0.3, seed=1)
        run_and_check(b2, oracle, kind, "c", "n", 65, 33, 17, 0.7, -0.3, seed=1)
        run_and_check(b2, oracle, kind, "C", "c", 65, 33, 17, 0.7, -0.3, seed=1)


def test_runtime_argument_errors_launch_nothing(b2):
    C = torch.ones(64, dtype=torch.float64, device="cuda")
    A = torch.ones(64, dtype=torch.float64, device="cuda")
    assert b2.b2_dgemm("N", "N", 4, 4, 4, 1.0, None, 4, A, 4, 0.0, C, 4, check=False) == -7
    assert b2.b2_dgemm("N", "N", 4, 4, 4, 1.0, A, 4, None, 4, 0.0, C, 4, check=False) == -9
    assert b2.b2_dgemm("N", "N", 4, 4, 4, 1.0, A, 4, A, 4, 0.0, None, 4, check=False) == -12
    assert b2.b2_dgemm("N", "N", 4, 4, 4, 1.0, A, 3, A, 4, 0.0, C, 4, check=False) == -8
    assert b2.b2_dgemm("N", "N", 4, 4, 4, 1.0, A, 4, A, 4, 0.0, C, 4, variant=99, check=False) == 1004
    torch.cuda.synchronize()
    assert (C == 1).all()


@pytest.mark.parametrize("kind", ["d", "s"])
def test_deterministic_bitwise(b2, kind):
    """Two runs of the same problem give the same bits (no races in the accumulation)."""
    tdt = torch.float64 if kind == "d" else torch.float32
    fn = b2.b2_dgemm if kind == "d" else b2.b2_sgemm
    m, n, k = 777, 513, 1031
    A, lda, B, ldb, C, ldc = synth.gemm_inputs("T", "N", m, n, k, "uniform", 77, tdt)
    outs = []
    for _ in range(2):
        Cd = C.cuda()
        fn("T", "N", m, n, k, 0.7, A.cuda(), lda, B.cuda(), ldb, -0.3, Cd, ldc)
        outs.append(Cd.cpu())
    assert torch.equal(outs[0].view(torch.uint8), outs[1].view(torch.uint8))


def test_sgemm_k_split_over_cluster(b2, oracle):
    """fp32 problems of about a wave of 128 x 64 tiles are launched with the k-loop of every tile split over a
    cluster of two CTAs (the second half reaches the first through distributed shared memory and is added in a
    fixed order): ragged sizes, all transposes, padded and aligned leading dimensions, exact on integer data,
    within the bound otherwise, the same bits on every run."""
    import json
    m, n, k = 1000, 1100, 777
    cfg = json.loads(b2.b2_gemm_query_config(1, "N", "N", m, n, k, m, k, m))
    if cfg["k_split"] < 2:
        pytest.skip("the selector does not split this problem on this device")
    for ta, tb in TRANS:
        run_and_check(b2, oracle, "s", ta, tb, m, n, k, 0.7, -0.3, seed=51, pad=True)
        run_and_check(b2, oracle, "s", ta, tb, m, n, k, 1.5, 0.5, dist="int9", seed=52, expect_exact=True)
    run_and_check(b2, oracle, "s", "N", "N", m, n, 129, 1.0, 0.0, seed=53)   # 9 slabs: too few to split, same entry
    A, lda, B, ldb, C, ldc = synth.gemm_inputs("N", "T", m, n, k, "uniform", 54, torch.float32)
    outs = []
    for _ in range(3):
        Cd = C.cuda()
        b2.b2_sgemm("N", "T", m, n, k, 0.7, A.cuda(), lda, B.cuda(), ldb, -0.3, Cd, ldc)
        outs.append(Cd.cpu())
    assert all(torch.equal(outs[0].view(torch.uint8), o.view(torch.uint8)) for o in outs[1:])


def test_dgemm_k_split_over_cluster(b2, oracle):
    """The fp64 tensor-core kernels with the k-loop of every tile split over a cluster of two or four CTAs
    (requested as variant + 256*s): ragged sizes, all transposes, padded and aligned leading dimensions, a k too
    short to give every CTA a slab; exact on integer data, within the bound otherwise, the same bits on every
    run; variants that cannot split decline without writing."""
    names = [b2.b2_variant_name(0, v) for v in range(nvariants(b2, "d"))]
    for v, name in enumerate(names):
        for split in (2, 4):
            if staged_by_tma(name) or "dfma" in name:
                C = torch.ones(64 * 64, dtype=torch.float64, device="cuda")
                rc = b2.b2_dgemm("N", "N", 64, 64, 64, 1.0, C, 64, C, 64, 0.0, C.clone(), 64, variant=v + 256 * split,
                                 check=False)
                assert rc == 1004, f"{name} accepted a k split"
                continue
            for ta, tb in TRANS:
                run_and_check(b2, oracle, "d", ta, tb, 333, 270, 145, 0.7, -0.3, seed=v, pad=True,
                              variant=v + 256 * split)
                run_and_check(b2, oracle, "d", ta, tb, 300, 260, 136, 1.5, 0.5, dist="int9", seed=v,
                              variant=v + 256 * split, expect_exact=True)
            run_and_check(b2, oracle, "d", "N", "N", 130, 70, 33, 1.0, 0.0, seed=3, variant=v + 256 * split)  # 3 slabs
            run_and_check(b2, oracle, "d", "N", "N", 65, 129, 7, 0.7, -0.3, seed=4, variant=v + 256 * split)   # 1 slab
    assert b2.b2_dgemm("N", "N", 64, 64, 64, 1.0, C, 64, C, 64, 0.0, C.clone(), 64, variant=2 + 256 * 3,
                       check=False) == 1004
    A, lda, B, ldb, C, ldc = synth.gemm_inputs("T", "N", 1001, 999, 1003, "uniform", 55, torch.float64)
    outs = []
    for _ in range(3):
        Cd = C.cuda()
        b2.b2_dgemm("T", "N", 1001, 999, 1003, 0.7, A.cuda(), lda, B.cuda(), ldb, -0.3, Cd, ldc, variant=2 + 512)
        outs.append(Cd.cpu())
    assert all(torch.equal(outs[0].view(torch.uint8), o.view(torch.uint8)) for o in outs[1:])


# ---- complex 4M ------------------------------------------------------------------------------------

def test_zgemm4m_small_full_all_transposes(b2, oracle):
    for ta, tb in TRANS:
        run_and_check(b2, oracle, "z", ta, tb, 301, 203, 157, 1 + 0.5j, 0j, seed=51, pad=True)
        run_and_check(b2, oracle, "z", ta, tb, 130, 70, 33, 0.3 - 0.8j, 0.25 + 0.75j, seed=52, pad=True)
        run_and_check(b2, oracle, "z", ta, tb, 130, 70, 33, 2 - 1j, 0.5 + 0.5j, dist="int9", seed=53,
                      expect_exact=True)
    run_and_check(b2, oracle, "z", "N", "N", 33, 17, 0, 1 + 1j, 0.5 - 0.5j, seed=54)
    run_and_check(b2, oracle, "z", "N", "N", 33, 17, 9, 0j, 0.5 - 0.5j, seed=55)
    run_and_check(b2, oracle, "z", "N", "N", 0, 17, 9, 1 + 0j, 0j, seed=56)


def test_zgemm_conjugate_transposes_and_3m(b2, oracle):
    """Every op pair with a conjugate transpose through 4M, and all nine pairs through 3M: integer data bit-exact
    against direct complex arithmetic, uniform data within 2*(2k+4)*u*S (4M) / 2*(3k+6)*u*S (3M) per component."""
    for ta in "NTC":
        for tb in "NTC":
            for kind in ("z", "z3"):
                if kind == "z" and "C" not in (ta, tb):
                    continue  # covered by test_zgemm4m_small_full_all_transposes
                run_and_check(b2, oracle, kind, ta, tb, 301, 203, 157, 1 + 0.5j, 0j, seed=61, pad=True)
                run_and_check(b2, oracle, kind, ta, tb, 130, 70, 33, 0.3 - 0.8j, 0.25 + 0.75j, seed=62, pad=True)
                run_and_check(b2, oracle, kind, ta, tb, 130, 70, 33, 2 - 1j, 0.5 + 0.5j, dist="int9", seed=63,
                              expect_exact=True)
    run_and_check(b2, oracle, "z3", "N", "N", 33, 17, 0, 1 + 1j, 0.5 - 0.5j, seed=64)
    run_and_check(b2, oracle, "z3", "C", "N", 33, 17, 5, 0j, 0.5 - 0.5j, seed=65)


def test_zgemm3m_4096_sampled(b2, oracle):
    cols = sample_columns(4096, tile=64, extra=8, seed=6)
    run_and_check(b2, oracle, "z3", "N", "N", 4096, 4096, 4096, 1 + 0.5j, 0j, dist="uniform", seed=5000, cols=cols)


def test_zgemm4m_argument_errors(b2):
    z = torch.zeros(64, dtype=torch.complex128, device="cuda")
    ws = torch.empty(1 << 16, dtype=torch.uint8, device="cuda")
    assert b2.b2_zgemm4m("X", "N", 4, 4, 4, 1, z, 4, z, 4, 0, z, 4, ws, check=False) == -1
    assert b2.b2_zgemm4m("N", "H", 4, 4, 4, 1, z, 4, z, 4, 0, z, 4, ws, check=False) == -2
    assert b2.b2_zgemm4m("N", "N", 4, 4, 4, 1, z, 4, z, 4, 0, z, 4, None, check=False) == 1003
    assert b2.b2_zgemm4m("N", "N", 4, 4, 4, 1, z, 4, z, 4, 0, z, 4, ws[:64], check=False) == 1003
    assert b2.b2_zgemm4m("N", "N", 4, 4, 4, 1, z, 4, z, 4, 0, z, 4, ws[8:], check=False) == 1003  # misaligned


# ---- host-buffer entry points ----------------------------------------------------------------------

@pytest.mark.parametrize("kind", ["d", "s"])
def test_host_entry_matches_oracle(b2, oracle, kind):
    tdt = torch.float64 if kind == "d" else torch.float32
    fn = b2.b2_dgemm_host if kind == "d" else b2.b2_sgemm_host
    u = 2.0 ** -53 if kind == "d" else 2.0 ** -24
    for ta, tb in TRANS:
        m, n, k = 301, 203, 157
        (ra, ca), (rb, cb) = synth.operand_shapes(ta, tb, m, n, k)
        A, lda, B, ldb, C, ldc = synth.gemm_inputs(ta, tb, m, n, k, "uniform", 61, tdt, ra + 5, rb + 3, m + 7)
        want = C.numpy().copy()
        oracle.ref_gemm(ta, tb, m, n, k, 0.7, A.numpy(), lda, B.numpy(), ldb, -0.3, want, ldc)
        _, S = oracle.ref_gemm_hi(ta, tb, m, n, k, 0.7, A.numpy(), lda, B.numpy(), ldb, -0.3, C.numpy(), ldc)
        ws = torch.empty(b2.b2_gemm_host_workspace_bytes(0 if kind == "d" else 1, ta, tb, m, n, k), dtype=torch.uint8,
                         device="cuda")
        Ch = C.clone().pin_memory()
        fn(ta, tb, m, n, k, 0.7, A.pin_memory(), lda, B.pin_memory(), ldb, -0.3, Ch, ldc, ws)
        got = Ch.numpy().reshape(n, ldc)
        assert got[:, m:].tobytes() == C.numpy().reshape(n, ldc)[:, m:].tobytes()
        err = np.abs(got[:, :m].astype(np.float64) - want.reshape(n, ldc)[:, :m].astype(np.float64))
        assert np.all(err <= 2 * k * u * S.reshape(n, m))


@pytest.mark.parametrize("kind", ["d", "s"])
def test_host_entry_large_k_chunks(b2, oracle, kind):
    """Large problems go up chunk by chunk along k and are accumulated as the chunks arrive (ragged last chunk and
    last panel, padded leading dimensions, all transposes); the old values of C are added at the end from a buffer
    of their own, and beta == 0 must not read C (NaN there).  Checked on a column sample: exact on integer data,
    within the bound otherwise."""
    tdt = torch.float64 if kind == "d" else torch.float32
    fn = b2.b2_dgemm_host if kind == "d" else b2.b2_sgemm_host
    u = 2.0 ** -53 if kind == "d" else 2.0 ** -24
    m, n, k = 2100, 2050, 2250
    assert b2.b2_gemm_host_workspace_bytes(0 if kind == "d" else 1, "N", "N", m, n, k) >= 4 * m * n * (8 if kind == "d" else 4)
    cols = sample_columns(n, tile=64, extra=6, seed=5)
    for ta, tb in TRANS:
        (ra, ca), (rb, cb) = synth.operand_shapes(ta, tb, m, n, k)
        for dist, alpha, beta in (("uniform", 0.7, -0.3), ("int9", 1.5, 0.5), ("int9", 1.0, 0.0)):
            A, lda, B, ldb, C, ldc = synth.gemm_inputs(ta, tb, m, n, k, dist, 63, tdt, ra + 5, rb + 3, m + 7)
            if beta == 0.0:
                C.fill_(float("nan"))
            want = C.numpy().copy()
            oracle.ref_gemm(ta, tb, m, n, k, alpha, A.numpy(), lda, B.numpy(), ldb, beta, want, ldc, cols=cols)
            ws = torch.empty(b2.b2_gemm_host_workspace_bytes(0 if kind == "d" else 1, ta, tb, m, n, k),
                             dtype=torch.uint8, device="cuda")
            Ch = C.clone().pin_memory()
            fn(ta, tb, m, n, k, alpha, A.pin_memory(), lda, B.pin_memory(), ldb, beta, Ch, ldc, ws)
            assert b2.b2_device_status() == 0
            got = Ch.numpy().reshape(n, ldc)
            assert got[:, m:].tobytes() == C.numpy().reshape(n, ldc)[:, m:].tobytes()  # padding rows untouched
            g, w_ = got[cols][:, :m], want.reshape(n, ldc)[cols][:, :m]
            if dist == "int9":
                assert g.tobytes() == w_.tobytes()
            else:
                _, S = oracle.ref_gemm_hi(ta, tb, m, n, k, alpha, A.numpy(), lda, B.numpy(), ldb, beta, C.numpy(), ldc,
                                          cols=cols)
                err = np.abs(g.astype(np.float64) - w_.astype(np.float64))
                assert np.all(err <= 2 * k * u * S.reshape(n, m)[cols])
            del ws


# ---- selector and probe ----------------------------------------------------------------------------

def test_query_config_reports_launch(b2):
    import json
    cfg = json.loads(b2.b2_gemm_query_config(0, "N", "N", 8192, 8192, 8192, 8192, 8192, 8192))
    assert cfg["micro_kernel"] == "dmma_tma" and cfg["grid"] == cfg["tiles_m"] * cfg["tiles_n"]
    odd = json.loads(b2.b2_gemm_query_config(0, "N", "N", 1001, 999, 1003, 1027, 1027, 1027))
    assert odd["micro_kernel"] == "dmma"
    assert cfg["tiles_m"] == -(-8192 // cfg["BM"]) and cfg["k_slabs"] == 8192 // cfg["kc"]
    cfg = json.loads(b2.b2_gemm_query_config(1, "T", "N", 1001, 999, 1003, 1027, 1027, 1027))
    assert cfg["micro_kernel"] == "ffma2" and cfg["vector_staging_if_pointers_aligned"] is False


def test_pipe_probe_rates(b2):
    from paper_1611_08035_b200 import pipes
    d = pipes.probe("dfma", 256, 1, 4000)
    t = pipes.probe("dmma_m16n8k4", 256, 1, 2000)
    f = pipes.probe("ffma", 256, 1, 4000)
    assert 55 <= d["fma_per_clk_per_sm"] <= 66 and 55 <= t["fma_per_clk_per_sm"] <= 66
    assert 110 <= f["fma_per_clk_per_sm"] <= 132


def test_instruction_mix_probes(b2):
    """The inner loops of the micro-kernels over resident slabs: the tensor-core mix runs at the pipe's rate, the
    packed-pair mixes below theirs (the shared-memory loads take issue slots from the pair instructions) and in
    the order of their loads per multiply-add: 16 x 8 above 8 x 8 above 4 x 4; the barrier costs a few percent."""
    from paper_1611_08035_b200 import pipes
    rate = lambda kind, cps, thr=128, **kw: pipes.probe(kind, thr, cps, 2000, **kw)["tflops"]
    dm = rate("mix_dmma_64x64", 2)
    f8, f8b = rate("mix_ffma2_8x8", 3), rate("mix_ffma2_8x8", 3, barrier=True)
    f16 = rate("mix_ffma2_16x8", 2)
    f4 = rate("mix_ffma2_4x4", 8, thr=64)
    assert 0.93 * 37.2 <= dm <= 1.02 * 37.2
    assert 0.78 * 74.4 <= f8 <= 0.95 * 74.4 and 0.93 * f8 <= f8b <= 1.01 * f8
    assert f4 < f8 < f16 <= 0.99 * 74.4


@pytest.mark.parametrize("kind", ["d", "s"])
def test_more_than_2_31_elements_of_c(b2, oracle, kind):
    """C with more than 2^31 elements (46400^2): column offsets no longer fit 32 bits even in elements.  k is short,
    so the run is cheap; the oracle evaluates a column sample (first, last, tile edges, around the 2^31-th element)
    on the compacted problem, which is the same arithmetic column by column."""
    tdt = torch.float64 if kind == "d" else torch.float32
    m = n = 46400
    k = 24
    assert m * n > 2 ** 31
    A, lda, B, ldb, _, _ = synth.gemm_inputs("N", "N", m, n, k, "int9", 9100, tdt)
    C = torch.full((m * n,), 7.0, dtype=tdt, device="cuda")
    fn = b2.b2_dgemm if kind == "d" else b2.b2_sgemm
    fn("N", "N", m, n, k, 1.5, A.cuda(), lda, B.cuda(), ldb, 0.5, C, m)
    assert b2.b2_device_status() == 0
    edge = (2 ** 31) // m  # the column that holds element number 2^31
    cols = sorted({0, 1, 63, 64, edge - 1, edge, edge + 1, n - 65, n - 64, n - 2, n - 1})
    Bn = B.numpy().reshape(n, ldb)[cols].copy().reshape(-1)
    want = np.full(m * len(cols), 7.0, dtype=A.numpy().dtype)
    oracle.ref_gemm("N", "N", m, len(cols), k, 1.5, A.numpy(), lda, Bn, ldb, 0.5, want, m)
    got = torch.stack([C[c * m:(c + 1) * m] for c in cols]).cpu().numpy().reshape(-1)
    assert got.tobytes() == want.tobytes()
    # nothing else moved: every element is an integer multiple of 0.5 within the range the data allow
    assert float(C.abs().max()) <= 1.5 * 16 * k + 3.5
