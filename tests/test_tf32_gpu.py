"""The TF32 tensor-core variants of the fp32 GEMM (b2_sgemm_tf32x1 / b2_sgemm_tf32x3) against their oracle.

Tolerances: bit-exact on integer-valued inputs (every TF32 product and fp32 partial sum is exact);
otherwise |C - C_ref| <= 2*(t*k + 2)*2^-24*S against the TF32 oracle of the same variant, t = 1 or 3 products per
k (the roundings of the operands are part of the definition; what differs is the fp32 accumulation of t*k terms
in the tensor core, whose additions may truncate, hence the factor 2, plus the two roundings of the alpha/beta
epilogue), and, against the wide fp32 oracle, the error the variant is reported with: 2^-10 * S for x1,
(2^-21 + 2*(3k+2)*2^-24) * S for the 3-term split."""
import itertools

import numpy as np
import pytest
import torch

from gpu_util import sample_columns
from paper_1611_08035_b200 import synth

pytestmark = pytest.mark.gpu
TRANS = list(itertools.product("NT", "NT"))


def run_tf32(b2, oracle, terms, ta, tb, m, n, k, alpha, beta, dist="uniform", seed=0, pad=False, cols=None,
             expect_exact=False):
    (ra, _), (rb, _) = synth.operand_shapes(ta, tb, m, n, k)
    lds = (synth.padded_ld(ra), synth.padded_ld(rb), synth.padded_ld(m)) if pad else (None, None, None)
    A, lda, B, ldb, C, ldc = synth.gemm_inputs(ta, tb, m, n, k, dist, seed, torch.float32, *lds)
    An, Bn, Cn = A.numpy(), B.numpy(), C.numpy()
    ws = torch.empty(max(256, b2.b2_sgemm_tf32_workspace_bytes(terms, m, n, k)), dtype=torch.uint8, device="cuda")
    Ad, Bd, Cd = A.cuda(), B.cuda(), C.cuda()
    b2.b2_sgemm_tf32(terms, ta, tb, m, n, k, alpha, Ad, lda, Bd, ldb, beta, Cd, ldc, ws)
    assert b2.b2_device_status() == 0
    assert torch.equal(Ad.cpu().view(torch.uint8), A.view(torch.uint8)) and torch.equal(Bd.cpu().view(torch.uint8), B.view(torch.uint8))
    got = Cd.cpu().numpy()
    if m == 0 or n == 0:
        assert got.tobytes() == Cn.tobytes()
        return
    want, S = oracle.ref_sgemm_tf32(terms, ta, tb, m, n, k, alpha, An, lda, Bn, ldb, beta, Cn, ldc, cols=cols)
    hi, _ = oracle.ref_gemm_hi(ta, tb, m, n, k, alpha, An, lda, Bn, ldb, beta, Cn, ldc, cols=cols)
    sel = list(range(n)) if cols is None else list(cols)
    G = got.reshape(n, ldc)
    assert G[:, m:].tobytes() == Cn.reshape(n, ldc)[:, m:].tobytes(), "padding rows of C were written"
    g = G[sel, :m].astype(np.float64)
    w = want.reshape(n, max(1, m))[sel, :m].astype(np.float64)
    h = hi.reshape(n, max(1, m))[sel, :m].astype(np.float64)
    Sv = S.reshape(n, max(1, m))[sel, :m]
    if expect_exact:
        assert np.array_equal(g, w), "integer-valued problem is not bit-exact"
        return
    assert np.all(np.abs(g - w) <= 2 * (terms * k + 2) * 2.0 ** -24 * Sv)
    level = 2.0 ** -10 if terms == 1 else (2.0 ** -21 + 2 * (3 * k + 2) * 2.0 ** -24)
    assert np.all(np.abs(g - h) <= level * Sv)


@pytest.mark.parametrize("terms", [1, 3])
def test_tf32_small_full_all_transposes(b2, oracle, terms):
    for ta, tb in TRANS:
        run_tf32(b2, oracle, terms, ta, tb, 333, 270, 145, 0.7, -0.3, seed=11, pad=True)
        run_tf32(b2, oracle, terms, ta, tb, 300, 520, 136, 1.0, 0.0, seed=12)          # wide-tile path (n > 256)
        run_tf32(b2, oracle, terms, ta, tb, 129, 65, 257, 1.5, 0.5, dist="int9", seed=13, pad=True, expect_exact=True)


@pytest.mark.parametrize("terms", [1, 3])
def test_tf32_edge_shapes(b2, oracle, terms):
    rng = np.random.default_rng(7)
    edge = [1, 2, 7, 31, 32, 33, 127, 128, 129, 255, 257]
    for trial in range(12):
        m, n, k = (int(rng.choice(edge)) for _ in range(3))
        ta, tb = TRANS[trial % 4]
        run_tf32(b2, oracle, terms, ta, tb, m, n, k, 0.7, -0.3, seed=trial, pad=bool(trial % 2))
        run_tf32(b2, oracle, terms, ta, tb, m, n, k, 1.5, 0.5, dist="int9", seed=trial, expect_exact=True)
    for (m, n, k) in [(5, 3, 0), (0, 7, 9), (7, 0, 9)]:
        run_tf32(b2, oracle, terms, "N", "N", m, n, k, 1.0, 0.5, seed=1)


@pytest.mark.parametrize("terms", [1, 3])
def test_tf32_large_sampled(b2, oracle, terms):
    size = 4096
    cols = sample_columns(size, tile=128, extra=16, seed=terms)
    run_tf32(b2, oracle, terms, "N", "N", size, size, size, 1.5, 0.5, seed=2100, cols=cols)
    run_tf32(b2, oracle, terms, "N", "N", size, size, size, 1.5, 0.5, dist="int9", seed=2100, cols=cols, expect_exact=True)


@pytest.mark.parametrize("terms", [1, 3])
def test_tf32_ragged_wide_tiles_both_residencies(b2, oracle, terms):
    """128 x 256 tiles with ragged last tile rows and columns, in both launch forms: 12 x 12 = 144 tiles (one wave,
    one CTA per SM with the 4-stage ring) and 16 x 13 = 208 tiles (more than one wave: two CTAs per SM, 2-stage rings)."""
    run_tf32(b2, oracle, terms, "N", "T", 1500, 3000, 100, 0.7, -0.3, seed=31)
    run_tf32(b2, oracle, terms, "T", "N", 2000, 3100, 70, 1.5, 0.5, dist="int9", seed=32, expect_exact=True)
    run_tf32(b2, oracle, terms, "N", "N", 2000, 3100, 70, 0.7, -0.3, seed=33, pad=True)


def test_tf32_long_k_several_waves(b2, oracle):
    """More than 512 k-slabs and more than one wave of ragged 128 x 256 tiles: the launch form with one CTA per SM
    and the 4-stage ring, whose slots and barrier phases wrap many times (beta != 0 and integer data)."""
    m, n, k = 2000, 3100, 5500   # three-term: 516 slabs, 16 x 13 = 208 tiles on 148 CTAs
    cols = sample_columns(n, tile=256, extra=8, seed=5)
    run_tf32(b2, oracle, 3, "N", "N", m, n, k, 0.7, -0.3, seed=41, cols=cols)
    run_tf32(b2, oracle, 3, "T", "T", m, n, k, 1.5, 0.5, dist="int9", seed=42, cols=cols, expect_exact=True)
    m, n, k = 2500, 5000, 16500  # one-term: 516 slabs, 20 x 20 = 400 tiles
    cols = sample_columns(n, tile=256, extra=4, seed=6)
    run_tf32(b2, oracle, 1, "N", "T", m, n, k, 1.5, 0.5, dist="int9", seed=43, cols=cols, expect_exact=True)


def test_tf32_quick_returns_and_errors(b2):
    m, n, k = 40, 30, 20
    A, lda, B, ldb, C, ldc = synth.gemm_inputs("N", "N", m, n, k, "uniform", 5, torch.float32)
    ws = torch.empty(b2.b2_sgemm_tf32_workspace_bytes(1, m, n, k), dtype=torch.uint8, device="cuda")
    nan = torch.full_like(A, float("nan")).cuda()
    Cd = C.cuda()
    b2.b2_sgemm_tf32(1, "N", "N", m, n, k, 0.0, nan, lda, torch.full_like(B, float("nan")).cuda(), ldb, 0.5, Cd, ldc, ws)
    assert torch.equal(Cd.cpu(), 0.5 * C)
    Cd = torch.full_like(C, float("nan")).cuda()
    b2.b2_sgemm_tf32(1, "N", "N", m, n, k, 1.0, A.cuda(), lda, B.cuda(), ldb, 0.0, Cd, ldc, ws)
    assert torch.isfinite(Cd.cpu()).all()
    assert b2.b2_sgemm_tf32(1, "N", "N", m, n, k, 1.0, A.cuda(), lda, B.cuda(), ldb, 0.0, Cd, ldc, None, check=False) == 1003
    assert b2.b2_sgemm_tf32(3, "N", "N", m, n, k, 1.0, A.cuda(), lda, B.cuda(), ldb, 0.0, Cd, ldc, ws, check=False) == 1003
    assert b2.b2_sgemm_tf32(1, "N", "N", m, n, k, 1.0, A.cuda(), m - 1, B.cuda(), ldb, 0.0, Cd, ldc, ws, check=False) == -8
    assert b2.b2_sgemm_tf32_workspace_bytes(2, m, n, k) == 0
    assert b2.b2_device_status() == 0
