"""SYRK and strided-batched GEMM through the C-ABI against their oracles.  Tolerances as for GEMM: bit-exact on
integer-valued inputs, |C - C_ref| <= 2*k*u*S otherwise, with S from the wide GEMM oracle of the same products."""
import itertools

import numpy as np
import pytest
import torch

from helpers import U
from paper_1611_08035_b200 import synth

pytestmark = pytest.mark.gpu
DT = {"d": (torch.float64, np.float64), "s": (torch.float32, np.float32)}


def run_syrk(b2, oracle, kind, uplo, trans, n, k, alpha, beta, dist="uniform", seed=0, pad=False, exact=False):
    tdt, ndt = DT[kind]
    ra, ca = (n, k) if trans == "N" else (k, n)
    lda = synth.padded_ld(ra) if pad else max(1, ra)
    ldc = synth.padded_ld(n) if pad else max(1, n)
    A = synth.matrix(ra, ca, lda, dist, seed, tdt)
    C = synth.matrix(n, n, ldc, dist, seed + 5, tdt, poison=synth.C_SENTINEL)
    want = C.numpy().copy()
    oracle.ref_syrk(uplo, trans, n, k, alpha, A.numpy(), lda, beta, want, ldc)
    Ad, Cd = A.cuda(), C.cuda()
    b2.b2_syrk(uplo, trans, n, k, alpha, Ad, lda, beta, Cd, ldc)
    assert b2.b2_device_status() == 0
    got = Cd.cpu().numpy()
    assert torch.equal(Ad.cpu().view(torch.uint8), A.view(torch.uint8))
    if n == 0:
        assert got.tobytes() == C.numpy().tobytes()
        return
    G, W, C0 = (x.reshape(n, ldc) for x in (got, want, C.numpy()))
    assert G[:, n:].tobytes() == C0[:, n:].tobytes()
    tri = (np.tril if uplo == "L" else np.triu)(np.ones((n, n), bool)).T  # [col, row] indexing of the storage
    g, w = G[:, :n], W[:, :n]
    assert g[~tri].tobytes() == C0[:, :n][~tri].tobytes(), "the other triangle was written"
    if exact:
        assert g[tri].tobytes() == w[tri].tobytes()
        return
    _, S = oracle.ref_gemm_hi(trans, "T" if trans == "N" else "N", n, n, k, alpha, A.numpy(), lda, A.numpy(), lda, beta,
                              C.numpy(), ldc)
    err = np.abs(g.astype(np.float64) - w.astype(np.float64))
    bad = (err > 2 * k * U[np.dtype(ndt)] * S.reshape(n, n)) & tri
    if bad.any():
        where = np.argwhere(bad)
        raise AssertionError(f"{int(bad.sum())} elements of the triangle exceed the bound; first (col, row): "
                             f"{where[:8].tolist()}, got {g[bad][:4]}, want {w[bad][:4]}, old {C0[:, :n][bad][:4]}")


@pytest.mark.parametrize("kind", ["d", "s"])
def test_syrk_shapes_and_triangles(b2, oracle, kind):
    for uplo, trans in itertools.product("LU", "NT"):
        run_syrk(b2, oracle, kind, uplo, trans, 333, 145, 0.7, -0.3, seed=1, pad=True)       # cp.async path
        run_syrk(b2, oracle, kind, uplo, trans, 300, 136, 1.0, 0.0, seed=2)                   # aligned (TMA for fp64)
        run_syrk(b2, oracle, kind, uplo, trans, 257, 130, 1.5, 0.5, dist="int9", seed=3, exact=True)
    for n, k in [(1, 1), (1, 50), (65, 1), (64, 64), (129, 17), (5, 0), (0, 7), (31, 300)]:
        run_syrk(b2, oracle, kind, "L", "N", n, k, -1.0, 1.0, seed=n + k, pad=True)
        run_syrk(b2, oracle, kind, "U", "T", n, k, -1.0, 1.0, seed=n + k)


def test_syrk_large_trailing_update_shape(b2, oracle):
    """The rank-k trailing update of a blocked Cholesky: n = 4096, k = 128, alpha = -1, beta = 1."""
    run_syrk(b2, oracle, "d", "L", "N", 4096, 128, -1.0, 1.0, dist="normal", seed=9)


def test_syrk_quick_returns_and_errors(b2):
    n, k = 40, 20
    C = synth.matrix(n, n, n, "uniform", 3, torch.float64)
    nanA = torch.full((n * k,), float("nan"), dtype=torch.float64, device="cuda")
    Cd = C.cuda()
    b2.b2_syrk("L", "N", n, k, 0.0, nanA, n, 0.5, Cd, n)
    got, c0 = Cd.cpu().view(n, n).T, C.view(n, n).T
    assert torch.equal(torch.tril(got), torch.tril(0.5 * c0)) and torch.equal(torch.triu(got, 1), torch.triu(c0, 1))
    z = torch.zeros(64, dtype=torch.float64, device="cuda")
    assert b2.b2_syrk("X", "N", 2, 2, 1.0, z, 2, 0.0, z, 2, check=False) == -1
    assert b2.b2_syrk("L", "Q", 2, 2, 1.0, z, 2, 0.0, z, 2, check=False) == -2
    assert b2.b2_syrk("L", "N", -1, 2, 1.0, z, 2, 0.0, z, 2, check=False) == -3
    assert b2.b2_syrk("L", "N", 2, 2, 1.0, None, 2, 0.0, z, 2, check=False) == -6
    assert b2.b2_syrk("L", "N", 3, 2, 1.0, z, 2, 0.0, z, 3, check=False) == -7
    assert b2.b2_syrk("L", "N", 3, 2, 1.0, z, 3, 0.0, None, 3, check=False) == -9
    assert b2.b2_syrk("L", "N", 3, 2, 1.0, z, 3, 0.0, z, 2, check=False) == -10


@pytest.mark.parametrize("kind", ["d", "s"])
def test_strided_batched(b2, oracle, kind):
    tdt, ndt = DT[kind]
    for (ta, tb), (m, n, k, batch), shared_b in [(("N", "N"), (70, 50, 33, 7), False), (("T", "N"), (129, 65, 40, 3), True),
                                                 (("N", "T"), (16, 16, 16, 300), False), (("T", "T"), (33, 200, 9, 2), False)]:
        (ra, ca), (rb, cb) = synth.operand_shapes(ta, tb, m, n, k)
        lda, ldb, ldc = ra + 1, rb + 2, m + 3
        sa, sb, sc = lda * ca + 5, (0 if shared_b else ldb * cb + 1), ldc * n + 7
        A = synth.matrix(1, sa * batch, 1, "uniform", 1, tdt)
        B = synth.matrix(1, max(sb * batch, ldb * cb), 1, "uniform", 2, tdt)
        C = synth.matrix(1, sc * batch, 1, "uniform", 3, tdt)
        want = C.numpy().copy()
        oracle.ref_gemm_strided_batched(ta, tb, m, n, k, 0.7, A.numpy(), lda, sa, B.numpy(), ldb, sb, -0.3, want, ldc, sc, batch)
        Cd = C.cuda()
        b2.b2_gemm_strided_batched(ta, tb, m, n, k, 0.7, A.cuda(), lda, sa, B.cuda(), ldb, sb, -0.3, Cd, ldc, sc, batch)
        got = Cd.cpu().numpy()
        u = U[np.dtype(ndt)]
        for b in range(batch):
            _, S = oracle.ref_gemm_hi(ta, tb, m, n, k, 0.7, A.numpy()[b * sa:], lda, B.numpy()[b * sb:], ldb, -0.3,
                                      C.numpy()[b * sc:], ldc)
            g = got[b * sc:b * sc + ldc * n].reshape(n, ldc)
            w = want[b * sc:b * sc + ldc * n].reshape(n, ldc)
            assert g[:, m:].tobytes() == w[:, m:].tobytes()
            assert np.all(np.abs(g[:, :m].astype(np.float64) - w[:, :m].astype(np.float64)) <= 2 * k * u * S.reshape(n, m))
            assert got[b * sc + ldc * n:(b + 1) * sc].tobytes() == C.numpy()[b * sc + ldc * n:(b + 1) * sc].tobytes()
    z = torch.zeros(4096, dtype=tdt, device="cuda")
    assert b2.b2_gemm_strided_batched("N", "N", 4, 4, 4, 1.0, z, 4, 16, z, 4, 16, 0.0, z, 4, 8, 2, check=False) == -16
    assert b2.b2_gemm_strided_batched("N", "N", 4, 4, 4, 1.0, z, 4, -1, z, 4, 16, 0.0, z, 4, 16, 2, check=False) == -9
    assert b2.b2_gemm_strided_batched("N", "N", 4, 4, 4, 1.0, z, 4, 16, z, 4, 16, 0.0, z, 4, 16, -1, check=False) == -17
    assert b2.b2_gemm_strided_batched("N", "N", 4, 4, 4, 1.0, z, 4, 16, z, 4, 16, 0.0, z, 4, 16, 0) == 0


# ---- split-K -------------------------------------------------------------------------------------------

def run_splitk(b2, oracle, kind, ta, tb, m, n, k, alpha, beta, splits, dist="uniform", seed=0, pad=False, exact=False):
    """The oracle is the plain GEMM definition: split-K only fixes another summation order."""
    tdt, ndt = DT[kind]
    (ra, _), (rb, _) = synth.operand_shapes(ta, tb, m, n, k)
    lds = (synth.padded_ld(ra), synth.padded_ld(rb), synth.padded_ld(m)) if pad else (None, None, None)
    A, lda, B, ldb, C, ldc = synth.gemm_inputs(ta, tb, m, n, k, dist, seed, tdt, *lds)
    want = C.numpy().copy()
    oracle.ref_gemm(ta, tb, m, n, k, alpha, A.numpy(), lda, B.numpy(), ldb, beta, want, ldc)
    need = b2.b2_gemm_splitk_workspace_bytes(tdt, m, n, k, splits)
    ws = torch.empty(max(256, need), dtype=torch.uint8, device="cuda")
    outs = []
    for _ in range(2):
        Cd = C.cuda()
        b2.b2_gemm_splitk(ta, tb, m, n, k, alpha, A.cuda(), lda, B.cuda(), ldb, beta, Cd, ldc, splits, ws)
        assert b2.b2_device_status() == 0
        outs.append(Cd.cpu().numpy())
    assert outs[0].tobytes() == outs[1].tobytes(), "two runs differ"
    got = outs[0]
    if m == 0 or n == 0:
        assert got.tobytes() == C.numpy().tobytes()
        return
    G, W, C0 = (x.reshape(n, ldc) for x in (got, want, C.numpy()))
    assert G[:, m:].tobytes() == C0[:, m:].tobytes(), "padding rows of C were written"
    if exact:
        assert G[:, :m].tobytes() == W[:, :m].tobytes()
        return
    _, S = oracle.ref_gemm_hi(ta, tb, m, n, k, alpha, A.numpy(), lda, B.numpy(), ldb, beta, C.numpy(), ldc)
    err = np.abs(G[:, :m].astype(np.float64) - W[:, :m].astype(np.float64))
    assert np.all(err <= 2 * max(k, 1) * U[np.dtype(ndt)] * S.reshape(n, max(1, m))[:, :m])


@pytest.mark.parametrize("kind", ["d", "s"])
def test_splitk_matches_the_plain_definition(b2, oracle, kind):
    for ta, tb in itertools.product("NT", "NT"):
        run_splitk(b2, oracle, kind, ta, tb, 100, 70, 2000, 0.7, -0.3, splits=0, seed=1, pad=True)
        run_splitk(b2, oracle, kind, ta, tb, 64, 64, 4096, 1.5, 0.5, splits=7, dist="int9", seed=2, exact=True)
        run_splitk(b2, oracle, kind, ta, tb, 130, 33, 1000, 1.0, 0.0, splits=5, seed=3)          # ragged last chunk
    for (m, n, k, splits) in [(1, 1, 5000, 0), (17, 9, 31, 4), (17, 9, 31, 40), (50, 60, 16, 3), (8, 8, 0, 4),
                              (0, 5, 100, 2), (33, 65, 257, 1), (256, 256, 8192, 0)]:
        run_splitk(b2, oracle, kind, "N", "N", m, n, k, -1.0, 1.0, splits=splits, dist="int9", seed=m + k, exact=True)


def test_splitk_plan_and_workspace_errors(b2):
    assert b2.b2_gemm_splitk_auto(256, 256, 65536) == 37   # 16 tiles of 64 x 64 on 592 resident slots
    assert b2.b2_gemm_splitk_auto(8192, 8192, 8192) == 1
    assert b2.b2_gemm_splitk_auto(64, 64, 1024) == 4       # chunks stay at least 256 deep
    assert b2.b2_gemm_splitk_workspace_bytes(torch.float64, 100, 10, 4096, 4) == 4 * 100 * 10 * 8
    assert b2.b2_gemm_splitk_workspace_bytes(torch.float32, 5, 10, 4096, 4) == 4 * 8 * 10 * 4
    assert b2.b2_gemm_splitk_workspace_bytes(torch.float64, 100, 10, 4096, 1) == 0
    A = torch.ones(64 * 1024, dtype=torch.float64, device="cuda")
    C = torch.zeros(64 * 64, dtype=torch.float64, device="cuda")
    ws = torch.empty(4 * 64 * 64 * 8, dtype=torch.uint8, device="cuda")
    args = ("N", "N", 64, 64, 1024, 1.0, A, 64, A, 1024, 0.0, C, 64)
    assert b2.b2_gemm_splitk(*args, splits=-1, workspace=ws, check=False) == -14
    assert b2.b2_gemm_splitk(*args, splits=4, workspace=None, check=False) == 1003
    assert b2.b2_gemm_splitk(*args, splits=4, workspace=ws[:1000], check=False) == 1003
    torch.cuda.synchronize()
    assert (C == 0).all()
    assert b2.b2_gemm_splitk(*args, splits=4, workspace=ws) == 0
    torch.cuda.synchronize()
    assert (C == 1024).all()
