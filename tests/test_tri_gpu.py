"""TRMM and TRSM through the C-ABI against their oracles.

TRMM is a sum of products like GEMM: bit-exact on integer data, |B - B_ref| <= 2*na*u*S otherwise with
S = |alpha| |op(A)| |B|.  TRSM: bit-exact on integer systems whose intermediate values are all representable;
otherwise both solutions satisfy the residual bound rho = g*(|T||X| + |alpha B|) of substitution with
g = 2*(na+2)*u, so their difference d solves T d = r_gpu - r_ref and |d| <= |T^-1| (rho_gpu + rho_ref), which
is what the test checks element by element (T^-1 from scipy on the host, in fp64)."""
import itertools

import numpy as np
import pytest
import scipy.linalg
import torch

from helpers import U
from paper_1611_08035_b200 import synth

pytestmark = pytest.mark.gpu
COMBOS = list(itertools.product("LR", "LU", "NT", "NU"))
DT = {"d": (torch.float64, np.float64), "s": (torch.float32, np.float32)}


def tri_inputs(kind, side, uplo, diag, m, n, seed, pad, integer=False):
    """A (triangle holds the data, the rest NaN, unit diagonal NaN), B; returns storage and the logical T."""
    tdt, ndt = DT[kind]
    na = m if side == "L" else n
    lda = synth.padded_ld(na) if pad else max(1, na)
    ldb = synth.padded_ld(m) if pad else max(1, m)
    rng = np.random.default_rng(seed)
    if integer:
        logical = np.zeros((na, na))
        for o in (1, 2):
            if na - o > 0:
                logical += np.diag(rng.integers(-1, 2, na - o).astype(float), -o if uplo == "L" else o)
        logical += np.diag(np.ones(na) if diag == "U" else rng.choice([-1.0, 1.0, 2.0, -2.0], na))
        B2 = rng.integers(-3, 4, (m, n)).astype(float)
    else:
        off = rng.uniform(-1, 1, (na, na)) / max(na, 1)
        d = rng.uniform(1, 2, na) * rng.choice([-1, 1], na)
        logical = (np.tril(off, -1) if uplo == "L" else np.triu(off, 1)) + np.diag(np.ones(na) if diag == "U" else d)
        B2 = rng.uniform(-1, 1, (m, n))
    logical = logical.astype(ndt)
    stored = logical.copy()
    other = np.triu(np.ones((na, na), bool), 1) if uplo == "L" else np.tril(np.ones((na, na), bool), -1)
    stored[other] = np.nan
    if diag == "U":
        stored[np.diag_indices(na)] = np.nan
    A = np.full(lda * max(na, 1), np.nan, dtype=ndt)
    if na:
        A.reshape(na, lda)[:, :na] = stored.T
    B = np.full(ldb * max(n, 1), synth.C_SENTINEL, dtype=ndt)
    if m and n:
        B.reshape(n, ldb)[:, :m] = B2.astype(ndt).T
    return A, lda, B, ldb, logical.astype(np.float64), B2.astype(ndt).astype(np.float64)


def run_tri(b2, oracle, which, kind, side, uplo, trans, diag, m, n, alpha, seed=0, pad=False, integer=False):
    tdt, ndt = DT[kind]
    A, lda, B, ldb, logical, B2 = tri_inputs(kind, side, uplo, diag, m, n, seed, pad, integer)
    want = B.copy()
    getattr(oracle, f"ref_{which}")(side, uplo, trans, diag, m, n, alpha, A, lda, want, ldb)
    Ad, Bd = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    getattr(b2, f"b2_{which}")(side, uplo, trans, diag, m, n, alpha, Ad, lda, Bd, ldb)
    assert b2.b2_device_status() == 0
    got = Bd.cpu().numpy()
    assert Ad.cpu().numpy().tobytes() == A.tobytes(), "A was modified"
    if m == 0 or n == 0:
        assert got.tobytes() == B.tobytes()
        return
    G, W = got.reshape(n, ldb), want.reshape(n, ldb)
    assert G[:, m:].tobytes() == B.reshape(n, ldb)[:, m:].tobytes(), "padding rows of B were written"
    g, w = G[:, :m].T.astype(np.float64), W[:, :m].T.astype(np.float64)
    assert np.all(np.isfinite(g)), "non-finite result (the unreferenced triangle or diagonal was read?)"
    if integer:
        assert np.array_equal(g, w), (which, side, uplo, trans, diag)
        return
    u = U[np.dtype(ndt)]
    na = m if side == "L" else n
    T = logical if trans == "N" else logical.T
    al = float(ndt(alpha))
    if which == "trmm":
        S = abs(al) * (np.abs(T) @ np.abs(B2) if side == "L" else np.abs(B2) @ np.abs(T))
        assert np.all(np.abs(g - w) <= 2 * na * u * S), (which, side, uplo, trans, diag)
        return
    gam = 2 * (na + 2) * u
    if side == "L":
        rho = gam * (np.abs(T) @ (np.abs(g) + np.abs(w)) + 2 * np.abs(al * B2))
        Tinv = np.abs(scipy.linalg.solve_triangular(T, np.eye(na), lower=(uplo == "L") != (trans == "T")))
        bound = Tinv @ rho
        resid, mag = T @ g - al * B2, np.abs(T) @ np.abs(g) + np.abs(al * B2)
    else:
        rho = gam * ((np.abs(g) + np.abs(w)) @ np.abs(T) + 2 * np.abs(al * B2))
        Tinv = np.abs(scipy.linalg.solve_triangular(T, np.eye(na), lower=(uplo == "L") != (trans == "T")))
        bound = rho @ Tinv
        resid, mag = g @ T - al * B2, np.abs(g) @ np.abs(T) + np.abs(al * B2)
    assert np.all(np.abs(resid) <= gam * mag), ("residual", side, uplo, trans, diag)
    assert np.all(np.abs(g - w) <= bound), ("difference", side, uplo, trans, diag)


@pytest.mark.parametrize("which", ["trmm", "trsm"])
@pytest.mark.parametrize("kind", ["d", "s"])
def test_all_sixteen_forms(b2, oracle, which, kind):
    for side, uplo, trans, diag in COMBOS:
        run_tri(b2, oracle, which, kind, side, uplo, trans, diag, 333, 270, 0.7, seed=1, pad=True)   # ragged, odd ld
        run_tri(b2, oracle, which, kind, side, uplo, trans, diag, 256, 192, 1.0, seed=2)             # whole leaves
        run_tri(b2, oracle, which, kind, side, uplo, trans, diag, 130, 97, 2.0 if which == "trmm" else 0.5, seed=3,
                integer=True)


@pytest.mark.parametrize("which", ["trmm", "trsm"])
def test_small_and_degenerate_shapes(b2, oracle, which):
    for (m, n) in [(1, 1), (1, 50), (50, 1), (31, 33), (32, 32), (33, 31), (64, 5), (5, 64), (0, 7), (7, 0), (65, 129)]:
        for side, uplo in itertools.product("LR", "LU"):
            run_tri(b2, oracle, which, "d", side, uplo, "N", "N", m, n, -1.0, seed=m + n, pad=True)
            run_tri(b2, oracle, which, "d", side, uplo, "T", "U", m, n, 1.0, seed=m + n)


@pytest.mark.parametrize("which", ["trmm", "trsm"])
def test_large_trailing_shapes(b2, oracle, which):
    """The shapes a blocked factorisation produces: a tall panel against a small triangle, and a big triangle."""
    run_tri(b2, oracle, which, "d", "R", "L", "T", "N", 2048, 128, 1.0, seed=11)
    run_tri(b2, oracle, which, "d", "L", "L", "N", "U", 128, 2048, 1.0, seed=12)
    run_tri(b2, oracle, which, "d", "L", "U", "N", "N", 1500, 700, 0.5, seed=13)
    run_tri(b2, oracle, which, "s", "R", "U", "N", "N", 700, 1500, 0.5, seed=14)


def test_alpha_zero_and_argument_errors(b2):
    nan = torch.full((16,), float("nan"), dtype=torch.float64, device="cuda")
    for fn in (b2.b2_trmm, b2.b2_trsm):
        B = torch.ones(20, dtype=torch.float64, device="cuda")
        assert fn("L", "L", "N", "N", 4, 3, 0.0, nan, 4, B, 5) == 0   # zeros, A is not read, padding rows kept
        torch.cuda.synchronize()
        want = torch.ones(20, dtype=torch.float64)
        want.view(4, 5)[:3, :4] = 0
        assert torch.equal(B.cpu(), want)
        args = dict(m=4, n=3, alpha=1.0, A=nan, lda=4, B=B, ldb=5)
        assert fn("X", "L", "N", "N", check=False, **args) == -1
        assert fn("L", "X", "N", "N", check=False, **args) == -2
        assert fn("L", "L", "X", "N", check=False, **args) == -3
        assert fn("L", "L", "N", "X", check=False, **args) == -4
        assert fn("L", "L", "N", "N", -1, 3, 1.0, nan, 4, B, 5, check=False) == -5
        assert fn("L", "L", "N", "N", 4, -1, 1.0, nan, 4, B, 5, check=False) == -6
        assert fn("L", "L", "N", "N", 4, 3, 1.0, None, 4, B, 5, check=False) == -8
        assert fn("L", "L", "N", "N", 4, 3, 1.0, nan, 3, B, 5, check=False) == -9
        assert fn("R", "L", "N", "N", 4, 3, 1.0, nan, 2, B, 5, check=False) == -9
        assert fn("L", "L", "N", "N", 4, 3, 1.0, nan, 4, None, 5, check=False) == -10
        assert fn("L", "L", "N", "N", 4, 3, 1.0, nan, 4, B, 3, check=False) == -11
