"""Shared machinery of the GPU parity tests: run one problem through the C-ABI and through the oracle on the
same seeded inputs and compare element by element (all of C, or a column sample for big problems)."""
from __future__ import annotations

import numpy as np
import torch

from helpers import U
from paper_1611_08035_b200 import synth

GUARD = 1024       # guard-band elements on each side of every device operand (a multiple of 256 bytes)
GUARD_BYTE = 0xA5  # as fp64/fp32 a large negative number no test produces

TORCH_DT = {"d": torch.float64, "s": torch.float32, "z": torch.complex128, "z3": torch.complex128}


def staged_by_tma(name: str) -> bool:
    """Variants whose operand tiles are fetched by the tensor memory accelerator: they need 16-byte aligned columns of
    A and B and decline everything else (and batches, triangles and k splits)."""
    return "tma" in name or "_ws_" in name


def declines_transposes(name: str, transa: str, transb: str) -> bool:
    """The TMA-staged fp32 kernel reads each operand in the layout it has in memory and has no pairing for the case
    where both are k-contiguous (A transposed, B not): it declines that case."""
    return name.startswith("ffma2_tma") and transa in "TtCc" and transb in "Nn"


def sample_columns(n: int, tile: int = 64, extra: int = 24, seed: int = 0):
    """First, last, both sides of every `tile` boundary hit by a coarse stride, plus seeded random columns."""
    cols = {0, n - 1}
    for b in range(tile, n, max(tile, (n // 8) // tile * tile)):
        cols.update({b - 1, b})
    rng = np.random.default_rng(seed)
    cols.update(int(c) for c in rng.integers(0, n, size=extra))
    return sorted(c for c in cols if 0 <= c < n)


def run_and_check(b2, oracle, kind, transa, transb, m, n, k, alpha, beta, dist="uniform", seed=0, pad=False,
                  variant=None, cols=None, c_dist=None, expect_exact=False, lds=None, offset=0, factor=None):
    """Returns the largest observed error/bound ratio.  kind: 'd', 's' (real), 'z' (4M complex) or 'z3' (3M).

    Checks: every compared element within 2*k*u*S (complex: 2*(2k+4)*u*S per component, 3M 2*(3k+6)*u*S); bit-exact when
    expect_exact; padding rows of C and unsampled nothing-else untouched; A and B unchanged.
    `offset` shifts every base pointer by that many elements (misaligned bases).  Every device operand sits
    between guard bands that must come back untouched."""
    tdt = TORCH_DT[kind]
    (ra, ca), (rb, cb) = synth.operand_shapes(transa, transb, m, n, k)
    if lds is not None:
        lda, ldb, ldc = lds
    elif pad:
        lda, ldb, ldc = synth.padded_ld(ra), synth.padded_ld(rb), synth.padded_ld(m)
    else:
        lda = ldb = ldc = None
    A, lda, B, ldb, C, ldc = synth.gemm_inputs(transa, transb, m, n, k, dist, seed, tdt, lda, ldb, ldc, c_dist=c_dist)
    An, Bn, Cn = A.numpy(), B.numpy(), C.numpy()

    guards = []

    def dev(x):
        """Device copy of x bracketed by guard bands: GUARD elements of a fixed byte pattern directly before and
        after it inside one allocation (the stand-in for a memory checker: a store before the first or past the
        last element of an operand lands in a band and is seen below).  The front band is a multiple of 256 bytes,
        so the operand keeps the alignment a fresh allocation has, then shifted by `offset` elements."""
        count = x.numel()
        buf = torch.empty(2 * GUARD + offset + count, dtype=x.dtype, device="cuda")
        buf.view(torch.uint8).fill_(GUARD_BYTE)
        body = buf[GUARD + offset:GUARD + offset + count]
        body.copy_(x)
        guards.append((buf, GUARD + offset, count))
        return buf, body

    Ah, Ad = dev(A)
    Bh, Bd = dev(B)
    Ch, Cd = dev(C)
    if kind == "z":
        ws = torch.empty(max(256, b2.b2_zgemm4m_workspace_bytes(transa, transb, m, n, k)), dtype=torch.uint8,
                         device="cuda")
        b2.b2_zgemm4m(transa, transb, m, n, k, alpha, Ad, lda, Bd, ldb, beta, Cd, ldc, ws)
    elif kind == "z3":
        ws = torch.empty(max(256, b2.b2_zgemm3m_workspace_bytes(transa, transb, m, n, k)), dtype=torch.uint8,
                         device="cuda")
        b2.b2_zgemm3m(transa, transb, m, n, k, alpha, Ad, lda, Bd, ldb, beta, Cd, ldc, ws)
    else:
        fn = b2.b2_dgemm if kind == "d" else b2.b2_sgemm
        rc = fn(transa, transb, m, n, k, alpha, Ad, lda, Bd, ldb, beta, Cd, ldc, variant=variant, check=False)
        if rc == 1004 and variant is not None:
            # a variant that needs 16-byte aligned operand columns (TMA staging) declines this problem:
            # nothing may have been launched or written
            name = b2.b2_variant_name(0 if kind == "d" else 1, variant)
            vec = 2 if kind == "d" else 4
            aligned = (Ad.data_ptr() % 16 == 0 and Bd.data_ptr() % 16 == 0 and lda % vec == 0 and ldb % vec == 0)
            assert staged_by_tma(name) and (not aligned or declines_transposes(name, transa, transb)), \
                f"{name} refused an aligned problem"
            torch.cuda.synchronize()
            assert Cd.cpu().numpy().tobytes() == Cn.tobytes(), "a refused call modified C"
            return None
        assert rc == 0, f"{fn.__name__} returned {rc}: {b2.strerror(rc)}"
    assert b2.b2_device_status() == 0, "a device-side wait timed out"
    torch.cuda.synchronize()
    got = Cd.cpu().numpy()
    for buf, start, count in guards:
        raw = buf.view(torch.uint8)
        es = buf.element_size()
        assert bool((raw[:start * es] == GUARD_BYTE).all()), "bytes before an operand were written"
        assert bool((raw[(start + count) * es:] == GUARD_BYTE).all()), "bytes behind an operand were written"
    assert torch.equal(Ad.cpu().view(torch.uint8), A.view(torch.uint8)), "A was modified"
    assert torch.equal(Bd.cpu().view(torch.uint8), B.view(torch.uint8)), "B was modified"

    want = Cn.copy()
    oracle.ref_gemm(transa, transb, m, n, k, alpha, An, lda, Bn, ldb, beta, want, ldc, cols=cols)
    _, S = oracle.ref_gemm_hi(transa, transb, m, n, k, alpha, An, lda, Bn, ldb, beta, Cn, ldc, cols=cols)
    if m == 0 or n == 0:
        assert got.tobytes() == Cn.tobytes()
        return 0.0
    sel = list(range(n)) if cols is None else list(cols)
    G = got.reshape(n, ldc)
    W = want.reshape(n, ldc)
    # padding rows of every column, and (for the GPU, which computes all columns) nothing outside m x n
    assert G[:, m:].tobytes() == Cn.reshape(n, ldc)[:, m:].tobytes(), "padding rows of C were written"
    g, w = G[sel, :m], W[sel, :m]
    Sv = S.reshape(n, max(1, m))[sel, :m]
    if expect_exact:
        assert g.tobytes() == w.tobytes(), "integer-valued problem is not bit-exact"
        return 0.0
    u = U[np.dtype(Cn.dtype)]
    if kind in ("z", "z3"):
        bound = 2.0 * ((2 * k + 4) if kind == "z" else (3 * k + 6)) * u * Sv
        err = np.maximum(np.abs(g.real - w.real), np.abs(g.imag - w.imag))
    else:
        bound = (2.0 * k * u if factor is None else factor) * Sv
        err = np.abs(g.astype(np.float64) - w.astype(np.float64))
    assert np.all(np.isfinite(g.view(np.float64) if kind in ("z", "z3") else g)), "non-finite result"
    bad = err > bound
    assert not bad.any(), f"{int(bad.sum())} elements exceed the bound; worst ratio " \
                          f"{float((err / np.maximum(bound, 1e-300)).max()):.3g}"
    return float((err / np.maximum(bound, 1e-300)).max())
