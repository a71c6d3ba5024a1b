"""Whole-matrix agreement between kernel variants at the full benchmark sizes.

On integer-valued data ({-4..4}, alpha = 1.5, beta = 0.5, k <= 8192) every partial sum is an exactly representable
integer, so there is ONE correct bit pattern whatever the order of summation, the tile shape, the staging path or
the pipe the multiply-adds run on.  Every variant of a data type must therefore produce the same bits over ALL of C,
launch after launch.  A column sample cannot replace this: a hand-off error between a producer and its consumers
in a staging ring that wraps hundreds of times may corrupt a handful of tiles in tens of thousands, which a few
dozen sampled columns rarely hit.  The comparison itself runs on the device; the oracle then checks a column
sample of the agreed result, which ties the whole matrix to the definition.
"""
import json

import numpy as np
import pytest
import torch

from gpu_util import declines_transposes, sample_columns, staged_by_tma
from paper_1611_08035_b200 import synth

pytestmark = pytest.mark.gpu


def _bits(x):
    return x.view(torch.int64 if x.element_size() == 8 else torch.int32)


def _assert_same(got, first, what):
    differing = int((_bits(got) != _bits(first)).sum())
    assert differing == 0, f"{what}: {differing} elements differ from the first variant"


def _oracle_sample(oracle, ta, tb, m, n, k, alpha, beta, A, lda, B, ldb, C0, ldc, got, seed, extra=8):
    cols = sample_columns(n, tile=64, extra=extra, seed=seed)
    want = C0.cpu().numpy()
    oracle.ref_gemm(ta, tb, m, n, k, alpha, A.cpu().numpy(), lda, B.cpu().numpy(), ldb, beta, want, ldc, cols=cols)
    g = got.cpu().numpy().reshape(n, ldc)[cols]
    assert g.tobytes() == want.reshape(n, ldc)[cols].tobytes(), "the agreed result differs from the oracle"


@pytest.mark.parametrize("size", [4096, 8192])
def test_fp64_every_tensor_core_variant_same_bits(b2, oracle, size):
    """cp.async-staged and TMA-staged DMMA variants (all tile shapes), three launches of each TMA-staged one, and
    the automatic choice, on the square benchmark problem."""
    m = n = k = size
    A, lda, B, ldb, C, ldc = synth.gemm_inputs("N", "N", m, n, k, "int9", 2200 + size, torch.float64, device="cuda")
    first = None
    names = [b2.b2_variant_name(0, v) for v in range(b2.b2_variant_count(0))]
    for v, name in list(enumerate(names)) + [(None, "auto")]:
        if v is not None and "dmma" not in name:
            continue
        for rep in range(3 if staged_by_tma(name) else 1):
            Cd = C.clone()
            b2.b2_dgemm("N", "N", m, n, k, 1.5, A, lda, B, ldb, 0.5, Cd, ldc, variant=v)
            assert b2.b2_device_status() == 0
            if first is None:
                first = Cd
            else:
                _assert_same(Cd, first, f"{name}, launch {rep}")
    _oracle_sample(oracle, "N", "N", m, n, k, 1.5, 0.5, A, lda, B, ldb, C, ldc, first, seed=size)


@pytest.mark.parametrize("ta,tb", [("N", "T"), ("T", "N"), ("T", "T")])
def test_fp64_transposed_staging_same_bits_4096(b2, oracle, ta, tb):
    """The transposed operand layouts (k-contiguous tiles in shared memory, other TMA boxes) at 4096^3."""
    m = n = k = 4096
    A, lda, B, ldb, C, ldc = synth.gemm_inputs(ta, tb, m, n, k, "int9", 2300, torch.float64, device="cuda")
    first = None
    for v in range(b2.b2_variant_count(0)):
        name = b2.b2_variant_name(0, v)
        if "dmma" not in name or "32x32" in name:
            continue
        for rep in range(2 if staged_by_tma(name) else 1):
            Cd = C.clone()
            b2.b2_dgemm(ta, tb, m, n, k, 1.5, A, lda, B, ldb, 0.5, Cd, ldc, variant=v)
            assert b2.b2_device_status() == 0
            if first is None:
                first = Cd
            else:
                _assert_same(Cd, first, f"{name} {ta}{tb}, launch {rep}")
    _oracle_sample(oracle, ta, tb, m, n, k, 1.5, 0.5, A, lda, B, ldb, C, ldc, first, seed=7)


def test_fp32_cluster_k_split_against_unsplit_2048(b2, oracle):
    """2048^3 fp32 is launched with the k-loop of each tile split over a cluster of two CTAs; an explicitly chosen
    variant is never split.  Same bits over the whole matrix, in all four transposes."""
    m = n = k = 2048
    cfg = json.loads(b2.b2_gemm_query_config(1, "N", "N", m, n, k, m, k, m))
    for ta in "NT":
        for tb in "NT":
            A, lda, B, ldb, C, ldc = synth.gemm_inputs(ta, tb, m, n, k, "int9", 2400, torch.float32, device="cuda")
            auto = C.clone()
            b2.b2_sgemm(ta, tb, m, n, k, 1.5, A, lda, B, ldb, 0.5, auto, ldc)
            for v in range(b2.b2_variant_count(1)):
                if declines_transposes(b2.b2_variant_name(1, v), ta, tb):
                    continue
                Cd = C.clone()
                b2.b2_sgemm(ta, tb, m, n, k, 1.5, A, lda, B, ldb, 0.5, Cd, ldc, variant=v)
                _assert_same(Cd, auto, f"{b2.b2_variant_name(1, v)} {ta}{tb} against the automatic (k_split "
                                       f"{cfg['k_split']}) launch")
            if ta == "N" and tb == "N":
                _oracle_sample(oracle, ta, tb, m, n, k, 1.5, 0.5, A, lda, B, ldb, C, ldc, auto, seed=11)


def test_fp32_every_fma_variant_same_bits_8192(b2, oracle):
    """8192^3 fp32: the kernel that transposes a k-contiguous B through registers, the one that copies it with
    cp.async, the scalar-FMA comparison kernel and the automatic choice."""
    m = n = k = 8192
    A, lda, B, ldb, C, ldc = synth.gemm_inputs("N", "N", m, n, k, "int9", 2500, torch.float32, device="cuda")
    first = None
    for v in [None] + [v for v in range(b2.b2_variant_count(1)) if "32x32" not in b2.b2_variant_name(1, v)]:
        Cd = C.clone()
        b2.b2_sgemm("N", "N", m, n, k, 1.5, A, lda, B, ldb, 0.5, Cd, ldc, variant=v)
        if first is None:
            first = Cd
        else:
            _assert_same(Cd, first, b2.b2_variant_name(1, v))
    _oracle_sample(oracle, "N", "N", m, n, k, 1.5, 0.5, A, lda, B, ldb, C, ldc, first, seed=13, extra=4)


@pytest.mark.parametrize("ta,tb", [("N", "N"), ("T", "T"), ("N", "T")])
def test_fp32_short_update_added_in_memory_8192(b2, oracle, ta, tb):
    """C := C - op(A) op(B) on 8192^2 with k = 128 in fp32: the automatic choice is the TMA-staged kernel, whose
    tiles are added to C in memory by bulk reductions (beta = 1) or leave by bulk stores (beta = 0); the cp.async
    kernel with the ordinary epilogue must give the same bits over the whole matrix."""
    m = n = 8192
    k = 128
    A, lda, B, ldb, C, ldc = synth.gemm_inputs(ta, tb, m, n, k, "int9", 2800, torch.float32, device="cuda")
    for beta in (1.0, 0.0):
        ref = C.clone()
        b2.b2_sgemm(ta, tb, m, n, k, -1.0, A, lda, B, ldb, beta, ref, ldc, variant=1)
        for rep in range(2):
            got = C.clone()
            b2.b2_sgemm(ta, tb, m, n, k, -1.0, A, lda, B, ldb, beta, got, ldc)
            assert b2.b2_device_status() == 0
            _assert_same(got, ref, f"automatic choice, beta {beta}, launch {rep}")
        tma = [v for v in range(b2.b2_variant_count(1)) if staged_by_tma(b2.b2_variant_name(1, v))][0]
        got = C.clone()
        b2.b2_sgemm(ta, tb, m, n, k, -1.0, A, lda, B, ldb, beta, got, ldc, variant=tma)
        _assert_same(got, ref, f"TMA-staged kernel, beta {beta}")
        if beta == 1.0:
            _oracle_sample(oracle, ta, tb, m, n, k, -1.0, 1.0, A, lda, B, ldb, C, ldc, ref, seed=19, extra=4)


@pytest.mark.parametrize("size", [4096, 8192])
def test_tf32_entries_against_the_fma_kernel_on_integer_data(b2, size):
    """Integers in {-4..4} are TF32 values and their sums stay below 2^24, so the one- and three-term tensor-core
    entries must give the bits of the FP32-FMA kernel over the whole matrix.  4096^3 runs both entries with two
    CTAs per SM; at 8192^3 the three-term entry (768 slabs) runs the one-CTA, four-stage form."""
    m = n = k = size
    A, lda, B, ldb, C, ldc = synth.gemm_inputs("N", "N", m, n, k, "int9", 2600 + size, torch.float32, device="cuda")
    ref = C.clone()
    b2.b2_sgemm("N", "N", m, n, k, 1.5, A, lda, B, ldb, 0.5, ref, ldc)
    for terms, fn in ((1, b2.b2_sgemm_tf32x1), (3, b2.b2_sgemm_tf32x3)):
        ws = torch.empty(b2.b2_sgemm_tf32_workspace_bytes(terms, m, n, k), dtype=torch.uint8, device="cuda")
        for rep in range(2):
            Cd = C.clone()
            fn("N", "N", m, n, k, 1.5, A, lda, B, ldb, 0.5, Cd, ldc, ws)
            assert b2.b2_device_status() == 0
            _assert_same(Cd, ref, f"tf32x{terms}, launch {rep}")
        del ws


def test_zgemm4m_planes_against_single_real_products_4096(b2, oracle):
    """The complex entry at 4096^3 on integer data, whole matrix: its result must equal, bit for bit, what the four
    plane products give when each is formed by one b2_dgemm call on planes split here with torch (alpha*A is exact
    on this data, and so is every later step)."""
    m = n = k = 4096
    alpha, beta = 2 - 1j, 0.5 + 0.5j
    A, lda, B, ldb, C, ldc = synth.gemm_inputs("N", "N", m, n, k, "int9", 2700, torch.complex128, device="cuda")
    ws = torch.empty(b2.b2_zgemm4m_workspace_bytes("N", "N", m, n, k), dtype=torch.uint8, device="cuda")
    got = C.clone()
    b2.b2_zgemm4m("N", "N", m, n, k, alpha, A, lda, B, ldb, beta, got, ldc, ws)
    assert b2.b2_device_status() == 0
    del ws
    Ap = alpha * A
    Apr, Api = Ap.real.contiguous(), Ap.imag.contiguous()
    Br, Bi = B.real.contiguous(), B.imag.contiguous()
    del Ap
    bc = beta * C
    Cr, Ci = bc.real.contiguous(), bc.imag.contiguous()
    del bc
    T = torch.empty_like(Cr)
    b2.b2_dgemm("N", "N", m, n, k, 1.0, Apr, lda, Br, ldb, 1.0, Cr, ldc)   # Cr = A'r Br + (beta C)r
    b2.b2_dgemm("N", "N", m, n, k, 1.0, Api, lda, Bi, ldb, 0.0, T, ldc)    # T = A'i Bi, by itself
    Cr -= T
    b2.b2_dgemm("N", "N", m, n, k, 1.0, Apr, lda, Bi, ldb, 1.0, Ci, ldc)   # Ci = A'r Bi + (beta C)i
    b2.b2_dgemm("N", "N", m, n, k, 1.0, Api, lda, Br, ldb, 0.0, T, ldc)    # T = A'i Br, by itself
    Ci += T
    differing = int((got.real != Cr).sum() + (got.imag != Ci).sum())
    assert differing == 0, f"{differing} components differ from the single real products"
    cols = sample_columns(n, tile=64, extra=4, seed=17)
    want = C.cpu().numpy()
    oracle.ref_gemm("N", "N", m, n, k, alpha, A.cpu().numpy(), lda, B.cpu().numpy(), ldb, beta, want, ldc, cols=cols)
    assert got.cpu().numpy().reshape(n, ldc)[cols].tobytes() == want.reshape(n, ldc)[cols].tobytes()
