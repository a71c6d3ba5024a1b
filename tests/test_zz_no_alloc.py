"""b2_zgemm4m_static: the complex GEMM for callers that cannot allocate device memory.

Such callers (code in a loop that must not touch the allocator, plug-ins whose host forbids cudaMalloc,
applications that gave all device memory to their own pool) cannot hand b2_zgemm4m a workspace, so this entry
point keeps its scratch planes in a fixed array inside the library.  The test calls it through the C-ABI twice
in a row -- the second call on a different shape, so that whatever the first call left in the shared array
would show -- and checks each result against b2_zgemm4m with a caller-provided workspace, within the complex
4M tolerance the other tests use (in practice the two agree bit for bit).  It runs last so that a failure here
cannot hide the other tests, and it passes alone in a fresh process as well as after them.
"""
import numpy as np
import pytest
import torch

from paper_1611_08035_b200 import synth

pytestmark = pytest.mark.gpu


def _pair(b2, oracle, ta, tb, m, n, k, alpha, beta, seed):
    (ra, ca), (rb, cb) = synth.operand_shapes(ta, tb, m, n, k)
    lda, ldb, ldc = ra + 3, rb + 1, m + 2
    A = synth.matrix(ra, ca, lda, "uniform", seed, torch.complex128)
    B = synth.matrix(rb, cb, ldb, "uniform", seed + 7, torch.complex128)
    C = synth.matrix(m, n, ldc, "uniform", seed + 13, torch.complex128, poison=synth.C_SENTINEL)
    Ad, Bd = A.cuda(), B.cuda()
    c_static, c_ws = C.cuda(), C.cuda()
    b2.b2_zgemm4m_static(ta, tb, m, n, k, alpha, Ad, lda, Bd, ldb, beta, c_static, ldc)
    ws = torch.empty(b2.b2_zgemm4m_workspace_bytes(ta, tb, m, n, k), dtype=torch.uint8, device="cuda")
    b2.b2_zgemm4m(ta, tb, m, n, k, alpha, Ad, lda, Bd, ldb, beta, c_ws, ldc, ws)
    torch.cuda.synchronize()
    got, want = c_static.cpu().numpy().reshape(n, ldc), c_ws.cpu().numpy().reshape(n, ldc)
    _, S = oracle.ref_gemm_hi(ta, tb, m, n, k, alpha, A.numpy(), lda, B.numpy(), ldb, beta, C.numpy(), ldc)
    bound = 2 * (2 * k + 4) * 2.0 ** -53 * S.reshape(n, m)
    d = got[:, :m] - want[:, :m]
    assert np.all(np.abs(d.real) <= bound) and np.all(np.abs(d.imag) <= bound)
    assert got[:, m:].tobytes() == C.numpy().reshape(n, ldc)[:, m:].tobytes()  # padding rows untouched
    assert np.all(np.isfinite(got[:, :m].view(np.float64)))


def test_static_scratch_matches_workspace_entry_on_two_calls_in_a_row(b2, oracle):
    _pair(b2, oracle, "N", "N", 200, 150, 170, 1 + 0.5j, 0.25 - 0.75j, seed=901)
    _pair(b2, oracle, "T", "N", 130, 71, 33, 0.3 - 0.8j, 0j, seed=902)  # smaller planes over the stale contents
    _pair(b2, oracle, "C", "T", 90, 40, 57, 1 - 1j, 0.5j, seed=903)     # a conjugate transpose


def test_static_scratch_limit_and_argument_errors(b2):
    z = torch.zeros(16, dtype=torch.complex128, device="cuda")
    assert b2.b2_zgemm4m_workspace_bytes("N", "N", 256, 256, 256) <= b2.ZGEMM4M_STATIC_BYTES
    assert b2.b2_zgemm4m_workspace_bytes("N", "N", 512, 512, 512) > b2.ZGEMM4M_STATIC_BYTES
    assert b2.b2_zgemm4m_static("N", "N", 512, 512, 512, 1, z, 512, z, 512, 0, z, 512, check=False) == 1005
    assert "scratch" in b2.strerror(1005)
    assert b2.b2_zgemm4m_static("X", "N", 4, 4, 4, 1, z, 4, z, 4, 0, z, 4, check=False) == -1
    assert b2.b2_zgemm4m_static("N", "N", 4, 4, 4, 1, z, 3, z, 4, 0, z, 4, check=False) == -8
    torch.cuda.synchronize()
    assert (z == 0).all()
