"""b2_zgemm4m_static: the complex GEMM for callers that cannot allocate device memory.

Such callers (code in a loop that must not touch the allocator, plug-ins whose host forbids cudaMalloc,
applications that gave all device memory to their own pool) cannot hand b2_zgemm4m a workspace, so this entry
point keeps its scratch planes in a fixed array inside the library.  The test calls it through the C-ABI several
times in a row -- later calls on different shapes, so that whatever an earlier call left in the shared array
would show -- and checks each result twice: against b2_zgemm4m with a caller-provided workspace (in practice
bit for bit) and against the CPU oracle directly, within the complex 4M tolerance the other tests use (bit-exact
on integer data).  It also covers the largest problem the array holds, the first one it does not, and the calls
that need no planes at all.  It runs last so that a failure here cannot hide the other tests, and it passes
alone in a fresh process as well as after them.
"""
import numpy as np
import pytest
import torch

from paper_1611_08035_b200 import synth

pytestmark = pytest.mark.gpu


def _pair(b2, oracle, ta, tb, m, n, k, alpha, beta, seed, dist="uniform"):
    (ra, ca), (rb, cb) = synth.operand_shapes(ta, tb, m, n, k)
    lda, ldb, ldc = ra + 3, rb + 1, m + 2
    A = synth.matrix(ra, ca, lda, dist, seed, torch.complex128)
    B = synth.matrix(rb, cb, ldb, dist, seed + 7, torch.complex128)
    C = synth.matrix(m, n, ldc, dist, seed + 13, torch.complex128, poison=synth.C_SENTINEL)
    Ad, Bd = A.cuda(), B.cuda()
    c_static, c_ws = C.cuda(), C.cuda()
    b2.b2_zgemm4m_static(ta, tb, m, n, k, alpha, Ad, lda, Bd, ldb, beta, c_static, ldc)
    ws = torch.empty(max(256, b2.b2_zgemm4m_workspace_bytes(ta, tb, m, n, k)), dtype=torch.uint8, device="cuda")
    b2.b2_zgemm4m(ta, tb, m, n, k, alpha, Ad, lda, Bd, ldb, beta, c_ws, ldc, ws)
    torch.cuda.synchronize()
    got, other = c_static.cpu().numpy().reshape(n, ldc), c_ws.cpu().numpy().reshape(n, ldc)
    want = C.numpy().copy()
    oracle.ref_gemm(ta, tb, m, n, k, alpha, A.numpy(), lda, B.numpy(), ldb, beta, want, ldc)
    want = want.reshape(n, ldc)
    assert got[:, m:].tobytes() == C.numpy().reshape(n, ldc)[:, m:].tobytes()  # padding rows untouched
    assert np.all(np.isfinite(got[:, :m].view(np.float64)))
    if dist == "int9":  # one correct bit pattern
        assert got[:, :m].tobytes() == want[:, :m].tobytes()
        assert got[:, :m].tobytes() == other[:, :m].tobytes()
        return
    _, S = oracle.ref_gemm_hi(ta, tb, m, n, k, alpha, A.numpy(), lda, B.numpy(), ldb, beta, C.numpy(), ldc)
    bound = 2 * (2 * k + 4) * 2.0 ** -53 * S.reshape(n, max(1, m))[:, :m]
    for ref in (want, other):
        d = got[:, :m] - ref[:, :m]
        assert np.all(np.abs(d.real) <= bound) and np.all(np.abs(d.imag) <= bound)


def test_static_scratch_matches_workspace_entry_on_two_calls_in_a_row(b2, oracle):
    _pair(b2, oracle, "N", "N", 200, 150, 170, 1 + 0.5j, 0.25 - 0.75j, seed=901)
    _pair(b2, oracle, "T", "N", 130, 71, 33, 0.3 - 0.8j, 0j, seed=902)  # smaller planes over the stale contents
    _pair(b2, oracle, "C", "T", 90, 40, 57, 1 - 1j, 0.5j, seed=903)     # a conjugate transpose
    _pair(b2, oracle, "N", "C", 64, 96, 80, 2 - 1j, 0.5 + 0.5j, seed=904, dist="int9")  # exact data, bit for bit


def _largest_square_that_fits(b2):
    s = 1
    while b2.b2_zgemm4m_workspace_bytes("N", "N", s + 1, s + 1, s + 1) <= b2.ZGEMM4M_STATIC_BYTES:
        s += 1
    return s


def test_static_scratch_at_its_limit(b2, oracle):
    """The largest cube whose planes still fit uses the array up to (almost) its last byte: an overrun of the
    fixed array would corrupt whatever the image keeps behind it or show up in the result.  One size further is
    refused with nothing launched."""
    s = _largest_square_that_fits(b2)
    assert 300 < s < 400
    assert b2.b2_zgemm4m_workspace_bytes("N", "N", s, s, s) > b2.ZGEMM4M_STATIC_BYTES - (256 << 10)
    _pair(b2, oracle, "N", "N", s, s, s, 1 + 0.5j, 0.25 - 0.75j, seed=905)
    _pair(b2, oracle, "N", "N", s, s, s, 1.5 + 0j, 0.5 + 0j, seed=906, dist="int9")
    z = torch.zeros((s + 1) * (s + 1), dtype=torch.complex128, device="cuda")
    assert b2.b2_zgemm4m_static("N", "N", s + 1, s + 1, s + 1, 1, z, s + 1, z, s + 1, 0, z, s + 1, check=False) == 1005
    torch.cuda.synchronize()
    assert (z == 0).all()


def test_static_scratch_limit_and_argument_errors(b2):
    z = torch.zeros(16, dtype=torch.complex128, device="cuda")
    assert b2.b2_zgemm4m_workspace_bytes("N", "N", 256, 256, 256) <= b2.ZGEMM4M_STATIC_BYTES
    assert b2.b2_zgemm4m_workspace_bytes("N", "N", 512, 512, 512) > b2.ZGEMM4M_STATIC_BYTES
    assert b2.b2_zgemm4m_static("N", "N", 512, 512, 512, 1, z, 512, z, 512, 0, z, 512, check=False) == 1005
    assert "scratch" in b2.strerror(1005)
    assert b2.b2_zgemm4m_static("X", "N", 4, 4, 4, 1, z, 4, z, 4, 0, z, 4, check=False) == -1
    assert b2.b2_zgemm4m_static("N", "N", 4, 4, 4, 1, z, 3, z, 4, 0, z, 4, check=False) == -8
    # the same answers as b2_zgemm4m on shapes beyond the limit: argument errors first, then the quick returns
    assert b2.b2_zgemm4m_static("N", "N", 4096, 4096, 4096, 1, z, 5, z, 4096, 0, z, 4096, check=False) == -8
    assert b2.b2_zgemm4m_static("N", "N", 0, 4096, 4096, 1, z, 1, z, 4096, 0, z, 1, check=False) == 0
    assert b2.b2_zgemm4m_static("N", "N", 4096, 0, 4096, 1, z, 4096, z, 4096, 0, z, 4096, check=False) == 0
    torch.cuda.synchronize()
    assert (z == 0).all()


def test_static_scratch_scale_only_calls_need_no_planes(b2, oracle):
    """alpha == 0 or k == 0 is C := beta*C: no plane is split, so the size limit does not apply; A and B are not
    read (NaN) and the result equals the oracle's bit for bit."""
    m, n, k = 900, 700, 800  # planes would need about 31 MB
    assert b2.b2_zgemm4m_workspace_bytes("N", "N", m, n, k) > b2.ZGEMM4M_STATIC_BYTES
    ldc = m + 1
    C = synth.matrix(m, n, ldc, "uniform", 907, torch.complex128, poison=synth.C_SENTINEL)
    nan = torch.full((m * k,), float("nan"), dtype=torch.complex128)
    for alpha, kk, beta in ((0j, k, 0.5 - 0.25j), (1 + 1j, 0, -1.5 + 0j), (0j, k, 0j)):
        Cd = C.cuda()
        rc = b2.b2_zgemm4m_static("N", "N", m, n, kk, alpha, nan.cuda(), m, nan.cuda(), max(1, kk), beta, Cd, ldc,
                                  check=False)
        assert rc == 0
        torch.cuda.synchronize()
        want = C.numpy().copy()
        oracle.ref_gemm("N", "N", m, n, kk, alpha, nan.numpy(), m, nan.numpy(), max(1, kk), beta, want, ldc)
        assert Cd.cpu().numpy().tobytes() == want.tobytes()
