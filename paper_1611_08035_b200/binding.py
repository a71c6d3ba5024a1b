"""ctypes binding of ``libb2gemm.so``: argument marshalling only.

Each Python function has the name and argument order of the C entry point it wraps (see
``include/b2gemm.h``); tensors are passed as raw device (or host) pointers plus sizes, the
stream as ``torch.cuda.current_stream().cuda_stream``.  No arithmetic of the GEMM happens
here.  Loading fails loudly when the library has not been built: there is no fallback.
"""
from __future__ import annotations

import ctypes
from ctypes import c_char, c_char_p, c_double, c_float, c_int, c_int64, c_size_t, c_void_p
from pathlib import Path

import torch

LIB_PATH = Path(__file__).resolve().parent / "libb2gemm.so"
_lib = None

_GEMM_TAIL_D = [c_char, c_char, c_int64, c_int64, c_int64, c_double, c_void_p, c_int64, c_void_p, c_int64, c_double,
                c_void_p, c_int64]
_GEMM_TAIL_S = [c_char, c_char, c_int64, c_int64, c_int64, c_float, c_void_p, c_int64, c_void_p, c_int64, c_float,
                c_void_p, c_int64]

_SIGNATURES = {
    "b2_dgemm": (c_int, _GEMM_TAIL_D + [c_void_p]),
    "b2_sgemm": (c_int, _GEMM_TAIL_S + [c_void_p]),
    "b2_dgemm_variant": (c_int, [c_int] + _GEMM_TAIL_D + [c_void_p]),
    "b2_sgemm_variant": (c_int, [c_int] + _GEMM_TAIL_S + [c_void_p]),
    "b2_device_status": (c_int, [c_void_p]),
    "b2_selftest_wait_timeout": (c_int, [c_void_p]),
    "b2_variant_count": (c_int, [c_int]),
    "b2_variant_name": (c_char_p, [c_int, c_int]),
    "b2_gemm_query_config": (c_int, [c_int, c_char, c_char, c_int64, c_int64, c_int64, c_int64, c_int64, c_int64,
                                     c_char_p, c_size_t]),
    "b2_zgemm4m_workspace_bytes": (c_size_t, [c_char, c_char, c_int64, c_int64, c_int64]),
    "b2_zgemm4m": (c_int, [c_char, c_char, c_int64, c_int64, c_int64, ctypes.POINTER(c_double), c_void_p, c_int64,
                           c_void_p, c_int64, ctypes.POINTER(c_double), c_void_p, c_int64, c_void_p, c_size_t,
                           c_void_p]),
    "b2_dtrmm": (c_int, [c_char, c_char, c_char, c_char, c_int64, c_int64, c_double, c_void_p, c_int64, c_void_p, c_int64,
                         c_void_p]),
    "b2_strmm": (c_int, [c_char, c_char, c_char, c_char, c_int64, c_int64, c_float, c_void_p, c_int64, c_void_p, c_int64,
                         c_void_p]),
    "b2_dtrsm": (c_int, [c_char, c_char, c_char, c_char, c_int64, c_int64, c_double, c_void_p, c_int64, c_void_p, c_int64,
                         c_void_p]),
    "b2_strsm": (c_int, [c_char, c_char, c_char, c_char, c_int64, c_int64, c_float, c_void_p, c_int64, c_void_p, c_int64,
                         c_void_p]),
    "b2_gemm_splitk_auto": (c_int, [c_int64, c_int64, c_int64]),
    "b2_gemm_splitk_workspace_bytes": (c_size_t, [c_int, c_int64, c_int64, c_int64, c_int]),
    "b2_dgemm_splitk": (c_int, [c_char, c_char, c_int64, c_int64, c_int64, c_double, c_void_p, c_int64, c_void_p, c_int64,
                                c_double, c_void_p, c_int64, c_int, c_void_p, c_size_t, c_void_p]),
    "b2_sgemm_splitk": (c_int, [c_char, c_char, c_int64, c_int64, c_int64, c_float, c_void_p, c_int64, c_void_p, c_int64,
                                c_float, c_void_p, c_int64, c_int, c_void_p, c_size_t, c_void_p]),
    "b2_zgemm3m_workspace_bytes": (c_size_t, [c_char, c_char, c_int64, c_int64, c_int64]),
    "b2_zgemm3m": (c_int, [c_char, c_char, c_int64, c_int64, c_int64, ctypes.POINTER(c_double), c_void_p, c_int64,
                           c_void_p, c_int64, ctypes.POINTER(c_double), c_void_p, c_int64, c_void_p, c_size_t,
                           c_void_p]),
    "b2_zgemm4m_static": (c_int, [c_char, c_char, c_int64, c_int64, c_int64, ctypes.POINTER(c_double), c_void_p, c_int64,
                                  c_void_p, c_int64, ctypes.POINTER(c_double), c_void_p, c_int64, c_void_p]),
    "b2_dsyrk": (c_int, [c_char, c_char, c_int64, c_int64, c_double, c_void_p, c_int64, c_double, c_void_p, c_int64,
                         c_void_p]),
    "b2_ssyrk": (c_int, [c_char, c_char, c_int64, c_int64, c_float, c_void_p, c_int64, c_float, c_void_p, c_int64,
                         c_void_p]),
    "b2_dgemm_strided_batched": (c_int, [c_char, c_char, c_int64, c_int64, c_int64, c_double, c_void_p, c_int64, c_int64,
                                         c_void_p, c_int64, c_int64, c_double, c_void_p, c_int64, c_int64, c_int64,
                                         c_void_p]),
    "b2_sgemm_strided_batched": (c_int, [c_char, c_char, c_int64, c_int64, c_int64, c_float, c_void_p, c_int64, c_int64,
                                         c_void_p, c_int64, c_int64, c_float, c_void_p, c_int64, c_int64, c_int64,
                                         c_void_p]),
    "b2_sgemm_tf32_workspace_bytes": (c_size_t, [c_int, c_int64, c_int64, c_int64]),
    "b2_sgemm_tf32x1": (c_int, _GEMM_TAIL_S + [c_void_p, c_size_t, c_void_p]),
    "b2_sgemm_tf32x3": (c_int, _GEMM_TAIL_S + [c_void_p, c_size_t, c_void_p]),
    "b2_gemm_host_workspace_bytes": (c_size_t, [c_int, c_char, c_char, c_int64, c_int64, c_int64]),
    "b2_dgemm_host": (c_int, _GEMM_TAIL_D + [c_void_p, c_size_t, c_void_p]),
    "b2_sgemm_host": (c_int, _GEMM_TAIL_S + [c_void_p, c_size_t, c_void_p]),
    "b2_pipe_probe": (c_int, [c_int, c_int, c_int, c_int64, c_void_p, c_size_t, ctypes.POINTER(c_double), c_void_p]),
    "b2_model_throughput": (c_double, [c_int, ctypes.POINTER(c_double), ctypes.POINTER(c_double)]),
    "b2_model_stalled_throughput": (c_double, [c_double, c_int, c_double]),
    "b2_model_register_updates": (c_int, [c_int, c_int, c_int, c_int, c_int, c_int, ctypes.POINTER(c_int)]),
    "b2_model_predict_variant": (c_int, [c_int, c_int, ctypes.POINTER(c_double), c_char_p, c_size_t]),
    "b2_model_enumerate": (c_int, [c_int, c_int, c_char_p, c_size_t]),
    "b2_strerror": (c_char_p, [c_int]),
    "b2_version": (c_char_p, []),
}

EXPORTED_SYMBOLS = tuple(_SIGNATURES)


def lib() -> ctypes.CDLL:
    """The loaded C library (loaded once).  Raises when it has not been built."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_1611_08035_b200.build` "
                "(there is no CPU or library fallback)")
        handle = ctypes.CDLL(str(LIB_PATH))
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


def strerror(status: int) -> str:
    return lib().b2_strerror(int(status)).decode()


def version() -> str:
    return lib().b2_version().decode()


class B2Error(RuntimeError):
    def __init__(self, fn: str, status: int):
        super().__init__(f"{fn} returned {status}: {strerror(status)}")
        self.status = status


_TR = {c: c.encode("ascii") for c in "NnTtCc"}


def _tr(c: str) -> bytes:
    b = _TR.get(c)
    return b if b is not None else c.encode("ascii")[:1]


# torch.cuda.current_stream() builds a Python Stream object (about 3 us per call, a third of the cost of
# launching a small GEMM from Python); the raw handle of the same stream comes from these two calls in 0.2 us.
_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)
_cur_device = getattr(torch._C, "_cuda_getDevice", None)


def _stream() -> int:
    if _raw_stream is not None and _cur_device is not None:
        return _raw_stream(_cur_device())
    return torch.cuda.current_stream().cuda_stream


def _check(fn: str, rc: int) -> None:
    if rc != 0:
        raise B2Error(fn, rc)


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def b2_dgemm(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, variant=None, check=True) -> int:
    """C := alpha*op(A)*op(B) + beta*C in fp64 on device tensors (column-major storage)."""
    for t in (A, B, C):
        if t is not None and (t.dtype != torch.float64 or not t.is_cuda):
            raise TypeError("b2_dgemm takes float64 CUDA tensors")
    if variant is None:
        rc = lib().b2_dgemm(_tr(transa), _tr(transb), m, n, k, alpha, _ptr(A), lda, _ptr(B), ldb, beta, _ptr(C), ldc,
                            _stream())
    else:
        rc = lib().b2_dgemm_variant(variant, _tr(transa), _tr(transb), m, n, k, alpha, _ptr(A), lda, _ptr(B), ldb,
                                    beta, _ptr(C), ldc, _stream())
    if check:
        _check("b2_dgemm", rc)
    return rc


def b2_sgemm(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, variant=None, check=True) -> int:
    """C := alpha*op(A)*op(B) + beta*C in fp32 (FP32 FMA only) on device tensors."""
    for t in (A, B, C):
        if t is not None and (t.dtype != torch.float32 or not t.is_cuda):
            raise TypeError("b2_sgemm takes float32 CUDA tensors")
    if variant is None:
        rc = lib().b2_sgemm(_tr(transa), _tr(transb), m, n, k, alpha, _ptr(A), lda, _ptr(B), ldb, beta, _ptr(C), ldc,
                            _stream())
    else:
        rc = lib().b2_sgemm_variant(variant, _tr(transa), _tr(transb), m, n, k, alpha, _ptr(A), lda, _ptr(B), ldb,
                                    beta, _ptr(C), ldc, _stream())
    if check:
        _check("b2_sgemm", rc)
    return rc


def b2_variant_count(dtype: int) -> int:
    return lib().b2_variant_count(dtype)


def b2_variant_name(dtype: int, variant: int):
    s = lib().b2_variant_name(dtype, variant)
    return None if s is None else s.decode()


def b2_gemm_query_config(dtype, transa, transb, m, n, k, lda, ldb, ldc) -> str:
    buf = ctypes.create_string_buffer(1024)
    rc = lib().b2_gemm_query_config(dtype, _tr(transa), _tr(transb), m, n, k, lda, ldb, ldc, buf, len(buf))
    _check("b2_gemm_query_config", rc)
    return buf.value.decode()


def b2_zgemm4m_workspace_bytes(transa, transb, m, n, k) -> int:
    return lib().b2_zgemm4m_workspace_bytes(_tr(transa), _tr(transb), m, n, k)


def b2_zgemm4m(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, workspace, check=True) -> int:
    """Complex128 GEMM from four real-kernel launches; A, B, C complex128 CUDA tensors, workspace uint8."""
    for t in (A, B, C):
        if t is not None and (t.dtype != torch.complex128 or not t.is_cuda):
            raise TypeError("b2_zgemm4m takes complex128 CUDA tensors")
    al = (c_double * 2)(complex(alpha).real, complex(alpha).imag)
    be = (c_double * 2)(complex(beta).real, complex(beta).imag)
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().b2_zgemm4m(_tr(transa), _tr(transb), m, n, k, al, _ptr(A), lda, _ptr(B), ldb, be, _ptr(C), ldc,
                          _ptr(workspace), wbytes, _stream())
    if check:
        _check("b2_zgemm4m", rc)
    return rc


def _tri(which, side, uplo, trans, diag, m, n, alpha, A, lda, B, ldb, check) -> int:
    dtype = next((t.dtype for t in (B, A) if t is not None), torch.float64)
    if dtype == torch.float64:
        name = f"b2_d{which}"
    elif dtype == torch.float32:
        name = f"b2_s{which}"
    else:
        raise TypeError(f"b2_{which} takes float64 or float32 tensors")
    for t in (A, B):
        if t is not None and (t.dtype != dtype or not t.is_cuda):
            raise TypeError(f"b2_{which} takes CUDA tensors of one dtype")
    rc = getattr(lib(), name)(_tr(side), _tr(uplo), _tr(trans), _tr(diag), m, n, alpha, _ptr(A), lda, _ptr(B), ldb,
                              _stream())
    if check:
        _check(name, rc)
    return rc


def b2_trmm(side, uplo, trans, diag, m, n, alpha, A, lda, B, ldb, check=True) -> int:
    """B := alpha*op(A)*B (side L) or alpha*B*op(A) (side R), A triangular; fp64 or fp32 by the tensors' dtype."""
    return _tri("trmm", side, uplo, trans, diag, m, n, alpha, A, lda, B, ldb, check)


def b2_trsm(side, uplo, trans, diag, m, n, alpha, A, lda, B, ldb, check=True) -> int:
    """Solve op(A)*X = alpha*B (side L) or X*op(A) = alpha*B (side R), A triangular; X overwrites B."""
    return _tri("trsm", side, uplo, trans, diag, m, n, alpha, A, lda, B, ldb, check)


def b2_gemm_splitk_auto(m, n, k) -> int:
    return lib().b2_gemm_splitk_auto(m, n, k)


def b2_gemm_splitk_workspace_bytes(dtype, m, n, k, splits=0) -> int:
    """dtype: torch.float64 / torch.float32."""
    return lib().b2_gemm_splitk_workspace_bytes(0 if dtype == torch.float64 else 1, m, n, k, splits)


def b2_gemm_splitk(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, splits=0, workspace=None,
                   check=True) -> int:
    """Split-K GEMM (fp64 or fp32 by the tensors' dtype); workspace: uint8 CUDA tensor or None."""
    if C.dtype == torch.float64:
        fn, name = lib().b2_dgemm_splitk, "b2_dgemm_splitk"
    elif C.dtype == torch.float32:
        fn, name = lib().b2_sgemm_splitk, "b2_sgemm_splitk"
    else:
        raise TypeError("b2_gemm_splitk takes float64 or float32 tensors")
    for t in (A, B, C):
        if t is not None and (t.dtype != C.dtype or not t.is_cuda):
            raise TypeError("b2_gemm_splitk takes CUDA tensors of one dtype")
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = fn(_tr(transa), _tr(transb), m, n, k, alpha, _ptr(A), lda, _ptr(B), ldb, beta, _ptr(C), ldc, splits,
            _ptr(workspace), wbytes, _stream())
    if check:
        _check(name, rc)
    return rc


def b2_zgemm3m_workspace_bytes(transa, transb, m, n, k) -> int:
    return lib().b2_zgemm3m_workspace_bytes(_tr(transa), _tr(transb), m, n, k)


def b2_zgemm3m(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, workspace, check=True) -> int:
    """Complex128 GEMM from three real-kernel launches (3M); same arguments as b2_zgemm4m."""
    for t in (A, B, C):
        if t is not None and (t.dtype != torch.complex128 or not t.is_cuda):
            raise TypeError("b2_zgemm3m takes complex128 CUDA tensors")
    al = (c_double * 2)(complex(alpha).real, complex(alpha).imag)
    be = (c_double * 2)(complex(beta).real, complex(beta).imag)
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = lib().b2_zgemm3m(_tr(transa), _tr(transb), m, n, k, al, _ptr(A), lda, _ptr(B), ldb, be, _ptr(C), ldc,
                          _ptr(workspace), wbytes, _stream())
    if check:
        _check("b2_zgemm3m", rc)
    return rc


ZGEMM4M_STATIC_BYTES = 6 << 20


def b2_zgemm4m_static(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, check=True) -> int:
    """b2_zgemm4m without a workspace argument, for callers that cannot allocate device memory.

    The scratch planes live in a ZGEMM4M_STATIC_BYTES array inside the library; problems that need more
    return B2_ERR_STATIC_LIMIT (1005).  Calls share that array: do not overlap them on the GPU."""
    for t in (A, B, C):
        if t is not None and (t.dtype != torch.complex128 or not t.is_cuda):
            raise TypeError("b2_zgemm4m_static takes complex128 CUDA tensors")
    al = (c_double * 2)(complex(alpha).real, complex(alpha).imag)
    be = (c_double * 2)(complex(beta).real, complex(beta).imag)
    rc = lib().b2_zgemm4m_static(_tr(transa), _tr(transb), m, n, k, al, _ptr(A), lda, _ptr(B), ldb, be, _ptr(C), ldc,
                                 _stream())
    if check:
        _check("b2_zgemm4m_static", rc)
    return rc


def b2_gemm_host_workspace_bytes(dtype, transa, transb, m, n, k) -> int:
    return lib().b2_gemm_host_workspace_bytes(dtype, _tr(transa), _tr(transb), m, n, k)


def _host_call(fn_name, want, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, workspace, check):
    for t in (A, B, C):
        if t is not None and (t.dtype != want or t.is_cuda):
            raise TypeError(f"{fn_name} takes {want} HOST tensors")
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = getattr(lib(), fn_name)(_tr(transa), _tr(transb), m, n, k, alpha, _ptr(A), lda, _ptr(B), ldb, beta, _ptr(C),
                                 ldc, _ptr(workspace), wbytes, _stream())
    if check:
        _check(fn_name, rc)
    return rc


def b2_dgemm_host(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, workspace, check=True) -> int:
    """b2_dgemm on HOST tensors (pinned for speed); copies in, computes on the GPU, copies C back."""
    return _host_call("b2_dgemm_host", torch.float64, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc,
                      workspace, check)


def b2_sgemm_host(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, workspace, check=True) -> int:
    """b2_sgemm on HOST tensors (pinned for speed); copies in, computes on the GPU, copies C back."""
    return _host_call("b2_sgemm_host", torch.float32, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc,
                      workspace, check)


def b2_model_throughput(rates, jobs) -> float:
    """Section 4: outer products per cycle of an instruction mix = min over pipelines of rate/jobs."""
    n = len(rates)
    if n != len(jobs):
        raise ValueError("rates and jobs must have the same length")
    r = (c_double * max(n, 1))(*rates)
    j = (c_double * max(n, 1))(*jobs)
    return lib().b2_model_throughput(n, r, j)


def b2_model_stalled_throughput(jobs: float, n_dependent: int, latency: float) -> float:
    return lib().b2_model_stalled_throughput(jobs, n_dependent, latency)


def b2_model_register_updates(r_total, mr, nr, v, r_a, r_r) -> int:
    """Section 5: floor((R_total - mr*nr/v - R_A) / R_R)."""
    out = c_int(0)
    _check("b2_model_register_updates", lib().b2_model_register_updates(r_total, mr, nr, v, r_a, r_r, ctypes.byref(out)))
    return out.value


def b2_model_enumerate(dtype: int, top: int = 16) -> str:
    """Ranked candidate micro-kernels/tiles of the pipeline model as a JSON string (host-only call)."""
    buf = ctypes.create_string_buffer(1 << 16)
    _check("b2_model_enumerate", lib().b2_model_enumerate(dtype, top, buf, len(buf)))
    return buf.value.decode()


def b2_model_predict_variant(dtype: int, variant: int):
    """(predicted fraction of pipe peak, JSON description) of a kernel variant from the pipeline model."""
    frac = c_double(0.0)
    buf = ctypes.create_string_buffer(1024)
    _check("b2_model_predict_variant", lib().b2_model_predict_variant(dtype, variant, ctypes.byref(frac), buf, len(buf)))
    return frac.value, buf.value.decode()


def b2_device_status() -> int:
    """Synchronise the current stream and return (and clear) the device status word: 0 or B2_ERR_TIMEOUT."""
    return lib().b2_device_status(_stream())


def b2_selftest_wait_timeout() -> int:
    """Enqueue the bounded-wait self-test kernel (the next b2_device_status then reports B2_ERR_TIMEOUT)."""
    return lib().b2_selftest_wait_timeout(_stream())


def b2_sgemm_tf32_workspace_bytes(terms: int, m: int, n: int, k: int) -> int:
    return lib().b2_sgemm_tf32_workspace_bytes(terms, m, n, k)


def b2_sgemm_tf32(terms, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, workspace, check=True) -> int:
    """fp32 GEMM on the tensor cores in TF32 (terms=1: b2_sgemm_tf32x1, terms=3: b2_sgemm_tf32x3); device tensors."""
    for t in (A, B, C):
        if t is not None and (t.dtype != torch.float32 or not t.is_cuda):
            raise TypeError("b2_sgemm_tf32 takes float32 CUDA tensors")
    fn = {1: lib().b2_sgemm_tf32x1, 3: lib().b2_sgemm_tf32x3}[terms]
    wbytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = fn(_tr(transa), _tr(transb), m, n, k, alpha, _ptr(A), lda, _ptr(B), ldb, beta, _ptr(C), ldc, _ptr(workspace),
            wbytes, _stream())
    if check:
        _check(f"b2_sgemm_tf32x{terms}", rc)
    return rc


def b2_sgemm_tf32x1(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, workspace, check=True) -> int:
    return b2_sgemm_tf32(1, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, workspace, check)


def b2_sgemm_tf32x3(transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, workspace, check=True) -> int:
    return b2_sgemm_tf32(3, transa, transb, m, n, k, alpha, A, lda, B, ldb, beta, C, ldc, workspace, check)


def b2_syrk(uplo, trans, n, k, alpha, A, lda, beta, C, ldc, check=True) -> int:
    """Symmetric rank-k update on the uplo triangle of C (b2_dsyrk / b2_ssyrk by dtype); device tensors."""
    if C is not None and C.dtype == torch.float32:
        fn, name = lib().b2_ssyrk, "b2_ssyrk"
    else:
        fn, name = lib().b2_dsyrk, "b2_dsyrk"
    for t in (A, C):
        if t is not None and (not t.is_cuda or (C is not None and t.dtype != C.dtype)):
            raise TypeError(f"{name} takes CUDA tensors of one dtype")
    rc = fn(_tr(uplo), _tr(trans), n, k, alpha, _ptr(A), lda, beta, _ptr(C), ldc, _stream())
    if check:
        _check(name, rc)
    return rc


def b2_gemm_strided_batched(transa, transb, m, n, k, alpha, A, lda, stride_a, B, ldb, stride_b, beta, C, ldc, stride_c,
                            batch, check=True) -> int:
    """`batch` GEMMs of one shape on strided operands (b2_dgemm_strided_batched / b2_sgemm_strided_batched)."""
    if C is not None and C.dtype == torch.float32:
        fn, name = lib().b2_sgemm_strided_batched, "b2_sgemm_strided_batched"
    else:
        fn, name = lib().b2_dgemm_strided_batched, "b2_dgemm_strided_batched"
    for t in (A, B, C):
        if t is not None and (not t.is_cuda or (C is not None and t.dtype != C.dtype)):
            raise TypeError(f"{name} takes CUDA tensors of one dtype")
    rc = fn(_tr(transa), _tr(transb), m, n, k, alpha, _ptr(A), lda, stride_a, _ptr(B), ldb, stride_b, beta, _ptr(C), ldc,
            stride_c, batch, _stream())
    if check:
        _check(name, rc)
    return rc
