"""Host threads that make their FIRST calls into the library at the same time.

The per-device caches (shared-memory attributes of every kernel, tensor-map encoder, status-word address, scratch
address, SM count) are filled on first use, and every host thread keeps its own short memory of the selector's
choices.  The header promises that threads may race on those first calls.  A race can only be provoked in a
process that has not called the library yet, so the body of this test runs in a child process: four threads wait
at a barrier and then call different entry points (fp64 through TMA, fp32 with a cluster split, the complex entry
on the library's own scratch, the TF32 entry), each on its own stream, several times; every result must equal,
bit for bit, what the same call gives afterwards from one thread.  ctypes drops the interpreter lock during a call,
so the calls do overlap.
"""
import subprocess
import sys
import textwrap

import pytest

pytestmark = pytest.mark.gpu

CHILD = textwrap.dedent(
    """
    import sys, threading
    import torch
    from paper_1611_08035_b200 import binding as b2, synth

    b2.lib()  # loads the shared object; no entry point has run yet
    dev = torch.device("cuda")
    m, n, k = 520, 392, 1040  # ragged against every tile; 16-byte aligned columns for the TMA paths

    def inputs(dt, seed):
        return synth.gemm_inputs("N", "T", m, n, k, "int9", seed, dt, device=dev)

    Ad, Bd, Cd = inputs(torch.float64, 1), inputs(torch.float32, 2), inputs(torch.complex128, 3)
    mz = 96
    Az = synth.gemm_inputs("N", "N", mz, mz, mz, "int9", 4, torch.complex128, device=dev)
    ws32 = torch.empty(b2.b2_sgemm_tf32_workspace_bytes(1, m, n, k), dtype=torch.uint8, device=dev)

    def dgemm(out):
        A, lda, B, ldb, C, ldc = Ad
        b2.b2_dgemm("N", "T", m, n, k, 1.5, A, lda, B, ldb, 0.5, out, ldc)

    def sgemm(out):
        A, lda, B, ldb, C, ldc = Bd
        b2.b2_sgemm("N", "T", m, n, k, 1.5, A, lda, B, ldb, 0.5, out, ldc)

    def zgemm(out):
        A, lda, B, ldb, C, ldc = Az
        b2.b2_zgemm4m_static("N", "N", mz, mz, mz, 2 - 1j, A, lda, B, ldb, 0.5 + 0.5j, out, ldc)

    def tf32(out):
        A, lda, B, ldb, C, ldc = Bd
        b2.b2_sgemm_tf32x1("N", "T", m, n, k, 1.5, A, lda, B, ldb, 0.5, out, ldc, ws32)

    jobs = [(dgemm, Ad[4]), (sgemm, Bd[4]), (zgemm, Az[4]), (tf32, Bd[4])]
    gate = threading.Barrier(len(jobs))
    results, errors = [None] * len(jobs), []

    def work(i):
        fn, C0 = jobs[i]
        try:
            stream = torch.cuda.Stream()
            outs = []
            gate.wait()
            with torch.cuda.stream(stream):
                for _ in range(8):
                    out = C0.clone()
                    fn(out)
                    outs.append(out)
            stream.synchronize()
            results[i] = outs
        except Exception as exc:  # reported by the parent
            errors.append(f"thread {i}: {exc!r}")

    threads = [threading.Thread(target=work, args=(i,)) for i in range(len(jobs))]
    [t.start() for t in threads]
    [t.join() for t in threads]
    if errors:
        print("\\n".join(errors)); sys.exit(2)
    if b2.b2_device_status() != 0:
        print("device status word set"); sys.exit(3)
    for i, (fn, C0) in enumerate(jobs):  # the same calls, one thread, afterwards
        ref = C0.clone()
        fn(ref)
        torch.cuda.synchronize()
        for r, out in enumerate(results[i]):
            if not torch.equal(out.view(torch.uint8), ref.view(torch.uint8)):
                print(f"job {i}, call {r}: differs from the single-threaded result"); sys.exit(4)
    print("ok")
    """
)


def test_first_calls_from_four_threads_at_once():
    res = subprocess.run([sys.executable, "-c", CHILD], capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, f"child failed ({res.returncode}):\n{res.stdout[-2000:]}\n{res.stderr[-2000:]}"
    assert res.stdout.strip().endswith("ok")
