"""The seeded input generator: splitmix64 against an independent big-integer implementation, determinism,
value ranges, leading-dimension independence, poison padding."""
import numpy as np
import torch

from paper_1611_08035_b200 import synth

M64 = (1 << 64) - 1


def splitmix_py(seed, i):
    z = (seed * 0x9E3779B97F4A7C15 + (i + 1) * 0x9E3779B97F4A7C15) & M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


def test_splitmix64_matches_big_integer_reference():
    idx = torch.tensor([0, 1, 2, 3, 1000, 2 ** 40 + 7], dtype=torch.int64)
    for seed in (0, 1, 1234567, 2 ** 63 + 11):
        got = synth.splitmix64(seed, idx).tolist()
        for i, g in zip(idx.tolist(), got):
            assert g & M64 == splitmix_py(seed, i)
    # the well-known first output of splitmix64 started from state 0
    z = [(synth.splitmix64(0, torch.tensor([0], dtype=torch.int64)).item()) & M64]
    assert z[0] == splitmix_py(0, 0) == 0xE220A8397B1DCDAF


def test_distributions_and_layout():
    A = synth.matrix(50, 40, 53, "uniform", 3).numpy().reshape(40, 53)
    assert np.all(np.isnan(A[:, 50:])) and np.all((A[:, :50] >= -1) & (A[:, :50] < 1))
    B = synth.matrix(50, 40, 50, "uniform", 3).numpy().reshape(40, 50)
    assert np.array_equal(A[:, :50], B)  # values do not depend on ld
    C = synth.matrix(50, 40, 64, "uniform", 3, chunk_cols=7).numpy().reshape(40, 64)
    assert np.array_equal(A[:, :50], C[:, :50])  # nor on chunking
    I = synth.matrix(300, 300, 300, "int9", 5).numpy()
    assert set(np.unique(I)) == set(float(v) for v in range(-4, 5))
    N = synth.matrix(400, 400, 400, "normal", 6).numpy()
    assert abs(N.mean()) < 0.02 and abs(N.std() - 1) < 0.02 and np.all(np.isfinite(N))
    F = synth.matrix(50, 40, 50, "uniform", 3, dtype=torch.float32).numpy().reshape(40, 50)
    assert np.array_equal(F, B.astype(np.float32))
    Z = synth.matrix(5, 4, 6, "uniform", 3, dtype=torch.complex128).numpy().reshape(4, 6)
    assert np.array_equal(Z[:, :5].real, synth.matrix(5, 4, 5, "uniform", 3).numpy().reshape(4, 5))
    assert np.array_equal(Z[:, :5].imag, synth.matrix(5, 4, 5, "uniform", 4).numpy().reshape(4, 5))
    S = synth.matrix(5, 4, 8, "uniform", 3, poison=synth.C_SENTINEL).numpy().reshape(4, 8)
    assert np.all(S[:, 5:] == synth.C_SENTINEL)
    assert np.float32(synth.C_SENTINEL) == synth.C_SENTINEL


def test_padded_ld_and_shapes():
    assert synth.padded_ld(1001) == 1027 and synth.padded_ld(999) == 1027 and synth.padded_ld(1003) == 1027
    assert synth.padded_ld(1024) == 1027 and synth.padded_ld(1) == 35
    assert synth.operand_shapes("N", "T", 3, 4, 5) == ((3, 5), (4, 5))
    assert synth.operand_shapes("T", "N", 3, 4, 5) == ((5, 3), (5, 4))
    A, lda, B, ldb, C, ldc = synth.gemm_inputs("T", "N", 3, 4, 5, "uniform", 1, c_dist="zero", ldc=6)
    assert (lda, ldb, ldc) == (5, 5, 6) and A.numel() == 15 and B.numel() == 20 and C.numel() == 24
    Cv = C.view(4, 6)
    assert (Cv[:, :3] == 0).all() and (Cv[:, 3:] == synth.C_SENTINEL).all()
