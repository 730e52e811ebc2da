"""The per-bin complex contraction alone (Table 1, the Cgemm row) against the
oracle's plain sum, in both arithmetic modes and on ragged shapes."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = {1: 1e-4, 2: 5e-3}


def run(bins, M, N, K, math, seed=0):
    import torch
    import oracle
    import paper_1412_7580_b200 as fc
    rng = np.random.default_rng([14127580, 55, seed, bins, M, N, K])
    lda = ldb = (K + 3) // 4 * 4
    ldc = (N + 3) // 4 * 4
    A = np.zeros((bins, 2, M, lda), np.float32)
    B = np.zeros((bins, 2, N, ldb), np.float32)
    A[..., :K] = rng.standard_normal((bins, 2, M, K), dtype=np.float32)
    B[..., :K] = rng.standard_normal((bins, 2, N, K), dtype=np.float32)
    # padding columns hold garbage that must never be read as data
    A[..., K:] = 1e30
    B[..., K:] = -1e30
    Ad, Bd = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    Cd = torch.full((bins, 2, M, ldc), float("nan"), device="cuda")
    status = torch.zeros(64, dtype=torch.int32, device="cuda")
    fc.fftconv_bin_contract(Ad, Bd, Cd, K, math=math, status_word=status)
    torch.cuda.synchronize()
    assert int(status[0].item()) == 0
    C = Cd.cpu().numpy().astype(np.float64)
    got = C[:, 0, :, :N] + 1j * C[:, 1, :, :N]
    Ac = A[:, 0, :, :K].astype(np.float64) + 1j * A[:, 1, :, :K].astype(np.float64)
    Bc = B[:, 0, :, :K].astype(np.float64) + 1j * B[:, 1, :, :K].astype(np.float64)
    ref = oracle.bin_contract(Ac, Bc, False, False)
    assert np.all(np.isfinite(got.real)) and np.all(np.isfinite(got.imag))
    # columns beyond N in the padded leading dimension stay untouched
    if ldc > N:
        assert np.all(np.isnan(C[..., N:]))
    return float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))


SHAPES = [
    # bins, M, N, K
    (3, 8, 8, 4), (5, 128, 128, 32), (7, 128, 64, 64), (4, 128, 256, 96), (2, 64, 64, 128),
    (3, 130, 70, 33), (2, 1, 1, 1), (9, 37, 129, 100), (2, 384, 384, 128), (300, 32, 48, 16),
    (2, 256, 96, 128), (1, 128, 384, 384),
]


@pytest.mark.parametrize("shape", SHAPES)
def test_contraction_fp32(shape):
    assert run(*shape, math=1) <= TOL[1]


@pytest.mark.parametrize("shape", SHAPES)
def test_contraction_tf32_tensor_cores(shape):
    assert run(*shape, math=2) <= TOL[2]


def test_tf32_many_tiles_per_cta():
    # more tiles than SMs: every CTA walks several tiles through both accumulator buffers
    assert run(700, 128, 128, 64, math=2, seed=3) <= TOL[2]
