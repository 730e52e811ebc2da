"""The per-bin complex contraction alone (Table 1, the Cgemm row) against the
oracle's plain sum, in both arithmetic modes and on ragged shapes."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

TOL = {1: 1e-4, 2: 5e-3}


def run(bins, M, N, K, math, seed=0, transA=False, transB=False, conjA=False, conjB=False):
    import torch
    import oracle
    import paper_1412_7580_b200 as fc
    rng = np.random.default_rng([14127580, 55, seed, bins, M, N, K])
    r4 = lambda v: (v + 3) // 4 * 4

    def operand(rows, trans, fill):
        """Logical [bins][rows][K] complex matrix, stored planar either as
        [2][bins][rows][ld>=K] or, transposed, as [2][bins][K][ld>=rows]."""
        re = rng.standard_normal((bins, rows, K), dtype=np.float32)
        im = rng.standard_normal((bins, rows, K), dtype=np.float32)
        if not trans:
            buf = np.full((2, bins, rows, r4(K)), fill, np.float32)   # padding must never be read as data
            buf[0, :, :, :K], buf[1, :, :, :K] = re, im
        else:
            buf = np.full((2, bins, K, r4(rows)), fill, np.float32)
            buf[0, :, :, :rows], buf[1, :, :, :rows] = re.transpose(0, 2, 1), im.transpose(0, 2, 1)
        return buf, re.astype(np.float64) + 1j * im.astype(np.float64)

    A, Ac = operand(M, transA, 1e30)
    B, Bc = operand(N, transB, -1e30)
    ldc = r4(N)
    Ad, Bd = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()
    Cd = torch.full((2, bins, M, ldc), float("nan"), device="cuda")
    status = torch.zeros(64, dtype=torch.int32, device="cuda")
    fc.fftconv_bin_contract(Ad, Bd, Cd, M, N, K, transA, transB, conjA, conjB, math=math,
                            status_word=status)
    torch.cuda.synchronize()
    assert int(status[0].item()) == 0
    C = Cd.cpu().numpy().astype(np.float64)
    got = C[0, :, :, :N] + 1j * C[1, :, :, :N]
    ref = oracle.bin_contract(Ac, Bc, conjA, conjB)
    assert np.all(np.isfinite(got.real)) and np.all(np.isfinite(got.imag))
    # padding columns of C (N..ldc-1) are scratch: untouched or zero, never data
    if ldc > N:
        pad = C[..., N:]
        assert np.all(np.isnan(pad) | (pad == 0))
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


# operand storage / conjugation as used by the three passes, plus the remaining combinations
FLAGS = [
    dict(transA=False, transB=False, conjA=False, conjB=True),    # fprop
    dict(transA=False, transB=True, conjA=False, conjB=False),    # bprop
    dict(transA=True, transB=True, conjA=True, conjB=False),      # accGrad
    dict(transA=True, transB=False, conjA=True, conjB=True),
]


@pytest.mark.parametrize("flags", FLAGS)
@pytest.mark.parametrize("math", [1, 2])
@pytest.mark.parametrize("shape", [(5, 128, 128, 64), (3, 130, 70, 33), (2, 37, 129, 100),
                                   (4, 64, 96, 128), (2, 8, 8, 4)])
def test_contraction_layouts_and_conjugates(shape, math, flags):
    assert run(*shape, math=math, seed=9, **flags) <= TOL[math]
