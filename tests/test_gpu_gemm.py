"""The library's own fp64 product (the contraction the set-up, the objective and the far parts of the sweep
are made of) against numpy, in all four operand layouts, on shapes that span several 128 x 128 tiles with
ragged edges in every dimension, through both the TMA-fed kernel and the cp.async kernel.  Inputs are small
integers so that every product and partial sum is exact in fp64: the result must match bit for bit
whatever the summation order."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def g():
    from paper_2607_27042_b200 import gptq2d
    return gptq2d


@pytest.mark.parametrize("tma", [3, 1, 0])
@pytest.mark.parametrize("M,N,K", [(128, 128, 16), (256, 384, 512), (130, 257, 75), (1, 1, 1), (300, 100, 1000),
                                   (127, 129, 17), (513, 8, 260)])
def test_gemm_all_layouts_exact(g, tma, M, N, K):
    rng = np.random.default_rng(M * 1000003 + N * 1009 + K)
    try:
        g.gptq2d_internal_test_hook(3, tma)
        for transa in (False, True):
            for transb in (False, True):
                opA = rng.integers(-8, 9, size=(M, K)).astype(np.float64)
                opB = rng.integers(-8, 9, size=(K, N)).astype(np.float64)
                C0 = rng.integers(-8, 9, size=(M, N)).astype(np.float64)
                # leading dimensions: padded, even (the TMA path needs 16-byte row pitches)
                def padded(a):
                    r, c = a.shape
                    buf = torch.full((r, c + 6 + (c & 1)), 7.0, dtype=torch.float64, device="cuda")
                    buf[:, :c] = torch.from_numpy(np.ascontiguousarray(a)).cuda()
                    return buf[:, :c]
                dA = padded(opA.T if transa else opA)
                dB = padded(opB.T if transb else opB)
                dC = padded(C0)
                g.gptq2d_internal_gemm(dA, dB, dC, transa=transa, transb=transb, alpha=2.0, beta=-1.0)
                torch.cuda.synchronize()
                want = 2.0 * (opA @ opB) - C0
                assert np.array_equal(dC.cpu().numpy(), want), (transa, transb)
    finally:
        g.gptq2d_internal_test_hook(3, 1)


def test_gemm_odd_leading_dimension_takes_the_fallback(g):
    rng = np.random.default_rng(5)
    A = rng.integers(-4, 5, size=(200, 131)).astype(np.float64)
    B = rng.integers(-4, 5, size=(131, 77)).astype(np.float64)
    dA, dB = torch.from_numpy(A).cuda(), torch.from_numpy(B).cuda()        # pitches 131 and 77 doubles: not 16-byte
    dC = torch.zeros((200, 77), dtype=torch.float64, device="cuda")
    g.gptq2d_internal_gemm(dA, dB, dC)
    torch.cuda.synchronize()
    assert np.array_equal(dC.cpu().numpy(), A @ B)
