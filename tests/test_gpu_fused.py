"""The sixteen-warp sweep kernel (far contractions fed by TMA beside the quadrant tasks on every SM) against
the CPU oracle.  It is not the default path (it measures slower than the eight-warp kernel); the test hook
forces it onto every shape its operands allow, so that ragged tiles, single rows / columns of tiles and
matrices with no far part at all go through it.  Z must be bit-exact against the oracle (nested Algorithm 5 on certified
inputs), E within 1e-9, runs repeatable bit for bit, and equal in Z to the eight-warp kernel."""
import numpy as np
import pytest
import torch

import oracle as O
from oracle import cref
from certify import MARGIN, certified_case
from paper_2607_27042_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def g():
    from paper_2607_27042_b200 import gptq2d
    return gptq2d


def _draw(m, n):
    def draw(seed):
        X, A, B = W.general_bases(m, n, seed)
        L, U, _, _ = O.feedback_factors(A, B)
        return X, L, U
    return draw


def _run(g, X, L, U, mode):
    try:
        g.gptq2d_internal_test_hook(4, mode)
        Z, E, mm, info = g.gptq2d_round(X, L, U, want_E=True, want_margin=True)
        torch.cuda.synchronize()
        g.check_info(info)
    finally:
        g.gptq2d_internal_test_hook(4, 0)
    return Z, E, float(mm.cpu()[0])


@pytest.mark.parametrize("m,n,seed", [(1, 1, 0), (64, 64, 1), (200, 330, 2), (515, 300, 3), (129, 1100, 4), (1100, 130, 5),
                                      (700, 900, 6), (1300, 1290, 7), (3, 1500, 8)])
def test_fused_kernel_forced_on_small_and_ragged_shapes(g, m, n, seed):
    (X, L, U), ref, _ = certified_case(_draw(m, n), cref.nested, seed)
    dX, dL, dU = (torch.from_numpy(a).cuda() for a in (X, L, U))
    Z, E, mm = _run(g, dX, dL, dU, 2)
    assert np.array_equal(Z.cpu().numpy().astype(np.int64), ref["Z"])
    assert np.max(np.abs(E.cpu().numpy() - ref["E"])) < 1e-9
    assert abs(mm - ref["margin"]) < 1e-9
    Z2, E2, mm2 = _run(g, dX, dL, dU, 2)
    assert torch.equal(Z, Z2) and torch.equal(E, E2) and mm == mm2
    Z0, E0, mm0 = _run(g, dX, dL, dU, 0)
    assert torch.equal(Z, Z0) and float((E - E0).abs().max()) < 1e-9


def test_fused_kernel_mid_size_with_library_factors(g):
    """Several waves of far parts (10 x 12 tiles, ragged), the library's own factors, objective."""
    for t in range(4):
        X, A, B = W.headline_like(1250, 1480, 21 + 1000 * t)
        L, U, _, _ = O.feedback_factors(A, B)
        ref = cref.nested(X, L, U)
        if ref["margin"] >= MARGIN:
            break
    else:
        pytest.fail("no certified seed")
    dX, dA, dB = (torch.from_numpy(a).cuda() for a in (X, A, B))
    Ld, Ud, _, _, finfo = g.gptq2d_factor(dA, dB)
    Z, E, mm = _run(g, dX, Ld, Ud, 2)
    g.check_info(finfo)
    Zh = Z.cpu().numpy().astype(np.int64)
    assert np.array_equal(Zh, ref["Z"])
    margin, Ecert = O.certificate_margin(X, Zh, L, U)
    assert margin >= MARGIN and abs(mm - margin) < 1e-9
    assert np.max(np.abs(E.cpu().numpy() - Ecert)) < 1e-8
    obj = float(g.gptq2d_objective(dX, Z, dA, dB).cpu()[0])
    want = O.objective(X, Zh, A, B)
    assert abs(obj - want) <= 1e-10 * want
    Z0, _, _ = _run(g, dX, Ld, Ud, 0)
    assert torch.equal(Z, Z0)


def test_fused_kernel_unaligned_factors_fall_back(g):
    """Odd leading dimensions cannot be described to the copy engine: the call must still be right."""
    (X, L, U), ref, _ = certified_case(_draw(300, 280), cref.nested, 31)
    Lp = torch.zeros((300, 301), dtype=torch.float64, device="cuda"); Lp[:, :300] = torch.from_numpy(L).cuda()
    Up = torch.zeros((280, 283), dtype=torch.float64, device="cuda"); Up[:, :280] = torch.from_numpy(U).cuda()
    Z, _, _ = _run(g, torch.from_numpy(X).cuda(), Lp[:, :300], Up[:, :280], 2)
    assert np.array_equal(Z.cpu().numpy().astype(np.int64), ref["Z"])
