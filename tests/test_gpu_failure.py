"""Failure handling on the GPU without faulting, trapping or hanging it: the failure is made on the host.

1. A bounded device-side wait is made to run out: the pipelined host entry is told (test hook) not to
   announce its last copy step, and the wait for a copy step is given a limit of a few milliseconds.
   The tasks that need the step give up, the kernel returns normally with GPTQ2D_ERR_DEVICE_TIMEOUT and
   the code of that wait, both streams drain, and the very next sweep on the same context is correct.
2. The workspace needs no clearing by the caller: filled with NaN bit patterns before the call, the
   sweeps give the same Z and E bit for bit (what must start at zero the call clears itself, and the
   E / C buffers are written before they are read).
"""
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


def test_bounded_wait_runs_out_and_the_context_stays_usable(g):
    (X, L, U), ref, _ = certified_case(_draw(1100, 700), cref.nested, 77)
    hX, hL, hU = (torch.from_numpy(np.ascontiguousarray(a)).pin_memory() for a in (X, L, U))
    hZ = torch.zeros((1100, 700), dtype=torch.int32).pin_memory()
    # a good call first (creates the copy stream, loads the kernels)
    g.gptq2d_round_host(hX, hL, hU, hZ=hZ)
    assert np.array_equal(hZ.numpy().astype(np.int64), ref["Z"])
    try:
        g.gptq2d_internal_test_hook(2, 20000)          # ~ a few milliseconds of polling
        g.gptq2d_internal_test_hook(1, 1)              # withhold the last copy step of the next call
        with pytest.raises(g.Gptq2dError) as ei:
            g.gptq2d_round_host(hX, hL, hU, hZ=hZ)
    finally:
        g.gptq2d_internal_test_hook(2, 0)
        g.gptq2d_internal_test_hook(1, 0)
    assert ei.value.status == 8                        # GPTQ2D_ERR_DEVICE_TIMEOUT
    assert ei.value.info[0] == 8 and ei.value.info[1] == -6, ei.value.info      # the wait for a copy step
    assert ei.value.info[2] == 3 + 2 - 1               # the step that never came: the last of the 3 x 2 block grid
    torch.cuda.synchronize()                           # nothing of the failed call is left running
    # the context is intact: the same call, unhooked, is correct again, and so is a resident sweep
    hZ.fill_(-5)
    g.gptq2d_round_host(hX, hL, hU, hZ=hZ)
    assert np.array_equal(hZ.numpy().astype(np.int64), ref["Z"])
    Z, _, _, info = g.gptq2d_round(torch.from_numpy(X).cuda(), torch.from_numpy(L).cuda(), torch.from_numpy(U).cuda())
    torch.cuda.synchronize()
    g.check_info(info)
    assert np.array_equal(Z.cpu().numpy().astype(np.int64), ref["Z"])


def _poison(nbytes):
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    ws.view(torch.int64)[: nbytes // 8] = 0x7FF8DEADBEEF0001     # a quiet NaN in every double
    return ws


@pytest.mark.parametrize("m,n,seed", [(200, 330, 1), (515, 300, 2), (129, 1100, 3)])
def test_poisoned_workspace_single(g, m, n, seed):
    (X, L, U), ref, _ = certified_case(_draw(m, n), cref.nested, seed)
    dX, dL, dU = (torch.from_numpy(a).cuda() for a in (X, L, U))
    Z0, E0, m0, i0 = g.gptq2d_round(dX, dL, dU, want_E=True, want_margin=True)
    nbytes = (g.gptq2d_round_workspace_bytes(m, n) + 7) // 8 * 8
    Z1, E1, m1, i1 = g.gptq2d_round(dX, dL, dU, want_E=True, want_margin=True, workspace=_poison(nbytes))
    torch.cuda.synchronize()
    g.check_info(i0); g.check_info(i1)
    assert np.array_equal(Z0.cpu().numpy().astype(np.int64), ref["Z"])
    assert torch.equal(Z0, Z1) and torch.equal(E0, E1) and float(m0[0]) == float(m1[0])


def test_poisoned_workspace_batched(g):
    shapes = [(64, 64), (200, 330), (130, 127), (300, 515)]
    batch = [certified_case(_draw(m, n), cref.nested, 10 + k)[0] for k, (m, n) in enumerate(shapes)]
    Xs = [torch.from_numpy(x).cuda() for x, _, _ in batch]
    Ls = [torch.from_numpy(l).cuda() for _, l, _ in batch]
    Us = [torch.from_numpy(u).cuda() for _, _, u in batch]
    Z0, E0, m0, i0 = g.gptq2d_round_batched(Xs, Ls, Us, want_E=True, want_margin=True)
    nbytes = (g.gptq2d_round_batched_workspace_bytes(Xs, Ls, Us, Z0, E0) + 7) // 8 * 8
    Z1, E1, m1, i1 = g.gptq2d_round_batched(Xs, Ls, Us, want_E=True, want_margin=True, workspace=_poison(nbytes))
    torch.cuda.synchronize()
    g.check_info(i0); g.check_info(i1)
    for b in range(len(shapes)):
        assert torch.equal(Z0[b], Z1[b]) and torch.equal(E0[b], E1[b]), shapes[b]
    assert torch.equal(m0, m1)
