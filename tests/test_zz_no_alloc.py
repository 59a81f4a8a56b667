"""The allocation-free entry point, gptq2d_round_static, against gptq2d_round.

Collected last on purpose (file name): if it fails, a run that stops at the first failure has
already exercised every other test.  It must pass alone in a fresh process and after the rest of
the suite, so it makes no assumption about what the library's shared scratch array holds.

Who needs this entry point: code that is not allowed to allocate device memory at the point
where it rounds -- a step that is captured into a CUDA graph, a region of a framework that bans
raw cudaMalloc, a latency-critical loop -- and so has no workspace to pass.  The scratch is a
static device array inside the library; the test checks that two calls in a row, which share
that array and inherit its previous contents, both reproduce the workspace-based entry point.
"""
import numpy as np
import pytest
import torch

from paper_2607_27042_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _dev(a):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=torch.float64).cuda()


def test_static_workspace_entry_matches_workspace_entry_twice_in_a_row():
    from paper_2607_27042_b200 import gptq2d as g
    assert g.gptq2d_round_static_max_dim() == 512
    # two different problems, so that the second call really meets the first one's leftovers:
    # a ragged multi-tile one and the largest size the static array admits
    cases = [W.gaussian_like(200, 330, seed=5), W.headline_like(512, 512, seed=6)]
    # One small call up front: the first call on a device looks up the array's address, and the first
    # launch of a kernel may make the driver load its code; neither belongs to the calls measured below.
    I8 = torch.eye(8, dtype=torch.float64, device="cuda")
    g.gptq2d_round_static(torch.zeros((8, 8), dtype=torch.float64, device="cuda"), I8, I8,
                          torch.zeros((8, 8), dtype=torch.int32, device="cuda"),
                          E=torch.zeros((8, 8), dtype=torch.float64, device="cuda"),
                          min_margin=torch.zeros(1, dtype=torch.float64, device="cuda"))
    torch.cuda.synchronize()
    for X, A, B in cases:
        m, n = X.shape
        dX, dA, dB = _dev(X), _dev(A), _dev(B)
        L, U, _, _, finfo = g.gptq2d_factor(dA, dB)
        Zref, Eref, mref, info = g.gptq2d_round(dX, L, U, want_E=True, want_margin=True)
        torch.cuda.synchronize()
        g.check_info(finfo); g.check_info(info)
        # every buffer is made here, before the call: the entry point and its wrapper allocate nothing
        Z = torch.full((m, n), -1, dtype=torch.int32, device="cuda")
        E = torch.zeros((m, n), dtype=torch.float64, device="cuda")
        mm = torch.zeros(1, dtype=torch.float64, device="cuda")
        sinfo = torch.zeros(4, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated()
        g.gptq2d_round_static(dX, L, U, Z, E=E, min_margin=mm, info=sinfo)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before
        # The driver's own count sees a raw cudaMalloc too.  It is taken around a REPEAT of the same call: the
        # first launch of a grid of a new size may make the driver grow its internal buffers once, which is
        # not an allocation of the entry point; a cudaMalloc inside the entry point would show on every call.
        free_before, _ = torch.cuda.mem_get_info()
        Z.fill_(-1)
        g.gptq2d_round_static(dX, L, U, Z, E=E, min_margin=mm, info=sinfo)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after >= free_before, (free_before, free_after)
        g.check_info(sinfo)
        assert torch.equal(Z, Zref)                                   # integers: bit-exact
        assert float((E - Eref).abs().max()) <= 1e-9                  # same bar as the parity tests
        assert abs(float(mm[0]) - float(mref[0])) <= 1e-9


def test_static_workspace_entry_rejects_oversize():
    from paper_2607_27042_b200 import gptq2d as g
    n = 513
    X = torch.zeros((n, n), dtype=torch.float64, device="cuda")
    I = torch.eye(n, dtype=torch.float64, device="cuda")
    Z = torch.zeros((n, n), dtype=torch.int32, device="cuda")
    with pytest.raises(g.Gptq2dError) as e:
        g.gptq2d_round_static(X, I, I, Z)
    assert e.value.status == 9
    assert "static workspace" in g.status_string(9)
