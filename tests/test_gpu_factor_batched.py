"""GPU parity of the batched set-up (gptq2d_factor_batched) against the CPU oracle's factors
(Section 3.1: L unit lower with (A^T A)^{-1} = L Lambda_L L^T, U unit upper with (B B^T)^{-1} = U^T Lambda_U U)."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2607_27042_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def g():
    from paper_2607_27042_b200 import gptq2d
    return gptq2d


def dev(a):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=torch.float64).cuda()


def check(g, shapes, seeds, with_identity=()):
    As, Bs, refs = [], [], []
    for b, ((m, n), seed) in enumerate(zip(shapes, seeds)):
        _, A, B = W.general_bases(m, n, seed)
        if b in with_identity:
            A = None
        As.append(None if A is None else dev(A))
        Bs.append(dev(B))
        refs.append(O.feedback_factors(np.eye(m) if A is None else A, B))
    Ls, Us, dLs, dUs, info = g.gptq2d_factor_batched(As, Bs, shapes=shapes)
    torch.cuda.synchronize()
    g.check_info(info)
    for b, (L, U, lamL, lamU) in enumerate(refs):
        gl, gu = Ls[b].cpu().numpy(), Us[b].cpu().numpy()
        sc = max(1.0, np.max(np.abs(L)), np.max(np.abs(U)))
        assert np.max(np.abs(gl - L)) < 1e-9 * sc, (b, shapes[b])
        assert np.max(np.abs(gu - U)) < 1e-9 * sc, (b, shapes[b])
        assert np.allclose(dLs[b].cpu().numpy(), 1.0 / lamL, rtol=1e-9), b
        assert np.allclose(dUs[b].cpu().numpy(), 1.0 / lamU, rtol=1e-9), b
        # exact ones on the diagonal, exact zeros in the opposite triangle
        assert np.array_equal(np.tril(gl), gl) and np.array_equal(np.diag(gl), np.ones(gl.shape[0]))
        assert np.array_equal(np.triu(gu), gu) and np.array_equal(np.diag(gu), np.ones(gu.shape[0]))
    return As, Bs, Ls, Us


def test_small_sides_of_every_size_class(g):
    shapes = [(1, 1), (1, 9), (9, 1), (17, 5), (64, 64), (100, 33), (128, 128), (127, 128), (33, 100), (2, 128)]
    check(g, shapes, seeds=range(len(shapes)), with_identity=(3,))


def test_mixed_small_and_large_sides_and_agreement_with_the_single_call(g):
    shapes = [(64, 64), (200, 90), (90, 300), (129, 129), (16, 16)]
    As, Bs, Ls, Us = check(g, shapes, seeds=[10, 11, 12, 13, 14])
    for b in range(len(shapes)):
        L1, U1, _, _, info = g.gptq2d_factor(As[b], Bs[b])
        torch.cuda.synchronize()
        g.check_info(info)
        assert float((L1 - Ls[b]).abs().max()) < 1e-10 * max(1.0, float(L1.abs().max()))
        assert float((U1 - Us[b]).abs().max()) < 1e-10 * max(1.0, float(U1.abs().max()))


def test_one_large_problem_among_small_ones_and_many_large_ones(g):
    """One problem of the blocked route takes gptq2d_factor's two-stream path; several of them are spread
    over a pool of streams (more problems than streams here, so slots are reused in order)."""
    check(g, [(64, 64), (300, 200), (5, 7)], seeds=[20, 21, 22])
    shapes = [(130 + 7 * b, 129 + 5 * b) for b in range(11)] + [(33, 33)]
    check(g, shapes, seeds=range(30, 30 + len(shapes)))


def test_two_hundred_config_c0_like_pairs_feed_the_batched_sweep(g):
    """The use the entry point exists for: factors of many 64 x 64 layers in one launch, then one batched sweep;
    every Z against the oracle's plain-C nested sweep where the certificate allows it."""
    from oracle import cref
    count = 200
    Xs, As, Bs, refs = [], [], [], []
    for b in range(count):
        X, A, B = W.make_config(0, seed=b)
        Xs.append(dev(X)); As.append(dev(A)); Bs.append(dev(B))
        refs.append((X, A, B))
    Ls, Us, _, _, finfo = g.gptq2d_factor_batched(As, Bs)
    Zs, _, mm, info = g.gptq2d_round_batched(Xs, Ls, Us, want_margin=True)
    torch.cuda.synchronize()
    g.check_info(finfo)
    g.check_info(info)
    checked = 0
    for b in range(0, count, 8):
        X, A, B = refs[b]
        L, U, _, _ = O.feedback_factors(A, B)
        ref = cref.nested(X, L, U)
        margin, _ = O.certificate_margin(X, ref["Z"], L, U)
        if margin >= 1e-9:
            assert np.array_equal(Zs[b].cpu().numpy().astype(np.int64), ref["Z"]), b
            assert abs(float(mm.cpu()[b]) - margin) < 1e-9
            checked += 1
    assert checked >= 15


def test_a_singular_basis_names_its_problem_and_the_others_are_still_factorised(g):
    shapes = [(20, 20), (30, 12), (40, 40)]
    As, Bs = [], []
    for b, (m, n) in enumerate(shapes):
        _, A, B = W.general_bases(m, n, 50 + b)
        if b == 1:
            A[:, 7] = 0.0                      # singular A: its Gram has a zero pivot
        As.append(dev(A)); Bs.append(dev(B))
    Ls, Us, _, _, info = g.gptq2d_factor_batched(As, Bs)
    torch.cuda.synchronize()
    vals = info.cpu().tolist()
    assert vals[0] == 5 and vals[2] == 0 and vals[3] == 1          # NOT_SPD, side A, problem 1
    for b in (0, 2):
        _, A, B = W.general_bases(*shapes[b], 50 + b)
        L, U, _, _ = O.feedback_factors(A, B)
        assert np.max(np.abs(Ls[b].cpu().numpy() - L)) < 1e-9 * max(1.0, np.max(np.abs(L)))
        assert np.max(np.abs(Us[b].cpu().numpy() - U)) < 1e-9 * max(1.0, np.max(np.abs(U)))


def test_the_multi_stream_set_up_is_bit_identical_to_the_one_stream_set_up(g):
    """With both bases given, gptq2d_factor runs the two sides on two streams and each side's chain of
    diagonal blocks ahead of its large updates on a third and fourth; with one basis it runs on the
    caller's stream alone.  Same kernels, same operands, so the outputs must agree bit for bit, run after
    run (a missing dependency between the streams would show up here)."""
    torch.manual_seed(3)
    for k, kb, reps in [(300, 337, 20), (640, 513, 10), (1500, 1200, 4)]:
        A = torch.randn(k, k, dtype=torch.float64, device="cuda") / k ** 0.5 + torch.eye(k, dtype=torch.float64, device="cuda")
        B = torch.randn(kb, kb, dtype=torch.float64, device="cuda") / kb ** 0.5 + torch.eye(kb, dtype=torch.float64, device="cuda")
        L0, _, dL0, _, i0 = g.gptq2d_factor(A, None, n=1)
        _, U0, _, dU0, i1 = g.gptq2d_factor(None, B, m=1)
        torch.cuda.synchronize()
        g.check_info(i0)
        g.check_info(i1)
        for _ in range(reps):
            L, U, dL, dU, info = g.gptq2d_factor(A, B)
            torch.cuda.synchronize()
            g.check_info(info)
            assert torch.equal(L, L0) and torch.equal(U, U0) and torch.equal(dL, dL0) and torch.equal(dU, dU0), k
