"""GPU parity of the reverse-order entry points (the same rounding taken from the last row and
column, Section 2 of the paper) against the CPU oracle's own reverse-order functions."""
import numpy as np
import pytest
import torch

import oracle as O
from oracle import cref
from paper_2607_27042_b200 import workloads as W

pytestmark = pytest.mark.gpu

MARGIN = 1e-9


@pytest.fixture(scope="module")
def g():
    from paper_2607_27042_b200 import gptq2d
    return gptq2d


def dev(a, dtype=torch.float64):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=dtype).cuda()


@pytest.mark.parametrize("m,n,seed", [(1, 1, 0), (1, 9, 1), (9, 1, 2), (8, 8, 3), (17, 5, 4), (40, 33, 5)])
def test_small_against_the_literal_reverse_sweep(g, m, n, seed):
    X, A, B = W.general_bases(m, n, seed)
    Lr, Ur, lamL, lamU = O.feedback_factors_reverse(A, B)
    ref = O.sweep_gptq2d_reverse(X, Lr, Ur)
    if ref["margin"] < MARGIN:
        pytest.skip("seed not certified")
    Z, E, mm, info = g.gptq2d_round_reverse(dev(X), dev(Lr), dev(Ur), want_E=True, want_margin=True)
    torch.cuda.synchronize()
    g.check_info(info)
    assert np.array_equal(Z.cpu().numpy().astype(np.int64), ref["Z"])
    assert np.max(np.abs(E.cpu().numpy() - ref["E"])) < 1e-9
    assert abs(float(mm.cpu()[0]) - ref["margin"]) < 1e-9
    # the factors, from the bases
    gLr, gUr, gdL, gdU, finfo = g.gptq2d_factor_reverse(dev(A), dev(B))
    torch.cuda.synchronize()
    g.check_info(finfo)
    sc = max(1.0, np.max(np.abs(Lr)), np.max(np.abs(Ur)))
    assert np.max(np.abs(gLr.cpu().numpy() - Lr)) < 1e-9 * sc
    assert np.max(np.abs(gUr.cpu().numpy() - Ur)) < 1e-9 * sc
    assert np.allclose(gdL.cpu().numpy(), 1.0 / lamL, rtol=1e-9)
    assert np.allclose(gdU.cpu().numpy(), 1.0 / lamU, rtol=1e-9)
    assert np.array_equal(np.triu(gLr.cpu().numpy()), gLr.cpu().numpy())        # exact zeros below
    assert np.array_equal(np.tril(gUr.cpu().numpy()), gUr.cpu().numpy())        # exact zeros above


@pytest.mark.parametrize("m,n,seed", [(130, 127, 0), (300, 515, 1), (700, 260, 2)])
def test_mid_size_against_the_reverse_certificate(g, m, n, seed):
    """Several tiles, ragged tails.  The oracle's Z comes from its plain-C nested sweep on the
    index-reversed problem (the identity the pins establish); the reverse certificate, which uses
    neither, then certifies the GPU's Z on the original problem."""
    X, A, B = W.general_bases(m, n, seed)
    Lr, Ur, _, _ = O.feedback_factors_reverse(A, B)
    ref = cref.nested(np.ascontiguousarray(X[::-1, ::-1]), np.ascontiguousarray(Lr[::-1, ::-1]),
                      np.ascontiguousarray(Ur[::-1, ::-1]))
    Zref = ref["Z"][::-1, ::-1]
    margin, Eref = O.certificate_margin_reverse(X, Zref, Lr, Ur)
    if margin < MARGIN:
        pytest.skip("seed not certified")
    gLr, gUr, _, _, finfo = g.gptq2d_factor_reverse(dev(A), dev(B))
    Z, E, mm, info = g.gptq2d_round_reverse(dev(X), gLr, gUr, want_E=True, want_margin=True)
    torch.cuda.synchronize()
    g.check_info(finfo)
    g.check_info(info)
    Zh = Z.cpu().numpy().astype(np.int64)
    assert np.array_equal(Zh, Zref)
    gm, Ecert = O.certificate_margin_reverse(X, Zh, Lr, Ur)
    assert gm >= MARGIN
    assert np.max(np.abs(E.cpu().numpy() - Ecert)) < 1e-8
    assert abs(float(mm.cpu()[0]) - margin) < 1e-8
    # and it is not the forward rounding
    L, U, _, _ = O.feedback_factors(A, B)
    Zf, _, _, finfo2 = g.gptq2d_round(dev(X), dev(L), dev(U))
    torch.cuda.synchronize()
    assert not np.array_equal(Zf.cpu().numpy(), Zh)


def test_strided_outputs_and_identity_bases(g):
    m, n = 70, 90
    X, A, B = W.general_bases(m, n, 9)
    # A = B = I: both orders are plain round-to-nearest
    Lr, Ur, _, _, finfo = g.gptq2d_factor_reverse(None, None, m=m, n=n)
    torch.cuda.synchronize()
    g.check_info(finfo)
    assert torch.equal(Lr, torch.eye(m, dtype=torch.float64, device="cuda"))
    assert torch.equal(Ur, torch.eye(n, dtype=torch.float64, device="cuda"))
    Zbig = torch.full((m, n + 7), -3, dtype=torch.int32, device="cuda")
    Z, _, _, info = g.gptq2d_round_reverse(dev(X), Lr, Ur, Z=Zbig[:, :n])
    torch.cuda.synchronize()
    g.check_info(info)
    assert np.array_equal(Zbig[:, :n].cpu().numpy(), np.rint(X).astype(np.int32))
    assert bool((Zbig[:, n:] == -3).all())


@pytest.mark.parametrize("m,n,seed", [(17, 5, 0), (200, 330, 1), (515, 300, 2)])
def test_fp32_stored_inputs_give_the_exact_trajectory_of_the_rounded_data(g, m, n, seed):
    """gptq2d_round_f32in: inputs kept in fp32, arithmetic in fp64.  The oracle is the fp64 oracle on the
    fp32-rounded data (exactly representable in fp64), so Z must be bit-exact against it."""
    X, A, B = W.general_bases(m, n, seed)
    L, U, _, _ = O.feedback_factors(A, B)
    X32, L32, U32 = (a.astype(np.float32) for a in (X, L, U))
    Xw, Lw, Uw = (a.astype(np.float64) for a in (X32, L32, U32))
    ref = cref.nested(Xw, Lw, Uw)
    margin, Eref = O.certificate_margin(Xw, ref["Z"], Lw, Uw)
    if margin < MARGIN:
        pytest.skip("seed not certified")
    Z, E, mm, info = g.gptq2d_round_f32in(torch.from_numpy(X32).cuda(), torch.from_numpy(L32).cuda(),
                                          torch.from_numpy(U32).cuda(), want_E=True, want_margin=True)
    torch.cuda.synchronize()
    g.check_info(info)
    assert np.array_equal(Z.cpu().numpy().astype(np.int64), ref["Z"])
    assert np.max(np.abs(E.cpu().numpy() - Eref)) < 1e-9
    assert abs(float(mm.cpu()[0]) - margin) < 1e-9
