"""GPU parity of the blocked sweep (Algorithm 4, Section 4 "Blocked GPTQ-2D") against the CPU oracle.

Small sizes: against the oracle's own Algorithm 4 and its literal Algorithm 3 (E element by element).
Mid sizes (several flush tiles, ragged tails, bands that leave the matrix on either side): Z against
the oracle's plain-C nested sweep, E and the margin against the integer-matrix certificate."""
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
def test_small_against_the_oracles_blocked_and_literal_sweeps(g, m, n, seed):
    X, A, B = W.general_bases(m, n, seed)
    L, U, _, _ = O.feedback_factors(A, B)
    ref = O.sweep_gptq2d(X, L, U)
    if ref["margin"] < MARGIN:
        pytest.skip("seed not certified")
    for w in sorted({1, 2, 3, 7, 16, min(64, m + n - 1), 64}):
        blk = O.sweep_blocked(X, L, U, w)
        assert np.array_equal(blk["Z"], ref["Z"])
        Z, E, mm, info = g.gptq2d_round_blocked(dev(X), dev(L), dev(U), w, want_E=True, want_margin=True)
        torch.cuda.synchronize()
        g.check_info(info)
        assert np.array_equal(Z.cpu().numpy().astype(np.int64), ref["Z"]), w
        assert np.max(np.abs(E.cpu().numpy() - blk["E"])) < 1e-10, w
        assert abs(float(mm.cpu()[0]) - ref["margin"]) < 1e-10, w


@pytest.mark.parametrize("m,n,seed,widths", [
    (130, 127, 0, (1, 5, 32, 64)),
    (300, 515, 1, (8, 24, 64)),
    (700, 260, 2, (16, 63, 64)),
    (64, 1030, 3, (64,)),
    (1030, 64, 4, (33, 64)),
])
def test_mid_size_against_the_certificate(g, m, n, seed, widths):
    X, A, B = W.general_bases(m, n, seed)
    L, U, _, _ = O.feedback_factors(A, B)
    ref = cref.nested(X, L, U)
    margin, Eref = O.certificate_margin(X, ref["Z"], L, U)
    if margin < MARGIN:
        pytest.skip("seed not certified")
    dX, dL, dU = dev(X), dev(L), dev(U)
    for w in widths:
        Z, E, mm, info = g.gptq2d_round_blocked(dX, dL, dU, w, want_E=True, want_margin=True)
        torch.cuda.synchronize()
        g.check_info(info)
        Zh = Z.cpu().numpy().astype(np.int64)
        assert np.array_equal(Zh, ref["Z"]), w
        assert np.max(np.abs(E.cpu().numpy() - Eref)) < 1e-8, w
        assert abs(float(mm.cpu()[0]) - margin) < 1e-8, w


def test_config_c1_and_garbage_in_the_unused_triangles(g):
    """c1 (256 x 256) for widths 32 and 64; the upper part of L and the lower part of U, diagonals
    included, are never read, so NaNs there change nothing."""
    X, A, B = W.make_config(1, seed=0)
    L, U, _, _ = O.feedback_factors(A, B)
    ref = cref.nested(X, L, U)
    margin, _ = O.certificate_margin(X, ref["Z"], L, U)
    assert margin >= MARGIN
    Lg = L.copy()
    Ug = U.copy()
    Lg[np.triu_indices(L.shape[0])] = np.nan
    Ug[np.tril_indices(U.shape[0])] = np.nan
    for w in (32, 64):
        Z, _, mm, info = g.gptq2d_round_blocked(dev(X), dev(Lg), dev(Ug), w, want_margin=True)
        torch.cuda.synchronize()
        g.check_info(info)
        assert np.array_equal(Z.cpu().numpy().astype(np.int64), ref["Z"])
        assert abs(float(mm.cpu()[0]) - margin) < 1e-9


def test_strided_operands_and_untouched_padding(g):
    m, n = 150, 200
    X, A, B = W.general_bases(m, n, 11)
    L, U, _, _ = O.feedback_factors(A, B)
    ref = cref.nested(X, L, U)
    margin, _ = O.certificate_margin(X, ref["Z"], L, U)
    if margin < MARGIN:
        pytest.skip("seed not certified")
    Xb = torch.full((m, n + 3), 7.0, dtype=torch.float64, device="cuda")
    Xb[:, :n] = dev(X)
    Lb = torch.zeros((m, m + 5), dtype=torch.float64, device="cuda")
    Lb[:, :m] = dev(L)
    Zb = torch.full((m, n + 7), -3, dtype=torch.int32, device="cuda")
    Eb = torch.full((m, n + 2), 9.0, dtype=torch.float64, device="cuda")
    _, _, _, info = g.gptq2d_round_blocked(Xb[:, :n], Lb[:, :m], dev(U), 48, Z=Zb[:, :n], E=Eb[:, :n])
    torch.cuda.synchronize()
    g.check_info(info)
    assert np.array_equal(Zb[:, :n].cpu().numpy().astype(np.int64), ref["Z"])
    assert bool((Zb[:, n:] == -3).all()) and bool((Eb[:, n:] == 9.0).all())


def test_width_out_of_range_and_data_errors(g):
    X = torch.zeros((4, 4), dtype=torch.float64, device="cuda")
    I4 = torch.eye(4, dtype=torch.float64, device="cuda")
    assert g.gptq2d_round_blocked_workspace_bytes(4, 4, 0) == 0
    assert g.gptq2d_round_blocked_workspace_bytes(4, 4, g.BLOCKED_MAX_WIDTH + 1) == 0
    for w in (0, g.BLOCKED_MAX_WIDTH + 1):
        with pytest.raises(g.Gptq2dError):
            g.gptq2d_round_blocked(X, I4, I4, w, workspace=torch.empty(1 << 20, dtype=torch.uint8, device="cuda"))
    Xn = X.clone()
    Xn[2, 1] = float("nan")
    _, _, _, info = g.gptq2d_round_blocked(Xn, I4, I4, 2)
    torch.cuda.synchronize()
    vals = info.cpu().tolist()
    assert vals[0] == 6 and (vals[1], vals[2]) == (2, 1)
    Xo = X.clone()
    Xo[3, 3] = 3e9
    _, _, _, info = g.gptq2d_round_blocked(Xo, I4, I4, 64)
    torch.cuda.synchronize()
    vals = info.cpu().tolist()
    assert vals[0] == 7 and (vals[1], vals[2]) == (3, 3)
