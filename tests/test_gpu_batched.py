"""GPU parity of the batched sweep (many matrices, one launch) through the C ABI.

Each matrix of a batch must get exactly what Algorithm 3 gives it alone: Z is compared bit for
bit with the CPU oracle (quartic definition for the small ones, nested Algorithm 5 plus the
certificate for the larger ones) and, as a second check, with the single-matrix entry point.
"""
import numpy as np
import pytest
import torch

import oracle as O
from oracle import cref
from paper_2607_27042_b200 import workloads as W
from certify import MARGIN, certified_case

pytestmark = pytest.mark.gpu



@pytest.fixture(scope="module")
def g():
    from paper_2607_27042_b200 import gptq2d
    return gptq2d


def dev(a, dtype=torch.float64):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=dtype).cuda()


def _draw(m, n):
    def draw(seed):
        X, A, B = W.general_bases(m, n, seed)
        L, U, _, _ = O.feedback_factors(A, B)
        return X, L, U
    return draw


def make_batch(shapes, seed0, oracle=None):
    """One certified input per shape: the oracle alone (quartic definition up to 4096 entries per side
    product, nested Algorithm 5 above) picks the first seed of seed0 + k, + 1000, ... that passes."""
    out = []
    for k, (m, n) in enumerate(shapes):
        orc = oracle or (cref.vec_sweep if m * n <= 70000 else cref.nested)
        inputs, ref, _ = certified_case(_draw(m, n), orc, seed0 + k)
        out.append(inputs)
    return out


def run_batched(g, batch, want_E=True):
    Xs = [dev(x) for x, _, _ in batch]
    Ls = [dev(l) for _, l, _ in batch]
    Us = [dev(u) for _, _, u in batch]
    Zs, Es, mm, info = g.gptq2d_round_batched(Xs, Ls, Us, want_E=want_E, want_margin=True)
    torch.cuda.synchronize()
    g.check_info(info)
    return ([z.cpu().numpy().astype(np.int64) for z in Zs],
            [e.cpu().numpy() for e in Es] if Es is not None else None, mm.cpu().numpy())


def test_mixed_shapes_bit_exact_against_the_quartic_oracle(g):
    shapes = [(64, 64), (1, 1), (1, 9), (9, 1), (17, 5), (65, 63), (100, 130), (129, 257), (200, 75), (8, 8),
              (130, 127), (256, 256)]
    batch = make_batch(shapes, seed0=100)
    Zs, Es, mm = run_batched(g, batch)
    for b, (X, L, U) in enumerate(batch):
        ref = cref.vec_sweep(X, L, U)
        assert ref["margin"] >= MARGIN               # make_batch certified it
        assert abs(mm[b] - ref["margin"]) < 1e-9, b
        assert np.array_equal(Zs[b], ref["Z"]), (b, shapes[b])
        assert np.max(np.abs(Es[b] - ref["E"])) < 1e-9, b


def test_batch_equals_single_calls_and_certificate_at_mid_size(g):
    # several tile-waves per matrix, ragged tails, different shapes in flight at once
    shapes = [(300, 515), (515, 300), (384, 384), (130, 1100), (700, 3), (257, 640)]
    batch = make_batch(shapes, seed0=200)
    Zs, Es, mm = run_batched(g, batch)
    for b, (X, L, U) in enumerate(batch):
        ref = cref.nested(X, L, U)
        margin, _ = O.certificate_margin(X, ref["Z"], L, U)
        assert margin >= MARGIN, (b, shapes[b])
        assert np.array_equal(Zs[b], ref["Z"]), (b, shapes[b])
        assert O.certificate_margin(X, Zs[b], L, U)[0] >= MARGIN
        Z1, E1, m1, info = g.gptq2d_round(dev(X), dev(L), dev(U), want_E=True, want_margin=True)
        torch.cuda.synchronize()
        g.check_info(info)
        assert np.array_equal(Z1.cpu().numpy(), Zs[b])
        assert np.array_equal(E1.cpu().numpy(), Es[b])          # same arithmetic, same order
        assert float(m1.cpu()[0]) == mm[b]


def test_many_small_matrices_and_repeatability(g):
    shapes = [(64, 64)] * 150 + [(40, 200)] * 30 + [(128, 128)] * 20
    batch = make_batch(shapes, seed0=1000)
    Zs, _, mm = run_batched(g, batch, want_E=False)
    Zs2, _, mm2 = run_batched(g, batch, want_E=False)
    for b, (X, L, U) in enumerate(batch):
        assert np.array_equal(Zs[b], Zs2[b])
        assert mm[b] == mm2[b]
        if b % 10 == 0:
            assert np.array_equal(Zs[b], cref.vec_sweep(X, L, U)["Z"]), b
        else:
            assert O.certificate_margin(X, Zs[b], L, U)[0] >= MARGIN, b


def test_c1_replicas_with_strides_and_views(g):
    # the batch may be views into shared allocations (strided rows), as a layer stack would be
    X, A, B = W.make_config(1, seed=0)
    L, U, _, _ = O.feedback_factors(A, B)
    ref = cref.vec_sweep(X, L, U)
    assert ref["margin"] >= MARGIN
    k = 5
    Xbig = torch.zeros((k, 256, 300), dtype=torch.float64, device="cuda")
    Zbig = torch.zeros((k, 256, 272), dtype=torch.int32, device="cuda")
    Xbig[:, :, :256] = dev(X)
    dL, dU = dev(L), dev(U)
    Xs = [Xbig[b, :, :256] for b in range(k)]
    Zs = [Zbig[b, :, :256] for b in range(k)]
    _, _, mm, info = g.gptq2d_round_batched(Xs, [dL] * k, [dU] * k, Zs=Zs, want_margin=True)
    torch.cuda.synchronize()
    g.check_info(info)
    for b in range(k):
        assert np.array_equal(Zbig[b, :, :256].cpu().numpy(), ref["Z"])
        assert int(Zbig[b, :, 256:].abs().max()) == 0
        assert abs(float(mm[b]) - ref["margin"]) < 1e-9


def test_data_error_names_the_matrix(g):
    shapes = [(64, 64), (100, 130), (200, 75), (65, 63)]
    batch = make_batch(shapes, seed0=300)
    bad = 2
    batch[bad][0][150, 40] = np.nan
    Xs = [dev(x) for x, _, _ in batch]
    Ls = [dev(l) for _, l, _ in batch]
    Us = [dev(u) for _, _, u in batch]
    _, _, _, info = g.gptq2d_round_batched(Xs, Ls, Us)
    torch.cuda.synchronize()
    vals = info.cpu().tolist()
    assert vals[0] == 6                         # NONFINITE
    assert vals[3] == bad and vals[1] == 150 and vals[2] == 40
    with pytest.raises(g.Gptq2dError):
        g.check_info(info)
    # the library stays usable afterwards
    good = make_batch([(64, 64), (65, 63)], seed0=400)
    Zs, _, _ = run_batched(g, good)
    for b, (X, L, U) in enumerate(good):
        assert np.array_equal(Zs[b], cref.vec_sweep(X, L, U)["Z"])
