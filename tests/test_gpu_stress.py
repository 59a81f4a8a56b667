"""Seeded random shapes through the tiled sweep: run-to-run bit-identity (a missing fence or a race in
the streamed hand-over between quadrants would break it), agreement with the untiled Algorithm-3
kernel (an independent implementation, itself checked against the oracle elsewhere), and the CPU
oracle on a subset."""
import numpy as np
import pytest
import torch

import oracle as O
from oracle import cref
from certify import MARGIN

pytestmark = pytest.mark.gpu



@pytest.fixture(scope="module")
def g():
    from paper_2607_27042_b200 import gptq2d
    return gptq2d


def make(rng, m, n):
    X = rng.standard_normal((m, n)) * 4
    L = np.tril(rng.standard_normal((m, m)) * (0.3 / np.sqrt(m)), -1) + np.eye(m)
    U = np.triu(rng.standard_normal((n, n)) * (0.3 / np.sqrt(n)), 1) + np.eye(n)
    return X, L, U


def make_certified(rng, m, n):
    """Draws until the oracle alone (nested Algorithm 5) certifies the input: every shape is checked."""
    for _ in range(8):
        X, L, U = make(rng, m, n)
        ref = cref.nested(X, L, U)
        if ref["margin"] >= MARGIN:
            return X, L, U, ref
    raise AssertionError("no certified draw for %d x %d" % (m, n))


def test_random_shapes_repeatable_and_equal_to_the_untiled_kernel(g):
    rng = np.random.default_rng(2024)
    shapes = [(int(rng.integers(1, 1100)), int(rng.integers(1, 1100))) for _ in range(24)]
    shapes += [(128, 128), (129, 129), (64, 1300), (1300, 64), (127, 385), (1700, 1800)]
    kept = []
    for k, (m, n) in enumerate(shapes):
        X, L, U, ref = make_certified(rng, m, n)
        dX, dL, dU = (torch.from_numpy(a).cuda() for a in (X, L, U))
        Z1, E1, m1, i1 = g.gptq2d_round(dX, dL, dU, want_E=True, want_margin=True)
        Z2, E2, _, i2 = g.gptq2d_round(dX, dL, dU, want_E=True)
        Zu, Eu, mu, iu = g.gptq2d_round(dX, dL, dU, precision=g.FP64_UNTILED, want_E=True, want_margin=True)
        torch.cuda.synchronize()
        for i in (i1, i2, iu):
            g.check_info(i)
        assert torch.equal(Z1, Z2) and torch.equal(E1, E2), (m, n)
        assert abs(float(m1.cpu()[0]) - ref["margin"]) < 1e-9 and abs(float(mu.cpu()[0]) - ref["margin"]) < 1e-9
        assert float((E1 - Eu).abs().max()) < 1e-9, (m, n)
        assert torch.equal(Z1, Zu), (m, n)
        assert np.array_equal(Z1.cpu().numpy().astype(np.int64), ref["Z"]), (m, n)
        kept.append((dX, dL, dU, Z1))
    # the same matrices again, a dozen at a time, in batched launches and through the host entry
    for trial in range(3):
        idx = rng.permutation(len(kept))[:12]
        Zs, _, _, info = g.gptq2d_round_batched([kept[i][0] for i in idx], [kept[i][1] for i in idx],
                                                [kept[i][2] for i in idx])
        torch.cuda.synchronize()
        g.check_info(info)
        for k, i in enumerate(idx):
            assert torch.equal(Zs[k], kept[i][3]), (trial, tuple(kept[i][0].shape))
    for i in rng.permutation(len(kept))[:6]:
        dX, dL, dU, Z1 = kept[i]
        hZ, _ = g.gptq2d_round_host(dX.cpu().pin_memory(), dL.cpu().pin_memory(), dU.cpu().pin_memory())
        assert torch.equal(hZ, Z1.cpu()), tuple(dX.shape)


def test_random_shapes_and_widths_through_the_blocked_sweep(g):
    """Algorithm 4 on seeded random shapes and block widths against the oracle's plain-C nested sweep
    (Z bit-exact where the certificate's margin allows it, E and the margin always), and run-to-run
    bit-identity (the CTAs of a block recompute each other's rows: the copies must agree bit for bit)."""
    rng = np.random.default_rng(4)
    cases = [(int(rng.integers(1, 500)), int(rng.integers(1, 500)), int(rng.integers(1, 65))) for _ in range(16)]
    cases += [(64, 64, 64), (65, 63, 63), (128, 129, 17), (1, 300, 64), (300, 1, 5), (257, 511, 64)]
    for (m, n, w) in cases:
        X, L, U, ref = make_certified(rng, m, n)
        margin, Eref = O.certificate_margin(X, ref["Z"], L, U)
        assert margin >= MARGIN
        dX, dL, dU = (torch.from_numpy(a).cuda() for a in (X, L, U))
        Z1, E1, m1, i1 = g.gptq2d_round_blocked(dX, dL, dU, w, want_E=True, want_margin=True)
        Z2, E2, _, i2 = g.gptq2d_round_blocked(dX, dL, dU, w, want_E=True)
        torch.cuda.synchronize()
        g.check_info(i1)
        g.check_info(i2)
        assert torch.equal(Z1, Z2) and torch.equal(E1, E2), (m, n, w)
        assert np.array_equal(Z1.cpu().numpy().astype(np.int64), ref["Z"]), (m, n, w)
        assert np.max(np.abs(E1.cpu().numpy() - Eref)) < 1e-9, (m, n, w)
        assert abs(float(m1.cpu()[0]) - margin) < 1e-9, (m, n, w)
