"""GPU parity at the full sizes of configurations c2-c4, in the launch configuration the
benchmark times.  The quartic definition cannot run here; Z is checked through the
certificate, which is necessary and sufficient at any size: an integer matrix Z is the
trajectory iff E = L^{-1} (Z - X) U^{-1} has every |E_ij| < 1/2 (oracle.certificate_margin),
with the ORACLE's factors, plus sampled entries recomputed one by one from Eq. 11."""
import hashlib
import json
import os

import numpy as np
import pytest
import torch

import oracle as O
from oracle import cref
from certify import MARGIN, classify_certificate
from paper_2607_27042_b200 import workloads as W

pytestmark = pytest.mark.gpu


def dev(a):
    return torch.as_tensor(np.ascontiguousarray(a), dtype=torch.float64).cuda()


# The seed each configuration is graded on, and how it was chosen.
#  * tests/golden/certified_seeds.json (written by tests/golden/make_certified_seeds.py, which calls only
#    the oracle: the plain-C nested sweep, Algorithm 5, on the oracle's own factors) holds, per configuration,
#    the first seed of 0, 1000, ... whose ORACLE margin is >= 1e-9 and a SHA-256 of the oracle's Z.  Where a
#    row exists the GPU's Z must hash to it: bit-exact parity at full size against a sweep that shares
#    nothing with the kernel.  (The nested sweep is sequential -- minutes at c3, the better part of an hour
#    per seed at c4 -- hence stored, not recomputed per run.)
#  * c2 is also swept by the nested oracle live, in the test.
#  * In every case the certificate (necessary and sufficient, oracle factors) is evaluated on the GPU's Z.
#    Only a genuine near-tie, |margin| < 1e-9, may move on to the next seed; a margin <= -1e-9 means Z is
#    not the trajectory of Theorem 1 / Eq. 11 and fails the test at once.
# The seeds are fixed here so that a run that quietly graded another seed cannot pass.
GRADED_SEED = {2: 0, 3: 0, 4: 1000}
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "certified_seeds.json")


def z_digest(Z):
    return hashlib.sha256(np.ascontiguousarray(Z, dtype="<i4").tobytes()).hexdigest()


@pytest.mark.parametrize("index", [2, 3, 4])
def test_full_config_certificate(index):
    from paper_2607_27042_b200 import gptq2d as g
    golden = json.load(open(GOLDEN)).get("c%d" % index) if os.path.exists(GOLDEN) else None
    if golden is not None:
        assert golden["seed"] == GRADED_SEED[index] and golden["margin"] >= MARGIN
    used = None
    for t in range(6):
        seed = 1000 * t
        if golden is not None and seed < golden["seed"]:
            continue                                      # the oracle alone found this seed within 1e-9 of a tie
        X, A, B = W.make_config(index, seed=seed)
        L, U, lamL, lamU = O.feedback_factors(A, B)
        Zref = None
        if index == 2:
            ref = cref.nested(X, L, U)
            if ref["margin"] < MARGIN:
                continue                                  # the oracle itself sits within 1e-9 of a tie
            Zref = ref["Z"]
        dX, dA, dB = dev(X), dev(A), dev(B)
        Ld, Ud, dL, dU, info = g.gptq2d_factor(dA, dB)
        Z, E, mm, info2 = g.gptq2d_round(dX, Ld, Ud, want_E=True, want_margin=True)
        torch.cuda.synchronize()
        g.check_info(info); g.check_info(info2)
        Zh = Z.cpu().numpy().astype(np.int64)
        margin, Ecert = O.certificate_margin(X, Zh, L, U)
        # the kernel's own margin must agree with the certificate whatever the verdict is
        assert abs(float(mm.cpu()[0]) - margin) < 1e-8, (index, seed, margin)
        verdict = classify_certificate(margin)
        assert verdict != "wrong", "c%d seed %d: certificate margin %.3e: Z is not the trajectory" % (index, seed, margin)
        if Zref is not None:
            assert verdict == "certified", (index, seed, margin)
            assert np.array_equal(Zh, Zref), "c%d seed %d: Z differs from the nested oracle" % (index, seed)
        if golden is not None:
            assert verdict == "certified", (index, seed, margin)
            assert z_digest(Zh) == golden["z_sha256"], "c%d seed %d: Z differs from the oracle's stored Z" % (index, seed)
            assert abs(margin - golden["margin"]) < 1e-8
        if verdict == "certified":
            used = seed
            break
    assert used is not None, "no seed with margin >= 1e-9"
    print("c%d graded on seed %d, certificate margin %.3e%s" % (index, used, margin,
                                                                 ", Z equal to the oracle's stored Z" if golden else ""))
    assert used == GRADED_SEED[index], "c%d was graded on seed %d, expected %d" % (index, used, GRADED_SEED[index])
    assert np.max(np.abs(Ecert)) < 0.5
    Eh = E.cpu().numpy()
    assert np.max(np.abs(Eh - Ecert)) < 1e-7
    assert np.max(np.abs(Ld.cpu().numpy() - L)) < 1e-8 * max(1.0, np.max(np.abs(L)))
    # sampled entries, one by one: Y_ij = X_ij + (L E U)_ij without the entry's own error,
    # and Z_ij must be its nearest integer
    rng = np.random.default_rng(index)
    m, n = X.shape
    for _ in range(64):
        i, j = int(rng.integers(m)), int(rng.integers(n))
        y = X[i, j] + L[i, :i + 1] @ Ecert[:i + 1, :j + 1] @ U[:j + 1, j] - Ecert[i, j]
        assert Zh[i, j] == int(np.rint(y))
    # the blocked sweep (Algorithm 4) must land on the same certified Z
    Zb, _, mb, infob = g.gptq2d_round_blocked(dX, Ld, Ud, 64, want_margin=True)
    torch.cuda.synchronize()
    g.check_info(infob)
    assert np.array_equal(Zb.cpu().numpy().astype(np.int64), Zh)
    assert abs(float(mb.cpu()[0]) - margin) < 1e-8
    del Zb
    obj = float(g.gptq2d_objective(dX, Z, dA, dB).cpu()[0])
    want = O.objective(X, Zh, A, B)
    assert abs(obj - want) <= 1e-10 * want
    assert want < O.objective(X, np.rint(X), A, B)
