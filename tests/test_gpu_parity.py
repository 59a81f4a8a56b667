"""GPU parity: the CUDA path through the C ABI against the CPU oracle, element by element.

Bar: Z bit-exact on inputs whose oracle margin (distance of the closest pre-rounding value
from a tie) is at least 1e-9; objective within 1e-10 relative; factors within 1e-9 absolute
scaled by the factor's magnitude (fp64 Cholesky-type error bound times the condition of the
configurations, far inside the margin).
"""
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


def gpu_round(g, X, L, U, precision=0, want_E=True):
    Z, E, mm, info = g.gptq2d_round(dev(X), dev(L), dev(U), precision=precision, want_E=want_E, want_margin=True)
    torch.cuda.synchronize()
    g.check_info(info)
    return Z.cpu().numpy().astype(np.int64), (E.cpu().numpy() if E is not None else None), float(mm.cpu()[0])


def oracle_small(X, L, U):
    """Quartic definition for small sizes (plain C restatement of Algorithm 1 on vec(X))."""
    return cref.vec_sweep(X, L, U)


# ------------------------------------------------------------------ the sweep, oracle factors
@pytest.mark.parametrize("precision", [0, 2, 3])
@pytest.mark.parametrize("m,n,seed", [(1, 1, 0), (1, 9, 1), (9, 1, 2), (8, 8, 3), (17, 5, 4), (64, 64, 5),
                                      (65, 63, 6), (100, 130, 7), (129, 257, 8), (200, 75, 9)])
def test_sweep_small_and_ragged_general_bases(g, m, n, seed, precision):
    X, A, B = W.general_bases(m, n, seed)
    L, U, _, _ = O.feedback_factors(A, B)
    ref = oracle_small(X, L, U)
    if ref["margin"] < MARGIN:
        pytest.skip("seed not certified")
    Z, E, mm = gpu_round(g, X, L, U, precision)
    assert np.array_equal(Z, ref["Z"])
    assert np.max(np.abs(E - ref["E"])) < 1e-9
    assert abs(mm - ref["margin"]) < 1e-9


def test_c0_bit_exact_against_explicit_kronecker_oracle(g):
    X, A, B = W.make_config(0, seed=0)
    ref = O.vec_sweep_explicit(X, A, B)           # the definition, 4096 x 4096 Kronecker Gram
    assert ref["margin"] >= MARGIN
    L, U, _, _ = O.feedback_factors(A, B)
    for precision in (0, 2, 3):
        Z, E, mm = gpu_round(g, X, L, U, precision)
        assert np.array_equal(Z, ref["Z"])
    # end to end with the library's own factors
    Ld, Ud, dL, dU, info = g.gptq2d_factor(dev(A), dev(B))
    Z2, _, _, info2 = g.gptq2d_round(dev(X), Ld, Ud)
    torch.cuda.synchronize()
    g.check_info(info); g.check_info(info2)
    assert np.array_equal(Z2.cpu().numpy().astype(np.int64), ref["Z"])


@pytest.mark.parametrize("variant", [None, "B=I", "A=B=I"])
def test_c1_bit_exact_and_reductions(g, variant):
    X, A, B = W.make_config(1, seed=0, variant=variant)
    L, U, lamL, lamU = O.feedback_factors(A, B)
    ref = oracle_small(X, L, U)                   # quartic vec-sweep over all 65536 coordinates
    assert ref["margin"] >= MARGIN
    Ld, Ud, dL, dU, info = g.gptq2d_factor(dev(A), dev(B))
    torch.cuda.synchronize()
    g.check_info(info)
    assert np.max(np.abs(Ld.cpu().numpy() - L)) < 1e-9 * max(1.0, np.max(np.abs(L)))
    assert np.max(np.abs(Ud.cpu().numpy() - U)) < 1e-9 * max(1.0, np.max(np.abs(U)))
    if variant == "A=B=I":
        assert torch.equal(Ld.cpu(), torch.eye(256, dtype=torch.float64))
        assert np.array_equal(ref["Z"], np.rint(X).astype(np.int64))
    if variant == "B=I":
        assert torch.equal(Ud.cpu(), torch.eye(256, dtype=torch.float64))
    for precision in (0, 2, 3):
        Z, E, mm, info = g.gptq2d_round(dev(X), Ld, Ud, precision=precision, want_E=True, want_margin=True)
        torch.cuda.synchronize()
        g.check_info(info)
        assert np.array_equal(Z.cpu().numpy().astype(np.int64), ref["Z"])
    obj = float(g.gptq2d_objective(dev(X), Z, dev(A), dev(B)).cpu()[0])
    want = O.objective(X, ref["Z"], A, B)
    assert abs(obj - want) <= 1e-10 * want + 1e-300
    closed = float((E.cpu().numpy() ** 2 * np.outer(dL.cpu().numpy(), dU.cpu().numpy())).sum())
    assert abs(closed - want) <= 1e-8 * want + 1e-300


# ------------------------------------------------------------------ factors on their own
@pytest.mark.parametrize("m,n,seed", [(5, 7, 0), (128, 128, 1), (130, 127, 2), (300, 515, 3), (1000, 260, 4)])
def test_factor_general_bases(g, m, n, seed):
    X, A, B = W.general_bases(m, n, seed)
    if max(m, n) > 64:      # keep the Grams reasonably conditioned at size
        A = A + np.sqrt(m) * np.eye(m)
        B = B + np.sqrt(n) * np.eye(n)
    L, U, lamL, lamU = O.feedback_factors(A, B)
    Ld, Ud, dL, dU, info = g.gptq2d_factor(dev(A), dev(B))
    torch.cuda.synchronize()
    g.check_info(info)
    Ld, Ud = Ld.cpu().numpy(), Ud.cpu().numpy()
    assert np.array_equal(np.diag(Ld), np.ones(m)) and np.array_equal(np.triu(Ld, 1), np.zeros((m, m)))
    assert np.array_equal(np.diag(Ud), np.ones(n)) and np.array_equal(np.tril(Ud, -1), np.zeros((n, n)))
    assert np.max(np.abs(Ld - L)) < 1e-10 * max(1.0, np.max(np.abs(L)))
    assert np.max(np.abs(Ud - U)) < 1e-10 * max(1.0, np.max(np.abs(U)))
    assert np.allclose(dL.cpu().numpy(), 1 / lamL, rtol=1e-10)
    assert np.allclose(dU.cpu().numpy(), 1 / lamU, rtol=1e-10)


def test_factor_triangular_shortcut_needs_no_oracle(g):
    # B upper triangular => U = diag(B) B^{-1}; A lower triangular => L = A^{-1} diag(A)
    rng = np.random.default_rng(3)
    B = np.triu(rng.standard_normal((150, 150))) + 12 * np.eye(150)
    A = np.tril(rng.standard_normal((140, 140))) + 12 * np.eye(140)
    Ld, Ud, _, _, info = g.gptq2d_factor(dev(A), dev(B))
    torch.cuda.synchronize()
    g.check_info(info)
    assert np.allclose(Ud.cpu().numpy(), np.diag(np.diag(B)) @ np.linalg.inv(B), atol=1e-11)
    assert np.allclose(Ld.cpu().numpy(), np.linalg.inv(A) @ np.diag(np.diag(A)), atol=1e-11)


@pytest.mark.parametrize("m,n", [(1, 1), (15, 17), (16, 33), (127, 129), (130, 257), (300, 515)])
def test_factor_orders_around_the_block_sizes(g, m, n):
    """Orders just below, at and above the 16-row blocks of the diagonal-block kernel and the 128-row blocks of the
    factorisation, against the oracle's factors."""
    rng = np.random.default_rng(1000 * m + n)
    A = rng.standard_normal((m, m)) / np.sqrt(m) + 2 * np.eye(m)
    B = rng.standard_normal((n, n)) / np.sqrt(n) + 2 * np.eye(n)
    L, U, lamL, lamU = O.feedback_factors(A, B)
    Ld, Ud, dL, dU, info = g.gptq2d_factor(dev(A), dev(B))
    torch.cuda.synchronize()
    g.check_info(info)
    assert np.max(np.abs(Ld.cpu().numpy() - L)) < 1e-11 and np.max(np.abs(Ud.cpu().numpy() - U)) < 1e-11
    assert np.allclose(dL.cpu().numpy(), 1 / lamL, rtol=1e-11) and np.allclose(dU.cpu().numpy(), 1 / lamU, rtol=1e-11)


def test_factor_two_level_blocking_ragged(g):
    """Orders of 44 block rows and more take the two-level route of the set-up (128-row steps inside outer blocks
    of 512 rows, rank-512 updates above them); 5700 and 5889 give ragged last blocks at both levels and one side
    with a last outer block of a single block row."""
    m, n = 5700, 5889
    X, A, B = W.general_bases(m, n, 5)
    A = A + np.sqrt(m) * np.eye(m)
    B = B + np.sqrt(n) * np.eye(n)
    L, U, lamL, lamU = O.feedback_factors(A, B)
    Ld, Ud, dL, dU, info = g.gptq2d_factor(dev(A), dev(B))
    torch.cuda.synchronize()
    g.check_info(info)
    Ld, Ud = Ld.cpu().numpy(), Ud.cpu().numpy()
    assert np.array_equal(np.diag(Ld), np.ones(m)) and np.array_equal(np.triu(Ld, 1), np.zeros((m, m)))
    assert np.array_equal(np.diag(Ud), np.ones(n)) and np.array_equal(np.tril(Ud, -1), np.zeros((n, n)))
    assert np.max(np.abs(Ld - L)) < 1e-10 * max(1.0, np.max(np.abs(L)))
    assert np.max(np.abs(Ud - U)) < 1e-10 * max(1.0, np.max(np.abs(U)))
    assert np.allclose(dL.cpu().numpy(), 1 / lamL, rtol=1e-10) and np.allclose(dU.cpu().numpy(), 1 / lamU, rtol=1e-10)


# ------------------------------------------------------------------ mid sizes: cubic oracle + certificate
@pytest.mark.parametrize("name,make", [
    ("c2_like", lambda s: W.llm_layer_like(384, 1408, s, samples=2048)),
    ("c3_like", lambda s: W.ill_conditioned_like(640, 640, s)),
    ("c4_like", lambda s: W.headline_like(768, 896, s)),
])
def test_mid_size_against_nested_oracle_and_certificate(g, name, make):
    for t in range(6):
        X, A, B = make(11 + 1000 * t)
        L, U, lamL, lamU = O.feedback_factors(A, B)
        ref = cref.nested(X, L, U)                # Algorithm 5: cubic, column-major, independent order
        if ref["margin"] >= MARGIN:
            break
    else:
        pytest.fail("no certified seed")
    Ld, Ud, dL, dU, info = g.gptq2d_factor(dev(A), dev(B))
    Z, E, mm, info2 = g.gptq2d_round(dev(X), Ld, Ud, want_E=True, want_margin=True)
    torch.cuda.synchronize()
    g.check_info(info); g.check_info(info2)
    Zh = Z.cpu().numpy().astype(np.int64)
    assert np.array_equal(Zh, ref["Z"])
    margin, Ecert = O.certificate_margin(X, Zh, L, U)
    assert margin >= MARGIN
    assert np.max(np.abs(E.cpu().numpy() - Ecert)) < 1e-8
    obj = float(g.gptq2d_objective(dev(X), Z, dev(A), dev(B)).cpu()[0])
    want = O.objective(X, Zh, A, B)
    assert abs(obj - want) <= 1e-10 * want
    # two runs and the untiled kernel must agree bit for bit (a missing fence would not)
    Z2, _, _, _ = g.gptq2d_round(dev(X), Ld, Ud)
    Z3, _, _, _ = g.gptq2d_round(dev(X), Ld, Ud, precision=2)
    Z4, _, _, _ = g.gptq2d_round(dev(X), Ld, Ud, precision=3)          # pull form (Algorithm 6)
    torch.cuda.synchronize()
    assert torch.equal(Z, Z2) and torch.equal(Z, Z3) and torch.equal(Z, Z4)


# ------------------------------------------------------------------ thin shapes: one row / one column of tiles
@pytest.mark.parametrize("m,n,seed", [(3, 1500, 0), (1500, 3, 1), (130, 1100, 2), (1100, 130, 3), (1, 700, 4), (700, 1, 5)])
def test_thin_shapes_against_nested_oracle(g, m, n, seed):
    for t in range(6):
        X, A, B = W.gaussian_like(m, n, seed + 1000 * t, samples=2 * max(m, n))
        L, U, _, _ = O.feedback_factors(A, B)
        ref = cref.nested(X, L, U)
        if ref["margin"] >= MARGIN:
            break
    else:
        pytest.fail("no certified seed")
    Z, E, mm = gpu_round(g, X, L, U)
    assert np.array_equal(Z, ref["Z"])
    assert np.max(np.abs(E - ref["E"])) < 1e-8
    # repeated runs must be bit-identical (the schedule differs from run to run, the arithmetic must not)
    Z2, E2, _ = gpu_round(g, X, L, U)
    assert np.array_equal(Z, Z2) and np.array_equal(E, E2)


# ------------------------------------------------------------------ invariances on the GPU path
def test_transpose_and_translation_invariance(g):
    X, A, B = W.general_bases(150, 70, 12)
    A = A + 6 * np.eye(150); B = B + 4 * np.eye(70)
    L, U, _, _ = O.feedback_factors(A, B)
    if O.sweep_nested(X, L, U)["margin"] < MARGIN:
        pytest.skip("seed not certified")
    Z, _, _ = gpu_round(g, X, L, U)
    Lt, Ut, _, _ = O.feedback_factors(B.T.copy(), A.T.copy())
    Zt, _, _ = gpu_round(g, X.T.copy(), Lt, Ut)
    assert np.array_equal(Zt, Z.T)
    K = (np.arange(150 * 70).reshape(150, 70) % 37) - 18
    Zk, _, _ = gpu_round(g, X + K, L, U)
    assert np.array_equal(Zk, Z + K)
    Zi, Ei, _ = gpu_round(g, K.astype(np.float64), L, U)
    assert np.array_equal(Zi, K) and np.all(Ei == 0)


def test_strided_inputs_and_host_entry(g):
    X, A, B = W.general_bases(90, 140, 21)
    L, U, _, _ = O.feedback_factors(A, B)
    ref = oracle_small(X, L, U)
    if ref["margin"] < MARGIN:
        pytest.skip("seed not certified")
    # odd leading dimensions (8-byte aligned rows only)
    Xp = torch.zeros((90, 151), dtype=torch.float64, device="cuda"); Xp[:, :140] = dev(X)
    Lp = torch.zeros((90, 97), dtype=torch.float64, device="cuda"); Lp[:, :90] = dev(L)
    Up = torch.zeros((140, 143), dtype=torch.float64, device="cuda"); Up[:, :140] = dev(U)
    Zp = torch.full((90, 149), -7, dtype=torch.int32, device="cuda")
    Z, _, _, info = g.gptq2d_round(Xp[:, :140], Lp[:, :90], Up[:, :140], Z=Zp[:, :140])
    torch.cuda.synchronize()
    g.check_info(info)
    assert np.array_equal(Zp[:, :140].cpu().numpy().astype(np.int64), ref["Z"])
    assert bool((Zp[:, 140:] == -7).all())
    hX = torch.from_numpy(X).pin_memory(); hL = torch.from_numpy(L).pin_memory(); hU = torch.from_numpy(U).pin_memory()
    hZ, hinfo = g.gptq2d_round_host(hX, hL, hU)
    assert np.array_equal(hZ.numpy().astype(np.int64), ref["Z"])


@pytest.mark.parametrize("m,n,seed,pinned", [(1100, 700, 31, True), (700, 1100, 32, False), (1537, 1537, 33, True),
                                             (513, 40, 34, True)])
def test_host_entry_streams_inputs_while_sweeping(g, m, n, seed, pinned):
    """gptq2d_round_host sends X, L, U in 512 x 512 blocks while the kernel already runs (several copy
    steps, ragged last blocks); Z must be what the device entry point gives on resident inputs, which
    in turn is checked against the nested CPU oracle and the certificate."""
    X, A, B = W.general_bases(m, n, seed)
    L, U, _, _ = O.feedback_factors(A, B)
    ref = cref.nested(X, L, U)
    margin, _ = O.certificate_margin(X, ref["Z"], L, U)
    if margin < MARGIN:
        pytest.skip("seed not certified")
    hX, hL, hU = (torch.from_numpy(np.ascontiguousarray(a)) for a in (X, L, U))
    hZ = torch.full((m, n), -5, dtype=torch.int32)
    hE = torch.zeros((m, n), dtype=torch.float64)
    hmargin = torch.zeros(1, dtype=torch.float64)
    if pinned:
        hX, hL, hU, hZ, hE, hmargin = (t.pin_memory() for t in (hX, hL, hU, hZ, hE, hmargin))
    for rep in range(2):                      # the second call reuses the staging buffers of the first
        hZ.fill_(-5)
        g.gptq2d_round_host(hX, hL, hU, hZ=hZ, hE=hE, hmargin=hmargin)
        assert np.array_equal(hZ.numpy().astype(np.int64), ref["Z"]), rep
        assert abs(float(hmargin[0]) - margin) < 1e-9
    Zd, Ed, _ = gpu_round(g, X, L, U)
    assert np.array_equal(Zd, hZ.numpy())
    assert np.array_equal(Ed, hE.numpy())


def test_host_entry_reports_data_errors_and_stays_usable(g):
    """A NaN in X through the streamed host entry: the status words come back, nothing hangs (the copy
    stream's waits are released when the kernel ends), and the next call is fine."""
    m, n = 700, 900
    X, A, B = W.general_bases(m, n, 77)
    L, U, _, _ = O.feedback_factors(A, B)
    hX, hL, hU = (torch.from_numpy(np.ascontiguousarray(a)).pin_memory() for a in (X, L, U))
    hZ = torch.zeros((m, n), dtype=torch.int32).pin_memory()
    bad = hX.clone().pin_memory()
    bad[300, 500] = float("nan")
    with pytest.raises(g.Gptq2dError) as ei:
        g.gptq2d_round_host(bad, hL, hU, hZ=hZ)
    # the entry reported lies on the anti-diagonal of the first non-finite value, within one 8 x 8 leaf of it
    assert ei.value.status == 6
    assert ei.value.info[1] + ei.value.info[2] == 800 and abs(ei.value.info[1] - 300) < 8
    g.gptq2d_round_host(hX, hL, hU, hZ=hZ)
    Zd, _, _ = gpu_round(g, X, L, U, want_E=False)
    assert np.array_equal(Zd, hZ.numpy())


def test_two_streams_two_workspaces(g):
    """Calls on different streams with their own workspaces may be in flight together (the persistent
    launches take turns on the device); neither disturbs the other's result."""
    cases = []
    for (m, n, seed) in [(300, 515, 41), (515, 300, 42)]:
        X, A, B = W.general_bases(m, n, seed)
        L, U, _, _ = O.feedback_factors(A, B)
        ref = cref.nested(X, L, U)
        cases.append((dev(X), dev(L), dev(U), ref["Z"], O.certificate_margin(X, ref["Z"], L, U)[0]))
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    outs = []
    for rep in range(3):
        for (dX, dL, dU, _, _), st in zip(cases, streams):
            with torch.cuda.stream(st):
                outs.append(g.gptq2d_round(dX, dL, dU, stream=st))
    torch.cuda.synchronize()
    for k, (Z, _, _, info) in enumerate(outs):
        g.check_info(info)
        _, _, _, Zref, margin = cases[k % 2]
        assert margin >= MARGIN, "input not certified by the oracle: pick another seed"
        assert np.array_equal(Z.cpu().numpy().astype(np.int64), Zref)


# ------------------------------------------------------------------ error behaviour (host-made failures only)
def test_argument_and_data_errors(g):
    X, A, B = W.general_bases(20, 30, 1)
    L, U, _, _ = O.feedback_factors(A, B)
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(g.Gptq2dError) as e:
        g.gptq2d_round(dev(X), dev(L), dev(U), workspace=small)
    assert e.value.status == 2
    with pytest.raises(g.Gptq2dError) as e:
        g.gptq2d_round(dev(X), dev(L), dev(U), precision=9)
    assert e.value.status == 1
    Xn = X.copy(); Xn[3, 4] = np.nan
    _, _, _, info = g.gptq2d_round(dev(Xn), dev(L), dev(U))
    torch.cuda.synchronize()
    assert info.cpu().tolist()[:3] == [6, 3, 4]
    Xb = X.copy(); Xb[0, 0] = 3e9
    _, _, _, info = g.gptq2d_round(dev(Xb), dev(L), dev(U))
    torch.cuda.synchronize()
    assert info.cpu().tolist()[0] == 7
    As = A.copy(); As[:, 5] = As[:, 6]             # singular basis => Gram not positive definite
    _, _, _, _, info = g.gptq2d_factor(dev(As), dev(B))
    torch.cuda.synchronize()
    assert info.cpu().tolist()[0] == 5 and info.cpu().tolist()[2] == 0
    # the context is still usable afterwards
    Z, _, _ = gpu_round(g, X, L, U)
    assert Z.shape == (20, 30)


def test_fp32_mode_reports_a_small_mismatch_fraction(g):
    X, A, B = W.headline_like(256, 256, 3)
    L, U, _, _ = O.feedback_factors(A, B)
    Z64, _, _ = gpu_round(g, X, L, U, 0)
    Z32, _, _ = gpu_round(g, X, L, U, 1)
    frac = float(np.mean(Z64 != Z32))
    assert frac < 0.01
