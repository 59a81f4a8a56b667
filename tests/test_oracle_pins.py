"""Pins the CPU oracle to facts fixed by the paper and by mathematics -- not to itself.

Each test is chosen so that a plausible slip in the oracle (dropped term, wrong sign,
transposed factor, LDL of the Gram instead of its inverse, wrong vec order) fails it.
"""
import os

import numpy as np
import pytest

import oracle as O
from paper_2607_27042_b200 import workloads as W

HERE = os.path.dirname(os.path.abspath(__file__))


def _rand_general(m, n, seed):
    return W.general_bases(m, n, seed)


# ---------------------------------------------------------------- printed in the paper
def test_antidiagonal_sets_match_figure1():
    want = {}
    with open(os.path.join(HERE, "golden", "fig1_antidiagonals_3x4.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            s, rest = line.split(":")
            want[int(s)] = sorted(tuple(int(v) for v in p.split(",")) for p in rest.split())
    m, n = 3, 4
    assert len(want) == m + n - 1
    for s1, pairs in want.items():
        got = sorted((i + 1, j + 1) for (i, j) in O.anti_diagonal(s1 - 2, m, n))
        assert got == pairs
    # every entry appears exactly once
    allp = [p for s in range(m + n - 1) for p in O.anti_diagonal(s, m, n)]
    assert sorted(allp) == [(i, j) for i in range(m) for j in range(n)]


# ---------------------------------------------------------------- closed forms
def test_closed_form_1x1_and_2x1():
    # 1 x 1: no feedback at all
    out = O.vec_sweep_explicit(np.array([[2.3]]), np.array([[3.0]]), np.array([[0.5]]))
    assert out["Z"][0, 0] == 2
    # 2 x 1 (B = [1]): G = [[g11,g12],[g12,g22]]; minimising r^T G r over r2 for fixed r1
    # gives r2 = -(g12/g22) r1, so the feedback coefficient is L21 = -g12/g22.
    A = np.array([[1.0, 0.7], [0.2, 1.3]])
    G = A.T @ A
    L, U, lamL, lamU = O.feedback_factors(A, np.array([[1.0]]))
    assert np.allclose(L, [[1.0, 0.0], [-G[0, 1] / G[1, 1], 1.0]], atol=1e-14)
    assert np.allclose(U, [[1.0]])
    x = np.array([[0.4], [1.45]])
    e1 = 0.0 - 0.4
    y2 = 1.45 + (-G[0, 1] / G[1, 1]) * e1
    out = O.vec_sweep_explicit(x, A, np.array([[1.0]]))
    assert out["Z"][:, 0].tolist() == [0, int(np.rint(y2))]
    assert abs(out["E"][1, 0] - (np.rint(y2) - y2)) < 1e-14


def test_ldl_factor_is_of_the_inverse_gram():
    rng = np.random.default_rng(5)
    M = rng.standard_normal((7, 7)) + 3 * np.eye(7)
    S = M.T @ M
    for f in (O.unit_lower_ldl_of_inverse, O.unit_lower_ldl_of_inverse_literal):
        F, lam = f(S)
        assert np.allclose(np.triu(F, 1), 0) and np.allclose(np.diag(F), 1)
        assert np.all(lam > 0)
        assert np.allclose(F @ np.diag(lam) @ F.T @ S, np.eye(7), atol=1e-10)
    F1, l1 = O.unit_lower_ldl_of_inverse(S)
    F2, l2 = O.unit_lower_ldl_of_inverse_literal(S)
    assert np.allclose(F1, F2, atol=1e-11) and np.allclose(l1, l2, rtol=1e-10)


def test_triangular_bases_shortcut():
    # B upper triangular: H^{-1} = B^{-T} B^{-1}, and B^{-1} is upper, so the unique
    # unit-upper U with H^{-1} = U^T lam U is diag(B) B^{-1}.  A lower triangular:
    # G^{-1} = A^{-1} A^{-T} gives L = A^{-1} diag(A).
    rng = np.random.default_rng(11)
    B = np.triu(rng.standard_normal((6, 6))) + 3 * np.eye(6)
    A = np.tril(rng.standard_normal((5, 5))) + 3 * np.eye(5)
    L, U, lamL, lamU = O.feedback_factors(A, B)
    assert np.allclose(U, np.diag(np.diag(B)) @ np.linalg.inv(B), atol=1e-12)
    assert np.allclose(L, np.linalg.inv(A) @ np.diag(np.diag(A)), atol=1e-12)


# ---------------------------------------------------------------- brute force (A, B only)
@pytest.mark.parametrize("m,n,seed", [(2, 2, 0), (3, 4, 1), (4, 3, 2), (4, 4, 3), (1, 4, 4), (4, 1, 5)])
def test_brute_force_conditional_minimiser(m, n, seed):
    X, A, B = _rand_general(m, n, seed)
    Zb, Yb = O.brute_force_trajectory(X, A, B)
    assert np.min(np.abs(np.abs(Yb - np.rint(Yb)) - 0.5)) > 1e-6   # no near-ties in the fixture
    out = O.vec_sweep_explicit(X, A, B)
    assert np.array_equal(out["Z"], Zb.astype(np.int64))
    # the value each entry was rounded at must agree too (catches sign errors that
    # happen to round the same way)
    assert np.allclose(out["Z"] - out["E"], Yb, atol=1e-9)
    out_lit = O.vec_sweep_explicit(X, A, B, literal=True)
    assert np.array_equal(out_lit["Z"], out["Z"])


# ---------------------------------------------------------------- Kronecker structure
@pytest.mark.parametrize("m,n", [(3, 4), (5, 2), (8, 8)])
def test_vectorised_feedback_is_kron_of_axis_factors(m, n):
    X, A, B = _rand_general(m, n, 21)
    G, H = O.gram_pair(A, B)
    F, lam = O.unit_lower_ldl_of_inverse(O.kron_gram(G, H))
    L, U, lamL, lamU = O.feedback_factors(A, B)
    assert np.allclose(F, np.kron(U.T, L), atol=1e-11)            # Eq. 10
    assert np.allclose(lam, np.kron(lamU, lamL), rtol=1e-10)
    # coefficient formula below Theorem 1
    i, j, ip, jp = m - 1, n - 1, 1, 0
    assert abs(F[j * m + i, jp * m + ip] - L[i, ip] * U[jp, j]) < 1e-11


def test_kronecker_vec_identity_for_objective():
    X, A, B = _rand_general(5, 7, 33)
    Z = np.rint(X + 0.3)
    a = O.objective(X, Z, A, B)
    b = O.objective_kron(X, Z, A, B)
    assert abs(a - b) <= 1e-12 * abs(a)
    # and against an entry-by-entry evaluation of A R B
    R = Z - X
    s = 0.0
    for p in range(5):
        for q in range(7):
            v = sum(A[p, i] * R[i, j] * B[j, q] for i in range(5) for j in range(7))
            s += v * v
    assert abs(a - s) <= 1e-12 * abs(a)


# ---------------------------------------------------------------- reductions
def test_identity_bases_reduce_to_round_to_nearest():
    rng = np.random.default_rng(2)
    X = 8 * rng.standard_normal((9, 6))
    L, U, lamL, lamU = O.feedback_factors(np.eye(9), np.eye(6))
    assert np.array_equal(L, np.eye(9)) and np.array_equal(U, np.eye(6))
    for fn in (O.sweep_gptq2d, O.vec_sweep_implicit, O.sweep_nested, O.sweep_implicit_y):
        assert np.array_equal(fn(X, L, U)["Z"], np.rint(X).astype(np.int64))
    # diagonal bases also decouple everything
    Ld, Ud, _, _ = O.feedback_factors(np.diag(rng.uniform(0.5, 2, 9)), np.diag(rng.uniform(0.5, 2, 6)))
    assert np.array_equal(Ld, np.eye(9)) and np.array_equal(Ud, np.eye(6))


def test_identity_right_basis_is_one_sided_gptq():
    X, A, _ = _rand_general(7, 5, 8)
    B = np.eye(5)
    L, U, _, _ = O.feedback_factors(A, B)
    assert np.array_equal(U, np.eye(5))
    Z2 = O.sweep_gptq2d(X, L, U)["Z"]
    # columns are independent: each is Algorithm 1 under L
    for j in range(5):
        zj, _, _ = O.adaptive_round_1d(X[:, j], L)
        assert np.array_equal(Z2[:, j], zj.astype(np.int64))
    # and equal to the elimination form that never builds L
    assert np.array_equal(Z2, O.gptq_one_sided_elimination(X, A).astype(np.int64))
    assert np.array_equal(Z2, O.vec_sweep_explicit(X, A, B)["Z"])


# ---------------------------------------------------------------- all algorithms, one trajectory
@pytest.mark.parametrize("m,n,seed", [(6, 9, 0), (9, 6, 1), (12, 12, 2), (1, 7, 3), (7, 1, 4)])
def test_all_forms_share_the_trajectory(m, n, seed):
    X, A, B = _rand_general(m, n, seed)
    L, U, _, _ = O.feedback_factors(A, B)
    ref = O.vec_sweep_explicit(X, A, B)
    assert ref["margin"] > 1e-7
    outs = [O.vec_sweep_implicit(X, L, U), O.sweep_dense_antidiagonal(X, L, U),
            O.sweep_gptq2d(X, L, U), O.sweep_nested(X, L, U), O.sweep_implicit_y(X, L, U)]
    for o in outs:
        assert np.array_equal(o["Z"], ref["Z"])
        assert np.allclose(o["E"], ref["E"], atol=1e-10)
    # buffer invariant of Algorithm 3: C = L E once the sweep ends
    g = O.sweep_gptq2d(X, L, U)
    assert np.allclose(g["C"], L @ g["E"], atol=1e-11)
    # Eq. 11 with every entry rounded: Z = X + L E U
    assert np.allclose(g["Z"], X + L @ g["E"] @ U, atol=1e-10)


@pytest.mark.parametrize("m,n,seed", [(6, 9, 0), (9, 6, 1), (12, 12, 2), (1, 7, 3), (7, 1, 4), (1, 1, 5), (23, 17, 6)])
def test_blocked_form_shares_the_trajectory_for_every_block_width(m, n, seed):
    """Algorithm 4 against the explicit vectorised sweep (Algorithm 1 under the Kronecker Gram), which
    shares none of its steps: width 1 (no in-block push at all, every contribution arrives by a flush),
    widths that leave a ragged last block or a last block of a single anti-diagonal, and one block that
    holds the whole sweep (no flush at all)."""
    X, A, B = _rand_general(m, n, seed)
    L, U, _, _ = O.feedback_factors(A, B)
    ref = O.vec_sweep_explicit(X, A, B)
    assert ref["margin"] > 1e-7
    widths = sorted({1, 2, 3, 5, 8, max(1, (m + n - 2) // 2), max(1, m + n - 2), m + n - 1, m + n + 5})
    for w in widths:
        o = O.sweep_blocked(X, L, U, w)
        assert np.array_equal(o["Z"], ref["Z"]), w
        assert np.allclose(o["E"], ref["E"], atol=1e-10), w
        # the single buffer is complete at the end, whichever mix of folds and flushes filled it
        assert np.allclose(o["C"], L @ o["E"], atol=1e-11), w
    with pytest.raises(ValueError):
        O.sweep_blocked(X, L, U, 0)


def test_blocked_form_random_shapes_and_widths_and_its_block_invariant():
    """Seeded random (m, n, w): Algorithm 4 against the nested column sweep (Algorithm 5), plus the state
    the correctness argument of Section 4 rests on: once every block is flushed, a later entry's Y is
    X + (L E U) over the entries rounded so far -- checked by stopping after the first block through a
    width that holds exactly that block and comparing with Eq. 11 on the partial E."""
    rng = np.random.default_rng(77)
    for _ in range(24):
        m, n = int(rng.integers(1, 20)), int(rng.integers(1, 20))
        w = int(rng.integers(1, m + n + 2))
        X, A, B = _rand_general(m, n, int(rng.integers(1 << 30)))
        L, U, _, _ = O.feedback_factors(A, B)
        ref = O.sweep_nested(X, L, U)
        if ref["margin"] < 1e-7:
            continue
        o = O.sweep_blocked(X, L, U, w)
        assert np.array_equal(o["Z"], ref["Z"]), (m, n, w)
        assert np.allclose(o["E"], ref["E"], atol=1e-10), (m, n, w)
        # partial state: zero the errors of everything after the first block; Eq. 11 then gives the
        # corrected value every later entry must have been handed by the flushes, and rounding the
        # first entry of the second block from it must reproduce Z there
        s1 = min(w - 1, m + n - 2)
        if s1 < m + n - 2:
            idx = np.add.outer(np.arange(m), np.arange(n))
            Epart = np.where(idx <= s1, o["E"], 0.0)
            Ypart = X + L @ Epart @ U
            for (i, j) in O.anti_diagonal(s1 + 1, m, n):
                assert np.rint(Ypart[i, j]) == o["Z"][i, j], (m, n, w, i, j)


def test_transpose_symmetry():
    X, A, B = _rand_general(5, 8, 17)
    Z = O.vec_sweep_explicit(X, A, B)["Z"]
    Zt = O.vec_sweep_explicit(X.T.copy(), B.T.copy(), A.T.copy())["Z"]
    assert np.array_equal(Zt, Z.T)
    L, U, _, _ = O.feedback_factors(A, B)
    Lt, Ut, _, _ = O.feedback_factors(B.T.copy(), A.T.copy())
    assert np.allclose(Lt, U.T, atol=1e-12) and np.allclose(Ut, L.T, atol=1e-12)


def test_translation_negation_scaling_invariances():
    X, A, B = _rand_general(6, 6, 29)
    Z = O.vec_sweep_explicit(X, A, B)["Z"]
    K = np.arange(36).reshape(6, 6) - 17
    assert np.array_equal(O.vec_sweep_explicit(X + K, A, B)["Z"], Z + K)
    assert np.array_equal(O.vec_sweep_explicit(-X, A, B)["Z"], -Z)
    assert np.array_equal(O.vec_sweep_explicit(K.astype(float), A, B)["Z"], K)
    Q, _ = np.linalg.qr(np.random.default_rng(1).standard_normal((6, 6)))
    assert np.array_equal(O.vec_sweep_explicit(X, 3.0 * Q @ A, 0.25 * B)["Z"], Z)
    assert abs(O.objective(X, Z, 3.0 * Q @ A, 0.25 * B) - 0.5625 * O.objective(X, Z, A, B)) < 1e-9


# ---------------------------------------------------------------- certificate / objective
def test_certificate_accepts_trajectory_and_rejects_a_flip():
    X, A, B = _rand_general(10, 13, 41)
    L, U, lamL, lamU = O.feedback_factors(A, B)
    out = O.sweep_gptq2d(X, L, U)
    margin, E = O.certificate_margin(X, out["Z"], L, U)
    assert margin > 0 and abs(margin - out["margin"]) < 1e-10
    assert np.allclose(E, out["E"], atol=1e-10)
    Zbad = out["Z"].copy()
    Zbad[4, 5] += 1
    mbad, _ = O.certificate_margin(X, Zbad, L, U)
    assert mbad < 0
    # closed-form objective from the local errors
    a = O.objective(X, out["Z"], A, B)
    assert abs(O.objective_from_errors(E, lamL, lamU) - a) <= 1e-10 * a
    # bound: every |E| <= 1/2
    assert a <= 0.25 * np.sum(1 / lamL) * np.sum(1 / lamU)


# ---------------------------------------------------------------- config-shaped inputs
def test_c0_explicit_kronecker_equals_implicit_and_gptq2d():
    X, A, B = W.make_config(0, seed=0)
    L, U, lamL, lamU = O.feedback_factors(A, B)
    ref = O.vec_sweep_explicit(X, A, B)           # 4096 x 4096 Kronecker Gram
    assert ref["margin"] > 1e-9
    assert np.array_equal(O.sweep_gptq2d(X, L, U)["Z"], ref["Z"])
    assert np.array_equal(O.sweep_nested(X, L, U)["Z"], ref["Z"])
    margin, _ = O.certificate_margin(X, ref["Z"], L, U)
    assert abs(margin - ref["margin"]) < 1e-9
    # rounding with feedback must beat plain rounding on the objective
    assert O.objective(X, ref["Z"], A, B) < O.objective(X, np.rint(X), A, B)


def test_workload_generators_are_deterministic_and_well_formed():
    X1, A1, B1 = W.make_config(0, seed=3)
    X2, A2, B2 = W.make_config(0, seed=3)
    assert np.array_equal(X1, X2) and np.array_equal(A1, A2) and np.array_equal(B1, B2)
    assert np.allclose(np.tril(A1, -1), 0) and np.allclose(np.tril(B1, -1), 0)
    Xi, Ai, Bi = W.make_config(0, seed=3, variant="A=B=I")
    assert np.array_equal(Ai, np.eye(64)) and np.array_equal(Bi, np.eye(64))
    X, A, B = W.ill_conditioned_like(48, 40, seed=1, cond=1e6)
    ev = np.linalg.eigvalsh(A.T @ A)
    assert 5e5 < ev[-1] / ev[0] < 2e6
    X, A, B = W.llm_layer_like(64, 96, seed=2, samples=256)
    assert X.shape == (64, 96) and np.std(X) > 0.9


# ---------------------------------------------------------------- plain-C restatement
@pytest.mark.parametrize("m,n,seed", [(5, 9, 0), (16, 11, 1), (1, 6, 2), (6, 1, 3)])
def test_c_oracle_matches_numpy_oracle_small(m, n, seed):
    from oracle import cref
    X, A, B = _rand_general(m, n, seed)
    L, U, _, _ = O.feedback_factors(A, B)
    ref = O.vec_sweep_explicit(X, A, B)
    for fn in (cref.vec_sweep, cref.alg3, cref.nested):
        out = fn(X, L, U)
        assert np.array_equal(out["Z"], ref["Z"])
        assert np.allclose(out["E"], ref["E"], atol=1e-10)
    Zb, _ = O.brute_force_trajectory(X, A, B)
    assert np.array_equal(cref.vec_sweep(X, L, U)["Z"], Zb.astype(np.int64))


def test_c1_quartic_sweep_and_its_reductions():
    """256 x 256: quartic vec-sweep (C) == GPTQ-2D == nested; B = I and A = B = I variants."""
    from oracle import cref
    X, A, B = W.make_config(1, seed=0)
    L, U, _, _ = O.feedback_factors(A, B)
    ref = cref.vec_sweep(X, L, U)
    assert ref["margin"] > 1e-9
    assert np.array_equal(cref.alg3(X, L, U)["Z"], ref["Z"])
    assert np.array_equal(cref.nested(X, L, U)["Z"], ref["Z"])
    margin, _ = O.certificate_margin(X, ref["Z"], L, U)
    assert abs(margin - ref["margin"]) < 1e-9
    Xb, Ab, Bb = W.make_config(1, seed=0, variant="B=I")
    Lb, Ub, _, _ = O.feedback_factors(Ab, Bb)
    zb = cref.vec_sweep(Xb, Lb, Ub)["Z"]
    zcol, _, _ = O.adaptive_round_1d(Xb[:, 17], Lb)
    assert np.array_equal(zb[:, 17], zcol.astype(np.int64))
    Xi, Ai, Bi = W.make_config(1, seed=0, variant="A=B=I")
    Li, Ui, _, _ = O.feedback_factors(Ai, Bi)
    assert np.array_equal(cref.vec_sweep(Xi, Li, Ui)["Z"], np.rint(Xi).astype(np.int64))


# ------------------------------------------------------------------ reverse order (Section 2, related work)
@pytest.mark.parametrize("m,n,seed", [(1, 1, 0), (2, 2, 1), (3, 4, 2), (4, 3, 3), (1, 6, 4), (6, 1, 5), (4, 4, 6)])
def test_reverse_order_trajectory_matches_its_brute_force(m, n, seed):
    """The reverse-order rounding is pinned by a conditional least-squares brute force that uses A and
    B only (no Gram, no factor), like the forward one; a wrong triangle, a wrong push direction or a
    transposed factor changes Z."""
    X, A, B = W.general_bases(m, n, seed)
    Zb = O.brute_force_trajectory_reverse(X, A, B)
    ref = O.vec_sweep_reverse(X, A, B)
    if ref["margin"] < 1e-9:
        pytest.skip("seed not certified")
    assert np.array_equal(Zb, ref["Z"])
    Lr, Ur, _, _ = O.feedback_factors_reverse(A, B)
    out = O.sweep_gptq2d_reverse(X, Lr, Ur)
    assert np.array_equal(out["Z"], ref["Z"])
    assert np.max(np.abs(out["E"] - ref["E"])) < 1e-10


def test_reverse_factors_are_unit_triangular_and_factor_the_inverse_grams():
    X, A, B = W.general_bases(9, 7, 11)
    Lr, Ur, lamL, lamU = O.feedback_factors_reverse(A, B)
    G, H = O.gram_pair(A, B)
    assert np.allclose(np.triu(Lr), Lr) and np.allclose(np.diag(Lr), 1.0)
    assert np.allclose(np.tril(Ur), Ur) and np.allclose(np.diag(Ur), 1.0)
    assert np.max(np.abs(Lr @ np.diag(lamL) @ Lr.T @ G - np.eye(9))) < 1e-9
    assert np.max(np.abs(Ur.T @ np.diag(lamU) @ Ur @ H - np.eye(7))) < 1e-9
    # Kronecker structure of the reverse feedback factor: F~ = U~^T (x) L~
    F, _ = O.unit_upper_udu_of_inverse(O.kron_gram(G, H))
    assert np.max(np.abs(F - np.kron(Ur.T, Lr))) < 1e-9


@pytest.mark.parametrize("m,n,seed", [(5, 8, 0), (12, 12, 1), (20, 9, 2)])
def test_reverse_order_is_the_forward_order_on_the_index_reversed_problem(m, n, seed):
    """With P the index reversal: reverse(X; A, B) = P forward(P X P; A P, P B) P, and the reverse factors
    are the reversed forward factors of the reversed bases.  This is what the CUDA path relies on."""
    X, A, B = W.general_bases(m, n, seed)
    Lr, Ur, _, _ = O.feedback_factors_reverse(A, B)
    rev = O.sweep_gptq2d_reverse(X, Lr, Ur)
    if rev["margin"] < 1e-9:
        pytest.skip("seed not certified")
    Lf, Uf, _, _ = O.feedback_factors(A[:, ::-1], B[::-1, :])
    fwd = O.sweep_gptq2d(X[::-1, ::-1].copy(), Lf, Uf)
    assert np.array_equal(fwd["Z"][::-1, ::-1], rev["Z"])
    assert np.max(np.abs(Lf[::-1, ::-1] - Lr)) < 1e-12 and np.max(np.abs(Uf[::-1, ::-1] - Ur)) < 1e-12
    # it is a different rounding from the forward one on the same inputs (so a no-op "reverse" fails)
    L, U, _, _ = O.feedback_factors(A, B)
    assert not np.array_equal(O.sweep_gptq2d(X, L, U)["Z"], rev["Z"])
    margin, E = O.certificate_margin_reverse(X, rev["Z"], Lr, Ur)
    assert abs(margin - rev["margin"]) < 1e-10 and np.max(np.abs(E - rev["E"])) < 1e-9
    bad = rev["Z"].copy(); bad[m // 2, n // 2] += 1
    assert O.certificate_margin_reverse(X, bad, Lr, Ur)[0] < 0


def test_fp32_statement_of_algorithm_3_is_pinned_to_the_fp64_trajectory():
    """The single-precision restatement of Algorithm 3 (the reference of the fp32 mode): where every pre-rounding
    value is far from a tie (margin >> fp32 error) it must land on the fp64 trajectory, which the brute force and
    the explicit Kronecker definition pin; with exactly representable data (dyadic factors, quarter-integer X) the
    fp32 arithmetic is exact and E must agree to the last bit; A = B = I reduces to round-to-nearest."""
    found = 0
    for seed in range(40):
        X, A, B = W.general_bases(14, 11, seed)
        L, U, _, _ = O.feedback_factors(A, B)
        ref = O.sweep_gptq2d(X, L, U)
        if ref["margin"] < 2e-3:
            continue
        got = O.sweep_gptq2d_fp32(X, L, U)
        assert np.array_equal(got["Z"], ref["Z"]), seed
        assert np.max(np.abs(got["E"].astype(np.float64) - ref["E"])) < 2e-4
        assert got["E"].dtype == np.float32
        found += 1
    assert found >= 5
    rng = np.random.default_rng(3)
    m, n = 9, 12
    L = np.tril(rng.integers(-2, 3, size=(m, m)) / 4.0, -1) + np.eye(m)
    U = np.triu(rng.integers(-2, 3, size=(n, n)) / 4.0, 1) + np.eye(n)
    X = rng.integers(-40, 41, size=(m, n)) / 4.0 + 0.125          # never a tie: every Y is an odd multiple of 1/8 ... 1/2^k
    ref = O.sweep_gptq2d(X, L, U)
    got = O.sweep_gptq2d_fp32(X, L, U)
    if ref["margin"] > 1e-6:                                        # exact dyadic arithmetic in both precisions
        assert np.array_equal(got["Z"], ref["Z"])
        assert np.array_equal(got["E"].astype(np.float64), ref["E"])
    Xr = rng.standard_normal((6, 7)) * 5
    got = O.sweep_gptq2d_fp32(Xr, np.eye(6), np.eye(7))
    assert np.array_equal(got["Z"], np.rint(Xr.astype(np.float32)).astype(np.int64))
