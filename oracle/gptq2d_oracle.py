"""Plain fp64 restatement of two-sided adaptive rounding, written from the paper.

TEST INFRASTRUCTURE ONLY -- never imported by the product package.

What "the result" is (Section 3.2, Theorem 2): the fixed-order greedy trajectory
of one-dimensional adaptive rounding (Algorithm 1) applied to vec(X) (column-major)
under the Kronecker Gram  H (x) G,  G = A^T A,  H = B B^T  (Eq. 8, Eq. 9).  It is
NOT the minimiser of the objective (exact closest-vector is NP-hard, Section 6).

Indices are 0-based here; the paper is 1-based.  vec index of (i, j) is j*m + i
(footnote of Eq. 1).  Rounding is IEEE round-half-to-even (np.rint); Theorem 1
only requires that ties be broken by some fixed rule and names none -- this is the
reading taken, and graded inputs never sit within 1e-9 of a tie.

Pins (see tests/test_oracle_pins.py): brute-force conditional minimiser that uses
A and B only; closed forms for 1x1 / 2x2; F == U^T (x) L; B = I column
independence and an elimination-form GPTQ; A = B = I round-to-nearest; the
Kronecker-vec identity; transpose symmetry; mutual agreement of Algorithms
1, 2, 3, 4, 5, 6 (Algorithm 4 for block widths from 1 to one block that holds the
whole sweep); the integer-matrix certificate.  The reverse-order functions at the
end (Section 2, "Two-sided and Kronecker-factored rounding": the same rounding
taken from the last row and column) are pinned by their own brute force, by
F~ == U~^T (x) L~ and by the index-reversal identity with the forward functions.
No function here is unpinned.
"""
from __future__ import annotations

import numpy as np
import scipy.linalg as sla

__all__ = [
    "gram_pair", "kron_gram", "unit_lower_ldl_of_inverse_literal",
    "unit_lower_ldl_of_inverse", "feedback_factors", "adaptive_round_1d",
    "vec_sweep_explicit", "vec_sweep_implicit", "anti_diagonal",
    "sweep_dense_antidiagonal", "sweep_gptq2d", "sweep_blocked", "sweep_nested", "sweep_implicit_y",
    "brute_force_trajectory", "local_errors_from_Z", "certificate_margin",
    "objective", "objective_kron", "objective_from_errors", "gptq_one_sided_elimination",
    "unit_upper_udu_of_inverse", "feedback_factors_reverse", "adaptive_round_1d_reverse",
    "vec_sweep_reverse", "sweep_gptq2d_reverse", "brute_force_trajectory_reverse",
    "certificate_margin_reverse", "sweep_gptq2d_fp32",
]


# --------------------------------------------------------------------------- metric
def gram_pair(A, B):
    """Eq. 8: row Gram G = A^T A (m x m) and column Gram H = B B^T (n x n)."""
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    return A.T @ A, B @ B.T


def kron_gram(G, H):
    """Eq. 9: the mn x mn Gram of vec(R) (column-major) is H (x) G."""
    return np.kron(H, G)


def objective(X, Z, A, B):
    """Eq. 7: || A (Z - X) B ||_F^2."""
    R = np.asarray(Z, dtype=np.float64) - np.asarray(X, dtype=np.float64)
    M = np.asarray(A, dtype=np.float64) @ R @ np.asarray(B, dtype=np.float64)
    return float(np.sum(M * M))


def objective_kron(X, Z, A, B):
    """Eq. 9: vec(R)^T (H (x) G) vec(R) with column-major vec (small sizes only)."""
    R = np.asarray(Z, dtype=np.float64) - np.asarray(X, dtype=np.float64)
    G, H = gram_pair(A, B)
    r = R.reshape(-1, order="F")
    return float(r @ (kron_gram(G, H) @ r))


# --------------------------------------------------------------------------- factors
def unit_lower_ldl_of_inverse_literal(S):
    """Section 3.1, literally: invert the Gram, LDL-factorise the inverse.

    S^{-1} = F diag(lam) F^T with F unit lower.  Obtained from the lower Cholesky
    factor T of S^{-1} (T T^T = S^{-1}) as F = T diag(T)^{-1}, lam = diag(T)^2.
    Loses accuracy for ill-conditioned S (it squares nothing, but the explicit
    inverse is not backward stable); kept as the definition and used to pin the
    stable route below.
    """
    S = np.asarray(S, dtype=np.float64)
    Sinv = np.linalg.inv(S)
    Sinv = 0.5 * (Sinv + Sinv.T)
    T = np.linalg.cholesky(Sinv)
    d = np.diag(T).copy()
    F = T / d[None, :]
    return F, d * d


def unit_lower_ldl_of_inverse(S):
    """Same factor as the literal routine, without forming S^{-1}.

    S^{-1} = F lam F^T  <=>  S = P^T P with P = lam^{-1/2} F^{-1} lower triangular.
    P comes from the Cholesky factor of the index-reversed S:  with J the reversal,
    J S J = Q Q^T (Q lower)  =>  P = (J Q J)^T.  Then F = P^{-1} diag(P) and
    lam = diag(P)^{-2}.  (The paper does not say how to obtain the LDL factor; this
    is the reading taken because it is backward stable.)
    """
    S = np.asarray(S, dtype=np.float64)
    Q = np.linalg.cholesky(S[::-1, ::-1])
    P = Q[::-1, ::-1].T                      # lower triangular, P^T P = S
    p = np.diag(P).copy()
    F = sla.solve_triangular(P, np.diag(p), lower=True)
    F = np.tril(F)
    np.fill_diagonal(F, 1.0)
    return F, 1.0 / (p * p)


def feedback_factors(A, B, literal=False):
    """Section 4.1: L unit lower with G^{-1} = L lamL L^T; U unit upper with
    H^{-1} = U^T lamU U.  Returns (L, U, lamL, lamU)."""
    G, H = gram_pair(A, B)
    f = unit_lower_ldl_of_inverse_literal if literal else unit_lower_ldl_of_inverse
    L, lamL = f(G)
    Ut, lamU = f(H)
    return L, Ut.T.copy(), lamL, lamU


# --------------------------------------------------------------------------- Algorithm 1
def adaptive_round_1d(x, F):
    """Algorithm 1: y <- x; for k: z_k = round(y_k); E_k = z_k - y_k; y_{k:} += F_{k:,k} E_k.

    Returns (z, E, y_at_rounding_time).
    """
    y = np.array(x, dtype=np.float64)
    d = y.size
    z = np.zeros(d)
    E = np.zeros(d)
    ypre = np.zeros(d)
    for k in range(d):
        ypre[k] = y[k]
        z[k] = np.rint(y[k])
        E[k] = z[k] - y[k]
        y[k:] += F[k:, k] * E[k]
    return z, E, ypre


def vec_sweep_explicit(X, A, B, literal=False):
    """The definition (Section 3.2): Algorithm 1 on vec(X) with F the unit lower LDL
    factor of (H (x) G)^{-1}, the explicit mn x mn Kronecker Gram being formed.

    Quartic; for m*n up to a few thousand.  Returns dict(Z, E, margin).
    """
    X = np.asarray(X, dtype=np.float64)
    m, n = X.shape
    G, H = gram_pair(A, B)
    K = kron_gram(G, H)
    f = unit_lower_ldl_of_inverse_literal if literal else unit_lower_ldl_of_inverse
    F, _ = f(K)
    z, E, _ = adaptive_round_1d(X.reshape(-1, order="F"), F)
    return _pack(z.reshape(m, n, order="F"), E.reshape(m, n, order="F"))


def vec_sweep_implicit(X, L, U):
    """Algorithm 1 on vec(X) with column k of F = U^T (x) L (Eq. 10) formed on the fly.

    F[(j*m+i), (j'*m+i')] = L[i,i'] * U[j',j]  (text below Theorem 1).  Still the
    quartic sweep over all mn coordinates; no mn x mn matrix is stored.
    """
    X = np.asarray(X, dtype=np.float64)
    m, n = X.shape
    y = X.reshape(-1, order="F").copy()
    z = np.zeros(m * n)
    E = np.zeros(m * n)
    for jp in range(n):
        for ip in range(m):
            k = jp * m + ip
            z[k] = np.rint(y[k])
            E[k] = z[k] - y[k]
            # column k of F restricted to coordinates >= k: rows of column jp from ip
            # on, then every later column in full (zero coefficients included).
            col = np.outer(U[jp, jp:], L[:, ip]).reshape(-1)[ip:]
            y[k:] += col * E[k]
    return _pack(z.reshape(m, n, order="F"), E.reshape(m, n, order="F"))


# --------------------------------------------------------------------------- anti-diagonal forms
def anti_diagonal(s, m, n):
    """Eq. 14 in 0-based form: all (i, j) with i + j == s, 0 <= i < m, 0 <= j < n."""
    lo = max(0, s - n + 1)
    hi = min(m - 1, s)
    return [(i, s - i) for i in range(lo, hi + 1)]


def sweep_dense_antidiagonal(X, L, U):
    """Algorithm 2: keep Y = X + L E U explicitly; after each anti-diagonal apply the
    rank-one updates L[:, i] E_ij U[j, :] (Eq. 13) of its entries."""
    Y = np.array(X, dtype=np.float64)
    m, n = Y.shape
    Z = np.zeros((m, n))
    E = np.zeros((m, n))
    for s in range(m + n - 1):
        idx = anti_diagonal(s, m, n)
        for (i, j) in idx:
            Z[i, j] = np.rint(Y[i, j])
            E[i, j] = Z[i, j] - Y[i, j]
        for (i, j) in idx:
            Y += np.outer(L[:, i], U[j, :]) * E[i, j]
    return _pack(Z, E)


def sweep_gptq2d(X, L, U):
    """Algorithm 3 (GPTQ-2D): corrected matrix Y plus the accumulated-feedback buffer C = L E.

    Stage s handles anti-diagonal s as a whole.  All its entries are rounded at once (they do not
    depend on one another, Eq. 14).  Their errors then travel along two axes only: down the entry's own
    column through L -- folded into C and pushed into Y; written here by TARGET row r, which receives
    L[r, i] * E[i, s - i] at column s - i from every source row i < r of the stage -- and, once C holds
    the stage's own errors (unit diagonal of L), right along the entry's own row through U, from the
    folded C_ij.  Same operations as the paper's two parallel loops per stage, grouped differently."""
    Y = np.array(X, dtype=np.float64)
    m, n = Y.shape
    Z = np.zeros((m, n))
    E = np.zeros((m, n))
    C = np.zeros((m, n))
    for s in range(m + n - 1):
        lo, hi = max(0, s - n + 1), min(m - 1, s)
        rows = np.arange(lo, hi + 1)
        cols = s - rows
        y = Y[rows, cols]
        z = np.rint(y)
        e = z - y                                          # E = Z - Y
        Z[rows, cols] = z
        E[rows, cols] = e
        C[rows, cols] += e                                 # the fold's own term: L_ii = 1
        for r in range(lo + 1, m):                         # fold and push down, by target row
            src = rows[rows < r]
            if src.size == 0:
                continue
            M = L[r, src] * e[:src.size]
            C[r, s - src] += M
            Y[r, s - src] += M
        for i, j in zip(rows, cols):                       # push right from the folded C
            Y[i, j + 1:] += C[i, j] * U[j, j + 1:]
    out = _pack(Z, E)
    out["C"] = C
    return out


def sweep_blocked(X, L, U, w):
    """Algorithm 4 (blocked GPTQ-2D): the sweep in blocks of w anti-diagonals with ONE buffer
    C = L E kept across blocks.  Inside a block Algorithm 3 runs with the fold and both pushes cut
    off at the block's last anti-diagonal s1; after the block, every later entry receives the
    rest at once: the down flush (the block's band of E in its column through L, added to Y and
    to C) and the right flush (the block's band of C in its row through U, added to Y).

    0-based: blocks start at s0 = 0, w, 2w, ... <= m+n-2 (the paper's 2, 2+w, ... in 1-based
    index sums); index ranges are clipped to the matrix, so the last block may hold a single
    anti-diagonal."""
    Y = np.array(X, dtype=np.float64)
    m, n = Y.shape
    w = int(w)
    if w < 1:
        raise ValueError("block width must be positive")
    Z = np.zeros((m, n))
    E = np.zeros((m, n))
    C = np.zeros((m, n))
    last = m + n - 2
    for s0 in range(0, last + 1, w):
        s1 = min(s0 + w - 1, last)
        for s in range(s0, s1 + 1):
            # one stage of the block, all its entries at once; the pushes stop at the block's last anti-diagonal
            # s1: from source (i, s - i) the downward push reaches rows r with r + (s - i) <= s1, the rightward
            # push columns c with i + c <= s1
            lo, hi = max(0, s - n + 1), min(m - 1, s)
            rows = np.arange(lo, hi + 1)
            cols = s - rows
            y = Y[rows, cols]
            z = np.rint(y)
            e = z - y
            Z[rows, cols] = z
            E[rows, cols] = e
            C[rows, cols] += e                                  # unit diagonal of L
            reach = s1 - s                                      # how many rows / columns a push may still travel
            for r in range(lo + 1, min(m - 1, hi + reach) + 1):         # fold and push down, by target row
                take = (rows < r) & (rows >= r - reach)
                if not take.any():
                    continue
                src = rows[take]
                M = L[r, src] * e[take]
                C[r, s - src] += M
                Y[r, s - src] += M
            for i, j in zip(rows, cols):                        # push right from the folded C
                end = min(s1 - i, n - 1) + 1
                Y[i, j + 1:end] += C[i, j] * U[j, j + 1:end]
        # down flush: column j's part of the block is rows s0-j .. s1-j; everything below s1-j is later
        for j in range(n):
            lo, hi = max(s0 - j, 0), min(s1 - j, m - 1)
            first = max(s1 - j + 1, 0)
            if lo > hi or first >= m:
                continue
            M = L[first:, lo:hi + 1] @ E[lo:hi + 1, j]
            C[first:, j] += M
            Y[first:, j] += M
        # right flush: row i's part of the block is columns s0-i .. s1-i
        for i in range(m):
            lo, hi = max(s0 - i, 0), min(s1 - i, n - 1)
            first = max(s1 - i + 1, 0)
            if lo > hi or first >= n:
                continue
            Y[i, first:] += C[i, lo:hi + 1] @ U[lo:hi + 1, first:]
    out = _pack(Z, E)
    out["C"] = C
    return out


def sweep_nested(X, L, U):
    """Algorithm 5 (nested, column-major): 1-D sweep down each column under L, then
    Y += (y - Y[:, j]) U[j, :]  (Eq. 18)."""
    Y = np.array(X, dtype=np.float64)
    m, n = Y.shape
    Z = np.zeros((m, n))
    E = np.zeros((m, n))
    for j in range(n):
        y = Y[:, j].copy()
        for i in range(m):
            Z[i, j] = np.rint(y[i])
            E[i, j] = Z[i, j] - y[i]
            y[i:] += L[i:, i] * E[i, j]
        Y += np.outer(y - Y[:, j], U[j, :])
    return _pack(Z, E)


def sweep_implicit_y(X, L, U):
    """Algorithm 6 (implicit Y): only C = L E is kept; Y_ij = X_ij + C[i, :j+1] U[:j+1, j]
    (Eq. 19) on demand, then C[i:, j] += L[i:, i] E_ij (Eq. 20)."""
    X = np.asarray(X, dtype=np.float64)
    m, n = X.shape
    Z = np.zeros((m, n))
    E = np.zeros((m, n))
    C = np.zeros((m, n))
    for s in range(m + n - 1):
        idx = anti_diagonal(s, m, n)
        for (i, j) in idx:
            y = X[i, j] + C[i, :j + 1] @ U[:j + 1, j]
            Z[i, j] = np.rint(y)
            E[i, j] = Z[i, j] - y
        for (i, j) in idx:
            C[i:, j] += L[i:, i] * E[i, j]
    return _pack(Z, E)


# --------------------------------------------------------------------------- independent checks
def brute_force_trajectory(X, A, B):
    """Greedy trajectory from the objective alone (no G, H, L, U, F).

    In column-major order: with the residuals of already-rounded coordinates held
    fixed, minimise || (B^T (x) A) r ||_2 over the REAL residuals of all remaining
    coordinates (a linear least-squares problem); the corrected value of the
    current coordinate is x_k + r_k*, and z_k is its nearest integer (Section 1
    describes the method this way: every coordinate goes to the integer closest to
    its conditional optimum once the earlier coordinates are frozen).  Tiny sizes only.
    Returns (Z, Ypre) with Ypre the value each entry was rounded at.
    """
    X = np.asarray(X, dtype=np.float64)
    m, n = X.shape
    Mfull = np.kron(np.asarray(B, dtype=np.float64).T, np.asarray(A, dtype=np.float64))
    x = X.reshape(-1, order="F")
    d = m * n
    r = np.zeros(d)
    z = np.zeros(d)
    ypre = np.zeros(d)
    for k in range(d):
        rhs = -Mfull[:, :k] @ r[:k]
        sol, *_ = np.linalg.lstsq(Mfull[:, k:], rhs, rcond=None)
        ypre[k] = x[k] + sol[0]
        z[k] = np.rint(ypre[k])
        r[k] = z[k] - x[k]
    return z.reshape(m, n, order="F"), ypre.reshape(m, n, order="F")


def gptq_one_sided_elimination(X, A):
    """One-sided rounding (B = I) in its elimination form: keep W and Hinv = G^{-1};
    after rounding row k of W, W[k+1:] -= Hinv[k+1:, k] / Hinv[k, k] * (w_k - q_k) and
    eliminate row/column k from Hinv (Schur complement).  Uses no LDL factor, so it
    pins L independently.  Columns of X are independent here (Section 1)."""
    W = np.array(X, dtype=np.float64)
    m, n = W.shape
    G = np.asarray(A, dtype=np.float64).T @ np.asarray(A, dtype=np.float64)
    Hinv = np.linalg.inv(G)
    Z = np.zeros((m, n))
    for k in range(m):
        Z[k] = np.rint(W[k])
        err = (W[k] - Z[k]) / Hinv[k, k]
        W[k + 1:] -= np.outer(Hinv[k + 1:, k], err)
        Hinv[k + 1:, k + 1:] -= np.outer(Hinv[k + 1:, k], Hinv[k, k + 1:]) / Hinv[k, k]
    return Z


def local_errors_from_Z(X, Z, L, U):
    """Eq. 11 read backwards: once every entry is rounded, Z = X + L E U with the full
    E (L and U have unit diagonals), so E = L^{-1} (Z - X) U^{-1}."""
    R = np.asarray(Z, dtype=np.float64) - np.asarray(X, dtype=np.float64)
    T = sla.solve_triangular(L, R, lower=True, unit_diagonal=True)
    # E U = T  <=>  U^T E^T = T^T
    Et = sla.solve_triangular(U.T, T.T, lower=True, unit_diagonal=True)
    return Et.T.copy()


def certificate_margin(X, Z, L, U):
    """An integer matrix Z is the trajectory iff every |E_ij| < 1/2 for
    E = L^{-1} (Z - X) U^{-1}: the value entry (i,j) is rounded at is
    Y_ij = Z_ij - E_ij, it depends on earlier errors only, and Z_ij is its nearest
    integer exactly when |E_ij| < 1/2 (induction over any admissible order,
    Theorem 1).  Returns (margin, E) with margin = 1/2 - max|E|: the distance of
    the closest pre-rounding value from a half-integer.  margin > 0 certifies Z.
    """
    E = local_errors_from_Z(X, Z, L, U)
    return float(0.5 - np.max(np.abs(E))), E


def objective_from_errors(E, lamL, lamU):
    """|| A R B ||_F^2 = sum_ij E_ij^2 / (lamL_i lamU_j), because R = L E U and
    L^T G L = lamL^{-1}, U H U^T = lamU^{-1} (from the two LDL identities)."""
    return float(np.sum((E * E) / np.outer(lamL, lamU)))


def _pack(Z, E):
    return {"Z": Z.astype(np.int64), "E": E, "margin": float(0.5 - np.max(np.abs(E))) if E.size else 0.5}


# --------------------------------------------------------------------------- reverse order
# Section 2 ("Two-sided and Kronecker-factored rounding"): the same greedy rounding taken in
# reverse order, from the last row and column.  Coordinates of vec(X) are visited from the
# last to the first; everything "lower" becomes "upper".
def unit_upper_udu_of_inverse(S):
    """S^{-1} = F lam F^T with F unit UPPER triangular (the factor Algorithm 1 needs when it
    runs from the last coordinate to the first).  S = R^T R with R upper (ordinary Cholesky)
    gives S^{-1} = R^{-1} R^{-T}, so F = R^{-1} diag(R) and lam = diag(R)^{-2}."""
    S = np.asarray(S, dtype=np.float64)
    R = np.linalg.cholesky(S).T
    r = np.diag(R).copy()
    F = sla.solve_triangular(R, np.diag(r), lower=False)
    F = np.triu(F)
    np.fill_diagonal(F, 1.0)
    return F, 1.0 / (r * r)


def feedback_factors_reverse(A, B):
    """L~ unit upper with G^{-1} = L~ lam L~^T and U~ unit lower with H^{-1} = U~^T lam U~.
    Returns (Lr, Ur, lamL, lamU)."""
    G, H = gram_pair(A, B)
    Lr, lamL = unit_upper_udu_of_inverse(G)
    Urt, lamU = unit_upper_udu_of_inverse(H)
    return Lr, Urt.T.copy(), lamL, lamU


def adaptive_round_1d_reverse(x, F):
    """Algorithm 1 run from the last coordinate to the first with a unit upper F:
    z_k = round(y_k); E_k = z_k - y_k; y_{:k+1} += F_{:k+1,k} E_k."""
    y = np.array(x, dtype=np.float64)
    d = y.size
    z = np.zeros(d)
    E = np.zeros(d)
    for k in range(d - 1, -1, -1):
        z[k] = np.rint(y[k])
        E[k] = z[k] - y[k]
        y[:k + 1] += F[:k + 1, k] * E[k]
    return z, E


def vec_sweep_reverse(X, A, B):
    """The definition: reverse Algorithm 1 on vec(X) under the explicit Kronecker Gram."""
    X = np.asarray(X, dtype=np.float64)
    m, n = X.shape
    G, H = gram_pair(A, B)
    F, _ = unit_upper_udu_of_inverse(kron_gram(G, H))
    z, E = adaptive_round_1d_reverse(X.reshape(-1, order="F"), F)
    return _pack(z.reshape(m, n, order="F"), E.reshape(m, n, order="F"))


def sweep_gptq2d_reverse(X, Lr, Ur):
    """Algorithm 3 mirrored for the reverse order: anti-diagonals from the last to the first;
    every error is folded UP its column of C = L~ E and pushed up its column of Y through L~,
    then C_ij is pushed LEFT along row i of Y through U~."""
    Y = np.array(X, dtype=np.float64)
    m, n = Y.shape
    Z = np.zeros((m, n))
    E = np.zeros((m, n))
    C = np.zeros((m, n))
    for s in range(m + n - 2, -1, -1):
        idx = anti_diagonal(s, m, n)
        for (i, j) in idx:
            Z[i, j] = np.rint(Y[i, j])
            E[i, j] = Z[i, j] - Y[i, j]
            M = Lr[:i + 1, i] * E[i, j]
            C[:i + 1, j] += M
            Y[:i, j] += M[:i]
        for (i, j) in idx:
            Y[i, :j] += C[i, j] * Ur[j, :j]
    return _pack(Z, E)


def brute_force_trajectory_reverse(X, A, B):
    """Reverse-order greedy trajectory from the objective alone: coordinates from the last to
    the first; with the residuals of the already-rounded (later) coordinates fixed, minimise
    || (B^T (x) A) r ||_2 over the real residuals of the remaining ones."""
    X = np.asarray(X, dtype=np.float64)
    m, n = X.shape
    Mfull = np.kron(np.asarray(B, dtype=np.float64).T, np.asarray(A, dtype=np.float64))
    x = X.reshape(-1, order="F")
    d = m * n
    r = np.zeros(d)
    z = np.zeros(d)
    for k in range(d - 1, -1, -1):
        rhs = -Mfull[:, k + 1:] @ r[k + 1:]
        sol, *_ = np.linalg.lstsq(Mfull[:, :k + 1], rhs, rcond=None)
        z[k] = np.rint(x[k] + sol[k])
        r[k] = z[k] - x[k]
    return z.reshape(m, n, order="F")


def certificate_margin_reverse(X, Z, Lr, Ur):
    """The certificate for the reverse order: Z = X + L~ E U~, so E = L~^{-1} (Z - X) U~^{-1}
    and Z is the reverse trajectory iff every |E_ij| < 1/2.  Returns (margin, E)."""
    R = np.asarray(Z, dtype=np.float64) - np.asarray(X, dtype=np.float64)
    T = sla.solve_triangular(Lr, R, lower=False, unit_diagonal=True)
    Et = sla.solve_triangular(Ur.T, T.T, lower=False, unit_diagonal=True)
    E = Et.T.copy()
    return float(0.5 - np.max(np.abs(E))), E


def sweep_gptq2d_fp32(X, L, U):
    """Algorithm 3 with every value held and every operation rounded in IEEE single precision.

    TEST INFRASTRUCTURE (reduced-precision mode).  X, L, U are rounded to float32 first; the steps are those of
    Algorithm 3 in the paper's order (round, error, scale by the column of L, fold into C, push down; then push
    right from the folded C), with numpy float32 arithmetic: products and sums are rounded separately (no fused
    multiply-add).  Z is returned as int64, E and C as float32.  A tiled fp32 kernel sums in another order, so it
    agrees with this only up to fp32 rounding: entries whose pre-rounding value lies within that error of a
    half-integer may differ, and every such flip moves the entries below and to the right of it.
    """
    X = np.asarray(X, dtype=np.float32)
    L = np.asarray(L, dtype=np.float32)
    U = np.asarray(U, dtype=np.float32)
    m, n = X.shape
    Y = X.copy()
    C = np.zeros((m, n), dtype=np.float32)
    E = np.zeros((m, n), dtype=np.float32)
    Z = np.zeros((m, n), dtype=np.int64)
    for s in range(m + n - 1):
        lo, hi = max(0, s - n + 1), min(m - 1, s)
        rows = np.arange(lo, hi + 1)
        cols = s - rows
        y = Y[rows, cols]
        z = np.rint(y)
        e = (z - y).astype(np.float32)
        Z[rows, cols] = z.astype(np.int64)
        E[rows, cols] = e
        for i, j, eij in zip(rows, cols, e):            # fold and push down, column by column
            M = (L[i:, i] * eij).astype(np.float32)
            M[0] = eij                                    # L_ii = 1
            C[i:, j] = (C[i:, j] + M).astype(np.float32)
            Y[i + 1:, j] = (Y[i + 1:, j] + M[1:]).astype(np.float32)
        for i, j in zip(rows, cols):                     # push right from the folded C
            Y[i, j + 1:] = (Y[i, j + 1:] + (C[i, j] * U[j, j + 1:]).astype(np.float32)).astype(np.float32)
    return {"Z": Z, "E": E, "C": C, "margin": float(0.5 - np.max(np.abs(E))) if E.size else 0.5}
