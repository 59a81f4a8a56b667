"""Seeded synthetic inputs (X, A, B) for two-sided rounding.

This module only manufactures inputs.  It contains none of the method's
arithmetic (no Gram inverses, no feedback factors, no rounding) and imports
neither the CUDA binding nor the CPU oracle, so both may be fed from it.

The paper runs no experiments and names no data set; its only hint is that the
bases may come from factors of Kronecker-factored Hessian approximations of a
network layer (Section 6).  The five configurations below stand in for that.

Generator: numpy PCG64, ``np.random.default_rng(seed)``.  Draw order is fixed:
X first, then everything for A, then everything for B.

"Upper Cholesky" of a Gram S means the upper-triangular R with R^T R = S.  With
A = R_A the row Gram A^T A equals the generated Gram.  With B = R_B the column
Gram B B^T = R_B R_B^T is a different SPD matrix with the same spectrum; this is
the literal reading of the configuration text and is what is generated.
"""
from __future__ import annotations

import numpy as np

CONFIG_NAMES = ("c0_64x64", "c1_256x256", "c2_1024x4096", "c3_4096x4096", "c4_8192x8192")
CONFIG_SHAPES = ((64, 64), (256, 256), (1024, 4096), (4096, 4096), (8192, 8192))


def upper_cholesky(S):
    """Upper-triangular R with R^T R = S."""
    return np.ascontiguousarray(np.linalg.cholesky(S).T)


def scaled_gaussian_gram(rng, k, samples, sigma_log, damping, chunk=4096):
    """S S^T / samples + damping * mean(diag) * I with S (k x samples) standard normal
    and row i scaled by exp(sigma_log * N(0,1)).  sigma_log = 0 draws no scales."""
    if sigma_log > 0.0:
        scales = np.exp(sigma_log * rng.standard_normal(k))
    else:
        scales = np.ones(k)
    gram = np.zeros((k, k))
    done = 0
    while done < samples:                      # column chunks bound the memory held
        c = min(chunk, samples - done)
        S = rng.standard_normal((k, c))
        S *= scales[:, None]
        gram += S @ S.T
        done += c
    gram /= samples
    gram = 0.5 * (gram + gram.T)
    gram[np.diag_indices(k)] += damping * float(np.mean(np.diag(gram)))
    return gram


def spectrum_gram(rng, k, cond):
    """Q diag(geomspace(1, 1/cond, k)) Q^T with Q from the QR of a Gaussian matrix."""
    Q, _ = np.linalg.qr(rng.standard_normal((k, k)))
    ev = np.geomspace(1.0, 1.0 / cond, k)
    gram = (Q * ev[None, :]) @ Q.T
    return 0.5 * (gram + gram.T)


def gaussian_like(m, n, seed, x_sigma=8.0, samples=512, sigma_log=1.0, damping=0.01):
    """The c0 / c1 recipe at any shape: X ~ N(0, x_sigma^2); A, B upper Cholesky of
    scaled Gaussian Grams."""
    rng = np.random.default_rng(seed)
    X = x_sigma * rng.standard_normal((m, n))
    A = upper_cholesky(scaled_gaussian_gram(rng, m, samples, sigma_log, damping))
    B = upper_cholesky(scaled_gaussian_gram(rng, n, samples, sigma_log, damping))
    return X, A, B


def llm_layer_like(m, n, seed, samples=4096, sigma_log=1.5, damping=0.01,
                   outlier_frac=1e-3, outlier_gain=20.0):
    """The c2 recipe: X = W / 0.02, W ~ N(0, 0.02^2) with a fraction of entries
    multiplied by outlier_gain; activation-style Grams with heavy-tailed channel
    scales."""
    rng = np.random.default_rng(seed)
    W = 0.02 * rng.standard_normal((m, n))
    mask = rng.random((m, n)) < outlier_frac
    W[mask] *= outlier_gain
    X = W / 0.02
    A = upper_cholesky(scaled_gaussian_gram(rng, m, samples, sigma_log, damping))
    B = upper_cholesky(scaled_gaussian_gram(rng, n, samples, sigma_log, damping))
    return X, A, B


def ill_conditioned_like(m, n, seed, cond=1e6, half_range=7.5):
    """The c3 recipe: X ~ Uniform(-half_range, half_range); Grams with a geometric
    spectrum of the given condition number."""
    rng = np.random.default_rng(seed)
    X = rng.uniform(-half_range, half_range, size=(m, n))
    A = upper_cholesky(spectrum_gram(rng, m, cond))
    B = upper_cholesky(spectrum_gram(rng, n, cond))
    return X, A, B


def headline_like(m, n, seed, x_sigma=4.0, samples=None, damping=0.01):
    """The c4 recipe: X ~ N(0, x_sigma^2); plain Gaussian Grams from 2*max(m,n)
    samples (8192 x 16384 at full size) with 1 % damping, no channel scales."""
    if samples is None:
        samples = 2 * max(m, n)
    rng = np.random.default_rng(seed)
    X = x_sigma * rng.standard_normal((m, n))
    A = upper_cholesky(scaled_gaussian_gram(rng, m, samples, 0.0, damping))
    B = upper_cholesky(scaled_gaussian_gram(rng, n, samples, 0.0, damping))
    return X, A, B


def make_config(index, seed=0, variant=None):
    """Inputs of configuration ``index`` (0..4) at full size.

    variant (c1 only in the configuration list, accepted everywhere):
      "B=I"   -> B replaced by the identity (one-sided reduction)
      "A=B=I" -> both bases replaced by the identity (round-to-nearest)
    """
    m, n = CONFIG_SHAPES[index]
    if index in (0, 1):
        X, A, B = gaussian_like(m, n, seed)
    elif index == 2:
        X, A, B = llm_layer_like(m, n, seed)
    elif index == 3:
        X, A, B = ill_conditioned_like(m, n, seed)
    elif index == 4:
        X, A, B = headline_like(m, n, seed)
    else:
        raise ValueError("configuration index must be 0..4")
    if variant == "B=I":
        B = np.eye(n)
    elif variant == "A=B=I":
        A = np.eye(m)
        B = np.eye(n)
    elif variant is not None:
        raise ValueError("unknown variant %r" % (variant,))
    return X, A, B


def general_bases(m, n, seed):
    """Small dense NON-triangular nonsingular A, B and a Gaussian X (edge-case tests:
    the method takes general bases, the five configurations happen to be triangular)."""
    rng = np.random.default_rng(seed)
    X = 3.0 * rng.standard_normal((m, n))
    A = rng.standard_normal((m, m)) + 2.0 * np.eye(m)
    B = rng.standard_normal((n, n)) + 2.0 * np.eye(n)
    return X, A, B
