"""fp64 CPU oracle for the ISOPO per-linear-layer hot path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  It shares no code with the CUDA path and
must never be imported by the product (`paper_2512_23353_b200`): only the test
suite, the smoke check and the benchmark's CPU-baseline leg may call it.

Everything is numpy float64.  A `numpy.matmul` / `numpy.linalg.eigh` call is
used as a single library step where the paper's listing uses the matching
torch call; there is no blocking, fusion or reordering beyond the listings.

Notation (paper's listing name in brackets):
  X   [T, d_in]   layer input activations of the packed microbatch  [act_in]
  dY  [T, d_out]  back-propagated output gradients delta            [grad_out]
  off [B+1]       sequence i owns token rows off[i] .. off[i+1]-1   [indices_by_sequence]
  G_i [d_out, d_in]  per-sequence log-prob gradient of the weight   [seq_logprob_grad]
  K   [B, B]      layer NTK  K_ij = <G_i, G_j>                      [ntk]
  A   [B]         advantages                                        [microbatch.advantages]
  c   [B]         transformed advantages (coefficients)
  dW  [d_out, d_in]  weight gradient  sum_i c_i G_i                 [mod.grad increment]

Readings of the paper taken where it is silent or ambiguous (each is restated
next to the function it affects):
  * Fisher norm from K alone: Eq. (F-norm-basic) with the B reduced
    per-sequence gradients as the sample set, normalised by the summed sample
    scale as Eq. (formal-F-norm) does:  F_i^2 = sum_j K_ij^2 / sum_j K_jj.
  * the coefficient multiplies G_i (the second `rescaling` listing returns
    `scaling * grad`); regularisation terms are absolute numbers supplied by
    the caller; no 1/n, 1/B or 1/T factor appears anywhere.

The token-sampled Fisher-norm estimator of Algorithm 1 (`sampled_fisher_norm_sq`) takes the sampled
row indices as an input; the K-only estimator above is the same formula with whole sequences as samples.

Pin status: every function below is pinned by closed forms, brute force and
invariants in tests/test_oracle_pins.py (the paper prints no numeric example).
"""

from __future__ import annotations

import numpy as np

REINFORCE = "reinforce"
NORMALISED = "normalised"          # Sec. 2.1 update  (p = -1)
NORMALISED_RAW = "normalised_raw"  # Eq. (F-norm-basic) without the scale normalisation
DIRECTION = "direction"            # Sec. 2.3 update  (r = -2)
EUCLID = "euclid"                  # q = -1 of the generalised re-scaling figure
GENERAL = "general"                # generalised re-scaling figure, free p, q, r
INTERACTING = "interacting"        # Sec. 3 / Algorithm 2

EPS_FIG3 = 1e-8                    # the constant inside `reg` of the generalised re-scaling figure


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def sequence_gradients(X, dY, off):
    """G_i = dY_i^T X_i for every sequence (Algorithm 1 and 2: `grad_out.T @ act_in`
    inside the loop over `indices_by_sequence`).  Returns [B, d_out, d_in]."""
    off = np.asarray(off, dtype=np.int64)
    B = off.shape[0] - 1
    G = np.empty((B, dY.shape[1], X.shape[1]), dtype=np.float64)
    for i in range(B):
        rows = slice(int(off[i]), int(off[i + 1]))
        G[i] = _f64(dY[rows]).T @ _f64(X[rows])
    return G


def ntk(G):
    """K_ij = sum(G_i * G_j), filled symmetrically (Algorithm 2, "make neural
    tangent kernel"; K = J J^T of Sec. 3)."""
    B = G.shape[0]
    K = np.empty((B, B), dtype=np.float64)
    for i in range(B):
        for j in range(i, B):
            K[i, j] = np.sum(G[i] * G[j])
            K[j, i] = K[i, j]
    return K


def fisher_norm_sq(K, normalise=True):
    """Squared Fisher norm of each sequence gradient, from K alone.

    Eq. (F-norm-basic): ||v||_F^2 ~ (1/n) sum_j (v . g_j)^2 with v = G_i and the
    samples g_j = G_j, so (v . g_j) = K_ij.  With `normalise` the estimate is
    divided by the average sample scale (1/n) sum_j ||g_j||^2 = tr(K)/n, as
    Eq. (formal-F-norm) does, giving sum_j K_ij^2 / sum_j K_jj.
    """
    K = _f64(K)
    B = K.shape[0]
    F2 = np.empty(B, dtype=np.float64)
    for i in range(B):
        F2[i] = np.sum(K[i] * K[i])
    if normalise:
        return F2 / np.trace(K)
    return F2 / B


def sampled_fisher_norm_sq(X, dY, off, sample_rows):
    """Squared Fisher norm of every sequence gradient from sampled token positions (Sec. 2.2,
    Eq. formal-F-norm with the "Efficient implementation" identities Eq. one and Eq. two).

    Sample j is the token gradient of row r_j = sample_rows[j] (drawn by the caller), the rank-one matrix
    g_j = dY[r_j] X[r_j]^T.  For v = G_i the estimator is
        F_i^2 = sum_j <G_i, g_j>^2 / sum_j ||g_j||^2,
    with <G_i, g_j> = dY[r_j] . (G_i X[r_j])      (Eq. one: the overlap with a rank-one matrix)
    and  ||g_j||^2  = ||dY[r_j]||^2 ||X[r_j]||^2  (Eq. two).
    Every G_i is materialised.  Returns F^2, [B].
    """
    X, dY = _f64(X), _f64(dY)
    off = np.asarray(off, dtype=np.int64)
    r = np.asarray(sample_rows, dtype=np.int64)
    x_s, d_s = X[r], dY[r]
    sample_norms_sq = np.sum(d_s * d_s, axis=1) * np.sum(x_s * x_s, axis=1)
    total = np.sum(sample_norms_sq)
    B = off.shape[0] - 1
    F2 = np.empty(B, dtype=np.float64)
    for i in range(B):
        lo, hi = int(off[i]), int(off[i + 1])
        G_i = dY[lo:hi].T @ X[lo:hi]
        overlaps = np.array([d_s[j] @ (G_i @ x_s[j]) for j in range(r.shape[0])])
        F2[i] = np.sum(overlaps ** 2) / total
    return F2


def sampled_coefficients(F2, A, lam=0.0):
    """Algorithm 1's re-scaling: c_i = A_i / sqrt(F_norm_i^2 + regularization)."""
    return _f64(A) / np.sqrt(_f64(F2) + lam)


def isopo_layer_sampled(X, dY, off, A, sample_rows, lam=0.0):
    """Algorithm 1 as printed: (X, dY, partition, A, sampled rows) -> (F_norm^2, c, dW)."""
    F2 = sampled_fisher_norm_sq(X, dY, off, sample_rows)
    c = sampled_coefficients(F2, A, lam)
    return F2, c, weight_gradient(sequence_gradients(X, dY, off), c)


def transform_advantages(K, A, variant, lam=0.0, pqr=None, regs=None):
    """Advantages -> per-sequence coefficients c, with dW = sum_i c_i G_i.

    REINFORCE    c_i = A_i
    NORMALISED   c_i = A_i / sqrt(F_i^2 + lam)             (display in Sec. 2.1)
    DIRECTION    c_i = A_i / (F_i^2 / ||G_i||^2 + lam)     (display in Sec. 2.3)
    EUCLID       c_i = A_i / sqrt(||G_i||^2 + lam)         (q = -1 in the generalised figure)
    GENERAL      c_i = A_i * reg2(F_i)^p * reg2(||G_i||)^q * reg2(F_i/||G_i||)^r
                 with reg2(v) = sqrt(v^2 + reg + 1e-8)     (generalised re-scaling figure;
                 `regs` = the three absolute regularisation terms, in that order)
    INTERACTING  c = U diag(1/(D + lam)) U^T A, K = U D U^T  (Algorithm 2; equals
                 (K + lam I)^{-1} A of the display in Sec. 3)
    ||G_i||^2 = K_ii.
    """
    K, A = _f64(K), _f64(A)
    n2 = np.diag(K).copy()
    if variant == REINFORCE:
        return A.copy()
    if variant == INTERACTING:
        D, U = np.linalg.eigh(K)
        return U @ ((1.0 / (D + lam)) * (U.T @ A))
    F2 = fisher_norm_sq(K, normalise=(variant != NORMALISED_RAW))
    if variant in (NORMALISED, NORMALISED_RAW):
        return A / np.sqrt(F2 + lam)
    if variant == DIRECTION:
        return A / (F2 / n2 + lam)
    if variant == EUCLID:
        return A / np.sqrt(n2 + lam)
    if variant == GENERAL:
        p, q, r = pqr
        reg_F, reg_G, reg_rel = (0.0, 0.0, 0.0) if regs is None else regs
        F = np.sqrt(F2)
        Gn = np.sqrt(n2)
        rel = F / Gn

        def reg2(val, reg):
            return np.sqrt(val ** 2 + reg + EPS_FIG3)

        return A * reg2(F, reg_F) ** p * reg2(Gn, reg_G) ** q * reg2(rel, reg_rel) ** r
    raise ValueError(f"unknown variant {variant!r}")


def spectral_coefficients(K, A, lam=0.0, rel_cutoff=0.0):
    """The interacting transform in the spectral form Algorithm 2 prints, with its spectrum returned:
    K = U D U^T (symmetric eigendecomposition), preconditioner 1 / (D + lam) per eigen-direction,
    c = U (preconditioner * (U^T A)).  Directions whose eigenvalue is not above rel_cutoff * max(D) are
    left out of the sum (rel_cutoff = 0 and a positive definite K: every direction, i.e. the
    interacting variant; lam = 0 with a cut-off: the pseudo-inverse on the kept range).
    Returns (c, D sorted from the largest down)."""
    K, A = _f64(K), _f64(A)
    D, U = np.linalg.eigh(K)
    keep = D > rel_cutoff * np.max(D)
    pre = np.where(keep, 1.0 / np.where(keep, D + lam, 1.0), 0.0)
    return U @ (pre * (U.T @ A)), D[::-1].copy()


def regulariser_means(K):
    """Microbatch means of the quantities the relative regulariser is added to (generalised
    re-scaling figure: `reg(val) = val + regularization * expectation(val)`):
    (mean_i F_i^2, mean_i ||G_i||^2, mean_i F_i^2/||G_i||^2).  mean_i ||G_i||^2 = tr K / B is also the
    mean eigenvalue `mean(D)` that the interacting experiment regularises with."""
    K = _f64(K)
    F2 = fisher_norm_sq(K)
    n2 = np.diag(K)
    return np.array([np.mean(F2), np.mean(n2), np.mean(F2 / n2)])


def ema_update(state, means, decay):
    """Running mean over microbatches ("EMA over minibatches with 0.9 decay").  state = (values[3],
    number of updates); the first update takes the means themselves."""
    values, n = state
    means = _f64(means)
    if n == 0:
        return means.copy(), 1
    return decay * _f64(values) + (1.0 - decay) * means, n + 1


def weight_gradient(G, c):
    """dW = sum_i c_i G_i (Algorithm 1: `grad += advantages[seq_id] * rescaled
    seq_logprob_grad`; Algorithm 2: `stack(seq_grads, -1) @ advantages_preconditioned`)."""
    G, c = _f64(G), _f64(c)
    dW = np.zeros(G.shape[1:], dtype=np.float64)
    for i in range(G.shape[0]):
        dW += c[i] * G[i]
    return dW


def isopo_layer(X, dY, off, A, variant, lam=0.0, pqr=None, regs=None):
    """Whole per-layer path: (X, dY, partition, A) -> (K, c, dW)."""
    G = sequence_gradients(X, dY, off)
    K = ntk(G)
    c = transform_advantages(K, A, variant, lam, pqr, regs)
    return K, c, weight_gradient(G, c)
