"""Pins for the fp64 oracle: closed forms, brute force on tiny inputs, invariants and a
hand-worked example.  None of the expected values below comes from the oracle itself or
from the CUDA path."""

import itertools
import json
import os

import numpy as np
import pytest

from oracle import isopo_oracle as orc

HERE = os.path.dirname(os.path.abspath(__file__))


def _problem(seed, B=5, d_in=6, d_out=4, lo=1, hi=7):
    rng = np.random.default_rng(seed)
    L = rng.integers(lo, hi + 1, size=B)
    off = np.concatenate([[0], np.cumsum(L)]).astype(np.int64)
    T = int(off[-1])
    X = rng.standard_normal((T, d_in))
    dY = rng.standard_normal((T, d_out))
    A = rng.standard_normal(B)
    return X, dY, off, A


def _G_bruteforce(X, dY, off):
    """Four nested Python loops, no matmul."""
    B = len(off) - 1
    G = np.zeros((B, dY.shape[1], X.shape[1]))
    for i in range(B):
        for t in range(off[i], off[i + 1]):
            for m in range(dY.shape[1]):
                for n in range(X.shape[1]):
                    G[i, m, n] += dY[t, m] * X[t, n]
    return G


def _gauss_solve(M, b):
    """Gaussian elimination with partial pivoting, written out (independent of eigh)."""
    M = np.array(M, dtype=np.float64)
    b = np.array(b, dtype=np.float64)
    n = len(b)
    for k in range(n):
        p = k + int(np.argmax(np.abs(M[k:, k])))
        if p != k:
            M[[k, p]] = M[[p, k]]
            b[[k, p]] = b[[p, k]]
        for r in range(k + 1, n):
            f = M[r, k] / M[k, k]
            M[r, k:] -= f * M[k, k:]
            b[r] -= f * b[k]
    x = np.zeros(n)
    for k in range(n - 1, -1, -1):
        x[k] = (b[k] - M[k, k + 1:] @ x[k + 1:]) / M[k, k]
    return x


# ----------------------------------------------------------------------------- hand example

def test_hand_worked_example():
    with open(os.path.join(HERE, "golden", "hand_example.json")) as f:
        g = json.load(f)
    X, dY, off, A = np.array(g["X"], float), np.array(g["dY"], float), np.array(g["offsets"]), np.array(g["A"], float)
    G = orc.sequence_gradients(X, dY, off)
    np.testing.assert_allclose(G, np.array(g["G"], float), rtol=0, atol=0)
    K = orc.ntk(G)
    np.testing.assert_allclose(K, np.array(g["K"], float), rtol=0, atol=0)
    F2 = np.array(g["F2_num"], float) / g["F2_den"]
    np.testing.assert_allclose(orc.fisher_norm_sq(K), F2, rtol=1e-15)
    np.testing.assert_allclose(orc.transform_advantages(K, A, orc.NORMALISED, 0.0), A / np.sqrt(F2), rtol=1e-15)
    np.testing.assert_allclose(orc.transform_advantages(K, A, orc.DIRECTION, 0.0),
                               A * np.array([8.0, 244.0]) / F2, rtol=1e-15)
    np.testing.assert_allclose(orc.transform_advantages(K, A, orc.EUCLID, 1.0),
                               A / np.sqrt(np.array([9.0, 245.0])), rtol=1e-15)
    c = orc.transform_advantages(K, A, orc.INTERACTING, float(g["lam_interacting"]))
    np.testing.assert_allclose(c, np.array(g["c_interacting_num"], float) / g["c_interacting_den"], rtol=1e-12)
    _, c2, dW = orc.isopo_layer(X, dY, off, A, orc.INTERACTING, float(g["lam_interacting"]))
    np.testing.assert_allclose(c2, c, rtol=1e-15)
    np.testing.assert_allclose(dW, np.array(g["dW_interacting_num"], float) / g["dW_interacting_den"], rtol=1e-12)


# ----------------------------------------------------------------------------- G and K

@pytest.mark.parametrize("seed", [0, 1, 2])
def test_G_matches_four_loop_bruteforce_and_Kii_is_its_norm(seed):
    X, dY, off, _ = _problem(seed)
    G = orc.sequence_gradients(X, dY, off)
    Gb = _G_bruteforce(X, dY, off)
    np.testing.assert_allclose(G, Gb, rtol=1e-13, atol=1e-13)
    K = orc.ntk(G)
    for i in range(len(off) - 1):
        assert K[i, i] == pytest.approx(float(np.sum(Gb[i] ** 2)), rel=1e-13)


@pytest.mark.parametrize("seed", [3, 4])
def test_K_equals_rank_one_route(seed):
    """Each token gradient is rank one (Eq. one / Eq. two): <d_t x_t^T, d_s x_s^T> = (d_t.d_s)(x_t.x_s),
    so K_ij = sum_{t in i, s in j} (d_t.d_s)(x_t.x_s) without ever forming G."""
    X, dY, off, _ = _problem(seed)
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    B = len(off) - 1
    K2 = np.zeros((B, B))
    for i in range(B):
        for j in range(B):
            for t in range(off[i], off[i + 1]):
                for s in range(off[j], off[j + 1]):
                    K2[i, j] += float(dY[t] @ dY[s]) * float(X[t] @ X[s])
    np.testing.assert_allclose(K, K2, rtol=1e-12, atol=1e-12)


def test_single_token_sequences_give_hadamard_of_token_grams():
    rng = np.random.default_rng(5)
    T = 9
    X, dY = rng.standard_normal((T, 5)), rng.standard_normal((T, 3))
    off = np.arange(T + 1)
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    np.testing.assert_allclose(K, (dY @ dY.T) * (X @ X.T), rtol=1e-13, atol=1e-13)


def test_single_sequence_is_frobenius_norm_of_textbook_gemm():
    X, dY, off, _ = _problem(6, B=1, lo=11, hi=11)
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    assert K.shape == (1, 1)
    assert K[0, 0] == pytest.approx(np.linalg.norm(dY.T @ X, "fro") ** 2, rel=1e-13)


@pytest.mark.parametrize("seed", [7, 8])
def test_K_symmetric_psd_cauchy_schwarz(seed):
    X, dY, off, _ = _problem(seed, B=7)
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    assert np.array_equal(K, K.T)
    assert np.linalg.eigvalsh(K).min() >= -1e-12 * np.trace(K)
    for i, j in itertools.combinations(range(7), 2):
        assert K[i, j] ** 2 <= K[i, i] * K[j, j] * (1 + 1e-12)


def test_K_permutation_and_scaling():
    X, dY, off, _ = _problem(9, B=4)
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    perm = [2, 0, 3, 1]
    Xp = np.concatenate([X[off[i]:off[i + 1]] for i in perm])
    dYp = np.concatenate([dY[off[i]:off[i + 1]] for i in perm])
    offp = np.concatenate([[0], np.cumsum([off[i + 1] - off[i] for i in perm])])
    Kp = orc.ntk(orc.sequence_gradients(Xp, dYp, offp))
    np.testing.assert_allclose(Kp, K[np.ix_(perm, perm)], rtol=1e-13)
    K3 = orc.ntk(orc.sequence_gradients(X, -3.0 * dY, off))
    np.testing.assert_allclose(K3, 9.0 * K, rtol=1e-13)


def test_orthogonal_supports_give_exactly_diagonal_K():
    rng = np.random.default_rng(10)
    B, per = 3, 2
    L = [3, 1, 4]
    off = np.concatenate([[0], np.cumsum(L)])
    X = np.zeros((off[-1], B * per))
    for i in range(B):
        X[off[i]:off[i + 1], i * per:(i + 1) * per] = rng.standard_normal((L[i], per))
    dY = rng.standard_normal((off[-1], 3))
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    assert np.count_nonzero(K - np.diag(np.diag(K))) == 0
    assert np.all(np.diag(K) > 0)


# ----------------------------------------------------------------------------- simple variants

@pytest.mark.parametrize("seed", [11, 12])
def test_normalised_variant_gives_unit_fisher_norm(seed):
    """With lam = 0 the re-scaled gradient w_i = c_i G_i / A_i has estimated Fisher norm 1:
    sum_j <w_i, G_j>^2 / sum_j ||G_j||^2 = 1, recomputed here from explicit G (not from K)."""
    X, dY, off, A = _problem(seed, B=6)
    Gb = _G_bruteforce(X, dY, off)
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    c = orc.transform_advantages(K, A, orc.NORMALISED, 0.0)
    den = sum(float(np.sum(Gb[j] ** 2)) for j in range(6))
    for i in range(6):
        w = (c[i] / A[i]) * Gb[i]
        num = sum(float(np.sum(w * Gb[j])) ** 2 for j in range(6))
        assert num / den == pytest.approx(1.0, rel=1e-12)


def test_fisher_norm_bounds_and_diagonal_closed_form():
    X, dY, off, _ = _problem(13, B=6)
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    F2 = orc.fisher_norm_sq(K)
    d = np.diag(K)
    assert np.all(F2 <= d * (1 + 1e-12))
    assert np.all(F2 >= d ** 2 / np.trace(K) * (1 - 1e-12))
    Kd = np.diag([2.0, 5.0, 0.5])
    np.testing.assert_allclose(orc.fisher_norm_sq(Kd), np.array([4.0, 25.0, 0.25]) / 7.5, rtol=1e-15)
    np.testing.assert_allclose(orc.fisher_norm_sq(Kd, normalise=False), np.array([4.0, 25.0, 0.25]) / 3.0, rtol=1e-15)


def test_simple_variants_single_sequence_and_large_lambda():
    K = np.array([[3.0]])
    A = np.array([-0.7])
    assert orc.transform_advantages(K, A, orc.NORMALISED, 0.25)[0] == pytest.approx(-0.7 / np.sqrt(3.25), rel=1e-15)
    assert orc.transform_advantages(K, A, orc.EUCLID, 0.25)[0] == pytest.approx(-0.7 / np.sqrt(3.25), rel=1e-15)
    assert orc.transform_advantages(K, A, orc.DIRECTION, 0.25)[0] == pytest.approx(-0.7 / 1.25, rel=1e-15)
    X, dY, off, A = _problem(14, B=5)
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    lam = 1e12 * np.trace(K)
    c = orc.transform_advantages(K, A, orc.NORMALISED, lam)
    np.testing.assert_allclose(np.sqrt(lam) * c, A, rtol=1e-10)   # behaves like norm clipping (Sec. 2.1)
    np.testing.assert_allclose(orc.transform_advantages(K, A, orc.REINFORCE), A, rtol=0)


def test_normalised_update_is_invariant_to_gradient_scale():
    X, dY, off, A = _problem(15, B=4)
    _, _, dW1 = orc.isopo_layer(X, dY, off, A, orc.NORMALISED, 0.0)
    _, _, dW2 = orc.isopo_layer(X, 17.0 * dY, off, A, orc.NORMALISED, 0.0)
    np.testing.assert_allclose(dW1, dW2, rtol=1e-12, atol=1e-14)


def test_general_rescaling_presets():
    """p = -1 reproduces the Sec. 2.1 update and r = -2 the Sec. 2.3 update (figure caption),
    up to the 1e-8 inside `reg`; q = -1 is Euclidean normalisation."""
    X, dY, off, A = _problem(16, B=5, d_in=8, d_out=8, lo=4, hi=9)
    K = orc.ntk(orc.sequence_gradients(X, 10 * dY, off))
    tol = dict(rtol=1e-7)
    np.testing.assert_allclose(orc.transform_advantages(K, A, orc.GENERAL, pqr=(-1, 0, 0)),
                               orc.transform_advantages(K, A, orc.NORMALISED, 0.0), **tol)
    np.testing.assert_allclose(orc.transform_advantages(K, A, orc.GENERAL, pqr=(0, 0, -2)),
                               orc.transform_advantages(K, A, orc.DIRECTION, 0.0), **tol)
    np.testing.assert_allclose(orc.transform_advantages(K, A, orc.GENERAL, pqr=(0, -1, 0)),
                               orc.transform_advantages(K, A, orc.EUCLID, 0.0), **tol)
    lamF = 0.3 * np.mean(orc.fisher_norm_sq(K))
    np.testing.assert_allclose(orc.transform_advantages(K, A, orc.GENERAL, pqr=(-1, 0, 0), regs=(lamF, 0, 0)),
                               orc.transform_advantages(K, A, orc.NORMALISED, lamF), **tol)
    # mixed exponents, written out independently
    F = np.sqrt((K ** 2).sum(1) / np.trace(K))
    n = np.sqrt(np.diag(K))
    want = A * (F * F + 0.5 + 1e-8) ** (-0.25) * (n * n + 2.0 + 1e-8) ** 0.5 * ((F / n) ** 2 + 0.1 + 1e-8) ** (-1.0)
    got = orc.transform_advantages(K, A, orc.GENERAL, pqr=(-0.5, 1.0, -2.0), regs=(0.5, 2.0, 0.1))
    np.testing.assert_allclose(got, want, rtol=1e-13)


# ----------------------------------------------------------------------------- interacting variant

@pytest.mark.parametrize("seed", [17, 18])
def test_interacting_solves_regularised_system(seed):
    X, dY, off, A = _problem(seed, B=6)
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    lam = 1e-3 * np.mean(np.diag(K))
    c = orc.transform_advantages(K, A, orc.INTERACTING, lam)
    assert np.linalg.norm((K + lam * np.eye(6)) @ c - A) <= 1e-12 * np.linalg.norm(A) * np.linalg.cond(K + lam * np.eye(6))
    np.testing.assert_allclose(c, _gauss_solve(K + lam * np.eye(6), A), rtol=1e-9)


def test_interacting_special_cases():
    A = np.array([1.0, -2.0, 0.5])
    Kd = np.diag([2.0, 5.0, 0.5])
    np.testing.assert_allclose(orc.transform_advantages(Kd, A, orc.INTERACTING, 0.5), A / np.array([2.5, 5.5, 1.0]), rtol=1e-14)
    assert orc.transform_advantages(np.array([[3.0]]), np.array([2.0]), orc.INTERACTING, 1.0)[0] == pytest.approx(0.5, rel=1e-15)
    # lam -> infinity: lam * c -> A with error <= ||K|| ||A|| / lam (scaled REINFORCE)
    X, dY, off, A = _problem(19, B=5)
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    for lam in (1e6, 1e9):
        lam_abs = lam * np.linalg.norm(K, 2)
        c = orc.transform_advantages(K, A, orc.INTERACTING, lam_abs)
        assert np.linalg.norm(lam_abs * c - A) <= np.linalg.norm(K, 2) * np.linalg.norm(A) / lam_abs * (1 + 1e-6) + 1e-15


def test_interacting_duplicate_sequences_get_equal_coefficients():
    X, dY, off, A = _problem(20, B=3, lo=3, hi=3)
    X2 = np.concatenate([X, X[off[1]:off[2]]])
    dY2 = np.concatenate([dY, dY[off[1]:off[2]]])
    off2 = np.concatenate([off, [off[-1] + 3]])
    A2 = np.concatenate([A, [A[1]]])
    K = orc.ntk(orc.sequence_gradients(X2, dY2, off2))
    c = orc.transform_advantages(K, A2, orc.INTERACTING, 0.1)
    assert c[1] == pytest.approx(c[3], rel=1e-10)


def test_interacting_update_is_the_parameter_space_ridge_solution():
    """v = J^T (K + lam I)^{-1} A (Sec. 3) equals (J^T J + lam I)^{-1} J^T A, the maximiser of
    v.(J^T A) - (1/2)||J v||^2 - (lam/2)||v||^2; checked with an N x N solve on a tiny layer."""
    X, dY, off, A = _problem(21, B=4, d_in=3, d_out=2)
    lam = 0.37
    K, c, dW = orc.isopo_layer(X, dY, off, A, orc.INTERACTING, lam)
    J = _G_bruteforce(X, dY, off).reshape(4, -1)
    v = _gauss_solve(J.T @ J + lam * np.eye(J.shape[1]), J.T @ A)
    np.testing.assert_allclose(dW.reshape(-1), v, rtol=1e-9, atol=1e-12)
    np.testing.assert_allclose(J @ v + lam * c, A, rtol=1e-9, atol=1e-12)


# ----------------------------------------------------------------------------- dW

def test_weight_gradient_special_cases():
    X, dY, off, A = _problem(22, B=5)
    G = orc.sequence_gradients(X, dY, off)
    K = orc.ntk(G)
    np.testing.assert_allclose(orc.weight_gradient(G, np.ones(5)), dY.T @ X, rtol=1e-12, atol=1e-12)
    e2 = np.zeros(5)
    e2[2] = 1.0
    np.testing.assert_allclose(orc.weight_gradient(G, e2), _G_bruteforce(X, dY, off)[2], rtol=1e-12, atol=1e-12)
    c1, c2 = np.random.default_rng(0).standard_normal((2, 5))
    np.testing.assert_allclose(orc.weight_gradient(G, 2 * c1 - 3 * c2),
                               2 * orc.weight_gradient(G, c1) - 3 * orc.weight_gradient(G, c2), rtol=1e-12, atol=1e-12)
    dW = orc.weight_gradient(G, c1)
    np.testing.assert_allclose([np.sum(dW * G[j]) for j in range(5)], K @ c1, rtol=1e-12)
    # REINFORCE: dW = (A o dY)^T X with A broadcast over each sequence's tokens
    _, c, dWr = orc.isopo_layer(X, dY, off, A, orc.REINFORCE)
    a_tok = np.repeat(A, np.diff(off))
    np.testing.assert_allclose(dWr, (a_tok[:, None] * dY).T @ X, rtol=1e-12, atol=1e-12)


# ----------------------------------------------------------------------------- planted mistakes are caught

# ----------------------------------------------------------------------------- Algorithm 1's sampled estimator
def _sampled_bruteforce(X, dY, off, rows):
    """Eq. (formal-F-norm) from its words: sum_j (v . g^(j))^2 / sum_j ||g^(j)||^2 with v = G_i as an
    explicit matrix (four-loop brute force) and every g^(j) = g_out_j a_in_j^T built as an explicit matrix."""
    G = _G_bruteforce(X, dY, off)
    gs = [np.outer(dY[j], X[j]) for j in rows]
    den = sum(float(np.sum(g * g)) for g in gs)
    return np.array([sum(float(np.sum(G[i] * g)) ** 2 for g in gs) / den for i in range(len(off) - 1)])


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_sampled_estimator_equals_explicit_rank_one_sum(seed):
    X, dY, off, _ = _problem(40 + seed)
    rng = np.random.default_rng(seed)
    rows = rng.permutation(int(off[-1]))[: max(1, int(off[-1]) // 2)]
    np.testing.assert_allclose(orc.sampled_fisher_norm_sq(X, dY, off, rows), _sampled_bruteforce(X, dY, off, rows),
                               rtol=1e-11)


def test_sampled_estimator_hand_example():
    # one sequence of two tokens, 1 x 1 layer: G = 2*3 + (-1)*4 = 2; sample = token 1: g0 = -1, a0 = 4
    # numerator (g0 * G * a0)^2 = (-8)^2 = 64, denominator (|g0| |a0|)^2 = 16  ->  F^2 = 4 = G^2
    X = np.array([[3.0], [4.0]])
    dY = np.array([[2.0], [-1.0]])
    F2 = orc.sampled_fisher_norm_sq(X, dY, [0, 2], [1])
    np.testing.assert_allclose(F2, [4.0], rtol=1e-14)
    np.testing.assert_allclose(orc.sampled_coefficients(F2, [3.0], lam=5.0), [1.0], rtol=1e-14)  # 3 / sqrt(4 + 5)


def test_sampled_estimator_with_all_tokens_of_single_token_sequences_is_the_K_only_estimator():
    """If every sequence is one token and every token is sampled, the position-wise samples ARE the
    sequence gradients, so Algorithm 1's estimate must equal sum_j K_ij^2 / sum_j K_jj."""
    rng = np.random.default_rng(5)
    T = 9
    X, dY = rng.standard_normal((T, 5)), rng.standard_normal((T, 3))
    off = np.arange(T + 1)
    K = (dY @ dY.T) * (X @ X.T)  # closed form for single-token sequences
    want = np.sum(K * K, axis=1) / np.trace(K)
    np.testing.assert_allclose(orc.sampled_fisher_norm_sq(X, dY, off, np.arange(T)), want, rtol=1e-11)
    np.testing.assert_allclose(orc.fisher_norm_sq(K), want, rtol=1e-12)


def test_sampled_estimator_invariances_and_bound():
    X, dY, off, A = _problem(77, B=6)
    T = int(off[-1])
    rows = np.array([0, T - 1, T // 2, 1])
    F2 = orc.sampled_fisher_norm_sq(X, dY, off, rows)
    # order of the samples does not matter; a repeated sample set gives the same ratio
    np.testing.assert_allclose(orc.sampled_fisher_norm_sq(X, dY, off, rows[::-1]), F2, rtol=1e-12)
    np.testing.assert_allclose(orc.sampled_fisher_norm_sq(X, dY, off, np.concatenate([rows, rows])), F2, rtol=1e-12)
    # Cauchy-Schwarz: (G . g^(j))^2 <= ||G||^2 ||g^(j)||^2, hence F_i^2 <= ||G_i||^2 = K_ii
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    assert np.all(F2 <= np.diag(K) * (1 + 1e-12))
    # scaling the back-propagated gradients by s scales G_i by s and every sample by s: F^2 scales by s^2
    np.testing.assert_allclose(orc.sampled_fisher_norm_sq(X, 3.0 * dY, off, rows), 9.0 * F2, rtol=1e-12)
    # a sample orthogonal to a sequence's gradient contributes nothing to it: d_in-disjoint supports
    Xo, dYo = np.zeros((4, 4)), np.ones((4, 2))
    Xo[0, 0] = Xo[1, 1] = 1.0   # sequence 0 lives on input coordinates 0, 1
    Xo[2, 2] = Xo[3, 3] = 1.0   # sequence 1 on 2, 3
    F2o = orc.sampled_fisher_norm_sq(Xo, dYo, [0, 2, 4], [0])   # the only sample is a token of sequence 0
    assert F2o[1] == 0.0 and F2o[0] > 0.0
    # the whole Algorithm-1 layer: dW = sum_i A_i / sqrt(F_i^2 + reg) G_i
    F2b, c, dW = orc.isopo_layer_sampled(X, dY, off, A, rows, lam=0.3)
    G = _G_bruteforce(X, dY, off)
    np.testing.assert_allclose(dW, sum(A[i] / np.sqrt(F2[i] + 0.3) * G[i] for i in range(6)), rtol=1e-11)


# ----------------------------------------------------------------------------- relative regulariser
def test_regulariser_means_and_ema():
    X, dY, off, _ = _problem(91, B=7)
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    m = orc.regulariser_means(K)
    # mean ||G_i||^2 is the mean eigenvalue of K, the statistic the interacting experiment names
    np.testing.assert_allclose(m[1], np.mean(np.linalg.eigvalsh(K)), rtol=1e-12)
    # diagonal K: F_i^2 = K_ii^2 / tr K, F_i^2 / K_ii = K_ii / tr K, whose mean is exactly 1 / B
    Kd = np.diag([1.0, 2.0, 5.0])
    np.testing.assert_allclose(orc.regulariser_means(Kd), [30.0 / 8.0 / 3.0, 8.0 / 3.0, 1.0 / 3.0], rtol=1e-14)
    # EMA: first update takes the value; n equal updates stay there; the closed form of the geometric weights
    s = (np.zeros(3), 0)
    s = orc.ema_update(s, [4.0, 4.0, 4.0], 0.9)
    np.testing.assert_allclose(s[0], 4.0)
    for _ in range(5):
        s = orc.ema_update(s, [4.0, 4.0, 4.0], 0.9)
    np.testing.assert_allclose(s[0], 4.0, rtol=1e-14)
    s = orc.ema_update(s, [14.0, 4.0, 4.0], 0.9)
    s = orc.ema_update(s, [4.0, 4.0, 4.0], 0.9)
    np.testing.assert_allclose(s[0][0], 4.0 + 0.9 * 0.1 * 10.0, rtol=1e-14)
    assert s[1] == 8


# ----------------------------------------------------------------------------- spectral form of Algorithm 2

def test_spectral_form_two_by_two_closed_form():
    """K = [[a, b], [b, a]]: eigenvalues a + b and a - b on (1, 1)/sqrt2 and (1, -1)/sqrt2, so
    c = (A1 + A2)/(2 (a + b + lam)) (1, 1) + (A1 - A2)/(2 (a - b + lam)) (1, -1); with the small direction
    cut off only the first term stays."""
    a, b, lam = 3.0, 1.0, 0.25
    K, A = np.array([[a, b], [b, a]]), np.array([2.0, -1.0])
    c, D = orc.spectral_coefficients(K, A, lam)
    hi, lo = (A[0] + A[1]) / (2 * (a + b + lam)), (A[0] - A[1]) / (2 * (a - b + lam))
    np.testing.assert_allclose(D, [a + b, a - b], rtol=1e-14)
    np.testing.assert_allclose(c, [hi + lo, hi - lo], rtol=1e-13)
    c_cut, _ = orc.spectral_coefficients(K, A, lam, rel_cutoff=0.6)  # 2 <= 0.6 * 4: dropped
    np.testing.assert_allclose(c_cut, [hi, hi], rtol=1e-13)
    c_keep, _ = orc.spectral_coefficients(K, A, lam, rel_cutoff=0.4)  # 2 > 0.4 * 4: kept
    np.testing.assert_allclose(c_keep, c, rtol=1e-14)


@pytest.mark.parametrize("seed", [41, 42])
def test_spectral_form_equals_elimination_and_its_spectrum_has_the_trace_and_determinant(seed):
    X, dY, off, A = _problem(seed, B=6)
    K = orc.ntk(orc.sequence_gradients(X, dY, off))
    lam = 1e-2 * np.mean(np.diag(K))
    c, D = orc.spectral_coefficients(K, A, lam)
    np.testing.assert_allclose(c, _gauss_solve(K + lam * np.eye(6), A), rtol=1e-9)
    assert np.all(np.diff(D) <= 0)
    assert np.sum(D) == pytest.approx(np.trace(K), rel=1e-12)
    # product of the shifted eigenvalues = determinant of the shifted matrix, by elimination pivots
    M = K + lam * np.eye(6)
    piv = 1.0
    M = M.copy()
    for k in range(6):
        piv *= M[k, k]
        M[k + 1:] -= np.outer(M[k + 1:, k] / M[k, k], M[k])
    assert np.prod(D + lam) == pytest.approx(piv, rel=1e-9)


def test_spectral_form_with_cutoff_on_a_rank_deficient_kernel_is_the_pseudo_inverse():
    """Two copies of every sequence: K has rank B/2.  With lam = 0 and the null directions cut off the
    result is the minimum-norm solution K^+ A (numpy's pinv, computed from the SVD)."""
    X, dY, off, A = _problem(43, B=3)
    G = orc.sequence_gradients(X, dY, off)
    K = orc.ntk(np.concatenate([G, G]))
    A2 = np.concatenate([A, 0.5 * A])
    c, D = orc.spectral_coefficients(K, A2, 0.0, rel_cutoff=1e-9)
    assert np.sum(D > 1e-9 * D[0]) == 3
    np.testing.assert_allclose(c, np.linalg.pinv(K, rcond=1e-9) @ A2, rtol=1e-8, atol=1e-12 * np.abs(c).max())
    np.testing.assert_allclose(c[:3], c[3:], rtol=1e-8)  # symmetric in the copies


def test_pins_catch_planted_mistakes(monkeypatch):
    """Each mistake planted in the oracle (an off-by-one partition, a one-sided kernel fill, a
    dropped normalisation, a wrong regulariser sign) makes a pin above fail."""
    true_seq, true_ntk, true_f2, true_tr = (orc.sequence_gradients, orc.ntk, orc.fisher_norm_sq,
                                            orc.transform_advantages)

    def seq_off_by_one(X, dY, off):
        off = np.asarray(off).copy()
        off[1:-1] += 1
        return true_seq(X, dY, off)

    def ntk_one_sided(G):
        return np.triu(true_ntk(G))

    def f2_unnormalised(K, normalise=True):
        return true_f2(K, normalise=False)

    def transform_wrong_sign(K, A, variant, lam=0.0, pqr=None, regs=None):
        return true_tr(K, A, variant, -lam, pqr, regs)

    true_sampled = orc.sampled_fisher_norm_sq

    def sampled_missing_normalisation(X, dY, off, rows):   # drops the division by sum_j ||g^(j)||^2
        Xs, dYs = np.asarray(X, float)[np.asarray(rows)], np.asarray(dY, float)[np.asarray(rows)]
        return true_sampled(X, dY, off, rows) * np.sum(np.sum(dYs * dYs, 1) * np.sum(Xs * Xs, 1))

    def sampled_transposed_samples(X, dY, off, rows):      # takes the samples' rows from the wrong end
        return true_sampled(X, dY, off, (int(np.asarray(off)[-1]) - 1) - np.asarray(rows))

    true_spec = orc.spectral_coefficients

    def spectral_cutoff_on_wrong_side(K, A, lam=0.0, rel_cutoff=0.0):  # keeps the small directions instead
        K, A = np.asarray(K, float), np.asarray(A, float)
        D, U = np.linalg.eigh(K)
        keep = D <= rel_cutoff * np.max(D) if rel_cutoff > 0 else np.ones_like(D, bool)
        return U @ (np.where(keep, 1.0 / (D + lam), 0.0) * (U.T @ A)), D[::-1].copy()

    def spectral_untransposed(K, A, lam=0.0, rel_cutoff=0.0):          # U (pre * (U A)) instead of U^T A
        K, A = np.asarray(K, float), np.asarray(A, float)
        D, U = np.linalg.eigh(K)
        return U @ ((1.0 / (D + lam)) * (U @ A)), D[::-1].copy()

    def spectral_ascending(K, A, lam=0.0, rel_cutoff=0.0):             # spectrum in eigh's order
        c, D = true_spec(K, A, lam, rel_cutoff)
        return c, D[::-1].copy()

    plants = [
        ("spectral_coefficients", spectral_cutoff_on_wrong_side, test_spectral_form_two_by_two_closed_form),
        ("spectral_coefficients", spectral_untransposed, lambda: test_spectral_form_equals_elimination_and_its_spectrum_has_the_trace_and_determinant(41)),
        ("spectral_coefficients", spectral_ascending, test_spectral_form_two_by_two_closed_form),
        ("sampled_fisher_norm_sq", sampled_missing_normalisation, test_sampled_estimator_hand_example),
        ("sampled_fisher_norm_sq", sampled_transposed_samples, lambda: test_sampled_estimator_equals_explicit_rank_one_sum(1)),
        ("sequence_gradients", seq_off_by_one, lambda: test_G_matches_four_loop_bruteforce_and_Kii_is_its_norm(0)),
        ("ntk", ntk_one_sided, lambda: test_K_equals_rank_one_route(3)),
        ("fisher_norm_sq", f2_unnormalised, lambda: test_normalised_variant_gives_unit_fisher_norm(11)),
        ("transform_advantages", transform_wrong_sign, lambda: test_interacting_solves_regularised_system(17)),
        ("transform_advantages", transform_wrong_sign, test_hand_worked_example),
    ]
    for name, wrong, pin in plants:
        monkeypatch.setattr(orc, name, wrong)
        with pytest.raises(AssertionError):
            pin()
        monkeypatch.undo()
        pin()
