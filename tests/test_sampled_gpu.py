"""GPU parity of isopo_sampled_coefficients (Algorithm 1's token-sampled Fisher-norm estimator and
re-scaling) against the fp64 oracle on the same bits and the same sampled rows.
Tolerances: 1e-5 (float32 inputs), 2e-2 (bfloat16 inputs, float32 accumulation)."""

import numpy as np
import pytest
import torch

from oracle import isopo_oracle as orc
from paper_2512_23353_b200 import workloads as wl
from tests._util import rel_fro, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2512_23353_b200 import binding
    return binding


def _inputs(Ls, d_in, d_out, dtype, seed, correlated=True):
    rng = np.random.default_rng(seed)
    off = np.concatenate([[0], np.cumsum(Ls)]).astype(np.int64)
    T = int(off[-1])
    w = wl.Workload("t", "bf16", len(Ls), "uniform", 1, 1, 4, "half", seed=seed)
    X, dY = wl.layer_inputs_host(w, wl.LayerShape("l", d_in, d_out), T, correlated)
    A = rng.standard_normal(len(Ls)).astype(np.float32)
    to = lambda a: torch.from_numpy(a).cuda().to(dtype)  # noqa: E731
    return to(X), to(dY), off, torch.from_numpy(A).cuda(), rng


def _run(b, X, dY, off, rows, A, lam):
    B, T = len(off) - 1, X.shape[0]
    code = b.BF16 if X.dtype == torch.bfloat16 else b.F32
    ws = b.alloc_sampled_workspace(code, T, X.shape[1], dY.shape[1], B, len(rows))
    c = torch.empty(B, device="cuda")
    F2 = torch.empty(B, device="cuda")
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.isopo_sampled_coefficients(X, dY, off, rows, A, lam, c, ws, info, F2)
    dW = torch.empty(dY.shape[1], X.shape[1], device="cuda")
    b.isopo_weight_grad(X, dY, c, off, dW, ws, info, b.PATH_GRAM, 0.0)   # the same workspace serves the GEMM
    torch.cuda.synchronize()
    assert int(info.item()) == 0
    return F2, c, dW


CASES = [
    # (lengths, d_in, d_out, n_samples)
    ([16, 40, 64, 21, 33, 50, 17, 64], 64, 64, 32),          # the tiny float32 layer shape
    ([1, 15, 16, 17, 63, 64, 65, 127, 129, 200], 256, 128, 100),
    ([50, 7, 300, 64, 1], 320, 200, 7),                      # fewer samples than one tile row, ragged widths
    ([33] * 9, 8, 8, 130),                                   # samples span two 128-row tiles; repeated rows allowed
    (list(range(120, 160)), 896, 128, 256),
]


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 1e-5), (torch.bfloat16, 2e-2)])
@pytest.mark.parametrize("case", range(len(CASES)))
def test_sampled_coefficients_match_algorithm_1(b, dtype, tol, case):
    Ls, d_in, d_out, n_s = CASES[case]
    X, dY, off, A, rng = _inputs(Ls, d_in, d_out, dtype, 300 + case)
    T = int(off[-1])
    rows = rng.permutation(T)[:n_s] if n_s <= T else rng.integers(0, T, size=n_s)
    F2_o = orc.sampled_fisher_norm_sq(to_f64(X), to_f64(dY), off, rows)
    lam = 1e-3 * float(np.mean(F2_o))
    F2, c, dW = _run(b, X, dY, off, rows, A, lam)
    assert rel_fro(F2.cpu().numpy(), F2_o) <= tol
    assert np.max(np.abs(F2.cpu().numpy() - F2_o) / F2_o) <= 2 * tol     # every sequence on its own
    c_o = orc.sampled_coefficients(F2_o, to_f64(A), lam)
    assert rel_fro(c.cpu().numpy(), c_o) <= tol
    G = orc.sequence_gradients(to_f64(X), to_f64(dY), off)
    assert rel_fro(dW.cpu().numpy(), orc.weight_gradient(G, to_f64(c))) <= tol
    assert rel_fro(dW.cpu().numpy(), orc.weight_gradient(G, c_o)) <= 2 * tol


def test_sampled_all_tokens_of_single_token_sequences_equals_K_route(b):
    """L_i = 1 and every token sampled: Algorithm 1's estimate is sum_j K_ij^2 / tr K, i.e. what
    isopo_transform_advantages(NORMALISED) computes from the K of isopo_layer_gram."""
    X, dY, off, A, _ = _inputs([1] * 150, 128, 64, torch.bfloat16, 9)
    F2, c, _ = _run(b, X, dY, off, np.arange(150), A, 0.0)
    res = b.isopo_layer(X, dY, off, A, b.VAR_NORMALISED, 0.0, b.PATH_GRAM)
    assert rel_fro(c.cpu().numpy(), res.coeffs.cpu().numpy()) <= 2e-2


def test_sampled_argument_checks(b):
    X, dY, off, A, _ = _inputs([5, 6], 8, 8, torch.float32, 1)
    ws = b.alloc_sampled_workspace(b.F32, 11, 8, 8, 2, 4)
    c = torch.empty(2, device="cuda")
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(b.IsopoError) as e:
        b.isopo_sampled_coefficients(X, dY, off, [0, 11], A, 0.0, c, ws, info)      # row index out of range
    assert e.value.status == b.ERR_INVALID_ARG
    with pytest.raises(b.IsopoError) as e:
        b.isopo_sampled_coefficients(X, dY, off, [0, 1, 2] * 400, A, 0.0, c, ws, info)  # workspace sized for 4 samples
    assert e.value.status == b.ERR_WORKSPACE
    assert b.isopo_sampled_workspace_bytes(b.F32, 11, 8, 8, 2, b.MAX_SAMPLES + 1) == 0


def test_non_finite_input_never_writes_past_the_sample_rows(b):
    """100 samples fill only part of the last 128-row tile of the estimator's tensor-core kernel.  The
    rows of that tile past the last sample are zero, but a non-finite activation among the column
    tokens turns 0 * inf into NaN; those rows have no place in M^T and must write nothing.  The
    workspace is followed by a guard region that has to stay as it was; the result may be NaN."""
    Ls = [40] * 40
    X, dY, off, A, rng = _inputs(Ls, 256, 128, torch.bfloat16, 77)
    T, B, n_s = int(off[-1]), len(Ls), 100
    X[T // 2, 5] = float("inf")
    dY[T // 3, 9] = float("nan")
    n = b.isopo_sampled_workspace_bytes(b.BF16, T, 256, 128, B, n_s)
    guard = 1 << 20
    raw = torch.full((n + 1024 + guard,), 0x5A, dtype=torch.uint8, device="cuda")
    shift = (-raw.data_ptr()) % 1024
    ws = raw[shift:shift + n]
    c = torch.empty(B, device="cuda")
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    rows = rng.permutation(T)[:n_s]
    b.isopo_sampled_coefficients(X, dY, off, rows, A, 0.0, c, ws, info)
    torch.cuda.synchronize()
    assert int(info.item()) == 0
    assert bool((raw[shift + n:] == 0x5A).all()), "the estimator wrote past its workspace"
    assert bool((raw[:shift] == 0x5A).all())
    # and the call still works on finite inputs afterwards, in the same workspace
    X[T // 2, 5] = 1.0
    dY[T // 3, 9] = 0.0
    b.isopo_sampled_coefficients(X, dY, off, rows, A, 0.0, c, ws, info)
    torch.cuda.synchronize()
    F2_o = orc.sampled_fisher_norm_sq(to_f64(X), to_f64(dY), off, rows)
    assert rel_fro(c.cpu().numpy(), orc.sampled_coefficients(F2_o, to_f64(A), 0.0)) <= 2e-2
