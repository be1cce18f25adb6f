"""GPU parity at the full sizes of the benchmark workloads, in the launch configuration bench.py
times (all sequences of the microbatch, auto path, one workspace).

Two kinds of check per workload:
  * a narrow projection (the k/v shape) in full: every entry of K, the coefficients of both
    variants and every entry of dW against the oracle;
  * a wide projection on sampled outputs the oracle can compute one by one from the definition:
    K_ij for all pairs of a sample of sequences (their G_i materialised in float64), and a
    sampled block dW[rows, cols] = sum_i c_i G_i[rows, cols] over ALL sequences (the oracle is
    given the matching columns of dY and X, which is exactly that block of every G_i).
Tolerance: relative Frobenius error <= 2e-2 (bf16 inputs, float32 accumulation).
"""

import numpy as np
import pytest
import torch

from oracle import isopo_oracle as orc
from paper_2512_23353_b200 import workloads as wl
from tests._util import rel_fro, to_f64

pytestmark = pytest.mark.gpu
TOL = 2e-2


@pytest.fixture(scope="module")
def b():
    from paper_2512_23353_b200 import binding
    return binding


def _layer(w, name):
    return next(l for l in w.layers if l.name == name)


def _run(b, w, layer, variant, lam_scale=1e-3):
    off, A_host = wl.microbatch(w)
    T, B = int(off[-1]), len(A_host)
    X, dY = wl.layer_inputs_device(w, layer, T)
    A = torch.from_numpy(A_host).cuda()
    ws = b.alloc_workspace(b.BF16, T, layer.d_in, layer.d_out, B, b.PATH_AUTO)
    K = torch.empty((B, B), dtype=torch.float32, device="cuda")
    c = torch.empty(B, dtype=torch.float32, device="cuda")
    dW = torch.empty((layer.d_out, layer.d_in), dtype=torch.float32, device="cuda")
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.isopo_layer_gram(X, dY, off, K, ws, info, b.PATH_AUTO)
    lam = lam_scale * float(torch.diagonal(K).mean().item())  # the caller's regulariser: 1e-3 * mean(diag K)
    b.isopo_transform_advantages(K, A, variant, lam, c, info)
    b.isopo_weight_grad(X, dY, c, off, dW, ws, info, b.PATH_AUTO, 0.0)
    torch.cuda.synchronize()
    assert int(info.item()) == 0
    return X, dY, off, A, K, c, dW, lam


@pytest.mark.parametrize("workload,name", [("llm_1p5b", "k_proj"), ("llm_7b", "v_proj")])
def test_narrow_projection_in_full(b, workload, name):
    w = wl.WORKLOADS[workload]
    layer = _layer(w, name)
    X, dY, off, A, K, c, dW, lam = _run(b, w, layer, b.VAR_INTERACTING)
    G = orc.sequence_gradients(to_f64(X), to_f64(dY), off)
    K_o = orc.ntk(G)
    assert rel_fro(K.cpu().numpy(), K_o) <= TOL
    c_o = orc.transform_advantages(K_o, to_f64(A), orc.INTERACTING, lam)
    cond = np.linalg.cond(K_o + lam * np.eye(len(A)))
    assert rel_fro(c.cpu().numpy(), c_o) <= TOL * max(1.0, cond / 1e3), cond
    assert rel_fro(dW.cpu().numpy(), orc.weight_gradient(G, to_f64(c))) <= TOL
    # the simple variant on the same K
    c2 = torch.empty_like(c)
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.isopo_transform_advantages(K, A, b.VAR_NORMALISED, lam, c2, info)
    torch.cuda.synchronize()
    assert rel_fro(c2.cpu().numpy(), orc.transform_advantages(K_o, to_f64(A), orc.NORMALISED, lam)) <= TOL


@pytest.mark.parametrize("workload,name,n_sample", [("llm_1p5b", "gate_proj", 10), ("llm_7b", "down_proj", 5)])
def test_wide_projection_sampled(b, workload, name, n_sample):
    w = wl.WORKLOADS[workload]
    layer = _layer(w, name)
    X, dY, off, A, K, c, dW, lam = _run(b, w, layer, b.VAR_NORMALISED)
    B = len(A)
    L = np.diff(off)
    rng = np.random.default_rng(7)
    # the shortest and the longest sequence, and a random few of the shorter half (oracle cost ~ length)
    order = np.argsort(L)
    pick = sorted({int(order[0]), int(order[-1]), *rng.choice(order[: B // 2], size=n_sample - 2, replace=False).tolist()})
    rows = torch.cat([torch.arange(int(off[i]), int(off[i + 1])) for i in pick]).cuda()
    off_s = np.concatenate([[0], np.cumsum([L[i] for i in pick])]).astype(np.int64)
    G_s = orc.sequence_gradients(to_f64(X[rows]), to_f64(dY[rows]), off_s)
    K_s = orc.ntk(G_s)
    K_gpu = K.cpu().numpy()[np.ix_(pick, pick)]
    assert rel_fro(K_gpu, K_s) <= TOL
    assert np.max(np.abs(np.diag(K_gpu) - np.diag(K_s)) / np.diag(K_s)) <= TOL
    # off-diagonal entries are tiny for independent tokens: measure them on the Cauchy-Schwarz scale sqrt(K_ii K_jj)
    assert np.max(np.abs(K_gpu - K_s) / np.sqrt(np.outer(np.diag(K_s), np.diag(K_s)))) <= TOL
    del G_s
    # a sampled block of dW over all sequences, with the GPU's own coefficients
    m_idx = torch.from_numpy(np.sort(rng.choice(layer.d_out, size=32, replace=False))).cuda()
    n_idx = torch.from_numpy(np.sort(rng.choice(layer.d_in, size=64, replace=False))).cuda()
    G_blk = orc.sequence_gradients(to_f64(X[:, n_idx]), to_f64(dY[:, m_idx]), off)
    dW_blk = orc.weight_gradient(G_blk, to_f64(c))
    got = dW[m_idx][:, n_idx].cpu().numpy()
    assert rel_fro(got, dW_blk) <= TOL
    # coefficients of the simple variant follow from the GPU's own K exactly as the oracle's formula says
    c_from_K = orc.transform_advantages(to_f64(K), to_f64(A), orc.NORMALISED, lam)
    assert rel_fro(c.cpu().numpy(), c_from_K) <= 1e-5
