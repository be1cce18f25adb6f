"""Tensor-parallel sharding of the layer path (output features split across ranks, one all-reduce of K).

CPU part: two gloo ranks, each with the oracle's partial K of its own columns of dY; after
tp.allreduce_K both hold the oracle's full K, and the row blocks of dW computed from the shards stack
to the full dW.  GPU part (one GPU): the two shards are run one after the other through the library,
their K summed on the device as the all-reduce would, and the result compared with the unsharded call
and with the oracle."""

import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from oracle import isopo_oracle as orc  # noqa: E402
from paper_2512_23353_b200 import tp  # noqa: E402


def _problem(seed=5, d_in=24, d_out=32):
    rng = np.random.default_rng(seed)
    Ls = rng.integers(1, 9, size=6)
    off = np.concatenate([[0], np.cumsum(Ls)]).astype(np.int64)
    T = int(off[-1])
    shared = rng.standard_normal((T, 2))
    X = rng.standard_normal((T, d_in)) + shared @ rng.standard_normal((2, d_in))
    dY = 0.1 * (rng.standard_normal((T, d_out)) + shared @ rng.standard_normal((2, d_out)))
    A = rng.standard_normal(len(Ls))
    return X, dY, off, A


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    X, dY, off, A = _problem()
    lo, hi = tp.shard_columns(dY.shape[1], rank, world)
    G_loc = orc.sequence_gradients(X, dY[:, lo:hi], off)
    K = torch.from_numpy(orc.ntk(G_loc))
    tp.allreduce_K(K)
    c = orc.transform_advantages(K.numpy(), A, orc.INTERACTING, 0.05)
    np.savez(os.path.join(out_dir, f"r{rank}.npz"), K=K.numpy(), c=c, dW=orc.weight_gradient(G_loc, c), lo=lo, hi=hi)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_sum_partial_K(tmp_path):
    port = 31500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    X, dY, off, A = _problem()
    G = orc.sequence_gradients(X, dY, off)
    K_o = orc.ntk(G)
    c_o = orc.transform_advantages(K_o, A, orc.INTERACTING, 0.05)
    dW_o = orc.weight_gradient(G, c_o)
    r = [np.load(tmp_path / f"r{k}.npz") for k in range(2)]
    for k in range(2):
        np.testing.assert_allclose(r[k]["K"], K_o, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(r[k]["c"], c_o, rtol=1e-9)
    assert (int(r[0]["lo"]), int(r[0]["hi"]), int(r[1]["lo"]), int(r[1]["hi"])) == (0, 16, 16, 32)
    np.testing.assert_allclose(np.vstack([r[0]["dW"], r[1]["dW"]]), dW_o, rtol=1e-9, atol=1e-12)


def test_shard_columns_covers_every_column_once():
    for d, world in ((32, 2), (8960, 8), (1536, 4), (24, 3), (40, 4)):
        spans = [tp.shard_columns(d, r, world) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == d
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        assert all((hi - lo) % 8 == 0 and hi > lo for lo, hi in spans)
    with pytest.raises(ValueError):
        tp.shard_columns(20, 0, 2)
    with pytest.raises(ValueError):
        tp.shard_columns(16, 0, 4)


def test_allreduce_is_identity_without_a_group():
    K = torch.arange(4.0).reshape(2, 2)
    assert torch.equal(tp.allreduce_K(K.clone()), K)


@pytest.mark.gpu
@pytest.mark.parametrize("route", ["materialise", "gram"])
def test_two_shards_on_one_gpu_equal_the_unsharded_layer(route):
    from paper_2512_23353_b200 import binding as b
    from tests._util import rel_fro, to_f64

    rng = np.random.default_rng(21)
    Ls = rng.integers(20, 200, size=24)
    off = np.concatenate([[0], np.cumsum(Ls)]).astype(np.int64)
    T = int(off[-1])
    shared = rng.standard_normal((T, 3)).astype(np.float32)
    X = torch.from_numpy(rng.standard_normal((T, 320), dtype=np.float32) + shared @ rng.standard_normal((3, 320)).astype(np.float32)).cuda().bfloat16()
    dY = torch.from_numpy(0.1 * (rng.standard_normal((T, 512), dtype=np.float32) + shared @ rng.standard_normal((3, 512)).astype(np.float32))).cuda().bfloat16()
    A = torch.from_numpy(rng.standard_normal(24).astype(np.float32)).cuda()
    path = b.PATH_MATERIALISE if route == "materialise" else b.PATH_GRAM
    full = b.isopo_layer(X, dY, off, A, b.VAR_INTERACTING, 0.0, path)  # K only; lambda follows from it
    lam = 1e-2 * float(torch.diagonal(full.K).mean().item())
    full = b.isopo_layer(X, dY, off, A, b.VAR_INTERACTING, lam, path)
    assert full.info == 0
    # the ranks' work, one after the other: partial K of each shard, summed as the all-reduce does
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    shards, K_sum = [], torch.zeros(24, 24, device="cuda")
    for r in range(2):
        lo, hi = tp.shard_columns(512, r, 2)
        dY_loc = dY[:, lo:hi].contiguous()
        ws = b.alloc_workspace(b.BF16, T, 320, hi - lo, 24, path)
        K_part = torch.empty(24, 24, device="cuda")
        b.isopo_layer_gram(X, dY_loc, off, K_part, ws, info, path)
        K_sum += K_part
        shards.append((dY_loc, ws))
    c = torch.empty(24, device="cuda")
    b.isopo_transform_advantages(K_sum, A, b.VAR_INTERACTING, lam, c, info)
    rows = []
    for dY_loc, ws in shards:
        dW_loc = torch.empty(dY_loc.shape[1], 320, device="cuda")
        b.isopo_weight_grad(X, dY_loc, c, off, dW_loc, ws, info, path, 0.0)
        rows.append(dW_loc)
    torch.cuda.synchronize()
    assert int(info.item()) == 0
    dW = torch.cat(rows)
    G = orc.sequence_gradients(to_f64(X), to_f64(dY), off)
    K_o = orc.ntk(G)
    assert rel_fro(K_sum.cpu().numpy(), K_o) <= 2e-2
    assert rel_fro(K_sum.cpu().numpy(), full.K.cpu().numpy()) <= 1e-4  # same products, other summation order
    assert rel_fro(dW.cpu().numpy(), orc.weight_gradient(G, to_f64(c))) <= 2e-2
    assert rel_fro(dW.cpu().numpy(), full.dW.cpu().numpy()) <= 2e-2
    # the single-rank form of the composed call is the plain layer
    one = tp.isopo_layer_tp(X, dY, off, A, b.VAR_INTERACTING, lam, path=path)
    assert one.info == 0 and rel_fro(one.dW.cpu().numpy(), full.dW.cpu().numpy()) <= 1e-3  # atomics order in K, through the solve
