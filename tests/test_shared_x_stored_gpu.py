"""GPU parity of isopo_layer_gram_shared_x_stored: the stored-gradient route for several projections that
read the same input.  One launch forms every projection's G_i; K and the weight gradient of each
projection are checked against the oracle (Alg. 2: per-layer NTK, dW = sum_i c_i G_i) and against one
isopo_layer_gram call per projection."""

import time

import numpy as np
import pytest
import torch

from oracle import isopo_oracle as orc
from tests._util import offdiag_rel_fro, rel_fro, report, to_f64

pytestmark = pytest.mark.gpu
TOL = 2e-2


@pytest.fixture(scope="module")
def b():
    from paper_2512_23353_b200 import binding
    return binding


def _case(Ls, d_in, d_outs, seed):
    rng = np.random.default_rng(seed)
    off = np.concatenate([[0], np.cumsum(Ls)]).astype(np.int64)
    T = int(off[-1])
    shared = rng.standard_normal((T, 3)).astype(np.float32)
    X = rng.standard_normal((T, d_in), dtype=np.float32) + shared @ rng.standard_normal((3, d_in)).astype(np.float32)
    dYs = [0.1 * (rng.standard_normal((T, d), dtype=np.float32) + shared @ rng.standard_normal((3, d)).astype(np.float32))
           for d in d_outs]
    to = lambda a: torch.from_numpy(a).cuda().bfloat16()  # noqa: E731
    return to(X), [to(d) for d in dYs], off


@pytest.mark.parametrize("Ls,d_in,d_outs", [
    ([1, 15, 16, 17, 63, 64, 65, 127, 129, 200], 256, [256, 512, 256]),  # ragged tails; every projection on 2-CTA tiles
    ([50, 7, 300, 64, 1], 320, [1000, 200]),                             # 8 and 2 row tiles, the last ones ragged
    ([700, 300, 1100], 1536, [1536, 256, 256]),                          # q / k / v of the 1.5B-class block
    (list(range(10, 50)), 896, [896, 128, 128]),                         # k / v with one row tile: one launch per projection
    ([33] * 9, 264, [256]),                                              # one projection
])
def test_shared_input_stored_route_matches_oracle(b, Ls, d_in, d_outs):
    X, dYs, off = _case(Ls, d_in, d_outs, 5000 + d_in)
    B, T = len(Ls), int(off[-1])
    Ks = [torch.full((B, B), float("nan"), device="cuda") for _ in d_outs]
    wss = [b.alloc_workspace(b.BF16, T, d_in, d, B, b.PATH_MATERIALISE) for d in d_outs]
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.isopo_layer_gram_shared_x_stored(X, dYs, off, Ks, wss, info)
    c = torch.linspace(-1.5, 2.0, B, device="cuda")
    for h, (dY, K, ws, d) in enumerate(zip(dYs, Ks, wss, d_outs)):
        dW = torch.full((d, d_in), float("nan"), device="cuda")
        b.isopo_weight_grad(X, dY, c, off, dW, ws, info, b.PATH_MATERIALISE, 0.0)   # the projection's own stored gradients
        torch.cuda.synchronize()
        assert int(info.item()) == 0
        G = orc.sequence_gradients(to_f64(X), to_f64(dY), off)
        K_o = orc.ntk(G)
        Kh = K.cpu().numpy()
        errs = dict(K=rel_fro(Kh, K_o), K_offdiag=offdiag_rel_fro(Kh, K_o) if B > 1 else 0.0,
                    dW=rel_fro(dW.cpu().numpy(), orc.weight_gradient(G, to_f64(c))))
        report(f"shared X, stored route, projection {h} ({d_in}->{d})", **errs)
        assert np.array_equal(Kh, Kh.T)
        assert max(errs.values()) <= TOL, errs
        K1 = torch.empty(B, B, device="cuda")
        ws1 = b.alloc_workspace(b.BF16, T, d_in, d, B, b.PATH_MATERIALISE)
        b.isopo_layer_gram(X, dY, off, K1, ws1, info, b.PATH_MATERIALISE)
        torch.cuda.synchronize()
        assert rel_fro(Kh, K1.cpu().numpy()) <= 1e-5  # the same stored values, another order of the float atomics
    assert int(info.item()) == 0


def test_shared_input_stored_route_argument_checks_and_time(b, capsys):
    from paper_2512_23353_b200 import workloads as wl
    w = wl.WORKLOADS["llm_1p5b"]
    off, _ = wl.microbatch(w)
    off = off[:65].copy()                       # the first 64 sequences of the 1.5B-class microbatch
    T, B = int(off[-1]), 64
    layers = {l.name: l for l in w.layers}
    X, dq = wl.layer_inputs_device(w, layers["q_proj"], T)
    _, dk = wl.layer_inputs_device(w, layers["k_proj"], T)
    _, dv = wl.layer_inputs_device(w, layers["v_proj"], T)
    dYs, d_outs = [dq, dk, dv], [1536, 256, 256]
    Ks = [torch.empty(B, B, device="cuda") for _ in d_outs]
    wss = [b.alloc_workspace(b.BF16, T, 1536, d, B, b.PATH_MATERIALISE) for d in d_outs]
    info = torch.zeros(1, dtype=torch.int32, device="cuda")

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(5):
            fn()
        torch.cuda.synchronize()
        return (time.perf_counter() - t0) / 5 * 1e3

    together = timed(lambda: b.isopo_layer_gram_shared_x_stored(X, dYs, off, Ks, wss, info))
    apart = timed(lambda: [b.isopo_layer_gram(X, dY, off, K, ws, info, b.PATH_MATERIALISE)
                           for dY, K, ws in zip(dYs, Ks, wss)])
    with capsys.disabled():
        print(f"\n[q/k/v of the 1.5B-class block, 64 sequences, T = {T}: shared X {together:.3f} ms, one call each {apart:.3f} ms]")
    assert int(info.item()) == 0
    with pytest.raises(b.IsopoError):
        b.isopo_layer_gram_shared_x_stored(X, dYs, off, Ks, [wss[0], wss[0], wss[2]], info)   # one workspace given twice
    with pytest.raises(b.IsopoError):
        b.isopo_layer_gram_shared_x_stored(X, dYs, off, Ks, [wss[0], wss[1], wss[2][:4096]], info)  # too small
    with pytest.raises(b.IsopoError):
        b.isopo_layer_gram_shared_x_stored(X.float(), [d.float() for d in dYs], off, Ks, wss, info)  # float32
