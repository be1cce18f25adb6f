"""GPU parity of isopo_layer_gram_shared_x: the Gram-route K of several projections that read the same
input, against the oracle per projection and against one isopo_layer_gram call per projection."""

import time

import numpy as np
import pytest
import torch

from oracle import isopo_oracle as orc
from tests._util import offdiag_rel_fro, rel_fro, to_f64

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
    ([1, 15, 16, 17, 63, 64, 65, 127, 129, 200], 256, [128, 64, 64]),   # ragged tails, three projections
    ([50, 7, 300, 64, 1], 320, [200, 72]),                              # widths off the 64-feature grid, two
    (list(range(10, 50)), 896, [896, 128, 128]),                        # q / k / v of the small-LLM block
    ([33] * 9, 8, [8]),                                                 # one projection: the plain Gram route
])
def test_shared_input_matches_oracle_and_single_calls(b, Ls, d_in, d_outs):
    X, dYs, off = _case(Ls, d_in, d_outs, 4000 + d_in)
    B, T = len(Ls), int(off[-1])
    Ks = [torch.full((B, B), float("nan"), device="cuda") for _ in d_outs]
    info = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = b.alloc_workspace(b.BF16, T, d_in, max(d_outs), B, b.PATH_GRAM)
    b.isopo_layer_gram_shared_x(X, dYs, off, Ks, ws, info)
    torch.cuda.synchronize()
    assert int(info.item()) == 0
    for dY, K, d in zip(dYs, Ks, d_outs):
        K_o = orc.ntk(orc.sequence_gradients(to_f64(X), to_f64(dY), off))
        Kh = K.cpu().numpy()
        assert np.array_equal(Kh, Kh.T)
        assert rel_fro(Kh, K_o) <= TOL and (B == 1 or offdiag_rel_fro(Kh, K_o) <= TOL)
        K1 = torch.empty(B, B, device="cuda")
        ws1 = b.alloc_workspace(b.BF16, T, d_in, d, B, b.PATH_GRAM)
        b.isopo_layer_gram(X, dY, off, K1, ws1, info, b.PATH_GRAM)
        torch.cuda.synchronize()
        assert rel_fro(Kh, K1.cpu().numpy()) <= 1e-4  # the same products, another order of the float atomics
    assert int(info.item()) == 0


def test_shared_input_argument_checks_and_time(b, capsys):
    Ls = np.random.default_rng(1).integers(16, 65, size=256).tolist()
    B = 256
    info = torch.zeros(1, dtype=torch.int32, device="cuda")

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(5):
            fn()
        torch.cuda.synchronize()
        return (time.perf_counter() - t0) / 5 * 1e3

    for name, d_outs in (("q/k/v", [896, 128, 128]), ("gate/up", [4864, 4864])):
        X, dYs, off = _case(Ls, 896, d_outs, 77)
        T = int(off[-1])
        Ks = [torch.empty(B, B, device="cuda") for _ in d_outs]
        ws = b.alloc_workspace(b.BF16, T, 896, max(d_outs), B, b.PATH_GRAM)
        together = timed(lambda: b.isopo_layer_gram_shared_x(X, dYs, off, Ks, ws, info))
        apart = timed(lambda: [b.isopo_layer_gram(X, dY, off, K, ws, info, b.PATH_GRAM) for dY, K in zip(dYs, Ks)])
        with capsys.disabled():
            print(f"\n[{name} of the short-rollouts block, T = {T}: shared X {together:.3f} ms, one call each {apart:.3f} ms]")
    assert int(info.item()) == 0
    with pytest.raises(b.IsopoError):
        b.isopo_layer_gram_shared_x(X, dYs * 2, off, Ks * 2, ws, info)          # four projections
    with pytest.raises(b.IsopoError):
        b.isopo_layer_gram_shared_x(X, dYs, off, Ks, ws[:4096], info)            # workspace too small
    with pytest.raises(b.IsopoError):
        b.isopo_layer_gram_shared_x(X.float(), [d.float() for d in dYs], off, Ks, ws, info)  # float32
