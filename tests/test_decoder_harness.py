"""The end-to-end harness (bench_decoder.py) on a toy decoder: every linear layer's weight gradient,
as the harness's backward hook produces it through the library, must equal the oracle's ISOPO layer
on the (X, dY) that reached that hook; and the plain arm must equal dY^T X."""

import importlib.util
import os
import types

import numpy as np
import pytest
import torch

from oracle import isopo_oracle as orc
from tests._util import rel_fro, to_f64

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _harness():
    spec = importlib.util.spec_from_file_location("bench_decoder", os.path.join(ROOT, "bench_decoder.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod


@pytest.mark.parametrize("route", ["stored", "sampled"])
def test_hooks_produce_the_oracles_layer_gradients(route):
    h = _harness()
    dev = torch.device("cuda", 0)
    args = types.SimpleNamespace(vocab=160, d_model=64, ffn=128, heads=2, layers=2)
    rng = np.random.default_rng(0)
    lengths = rng.integers(5, 40, size=6)
    mb = h.Microbatch(lengths, h.group_advantages(6, 3, rng), dev)
    ids = torch.randint(0, args.vocab, (mb.T,), device=dev)
    targets = torch.randint(0, args.vocab, (mb.T,), device=dev)
    model = h.Decoder(args, dev)
    isopo = h.IsopoState(mb, route, "interacting", 16, dev)
    isopo.reserve({(l.weight.shape[1], l.weight.shape[0]) for l in model.linears()})
    seen = {}
    inner = isopo.weight_grad

    def recording(name, X, dY, dW):
        seen[name] = (X.clone(), dY.clone())
        inner(name, X, dY, dW)

    isopo.weight_grad = recording
    for l in model.linears():
        l.isopo = isopo
    model.log_prob_sum(ids, targets, mb).backward()
    torch.cuda.synchronize()
    assert int(isopo.info.item()) == 0 and len(seen) == 2 * 7 + 1
    A = to_f64(mb.A)
    for l in model.linears():
        X, dY = (to_f64(t) for t in seen[l.name])
        if route == "sampled":
            _, _, dW_o = orc.isopo_layer_sampled(X, dY, mb.off, A, isopo.rows, 0.0)
        else:
            K = orc.ntk(orc.sequence_gradients(X, dY, mb.off))
            _, _, dW_o = orc.isopo_layer(X, dY, mb.off, A, orc.INTERACTING, 1e-3 * float(np.mean(np.diag(K))))
        assert rel_fro(l.dW.cpu().numpy(), dW_o) <= 2e-2, l.name
    # plain arm on the same model: dW = dY^T X of advantage-weighted log-probabilities
    for l in model.linears():
        l.isopo = None
        l.dW.zero_()
    seen.clear()
    model.log_prob_sum(ids, targets, mb, mb.tok_adv).backward()
    assert float(model.head.dW.abs().sum()) > 0.0
