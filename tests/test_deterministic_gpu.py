"""Deterministic mode: K of the bf16 stored-gradient route is normally reduced over the CTAs with float
atomics, so two runs differ in their last bits; with the mode on, per-CTA partial sums are added in a
fixed order and K, the coefficients and dW must be bit-identical from run to run - which tells a race
(results that differ) from rounding (results that do not).  The values still match the oracle."""

import numpy as np
import pytest
import torch

from oracle import isopo_oracle as orc
from tests._util import rel_fro, to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def b():
    from paper_2512_23353_b200 import binding
    return binding


@pytest.mark.parametrize("B,d_in,d_out", [(5, 320, 200), (70, 256, 128), (256, 512, 256)])
def test_two_runs_are_bit_identical(b, B, d_in, d_out):
    rng = np.random.default_rng(B)
    Ls = rng.integers(1, 40, size=B)
    off = np.concatenate([[0], np.cumsum(Ls)]).astype(np.int64)
    g = torch.Generator(device="cuda")
    g.manual_seed(B)
    X = torch.randn(int(off[-1]), d_in, device="cuda", generator=g).to(torch.bfloat16)
    dY = (0.1 * torch.randn(int(off[-1]), d_out, device="cuda", generator=g)).to(torch.bfloat16)
    A = torch.randn(B, device="cuda", generator=g)
    plain_bytes = b.isopo_workspace_bytes(b.BF16, int(off[-1]), d_in, d_out, B, b.PATH_MATERIALISE)
    b.isopo_set_deterministic(True)
    try:
        assert b.isopo_workspace_bytes(b.BF16, int(off[-1]), d_in, d_out, B, b.PATH_MATERIALISE) > plain_bytes
        runs = []
        for _ in range(3):
            res = b.isopo_layer(X, dY, off, A, b.VAR_INTERACTING, 1e-2, b.PATH_MATERIALISE)
            assert res.info == 0
            runs.append((res.K.clone(), res.coeffs.clone(), res.dW.clone()))
        for K, c, dW in runs[1:]:
            assert torch.equal(K, runs[0][0]) and torch.equal(c, runs[0][1]) and torch.equal(dW, runs[0][2])
        K = runs[0][0]
        assert torch.equal(K, K.T)
        G = orc.sequence_gradients(to_f64(X), to_f64(dY), off)
        assert rel_fro(K.cpu().numpy(), orc.ntk(G)) <= 2e-2
    finally:
        b.isopo_set_deterministic(False)
    assert b.isopo_workspace_bytes(b.BF16, int(off[-1]), d_in, d_out, B, b.PATH_MATERIALISE) == plain_bytes
