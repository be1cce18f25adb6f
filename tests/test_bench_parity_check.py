"""bench.py's own parity check (the `parity` record of the bench line) on the CPU: fed with the oracle's
outputs it must report errors at rounding level, and it must notice a wrong K, a wrong dW and
coefficients that do not follow from K - so that an `ok: true` in the bench line means something."""

import os
import sys
import types

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
from oracle import isopo_oracle as orc  # noqa: E402


def _layers(seed, variant, lam_scale=1e-3):
    rng = np.random.default_rng(seed)
    Ls = rng.integers(3, 20, size=12)
    off = np.concatenate([[0], np.cumsum(Ls)]).astype(np.int64)
    T = int(off[-1])
    A = rng.standard_normal(12)
    layers, lams = [], []
    for d_in, d_out in ((40, 24), (72, 96)):
        X, dY = rng.standard_normal((T, d_in)), 0.1 * rng.standard_normal((T, d_out))
        G = orc.sequence_gradients(X, dY, off)
        K = orc.ntk(G)
        lam = lam_scale * float(np.mean(np.diag(K)))
        c = orc.transform_advantages(K, A, variant, lam)
        layers.append({"layer": types.SimpleNamespace(name="l", d_in=d_in, d_out=d_out),
                       "X": torch.from_numpy(X), "dY": torch.from_numpy(dY), "K": torch.from_numpy(K),
                       "c": torch.from_numpy(c), "dW": torch.from_numpy(orc.weight_gradient(G, c))})
        lams.append(lam)
    return layers, off, torch.from_numpy(A), lams


def test_oracle_outputs_pass_and_planted_errors_show():
    for variant in (orc.INTERACTING, orc.NORMALISED):
        layers, off, A, lams = _layers(3, variant)
        rec = bench.parity_check(layers, off, A, lams, variant, n_seq=5)
        assert rec["K"] < 1e-12 and rec["dW"] < 1e-12 and rec["c_from_K"] < 1e-10, rec
        assert rec["projections"] == 2 and rec["sequences_in_K_sample"] == 5

        bad, off, A, lams = _layers(3, variant)
        i_short = int(np.argmin(np.diff(off)))
        bad[1]["K"][i_short, i_short] *= 1.05            # one diagonal entry of a sampled sequence
        assert bench.parity_check(bad, off, A, lams, variant, n_seq=5)["K"] > 1e-3

        bad, off, A, lams = _layers(3, variant)
        bad[0]["dW"] *= 1.03
        assert bench.parity_check(bad, off, A, lams, variant, n_seq=5)["dW"] > 2e-2

        bad, off, A, lams = _layers(3, variant)
        bad[0]["c"][4] += 0.1 * bad[0]["c"].abs().max()   # coefficients that no longer follow from K
        rec = bench.parity_check(bad, off, A, lams, variant, n_seq=5)
        assert rec["c_from_K"] > 1e-3 and rec["dW"] > 1e-3  # and the dW block was formed with other coefficients
