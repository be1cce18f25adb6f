"""Helpers shared by the tests: error measures and oracle adapters (no method arithmetic)."""

import numpy as np
import torch

from oracle import isopo_oracle as orc

VARIANT_NAME = {0: orc.REINFORCE, 1: orc.NORMALISED, 2: orc.DIRECTION, 3: orc.EUCLID, 4: orc.GENERAL,
                5: orc.INTERACTING, 6: orc.NORMALISED_RAW}


def rel_fro(got, want):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300))


def offdiag_rel_fro(got, want):
    got = np.asarray(got, dtype=np.float64).copy()
    want = np.asarray(want, dtype=np.float64).copy()
    np.fill_diagonal(got, 0.0)
    np.fill_diagonal(want, 0.0)
    return rel_fro(got, want)


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a float32/bfloat16 tensor to a float64 numpy array."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def oracle_layer(X, dY, off, A, variant_code, lam, pqr_regs=None):
    """Runs the fp64 oracle on the same bits the GPU sees."""
    pqr = regs = None
    if pqr_regs is not None:
        pqr, regs = tuple(pqr_regs[:3]), tuple(pqr_regs[3:])
    return orc.isopo_layer(to_f64(X), to_f64(dY), np.asarray(off), to_f64(A), VARIANT_NAME[variant_code], float(lam),
                           pqr, regs)


def report(label, **values):
    """One line per parity case with the measured errors and cond(K + lambda I) (shown by pytest -s or on failure)."""
    print("[parity] " + label + ": " + ", ".join(f"{k}={v:.3e}" for k, v in values.items()))
