"""Seeded synthetic microbatches with the shapes of LLM fine-tuning layers.

This module only draws inputs (sequence lengths, rewards -> advantages,
activations, output gradients).  It holds none of the method's arithmetic and
imports neither the CUDA binding nor the CPU oracle, so both sides can be fed
from it.

Small workloads are drawn on the host with numpy's PCG64; large ones draw X
and dY on the device with a seeded torch generator (the test then copies the
slices it needs back to the host for the oracle, so both sides see the same
bits).
"""

from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


@dataclass(frozen=True)
class LayerShape:
    name: str
    d_in: int
    d_out: int


@dataclass(frozen=True)
class Workload:
    """One ragged microbatch recipe."""
    name: str
    dtype: str                 # "f32" or "bf16"
    B: int
    len_law: str               # "uniform" or "loguniform"
    len_lo: int
    len_hi: int
    group: int                 # sequences per prompt group
    reward_p: str              # "half" (Bernoulli(0.5)) or "uniform" (p ~ U[0.1, 0.9] per group)
    layers: tuple = field(default_factory=tuple)
    seed: int = 0


def _block(d_model, ffn, kv):
    return (
        LayerShape("q_proj", d_model, d_model),
        LayerShape("k_proj", d_model, kv),
        LayerShape("v_proj", d_model, kv),
        LayerShape("o_proj", d_model, d_model),
        LayerShape("gate_proj", d_model, ffn),
        LayerShape("up_proj", d_model, ffn),
        LayerShape("down_proj", ffn, d_model),
    )


WORKLOADS = {
    # one 64 -> 64 fp32 layer, 8 sequences of 16..64 tokens
    "tiny_f32": Workload("tiny_f32", "f32", 8, "uniform", 16, 64, 4, "half",
                         (LayerShape("linear", 64, 64),), seed=1001),
    # small-LLM block: d_model 896, FFN 4864 (kv width 128 assumed), 64 sequences of 128..1024 tokens
    "small_llm": Workload("small_llm", "bf16", 64, "uniform", 128, 1024, 8, "uniform",
                          _block(896, 4864, 128), seed=1002),
    # short rollouts on the small-LLM block (256 sequences of 16..64 tokens): the regime where the Gram route is cheaper
    "short_rollouts": Workload("short_rollouts", "bf16", 256, "uniform", 16, 64, 8, "uniform",
                               _block(896, 4864, 128), seed=1006),
    # 1.5B-class block: d_model 1536, FFN 8960, GQA kv width 256, 32 prompts x 8 samples
    "llm_1p5b": Workload("llm_1p5b", "bf16", 256, "loguniform", 256, 4096, 8, "uniform",
                         _block(1536, 8960, 256), seed=1003),
    # 7B-class block: d_model 3584, FFN 18944, kv width 512, 64 sequences of 1024..8192 tokens
    "llm_7b": Workload("llm_7b", "bf16", 64, "uniform", 1024, 8192, 8, "uniform",
                       _block(3584, 18944, 512), seed=1004),
}


def sequence_lengths(w: Workload, rng: np.random.Generator, scale_div: int = 1) -> np.ndarray:
    """Lengths per the workload's law; `scale_div` shrinks every length (>= 1 token)."""
    if w.len_law == "uniform":
        L = rng.integers(w.len_lo, w.len_hi + 1, size=w.B)
    elif w.len_law == "loguniform":
        u = rng.uniform(np.log(w.len_lo), np.log(w.len_hi), size=w.B)
        L = np.clip(np.rint(np.exp(u)).astype(np.int64), w.len_lo, w.len_hi)
    else:
        raise ValueError(w.len_law)
    return np.maximum(1, L.astype(np.int64) // scale_div)


def offsets_from_lengths(L: np.ndarray) -> np.ndarray:
    off = np.zeros(L.shape[0] + 1, dtype=np.int64)
    np.cumsum(L, out=off[1:])
    return off


def group_advantages(w: Workload, rng: np.random.Generator) -> np.ndarray:
    """Group-relative advantages (r - mean_group) / (std_group + 1e-6) from Bernoulli rewards."""
    B, g = w.B, w.group
    n_groups = (B + g - 1) // g
    if w.reward_p == "half":
        p = np.full(n_groups, 0.5)
    else:
        p = rng.uniform(0.1, 0.9, size=n_groups)
    r = (rng.uniform(size=(n_groups, g)) < p[:, None]).astype(np.float64)
    A = (r - r.mean(axis=1, keepdims=True)) / (r.std(axis=1, keepdims=True) + 1e-6)
    return A.reshape(-1)[:B].astype(np.float32)


def microbatch(w: Workload, scale_div: int = 1):
    """(offsets int64 [B+1], advantages float32 [B]) for the workload's seed."""
    rng = np.random.default_rng(w.seed)
    off = offsets_from_lengths(sequence_lengths(w, rng, scale_div))
    A = group_advantages(w, rng)
    return off, A


def layer_inputs_host(w: Workload, layer: LayerShape, T: int, correlated: bool = False):
    """X ~ N(0, 1) [T, d_in] and dY ~ N(0, 0.1^2) [T, d_out] as float32 numpy arrays.

    `correlated` adds, to every token, a shared rank-4 component of the same
    energy, so that different sequences' gradients overlap strongly (K gets
    O(1) off-diagonal entries and the interacting solve becomes non-trivial).
    For bf16 workloads the caller rounds the arrays to bf16.
    """
    rng = np.random.default_rng([w.seed, layer.d_in, layer.d_out, 7])
    X = rng.standard_normal((T, layer.d_in), dtype=np.float32)
    dY = 0.1 * rng.standard_normal((T, layer.d_out), dtype=np.float32)
    if correlated:
        r = 4
        ux = rng.standard_normal((r, layer.d_in), dtype=np.float32)
        uy = rng.standard_normal((r, layer.d_out), dtype=np.float32)
        ax = rng.standard_normal((T, r), dtype=np.float32) / np.float32(np.sqrt(r))
        ay = rng.standard_normal((T, r), dtype=np.float32) / np.float32(np.sqrt(r))
        X = (X + ax @ ux).astype(np.float32)
        dY = (dY + np.float32(0.1) * (ay @ uy)).astype(np.float32)
    return X, dY


def layer_inputs_device(w: Workload, layer: LayerShape, T: int, device="cuda"):
    """Same distributions drawn on the device (torch, seeded) in the workload's dtype."""
    import torch

    gen = torch.Generator(device=device)
    gen.manual_seed(w.seed * 1000003 + layer.d_in * 131 + layer.d_out)
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    X = torch.empty((T, layer.d_in), device=device, dtype=dt)
    dY = torch.empty((T, layer.d_out), device=device, dtype=dt)
    X.normal_(0.0, 1.0, generator=gen)
    dY.normal_(0.0, 0.1, generator=gen)
    return X, dY
