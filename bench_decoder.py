#!/usr/bin/env python
"""End-to-end harness: backward pass of a random-init decoder with ISOPO on every linear layer
against the same backward with plain (REINFORCE) weight gradients.

This is the integration the paper describes (Algorithm 1 / 2 headers): backprop runs on
sum(log_prob) WITHOUT advantages, every linear layer stashes its input in the forward pass, and in
the backward pass the layer turns (X, dY, sequence partition, advantages) into its own weight
gradient through the library's three calls.  The input gradient dX = dY W is the ordinary one: the
transform is layer-local, so nothing but dW changes.  The REINFORCE arm backpropagates
sum_i A_i log_prob_i and forms dW = dY^T X with cuBLAS.

    python bench_decoder.py [--layers 24 --d-model 2048 --ffn 5632 --heads 16 --vocab 32000
                             --seqs 128 --len-lo 512 --len-hi 2048 --route stored|sampled
                             --variant interacting|normalised --steps 3]

Prints one JSON line with the times of both arms and their ratio.  Synthetic token ids and
group-normalised advantages (groups of 8); layers are recomputed in the backward pass (activation
checkpointing) so that the 24-layer model fits next to the stored per-sequence gradients.
PyTorch supplies the model around the linear layers (attention, norms, softmax); the library
supplies every ISOPO step.
"""

from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np
import torch
import torch.nn.functional as F
from torch.utils.checkpoint import checkpoint

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)


class Microbatch:
    """Packed ragged microbatch: offsets, advantages and what the linear layers need in backward."""

    def __init__(self, lengths, advantages, device):
        self.off = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int64)
        self.T, self.B = int(self.off[-1]), len(lengths)
        self.A = torch.from_numpy(np.asarray(advantages, dtype=np.float32)).to(device)
        seq = np.repeat(np.arange(self.B), lengths)
        self.tok_adv = self.A[torch.from_numpy(seq).to(device)]
        # packed token -> (sequence, position) for the padded attention layout
        self.Lmax = int(max(lengths))
        pos = np.concatenate([np.arange(l) for l in lengths])
        self.flat_index = torch.from_numpy(seq * self.Lmax + pos).to(device)


class IsopoState:
    """What the ISOPO arm shares between layers: binding, route, workspace, sample rows."""

    def __init__(self, mb: Microbatch, route: str, variant: str, n_samples: int, device):
        from paper_2512_23353_b200 import binding as b
        self.b, self.mb, self.route = b, mb, route
        self.variant = b.VAR_INTERACTING if variant == "interacting" else b.VAR_NORMALISED
        self.rows = np.random.default_rng(5).permutation(mb.T)[:n_samples].astype(np.int64)
        self.info = torch.zeros(1, dtype=torch.int32, device=device)
        self.ws = None
        self.device = device
        self.ema = {}      # per layer: running means of the relative regulariser
        self.K = torch.empty((mb.B, mb.B), dtype=torch.float32, device=device)
        self.c = torch.empty(mb.B, dtype=torch.float32, device=device)

    def reserve(self, shapes):
        b, mb = self.b, self.mb
        need = 0
        for d_in, d_out in shapes:
            if self.route == "sampled":
                need = max(need, b.isopo_sampled_workspace_bytes(b.BF16, mb.T, d_in, d_out, mb.B, len(self.rows)))
            else:
                need = max(need, b.isopo_workspace_bytes(b.BF16, mb.T, d_in, d_out, mb.B, b.PATH_AUTO))
        raw = torch.empty(need + 1024, dtype=torch.uint8, device=self.device)
        shift = (-raw.data_ptr()) % 1024
        self.ws = raw[shift:shift + need]

    def weight_grad(self, name, X, dY, dW):
        """dW += ISOPO weight gradient of this layer (regulariser: 1e-3 x the layer's running mean)."""
        b, mb = self.b, self.mb
        if self.route == "sampled":
            F2 = self.ema.setdefault(name, torch.zeros(mb.B, dtype=torch.float32, device=self.device))
            lam = 0.0  # Algorithm 1 with no regulariser (the non-interacting experiment ran without one)
            b.isopo_sampled_coefficients(X, dY, mb.off, self.rows, mb.A, lam, self.c, self.ws, self.info, F2)
            b.isopo_weight_grad(X, dY, self.c, mb.off, dW, self.ws, self.info, b.PATH_GRAM, 1.0)
            return
        state = self.ema.setdefault(name, torch.zeros(4, dtype=torch.float32, device=self.device))
        b.isopo_layer_gram(X, dY, mb.off, self.K, self.ws, self.info, b.PATH_AUTO)
        b.isopo_reg_ema_update(self.K, 0.9, state)
        b.isopo_transform_advantages_rel(self.K, mb.A, self.variant, 1e-3, state, self.c, self.info)
        b.isopo_weight_grad(X, dY, self.c, mb.off, dW, self.ws, self.info, b.PATH_AUTO, 1.0)


class HookedLinearFn(torch.autograd.Function):
    """y = x W^T.  Backward: dX = dY W as usual; dW by `mode`: plain dY^T X, or the ISOPO path."""

    @staticmethod
    def forward(ctx, x, layer):
        ctx.layer = layer
        ctx.save_for_backward(x)
        return x @ layer.weight.t()

    @staticmethod
    def backward(ctx, dY):
        (x,) = ctx.saved_tensors
        layer = ctx.layer
        dY = dY.contiguous()
        dX = dY @ layer.weight
        if layer.isopo is None:
            layer.dW.add_(dY.t() @ x)
        else:
            layer.isopo.weight_grad(layer.name, x, dY, layer.dW)
        return dX, None


class HookedLinear:
    def __init__(self, name, d_in, d_out, device, gen):
        self.name = name
        self.weight = (torch.randn(d_out, d_in, device=device, generator=gen) * d_in ** -0.5).to(torch.bfloat16)
        self.dW = torch.zeros(d_out, d_in, dtype=torch.float32, device=device)  # the "mod.grad" of the listings
        self.isopo = None

    def __call__(self, x):
        return HookedLinearFn.apply(x, self)


def rms_norm(x, eps=1e-6):
    return (x.float() * torch.rsqrt(x.float().pow(2).mean(-1, keepdim=True) + eps)).to(x.dtype)


class Block:
    def __init__(self, idx, d, ffn, heads, device, gen):
        self.heads, self.d = heads, d
        mk = lambda n, i, o: HookedLinear(f"L{idx}.{n}", i, o, device, gen)  # noqa: E731
        self.q, self.k, self.v, self.o = mk("q", d, d), mk("k", d, d), mk("v", d, d), mk("o", d, d)
        self.gate, self.up, self.down = mk("gate", d, ffn), mk("up", d, ffn), mk("down", ffn, d)

    def linears(self):
        return [self.q, self.k, self.v, self.o, self.gate, self.up, self.down]

    def attention(self, q, k, v, mb: Microbatch):
        # packed [T, d] -> padded [B, heads, Lmax, hd]; causal masking keeps sequences apart and the
        # padding (at the end of each row) out of every real token's window
        hd = self.d // self.heads

        def pad(t):
            buf = t.new_zeros(mb.B * mb.Lmax, self.d)
            buf.index_copy_(0, mb.flat_index, t)
            return buf.view(mb.B, mb.Lmax, self.heads, hd).transpose(1, 2)

        out = F.scaled_dot_product_attention(pad(q), pad(k), pad(v), is_causal=True)
        return out.transpose(1, 2).reshape(mb.B * mb.Lmax, self.d).index_select(0, mb.flat_index)

    def forward(self, h, mb):
        x = rms_norm(h)
        h = h + self.o(self.attention(self.q(x), self.k(x), self.v(x), mb))
        x = rms_norm(h)
        return h + self.down(F.silu(self.gate(x)) * self.up(x))


class Decoder:
    def __init__(self, args, device):
        gen = torch.Generator(device=device)
        gen.manual_seed(1005)
        self.embed = (torch.randn(args.vocab, args.d_model, device=device, generator=gen) * 0.02).to(torch.bfloat16)
        self.blocks = [Block(i, args.d_model, args.ffn, args.heads, device, gen) for i in range(args.layers)]
        self.head = HookedLinear("lm_head", args.d_model, args.vocab, device, gen)

    def linears(self):
        return [l for blk in self.blocks for l in blk.linears()] + [self.head]

    def log_prob_sum(self, ids, targets, mb, token_weights=None):
        """sum_t w_t log pi(target_t | prefix); w = 1 for the ISOPO arm, the advantages for REINFORCE."""
        h = self.embed[ids].requires_grad_(True)
        for blk in self.blocks:
            h = checkpoint(blk.forward, h, mb, use_reentrant=False)
        logits = self.head(rms_norm(h))
        logp = -F.cross_entropy(logits.float(), targets, reduction="none")
        return (logp * token_weights).sum() if token_weights is not None else logp.sum()


def group_advantages(B, group, rng):
    p = rng.uniform(0.1, 0.9, size=(B + group - 1) // group)
    r = (rng.uniform(size=(len(p), group)) < p[:, None]).astype(np.float64)
    A = (r - r.mean(1, keepdims=True)) / (r.std(1, keepdims=True) + 1e-6)
    return A.reshape(-1)[:B].astype(np.float32)


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=24)
    ap.add_argument("--d-model", type=int, default=2048)
    ap.add_argument("--ffn", type=int, default=5632)
    ap.add_argument("--heads", type=int, default=16)
    ap.add_argument("--vocab", type=int, default=32000)
    ap.add_argument("--seqs", type=int, default=128)
    ap.add_argument("--len-lo", type=int, default=512)
    ap.add_argument("--len-hi", type=int, default=2048)
    ap.add_argument("--route", default="stored", choices=["stored", "sampled"])
    ap.add_argument("--variant", default="interacting", choices=["interacting", "normalised"])
    ap.add_argument("--samples", type=int, default=128)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=1)
    return ap.parse_args(argv)


def run_decoder(args, dev=None):
    """Both arms on one device; returns the record that main() prints."""
    dev = dev or torch.device("cuda", torch.cuda.current_device())
    torch.cuda.set_device(dev)
    rng = np.random.default_rng(1005)
    lengths = rng.integers(args.len_lo, args.len_hi + 1, size=args.seqs)
    mb = Microbatch(lengths, group_advantages(args.seqs, 8, rng), dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(7)
    ids = torch.randint(0, args.vocab, (mb.T,), device=dev, generator=gen)
    targets = torch.randint(0, args.vocab, (mb.T,), device=dev, generator=gen)
    model = Decoder(args, dev)
    isopo = IsopoState(mb, args.route, args.variant, args.samples, dev)
    isopo.reserve({(l.weight.shape[1], l.weight.shape[0]) for l in model.linears()})

    def run(arm):
        for l in model.linears():
            l.isopo = isopo if arm == "isopo" else None
            l.dW.zero_()
        weights = None if arm == "isopo" else mb.tok_adv
        times = {"fwd": [], "bwd": []}
        for it in range(args.warmup + args.steps):
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            e[0].record()
            loss = model.log_prob_sum(ids, targets, mb, weights)
            e[1].record()
            loss.backward()
            e[2].record()
            torch.cuda.synchronize()
            if it >= args.warmup:
                times["fwd"].append(e[0].elapsed_time(e[1]))
                times["bwd"].append(e[1].elapsed_time(e[2]))
        if int(isopo.info.item()) != 0:
            raise SystemExit(f"device-side error: info={int(isopo.info.item()):#x}")
        return {k: float(np.median(v)) for k, v in times.items()}

    plain = run("reinforce")
    ours = run("isopo")
    out = {
        "harness": "decoder backward, ISOPO on every linear layer vs plain weight gradients",
        "config": {"layers": args.layers, "d_model": args.d_model, "ffn": args.ffn, "heads": args.heads,
                   "vocab": args.vocab, "B": mb.B, "tokens": mb.T, "route": args.route,
                   "variant": "normalised (Algorithm 1)" if args.route == "sampled" else args.variant,
                   "dtype": "bf16", "data": "synthetic", "recompute": "every block in backward"},
        "reinforce_ms": plain, "isopo_ms": ours,
        "backward_ratio": ours["bwd"] / plain["bwd"],
        "step_ratio": (ours["fwd"] + ours["bwd"]) / (plain["fwd"] + plain["bwd"]),
        "tokens_per_s_isopo": mb.T / ((ours["fwd"] + ours["bwd"]) * 1e-3),
        "peak_mem_gb": torch.cuda.max_memory_allocated() / 2 ** 30,
    }
    return out


def main():
    print(json.dumps(run_decoder(parse_args())))


if __name__ == "__main__":
    main()
