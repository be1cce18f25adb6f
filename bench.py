#!/usr/bin/env python
"""Benchmark of the ISOPO per-layer hot path on B200.

One "step" = the whole hot path (isopo_layer_gram -> isopo_transform_advantages -> isopo_weight_grad)
for the seven projections of one transformer block over one ragged synthetic microbatch: K for every
projection, then the coefficients of all seven in one batched transform launch, then every dW.  The
default workload is the 1.5B-class block (d_model 1536, FFN 8960, kv 256; 256 sequences with
log-uniform lengths in [256, 4096], ~355k tokens), the shapes the throughput target is quoted on.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs its own microbatch with no
data-path collective (the path shards by independent microbatches) and the time is the max over
ranks.  `--impl reference` times the fp64 CPU oracle on a bounded sample instead.
"""

from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

# profiles/dram_traffic_llm_1p5b_block_full_size.md: 80.3 GB measured over the seven launches of the block at full
# size (median of five one-pass captures on five boxes: 54.2, 56.0, 80.2, 80.6, 86.4 GB) / 51.5 GB algorithmic (inputs read once +
# stored gradients written once)
SEQ_GRAD_DRAM_OVER_ALGORITHMIC = 1.56
METRIC = "isopo_block_tokens_per_s"
UNIT = "tokens/s"
L2_BYTES = 126 * 1024 * 1024


# ------------------------------------------------------------------------------------------------
# helpers
# ------------------------------------------------------------------------------------------------

def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p["bf16_tflops_sustained"], "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU through NVML (every 5 ms, in a thread)
    while the timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, cuda_index: int):
        self.cuda_index = cuda_index
        self.samples = []
        self.stop_flag = threading.Event()
        self.thread = None
        self.error = None

    def _handle(self, nv):
        import torch
        props = torch.cuda.get_device_properties(self.cuda_index)
        try:
            bus = f"{props.pci_domain_id:08x}:{props.pci_bus_id:02x}:{props.pci_device_id:02x}.0"
            return nv.nvmlDeviceGetHandleByPciBusId(bus.encode())
        except Exception:
            return nv.nvmlDeviceGetHandleByIndex(self.cuda_index)

    def start(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = self._handle(nv)
            reasons_fn = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
            smax = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
        except Exception as e:  # no NVML: the bench line says so instead of inventing clocks
            self.error = f"NVML unavailable: {e}"
            return

        def pump():
            while not self.stop_flag.is_set():
                try:
                    self.samples.append((nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM), smax,
                                         nv.nvmlDeviceGetPowerUsage(h) / 1000.0, int(reasons_fn(h))))
                except Exception:
                    pass
                time.sleep(0.005)

        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self):
        if self.thread is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [self.error or "no samples"]}
        self.stop_flag.set()
        self.thread.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = [x[0] for x in self.samples]
        mask = 0
        for x in self.samples:
            mask |= x[3]
        return {"sm_mhz": statistics.median(sm), "sm_min_mhz": min(sm), "sm_max_mhz": self.samples[0][1],
                "power_w_max": max(x[2] for x in self.samples), "samples": len(sm),
                "reasons": sorted(name for bit, name in self.REASONS.items() if mask & bit)}


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def rank_workload(w, rank: int, world: int):
    """The microbatch recipe of one rank: the path shards by independent microbatches (K is defined
    per microbatch), so with several ranks each draws its own from a rank-dependent seed."""
    if world == 1:
        return w
    from dataclasses import replace
    return replace(w, seed=w.seed + 7919 * rank)


def reduce_over_ranks(elapsed_ms: float, tokens: float, device=None):
    """(max elapsed over ranks, total tokens over ranks); identity without a process group."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return elapsed_ms, tokens
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    n = torch.tensor([tokens], dtype=torch.float64, device=device)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), float(n.item())


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
# ------------------------------------------------------------------------------------------------

def oracle_sample(workload_name: str, n_seq: int, len_div: int):
    """Bounded sample of the workload for the CPU oracle: the first `n_seq` sequences with every
    length divided by `len_div`, all seven projections.  Returns (tokens, seconds, description)."""
    from oracle import isopo_oracle as orc
    from paper_2512_23353_b200 import workloads as wl

    w = wl.WORKLOADS[workload_name]
    off_full, A_full = wl.microbatch(w, scale_div=len_div)
    off = off_full[: n_seq + 1].copy()
    A = A_full[:n_seq].astype(np.float64)
    T = int(off[-1])
    inputs = []
    for layer in w.layers:
        X, dY = wl.layer_inputs_host(w, layer, T)
        inputs.append((X, dY))
    t0 = time.perf_counter()
    for X, dY in inputs:
        G = orc.sequence_gradients(X, dY, off)
        K = orc.ntk(G)
        lam = 1e-3 * float(np.mean(np.diag(K)))
        c = orc.transform_advantages(K, A, orc.INTERACTING, lam)
        orc.weight_gradient(G, c)
    dt = time.perf_counter() - t0
    desc = (f"{workload_name}: first {n_seq} of {w.B} sequences, lengths/{len_div} ({T} tokens), all "
            f"{len(w.layers)} projections, interacting variant, numpy float64")
    return T, dt, desc


def parity_check(layers, off, A, lam_by_layer, variant_name, n_seq=8):
    """The last timed step's outputs against the fp64 oracle, the cheap way: per projection, K_ij for all
    pairs of the `n_seq` shortest sequences (their G_i materialised in float64), one 32 x 64 block of dW over
    ALL sequences with the library's coefficients, and those coefficients against the oracle's transform of
    the library's K.  Relative Frobenius errors, the worst projection of each; tolerance 2e-2 (bf16) / 1e-5."""
    import torch

    from oracle import isopo_oracle as orc

    def f64(t):
        return t.detach().to("cpu").to(torch.float64).numpy()

    def rel(a, ref):
        return float(np.linalg.norm(np.asarray(a, np.float64) - ref) / max(np.linalg.norm(ref), 1e-300))

    L_len = np.diff(off)
    pick = sorted(np.argsort(L_len, kind="stable")[:n_seq].tolist())
    off_s = np.concatenate([[0], np.cumsum([L_len[i] for i in pick])]).astype(np.int64)
    rng = np.random.default_rng(11)
    worst = {"K": 0.0, "dW": 0.0, "c_from_K": 0.0}
    t0 = time.perf_counter()
    for L, lam in zip(layers, lam_by_layer):
        lay = L["layer"]
        rows = torch.cat([torch.arange(int(off[i]), int(off[i + 1])) for i in pick]).to(L["X"].device)
        G_s = orc.sequence_gradients(f64(L["X"][rows]), f64(L["dY"][rows]), off_s)
        worst["K"] = max(worst["K"], rel(f64(L["K"])[np.ix_(pick, pick)], orc.ntk(G_s)))
        del G_s
        m_idx = torch.from_numpy(np.sort(rng.choice(lay.d_out, size=min(32, lay.d_out), replace=False))).to(L["X"].device)
        n_idx = torch.from_numpy(np.sort(rng.choice(lay.d_in, size=min(64, lay.d_in), replace=False))).to(L["X"].device)
        G_blk = orc.sequence_gradients(f64(L["X"][:, n_idx]), f64(L["dY"][:, m_idx]), off)
        worst["dW"] = max(worst["dW"], rel(f64(L["dW"][m_idx][:, n_idx]), orc.weight_gradient(G_blk, f64(L["c"]))))
        worst["c_from_K"] = max(worst["c_from_K"],
                                rel(f64(L["c"]), orc.transform_advantages(f64(L["K"]), f64(A), variant_name, lam)))
    return {**worst, "sequences_in_K_sample": len(pick), "dW_block": "32 x 64 over all sequences",
            "projections": len(layers), "seconds": time.perf_counter() - t0}


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    times, tokens, desc = [], 0, ""
    for it in range(args.warmup + args.steps):
        tokens, dt, desc = oracle_sample(args.workload, args.cpu_seqs, args.cpu_len_div)
        if it >= args.warmup:
            times.append(dt)
    ms = 1000.0 * sum(times) / len(times)
    value = tokens / (ms / 1000.0)
    cores = cpu_threads()
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(out))


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------

def run_gpu(args):
    import torch

    from paper_2512_23353_b200 import binding as b
    from paper_2512_23353_b200 import workloads as wl

    rank, world, local = dist_env()
    if world != args.gpus:
        if world == 1 and args.gpus > 1:
            raise SystemExit("launch with torchrun for --gpus > 1")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    w = rank_workload(wl.WORKLOADS[args.workload], rank, world)
    off, A_host = wl.microbatch(w)
    if args.seqs:  # profiling aid: the first --seqs sequences only (keeps an ncu capture small)
        off, A_host = off[: args.seqs + 1].copy(), A_host[: args.seqs].copy()
    T, B = int(off[-1]), len(A_host)
    wanted = set(args.layers.split(",")) if args.layers else None
    w_layers = [l for l in w.layers if wanted is None or l.name in wanted]
    n_warm = args.warmup if args.short_warmup else max(args.warmup, 3)
    dt_code = b.BF16 if w.dtype == "bf16" else b.F32
    variant = b.VAR_INTERACTING if args.variant == "interacting" else b.VAR_NORMALISED

    sampled = args.route == "sampled"
    if args.deterministic:  # before any workspace is sized: the per-CTA partial sums of K live there
        b.isopo_set_deterministic(True)
    if args.store_format == "e4m3_split":  # before any workspace is sized or written
        b.isopo_set_store_format(b.STORE_E4M3_SPLIT)
    # Algorithm 1 draws its overlap samples with randperm: the bench draws them once, seeded, on the host
    sample_rows = np.random.default_rng(w.seed + 17).permutation(T)[: args.samples].astype(np.int64)
    # the stored route keeps every projection's workspace until the block's coefficients are known, so
    # that one batched launch solves for all of them; with --schedule single one workspace is reused
    batched = not sampled and args.schedule == "batched"
    layers = []
    ws_sizes = []
    for layer in w_layers:
        X, dY = wl.layer_inputs_device(w, layer, T, dev)
        if sampled:
            path = b.PATH_GRAM
            ws_sizes.append(b.isopo_sampled_workspace_bytes(dt_code, T, layer.d_in, layer.d_out, B, len(sample_rows)))
        else:
            path = b.isopo_choose_path(dt_code, T, layer.d_in, layer.d_out, B)
            ws_sizes.append(b.isopo_workspace_bytes(dt_code, T, layer.d_in, layer.d_out, B, path))
        layers.append({"layer": layer, "X": X, "dY": dY, "path": path,
                       "K": torch.empty((B, B), dtype=torch.float32, device=dev),
                       "c": torch.empty(B, dtype=torch.float32, device=dev),
                       "dW": torch.zeros((layer.d_out, layer.d_in), dtype=torch.float32, device=dev),
                       "lam": 0.0})

    def aligned(nbytes):
        raw = torch.empty(nbytes + 1024, dtype=torch.uint8, device=dev)
        shift = (-raw.data_ptr()) % 1024
        return raw[shift:shift + nbytes]

    if batched:
        for L, n in zip(layers, ws_sizes):
            L["ws"] = aligned(n)
    else:
        shared_ws = aligned(max(ws_sizes))
        for L in layers:
            L["ws"] = shared_ws
    A = torch.from_numpy(A_host).to(dev)
    info = torch.zeros(1, dtype=torch.int32, device=dev)

    def layer_calls(L):
        if sampled:  # Algorithm 1: coefficients from sampled token rows, then the folded weight-gradient GEMM
            b.isopo_sampled_coefficients(L["X"], L["dY"], off, sample_rows, A, L["lam"], L["c"], L["ws"], info, L["F2"])
        else:
            b.isopo_layer_gram(L["X"], L["dY"], off, L["K"], L["ws"], info, L["path"])
            b.isopo_transform_advantages(L["K"], A, variant, L["lam"], L["c"], info)
        b.isopo_weight_grad(L["X"], L["dY"], L["c"], off, L["dW"], L["ws"], info, L["path"], 0.0)

    def step():
        if not batched:
            for L in layers:
                layer_calls(L)
            return
        for L in layers:
            b.isopo_layer_gram(L["X"], L["dY"], off, L["K"], L["ws"], info, L["path"])
        b.isopo_transform_advantages_batched([L["K"] for L in layers], A, variant, [L["lam"] for L in layers],
                                             [L["c"] for L in layers], info)
        for L in layers:
            b.isopo_weight_grad(L["X"], L["dY"], L["c"], off, L["dW"], L["ws"], info, L["path"], 0.0)

    # the regulariser is an absolute number the caller carries from earlier minibatches:
    # 1e-3 * mean(diag K) (stored route) or 1e-3 * mean(F^2) (sampled route), taken once from an untimed pass
    for L in layers:
        L["F2"] = torch.zeros(B, dtype=torch.float32, device=dev)
    step()
    torch.cuda.synchronize()
    for L in layers:
        L["lam"] = 1e-3 * float((L["F2"] if sampled else torch.diagonal(L["K"])).mean().item())
    for _ in range(n_warm):
        step()
    torch.cuda.synchronize()
    if int(info.item()) != 0:
        raise SystemExit(f"device-side error during warm-up: info={int(info.item()):#x}")
    b.isopo_profile_collect()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    b.isopo_profile_enable(True)
    # a step whose inputs fit the L2 would be timed on cached data: flush between such steps (a 256 MB
    # fill, outside the timed intervals) and time every step with its own pair of events
    input_bytes = sum(L["X"].numel() * L["X"].element_size() + L["dY"].numel() * L["dY"].element_size()
                      for L in layers)
    flush = input_bytes < 2 * L2_BYTES
    if flush:
        flush_buf = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)
        marks = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                 for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    e0.record()
    for it in range(args.steps):
        if flush:
            flush_buf.fill_(it & 0xff)
            marks[it][0].record()
        step()
        if flush:
            marks[it][1].record()
    e1.record()
    barrier()
    clocks = sampler.stop()
    b.isopo_profile_enable(False)
    elapsed_ms = sum(a.elapsed_time(c) for a, c in marks) if flush else e0.elapsed_time(e1)
    prof = b.isopo_profile_collect()
    if int(info.item()) != 0:
        raise SystemExit(f"device-side error during the timed region: info={int(info.item()):#x}")
    elapsed_ms, total_tokens = reduce_over_ranks(elapsed_ms, float(T), dev)
    ms_per_step = elapsed_ms / args.steps
    value = total_tokens / (ms_per_step / 1000.0)

    # ---- the timed run's own outputs against the oracle (rank 0; stored route: K, c, dW are all there) ----
    parity = None
    if rank == 0 and not sampled and not args.skip_parity:
        from oracle import isopo_oracle as orc
        parity = parity_check(layers, off, A, [L["lam"] for L in layers],
                              orc.INTERACTING if args.variant == "interacting" else orc.NORMALISED)
        tol = 2e-2 if w.dtype == "bf16" else 1e-5
        parity["tolerance"] = tol
        parity["ok"] = bool(parity["K"] <= tol and parity["dW"] <= tol and parity["c_from_K"] <= max(tol * 1e-2, 1e-5))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    # ---- algorithmic work of one step (this rank) ----
    flops_dw = sum(2.0 * T * L["layer"].d_in * L["layer"].d_out for L in layers)
    flops_k = sum(float(B) * B * L["layer"].d_in * L["layer"].d_out for L in layers)
    flops_comb = sum(2.0 * B * L["layer"].d_in * L["layer"].d_out for L in layers)
    if not sampled:  # layers on the Gram route: token Grams instead of the K pass and the combine
        gram_layers = [L for L in layers if L["path"] == b.PATH_GRAM]
        flops_k = sum(float(B) * B * L["layer"].d_in * L["layer"].d_out for L in layers if L["path"] != b.PATH_GRAM) + \
            sum(float(L["layer"].d_in + L["layer"].d_out) * T * T for L in gram_layers)
        flops_comb = sum(2.0 * B * L["layer"].d_in * L["layer"].d_out for L in layers if L["path"] != b.PATH_GRAM)
    if sampled:
        flops_k = sum(2.0 * T * len(sample_rows) * (L["layer"].d_in + L["layer"].d_out) for L in layers)
        flops_comb = 0.0
    flops_step = flops_dw + flops_k + flops_comb
    step_tflops = flops_step / (ms_per_step * 1e-3) / 1e12

    # ---- roofline of the dominant kernel, from the events recorded inside the timed region ----
    dom = max(prof.items(), key=lambda kv: kv[1][0])[0] if prof else None
    roofline = None
    if dom == "k_bf16_weight_grad":
        ms_total, n = prof[dom]
        achieved = flops_dw * args.steps / (ms_total * 1e-3) / 1e12
        roofline = {"kernel": dom, "bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops_sustained"],
                    "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops_sustained"], "traffic": None,
                    "peak_source": f"{peaks['source']} sustained bf16 (burst {peaks['bf16_tflops']})",
                    "avg_launch_ms": ms_total / n, "launches": n}
    elif dom == "k_bf16_gram":
        # Gram route: (d_in + d_out) T^2 flop per layer (symmetric half of the two token Grams)
        ms_total, n = prof[dom]
        flops_gram = sum(float(L["layer"].d_in + L["layer"].d_out) * T * T for L in layers if L["path"] == b.PATH_GRAM)
        achieved = flops_gram * args.steps / (ms_total * 1e-3) / 1e12
        roofline = {"kernel": dom, "bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"],
                    "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"], "traffic": None,
                    "peak_source": f"{peaks['source']} burst bf16 (short kernels; sustained {peaks['bf16_tflops_sustained']})",
                    "avg_launch_ms": ms_total / n, "launches": n}
    elif dom == "k_bf16_seq_grad":
        ms_total, n = prof[dom]
        achieved = flops_dw * args.steps / (ms_total * 1e-3) / 1e12
        # DRAM bytes per launch: ncu's dram__bytes_read + write of this kernel over the seven projections of the
        # llm_1p5b block at full size (one-pass capture), as a ratio to the algorithmic bytes (inputs read once +
        # gradients written once) and applied to this run's average launch.
        alg_bytes = sum(2.0 * T * (L["layer"].d_in + L["layer"].d_out) + 2.0 * B * L["layer"].d_in * L["layer"].d_out
                        for L in layers) / len(layers)
        traffic = SEQ_GRAD_DRAM_OVER_ALGORITHMIC * alg_bytes
        roofline = {"kernel": dom, "bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops_sustained"],
                    "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops_sustained"], "traffic": traffic,
                    "traffic_unit": "bytes per launch (ncu dram__bytes_read+write at full size on llm_1p5b, median of five boxes: 1.56 x algorithmic)",
                    "peak_source": f"{peaks['source']} sustained bf16 (burst {peaks['bf16_tflops']})",
                    "avg_launch_ms": ms_total / n, "launches": n}
    elif dom is not None:
        ms_total, n = prof[dom]
        roofline = {"kernel": dom, "bound": "hbm", "achieved": None, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": None, "traffic": None, "avg_launch_ms": ms_total / n, "launches": n}
    kernels = {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] / args.steps} for k, v in prof.items()}
    # one pass over the stored gradients (layers on the stored route only)
    g_bytes = sum(2.0 * B * L["layer"].d_in * L["layer"].d_out for L in layers
                  if not sampled and L["path"] != b.PATH_GRAM)
    for name in ("k_bf16_ntk", "k_bf16_combine"):
        if name in kernels and kernels[name]["ms_per_step"] > 0:
            kernels[name]["hbm_gbs"] = g_bytes / (kernels[name]["ms_per_step"] * 1e-3) / 1e9
            kernels[name]["hbm_frac"] = kernels[name]["hbm_gbs"] / peaks["hbm_gbs"]

    # ---- per-projection breakdown (one more untimed pass, events per kernel) ----
    per_layer = []
    b.isopo_profile_enable(True)
    for L in layers:
        layer_calls(L)
        pl = b.isopo_profile_collect()
        per_layer.append({"layer": L["layer"].name, **{k: round(v[0], 4) for k, v in pl.items()}})
    b.isopo_profile_enable(False)

    # ---- plain dW GEMM (cuBLAS through torch) on the same inputs, same run ----
    # Timed the way the step is: the block's GEMMs one after the other, args.steps times, after three untimed
    # passes.  (A loop over one layer at a time starts each layer from an idle, cool GPU and lets the short
    # GEMMs run above the clock the power cap sustains; it read 1-5 % lower than this loop on the same box.)
    def block_loop(call):
        for _ in range(3):
            for L in layers:
                call(L)
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(args.steps):
            for L in layers:
                call(L)
        c.record()
        torch.cuda.synchronize()
        total = a.elapsed_time(c) / args.steps
        # per layer, from events inside a second, identical loop (the table only; not the headline figure)
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(len(layers) + 1)] for _ in range(args.steps)]
        for it in range(args.steps):
            ev[it][0].record()
            for k, L in enumerate(layers):
                call(L)
                ev[it][k + 1].record()
        torch.cuda.synchronize()
        by_layer = [sum(ev[it][k].elapsed_time(ev[it][k + 1]) for it in range(args.steps)) / args.steps
                    for k in range(len(layers))]
        return total, by_layer

    plain_ms, plain_by_layer = block_loop(lambda L: torch.matmul(L["dY"].t(), L["X"]))
    # for comparison only: one layer at a time, each in a loop of its own (see the note above)
    plain_isolated_ms = 0.0
    for L in layers:
        for _ in range(3):
            torch.matmul(L["dY"].t(), L["X"])
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(args.steps):
            torch.matmul(L["dY"].t(), L["X"])
        c.record()
        torch.cuda.synchronize()
        plain_isolated_ms += a.elapsed_time(c) / args.steps
    # the library's own plain GEMM: isopo_weight_grad on the GEMM route with every coefficient one
    # (bf16 workloads; the ratio above is quoted against the faster of the two, which is cuBLAS)
    own_plain_ms = None
    if w.dtype == "bf16":
        ones = torch.ones(B, dtype=torch.float32, device=dev)
        ws_g = aligned(max(b.isopo_workspace_bytes(dt_code, T, L["layer"].d_in, L["layer"].d_out, B, b.PATH_GRAM)
                           for L in layers))
        own_plain_ms, _ = block_loop(
            lambda L: b.isopo_weight_grad(L["X"], L["dY"], ones, off, L["dW"], ws_g, info, b.PATH_GRAM, 0.0))
        del ws_g
        b.isopo_profile_collect()
    overhead = ms_per_step / min(plain_ms, own_plain_ms) if own_plain_ms else ms_per_step / plain_ms

    # ---- the same step replayed from a CUDA graph (launch-bound workloads): extra figure, not the metric ----
    graph = None
    if args.graph:
        g = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        with torch.cuda.graph(g):
            step()
        for _ in range(3):
            g.replay()
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(args.steps):
            g.replay()
        c.record()
        torch.cuda.synchronize()
        if int(info.item()) != 0:
            raise SystemExit(f"device-side error during graph replay: info={int(info.item()):#x}")
        graph = {"ms_per_step": a.elapsed_time(c) / args.steps, "steps": args.steps,
                 "note": "one captured step replayed back to back; no L2 flush between replays"}

    # ---- end to end: host buffers, copies inside the timed region ----
    e2e = None
    if not args.skip_e2e:
        shapes = {}
        for L in layers:
            shapes.setdefault(("X", L["layer"].d_in), L["X"])
            shapes.setdefault(("dY", L["layer"].d_out), L["dY"])
        pinned = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True) for k, v in shapes.items()}
        for k, v in shapes.items():
            pinned[k].copy_(v)
        dW_host = {id(L): torch.empty(L["dW"].shape, dtype=torch.float32, pin_memory=True) for L in layers}
        h2d = sum(L["X"].numel() * L["X"].element_size() + L["dY"].numel() * L["dY"].element_size() for L in layers)
        d2h = sum(L["dW"].numel() * 4 for L in layers)

        # three streams: host -> device copies run ahead of the compute stream, results leave behind it;
        # events order every buffer's reuse (a layer's inputs are not overwritten before the previous
        # step's kernels on them are done, its dW not before the previous copy-out has left)
        comp = torch.cuda.current_stream()
        copy_s, out_s = torch.cuda.Stream(), torch.cuda.Stream()
        ready = {id(L): torch.cuda.Event() for L in layers}
        done = {id(L): torch.cuda.Event() for L in layers}
        left = {id(L): torch.cuda.Event() for L in layers}
        for L in layers:
            done[id(L)].record(comp)
            left[id(L)].record(comp)

        def e2e_step():
            for L in layers:
                with torch.cuda.stream(copy_s):
                    copy_s.wait_event(done[id(L)])
                    L["X"].copy_(pinned[("X", L["layer"].d_in)], non_blocking=True)
                    L["dY"].copy_(pinned[("dY", L["layer"].d_out)], non_blocking=True)
                    ready[id(L)].record(copy_s)
                comp.wait_event(ready[id(L)])
                comp.wait_event(left[id(L)])
                layer_calls(L)
                done[id(L)].record(comp)
                with torch.cuda.stream(out_s):
                    out_s.wait_event(done[id(L)])
                    dW_host[id(L)].copy_(L["dW"], non_blocking=True)
                    left[id(L)].record(out_s)

        e2e_step()
        torch.cuda.synchronize()
        n_e2e = max(1, min(args.steps, 3))
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(comp)
        copy_s.wait_event(a)
        for _ in range(n_e2e):
            e2e_step()
        for L in layers:
            comp.wait_event(left[id(L)])  # the last results have reached the host
        c.record(comp)
        torch.cuda.synchronize()
        e2e_ms = a.elapsed_time(c) / n_e2e
        e2e = {"value": T / (e2e_ms / 1000.0), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_ms, "steps": n_e2e}
        del pinned, dW_host

    # ---- the other route through the library on the same inputs: Algorithm 1 as printed (sampled Fisher norm) ----
    routes = None
    if not sampled and w.dtype == "bf16" and world == 1 and not args.skip_routes:
        s_ws = aligned(max(b.isopo_sampled_workspace_bytes(dt_code, T, L["layer"].d_in, L["layer"].d_out, B, len(sample_rows))
                           for L in layers))
        F2 = torch.zeros(B, dtype=torch.float32, device=dev)
        lam_s = {}

        def sampled_step():
            for L in layers:
                b.isopo_sampled_coefficients(L["X"], L["dY"], off, sample_rows, A, lam_s.get(id(L), 0.0), L["c"], s_ws, info, F2)
                b.isopo_weight_grad(L["X"], L["dY"], L["c"], off, L["dW"], s_ws, info, b.PATH_GRAM, 0.0)

        for L in layers:  # regulariser 1e-3 * mean(F^2), taken once from an untimed pass
            b.isopo_sampled_coefficients(L["X"], L["dY"], off, sample_rows, A, 0.0, L["c"], s_ws, info, F2)
            lam_s[id(L)] = 1e-3 * float(F2.mean().item())
        for _ in range(3):
            sampled_step()
        torch.cuda.synchronize()
        b.isopo_profile_collect()
        n_s = max(1, min(args.steps, 10))
        s_sampler = ClockSampler(local)
        b.isopo_profile_enable(True)
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        s_sampler.start()
        a.record()
        for _ in range(n_s):
            sampled_step()
        c.record()
        torch.cuda.synchronize()
        s_clocks = s_sampler.stop()
        b.isopo_profile_enable(False)
        s_prof = b.isopo_profile_collect()
        if int(info.item()) != 0:
            raise SystemExit(f"device-side error on the sampled route: info={int(info.item()):#x}")
        s_ms = a.elapsed_time(c) / n_s
        routes = {"sampled": {
            "what": "Algorithm 1 as printed: isopo_sampled_coefficients (%d seeded token samples) + isopo_weight_grad on "
                    "the GEMM route for each projection; normalised variant; same inputs, same run" % len(sample_rows),
            "ms_per_step": s_ms, "steps": n_s, "tokens_per_s": T / (s_ms * 1e-3),
            "overhead_vs_plain_dw_gemm": s_ms / plain_ms,
            "kernels": {k: {"ms_per_step": v[0] / n_s, "launches_per_step": v[1] / n_s} for k, v in s_prof.items()},
            "clocks": s_clocks}}
        del s_ws

    # ---- the stored route once more with the split e4m3 store (K pass on half the bytes), same inputs and workspaces ----
    if not sampled and w.dtype == "bf16" and world == 1 and not args.skip_routes and args.store_format == "bf16":
        b.isopo_set_store_format(b.STORE_E4M3_SPLIT)
        try:
            for _ in range(3):
                step()
            torch.cuda.synchronize()
            b.isopo_profile_collect()
            n_s = max(1, min(args.steps, 10))
            f_sampler = ClockSampler(local)
            b.isopo_profile_enable(True)
            a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            f_sampler.start()
            a.record()
            for _ in range(n_s):
                step()
            c.record()
            torch.cuda.synchronize()
            f_clocks = f_sampler.stop()
            b.isopo_profile_enable(False)
            f_prof = b.isopo_profile_collect()
            if int(info.item()) != 0:
                raise SystemExit(f"device-side error with the split store: info={int(info.item()):#x}")
            f_ms = a.elapsed_time(c) / n_s
            from oracle import isopo_oracle as orc
            f_parity = None if args.skip_parity else parity_check(
                layers, off, A, [L["lam"] for L in layers], orc.INTERACTING if args.variant == "interacting" else orc.NORMALISED)
            routes = routes or {}
            routes["stored_e4m3_split"] = {
                "what": "the stored route with isopo_set_store_format(ISOPO_STORE_E4M3_SPLIT): gradients kept as two e4m3 "
                        "planes, K pass on the high plane, diagonal of K from float32 sums in the gradient GEMM; same "
                        "inputs, workspaces and schedule, same run",
                "ms_per_step": f_ms, "steps": n_s, "tokens_per_s": T / (f_ms * 1e-3),
                "overhead_vs_plain_dw_gemm": f_ms / plain_ms,
                "kernels": {k: {"ms_per_step": v[0] / n_s, "launches_per_step": v[1] / n_s} for k, v in f_prof.items()},
                "parity": f_parity, "clocks": f_clocks}
        finally:
            b.isopo_set_store_format(b.STORE_BF16)

    # ---- the stored route with ONE workspace reused by every projection (what a backward pass with little spare
    #      memory does: gram, transform, weight gradient per layer; seven single solves instead of one batched) ----
    if batched and w.dtype == "bf16" and world == 1 and not args.skip_routes and args.store_format == "bf16":
        one_ws = aligned(max(ws_sizes))

        def one_ws_step():
            for L in layers:
                b.isopo_layer_gram(L["X"], L["dY"], off, L["K"], one_ws, info, L["path"])
                b.isopo_transform_advantages(L["K"], A, variant, L["lam"], L["c"], info)
                b.isopo_weight_grad(L["X"], L["dY"], L["c"], off, L["dW"], one_ws, info, L["path"], 0.0)

        for _ in range(3):
            one_ws_step()
        torch.cuda.synchronize()
        n_s = max(1, min(args.steps, 10))
        o_sampler = ClockSampler(local)
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        o_sampler.start()
        a.record()
        for _ in range(n_s):
            one_ws_step()
        c.record()
        torch.cuda.synchronize()
        o_clocks = o_sampler.stop()
        if int(info.item()) != 0:
            raise SystemExit(f"device-side error with one workspace: info={int(info.item()):#x}")
        o_ms = a.elapsed_time(c) / n_s
        routes = routes or {}
        routes["stored_one_workspace"] = {
            "what": "the stored route with one workspace reused by every projection and a transform launch per "
                    "projection (the headline step keeps all workspaces and solves the block in one launch); same inputs, same run",
            "ms_per_step": o_ms, "steps": n_s, "tokens_per_s": T / (o_ms * 1e-3), "overhead_vs_plain_dw_gemm": o_ms / plain_ms,
            "workspace_gb": max(ws_sizes) / 1e9, "headline_workspaces_gb": sum(ws_sizes) / 1e9, "clocks": o_clocks}
        del one_ws

    # ---- the oracle on this machine's host cores, bounded sample ----
    cpu = None
    if world == 1 and not args.skip_cpu:
        tok_s, dt_s, desc = oracle_sample(args.workload, args.cpu_seqs, args.cpu_len_div)
        cpu = {"value": tok_s / dt_s, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": desc,
               "seconds": dt_s}

    # ---- end-to-end decoder backward (library calls in every linear layer's hook) against plain gradients ----
    cfg_layers = [f"{L['layer'].name}:{L['layer'].d_in}->{L['layer'].d_out}" for L in layers]
    cfg_paths = ["gram" if L["path"] == b.PATH_GRAM else "materialise" for L in layers]
    decoder = None
    if world == 1 and not args.skip_decoder and args.workload == "llm_1p5b" and not args.layers and not args.seqs:
        import bench_decoder
        for L in layers:  # the block's tensors and workspaces go first: the decoder needs the memory
            L.clear()
        del layers
        torch.cuda.empty_cache()
        decoder = {}
        for route in ("stored", "sampled"):
            d_sampler = ClockSampler(local)
            d_sampler.start()
            rec = bench_decoder.run_decoder(bench_decoder.parse_args(["--route", route, "--steps", "2", "--warmup", "1"]), dev)
            rec["clocks"] = d_sampler.stop()
            decoder[route] = rec
            torch.cuda.empty_cache()

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": n_warm, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": args.workload, "B": B, "tokens": T,
                   "route": "sampled (Algorithm 1, %d token samples)" % len(sample_rows) if sampled else "stored gradients",
                   "variant": "normalised (Algorithm 1)" if sampled else args.variant,
                   "store_format": args.store_format, "deterministic": bool(args.deterministic),
                   "layers": cfg_layers, "paths": cfg_paths,
                   "l2": ("L2 flushed between steps (256 MB fill, untimed); every step timed by its own events"
                          if flush else "inputs larger than L2 (no flush needed)"),
                   "step": ("sampled_coefficients + weight_grad for each projection" if sampled else
                            "layer_gram for each projection, one transform_advantages_batched for all, weight_grad "
                            "for each projection" if batched else

                            "layer_gram + transform_advantages + weight_grad for each projection")},
        "clocks": clocks,
        "e2e": e2e,
        "cuda_graph": graph,
        "gpu_launches": int(sum(v[1] for v in prof.values())),
        "roofline": roofline,
        "cpu_baseline": cpu,
        "parity": parity,
        "routes": routes,
        "decoder": decoder,
        "step_tflops": step_tflops,
        "pct_bf16_peak_sustained": step_tflops / peaks["bf16_tflops_sustained"],
        "plain_dw_gemm_ms": plain_ms,
        "plain_dw_gemm_timing": "the block's GEMMs back to back, steps x block, one pair of events (as the step is timed)",
        "plain_dw_gemm_per_layer_loops_ms": plain_isolated_ms,
        "plain_dw_gemm_own_ms": own_plain_ms,
        "overhead_vs_plain_dw_gemm": overhead,
        "kernels": kernels,
        "per_layer_ms": [dict(pl, plain_dw_gemm=round(pm, 4)) for pl, pm in zip(per_layer, plain_by_layer)],
    }
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llm_1p5b")
    ap.add_argument("--variant", default="interacting", choices=["interacting", "normalised"])
    ap.add_argument("--route", default="stored", choices=["stored", "sampled"],
                    help="stored: K from materialised per-sequence gradients (both variants); sampled: Algorithm 1's "
                         "token-sampled Fisher norm + folded weight-gradient GEMM (non-interacting variant)")
    ap.add_argument("--samples", type=int, default=128, help="n_overlap_samples of the sampled route")
    ap.add_argument("--store-format", default="bf16", choices=["bf16", "e4m3_split"],
                    help="stored route: how the per-sequence gradients are kept (isopo_set_store_format)")
    ap.add_argument("--schedule", default="batched", choices=["batched", "single"],
                    help="stored route: batched = every projection keeps its workspace and one launch solves for all "
                         "their coefficients; single = one call per projection, one shared workspace")
    ap.add_argument("--deterministic", action="store_true",
                    help="stored route: K summed over the CTAs in a fixed order (isopo_set_deterministic)")
    ap.add_argument("--graph", action="store_true",
                    help="also capture one step in a CUDA graph and time its replays (reported under cuda_graph)")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-parity", action="store_true", help="do not check the timed run's outputs against the oracle")
    ap.add_argument("--skip-routes", action="store_true", help="do not also time the sampled route (Algorithm 1)")
    ap.add_argument("--skip-decoder", action="store_true", help="do not run the end-to-end decoder harness")
    ap.add_argument("--layers", default="", help="comma-separated projection names (default: all of the block)")
    ap.add_argument("--seqs", type=int, default=0, help="use only the first N sequences (profiling aid)")
    ap.add_argument("--short-warmup", action="store_true", help="allow fewer than 3 warm-up steps (profiling only)")
    ap.add_argument("--cpu-seqs", type=int, default=8)
    ap.add_argument("--cpu-len-div", type=int, default=8)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
