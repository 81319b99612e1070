#!/usr/bin/env python
"""Benchmark of the JoT denoising step on B200.

A step is one pass of the whole hot path over one batch: transformer forward over the canvas, LM head
fused with the online softmax statistics over the masked rows of the current block, acceptance /
freeze update.  Default workload: the LLaDA-8B-shaped random-init model, batch 1, prompt 128 + 256
masked tokens, semi-autoregressive blocks of 32 (seeded synthetic weights and tokens).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload llada8b|tiny]

Prints ONE JSON line.  With --gpus N > 1 (under torchrun) every rank runs an independent replica of the
workload (sequences are independent; there is no data-path collective) and rank 0 reports the aggregate.
--impl reference times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2602_11133_b200 import inputs  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

WORKLOADS = {
    # name: (geometry, B, P, G, T, block_len, (tau_max, tau_min, gamma, D))
    "llada8b": (inputs.LLADA_8B, 1, 128, 256, 256, 32, (30.0, 1.0, 0.5, 8)),
    "tiny": (inputs.TINY, 1, 32, 64, 64, 64, (90.0, 1.0, 0.5, 8)),
}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """SM clock and throttle reasons sampled through NVML (read-only queries) while the timed region runs."""
    REASONS = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40, "sw_power_cap": 0x4}

    def __init__(self, device: torch.device, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz, self.period = [], set(), None, period_s
        self.stop_flag = threading.Event()
        self.thread = None
        self.handle = None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(device.index or 0)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.handle = None

    def _loop(self):
        nv = self.nv
        while not self.stop_flag.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM)))
                bits = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
                for name, bit in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self.stop_flag.wait(self.period)

    def __enter__(self):
        if self.handle is not None:
            self.thread = threading.Thread(target=self._loop, daemon=True)
            self.thread.start()
        return self

    def __exit__(self, *exc):
        self.stop_flag.set()
        if self.thread:
            self.thread.join(timeout=2)

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def step_flops(g, n_layers, B, L, R):
    """Algorithmic flops of one step: body projections and attention over the canvas, LM head over R rows."""
    M = B * L
    d, hd = g.d_model, g.head_dim
    per_layer = 2 * M * d * g.qkv_rows + 2 * M * (g.n_q_heads * hd) * d + 2 * M * d * 2 * g.d_ff + 2 * M * g.d_ff * d
    attn = 4 * B * g.n_q_heads * L * L * hd
    return n_layers * (per_layer + attn), 2 * R * d * g.vocab


def weight_bytes(g, n_layers):
    per_layer = (g.qkv_rows * g.d_model + g.d_model * g.n_q_heads * g.head_dim + 3 * g.d_ff * g.d_model) * 2
    return n_layers * per_layer + g.vocab * g.d_model * 2


# ------------------------------------------------------------------------------------------------ CPU oracle
def time_oracle_sample(g, w_any, nl, B, P, G, block_len, params, sample_layers=2, reps=1):
    """Time the CPU oracle as it stands on a bounded sample: `sample_layers` transformer layers over the
    whole canvas, plus the LM head, statistics and acceptance over the first block's rows; extrapolate
    the body linearly to the model's depth.  Returns (seconds per full step, description, threads)."""
    from oracle import jot_oracle as jo
    from oracle import model_oracle as mo
    L = P + G
    sl = min(sample_layers, nl, len(w_any["layers"]))
    w_cpu = {k: v.cpu() for k, v in w_any.items() if k != "layers"}
    w_cpu["layers"] = [{k: v.cpu() for k, v in lw.items()} for lw in w_any["layers"][:sl]]
    prompt = inputs.prompt(0, B, P, g.vocab, g.mask_id)
    x = torch.cat([prompt, torch.full((B, G), g.mask_id, dtype=torch.int32)], dim=1)
    rows = [(b, i) for b in range(B) for i in range(P, P + block_len)]
    jp = jo.JotParams(*params)
    best_body, best_head = float("inf"), float("inf")
    for _ in range(reps):
        t0 = time.perf_counter()
        h = mo.hidden_states(g, w_cpu, x, True, sl)
        t1 = time.perf_counter()
        sel = torch.stack([h[b, i] for b, i in rows])
        logits = mo.lm_head_logits(sel, w_cpu["lm_head"])
        for b in range(B):
            xs = x[b].tolist()
            st = {i: jo.row_stats(logits[r].numpy(), g.mask_id) for r, (bb, i) in enumerate(rows) if bb == b}
            jo.accept_freeze(xs, st, jp, g.mask_id, P, P + block_len, 1)
        t2 = time.perf_counter()
        best_body, best_head = min(best_body, t1 - t0), min(best_head, t2 - t1)
    step_s = best_body * (nl / sl if sl else 0.0) + best_head
    desc = (f"{sl} of {nl} layers over the {B}x{L} canvas (body time scaled by {nl}/{sl}) + LM head, statistics and "
            f"acceptance over the {len(rows)} rows of the first block; float64")
    return step_s, desc, torch.get_num_threads()


# ------------------------------------------------------------------------------------------------ main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llada8b", choices=sorted(WORKLOADS))
    ap.add_argument("--layers", type=int, default=None, help="override depth (debugging only; invalid as a result)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    g, B, P, G, T, Lb, params = WORKLOADS[args.workload]
    L = P + G
    nl = g.n_layers if args.layers is None else args.layers

    if args.impl == "reference":
        if rank != 0:
            return 0
        return run_reference(args, g, nl, B, P, G, T, Lb, params)

    from paper_2602_11133_b200 import jot
    jot._lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    peaks, peaks_kind = load_peaks()
    weights = inputs.model_weights(g, seed=0, device=dev, n_layers=nl)
    model = jot.Model(g, weights, B, L)
    jp = jot.Params(*params)
    prompt_host = inputs.prompt(0, B, P, g.vocab, g.mask_id).pin_memory()
    canvas0 = torch.cat([prompt_host, torch.full((B, G), g.mask_id, dtype=torch.int32)], dim=1).to(dev)
    stats = jot.Stats.empty(B, L, dev)
    n_masked = torch.zeros(B, dtype=torch.int32, device=dev)

    def run_steps(n, tokens):
        """n denoising steps of the block schedule (one token per step by the schedule, early exits on top)."""
        for s in range(n):
            blk = min(s // Lb, G // Lb - 1)
            lo = P + blk * Lb
            model.denoise_step(tokens, lo, lo + Lb, out=stats)
            jot.accept_freeze(jp, g.mask_id, tokens, lo, lo + Lb, 1, stats, n_masked, step_index=s + 1)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    tokens = canvas0.clone()
    run_steps(args.warmup, tokens)
    tokens = canvas0.clone()
    barrier()
    launches0 = jot.launch_count()
    model.profile(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(dev) as clocks:
        ev0.record()
        run_steps(args.steps, tokens)
        ev1.record()
        barrier()
    ms = ev0.elapsed_time(ev1)
    prof = model.profile_read()
    model.profile(False)
    launches = jot.launch_count() - launches0

    # ---- end to end through the public call: host prompt -> jot_generate -> host tokens ----
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    d_prompt = prompt_host.to(dev, non_blocking=True)
    out, used, passes = model.generate(d_prompt, G, T, jp, Lb)
    host_out = out.cpu()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_tokens = host_out.shape[1] - P

    t_ms = torch.tensor([ms, e2e_s * 1e3], dtype=torch.float64, device=dev)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t_ms, op=dist.ReduceOp.MAX)
    ms_max, e2e_ms_max = t_ms.tolist()
    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return 0

    steps_per_s = world * args.steps / (ms_max / 1e3)
    body_flops, head_flops = step_flops(g, nl, B, L, B * Lb)
    # dominant kernel class by measured device time
    dom = max(prof, key=lambda k: prof[k][0])
    dom_ms, dom_n = prof[dom]
    M = B * L
    flops_per_launch = {
        "gemm_qkv": 2 * M * g.d_model * g.qkv_rows, "gemm_o": 2 * M * g.n_q_heads * g.head_dim * g.d_model,
        "gemm_gate_up": 2 * M * g.d_model * 2 * g.d_ff, "gemm_down": 2 * M * g.d_ff * g.d_model,
        "attention": 4 * B * g.n_q_heads * L * L * g.head_dim, "lm_head": 2 * B * Lb * g.d_model * g.vocab,
    }
    tensor_peak = peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"])
    if dom in flops_per_launch and dom_n:
        ach = flops_per_launch[dom] / (dom_ms / dom_n * 1e-3) / 1e12
        roofline = {"kernel": dom, "bound": "tensor", "achieved": round(ach, 2), "peak": tensor_peak,
                    "unit": "TFLOP/s", "frac": round(ach / tensor_peak, 4), "traffic": None,
                    "peak_kind": f"bf16 cuBLAS sustained, of {peaks_kind}", "avg_launch_ms": round(dom_ms / dom_n, 4),
                    "launches": dom_n}
    else:
        roofline = {"kernel": dom, "bound": "hbm", "achieved": None, "peak": peaks.get("hbm_gbs"), "unit": "GB/s",
                    "frac": None, "traffic": None}
    total_prof = sum(v[0] for v in prof.values()) or 1.0
    breakdown = {k: {"ms_per_step": round(v[0] / args.steps, 4), "share": round(v[0] / total_prof, 4),
                     "launches_per_step": round(v[1] / args.steps, 2)} for k, v in prof.items() if v[1]}
    for k, f in flops_per_launch.items():
        if k in breakdown and prof[k][1]:
            breakdown[k]["tflops"] = round(f / (prof[k][0] / prof[k][1] * 1e-3) / 1e12, 1)
    step_s = ms_max / 1e3 / args.steps
    whole = {"step_tflops": round((body_flops + head_flops) / step_s / 1e12, 1),
             "tensor_frac_of_" + peaks_kind: round((body_flops + head_flops) / step_s / 1e12 / tensor_peak, 4),
             "weight_stream_gbs": round(weight_bytes(g, nl) / step_s / 1e9, 1),
             "hbm_frac_of_" + peaks_kind: round(weight_bytes(g, nl) / step_s / 1e9 / peaks.get("hbm_gbs", 6650.0), 4)}

    cpu_step_s, cpu_desc, cpu_threads = time_oracle_sample(g, weights, nl, B, P, G, Lb, params)
    line = {
        "metric": "denoising_steps_per_s", "value": round(steps_per_s, 3), "unit": "steps/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_max / args.steps, 4),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {nl} layers d={g.d_model} heads={g.n_q_heads}/{g.n_kv_heads}x{g.head_dim} "
                               f"ff={g.d_ff} vocab={g.vocab}; batch {B} per GPU, prompt {P} + {G} masked, blocks of {Lb}, "
                               f"JoT ({params[0]:g},{params[1]:g},{params[2]:g},{params[3]})",
                   "l2": "inputs exceed L2: every step streams %.1f GB of weights" % (weight_bytes(g, nl) / 1e9),
                   "parallelism": "independent replicas" if world > 1 else "single GPU"},
        "clocks": clocks.summary(),
        "e2e": {"value": round(world * passes / (e2e_ms_max / 1e3), 3), "unit": "steps/s",
                "h2d_bytes_per_step": int(prompt_host.numel() * 4 / max(passes, 1)),
                "d2h_bytes_per_step": int(host_out.numel() * 4 / max(passes, 1) + 12),
                "call": "jot_generate from a pinned host prompt to host tokens", "forward_passes": passes,
                "steps_used": used, "generated_tokens_per_s": round(world * B * e2e_tokens / (e2e_ms_max / 1e3), 2)},
        "gpu_launches": int(launches),
        "roofline": roofline, "step_roofline": whole, "kernels": breakdown,
        "cpu_baseline": {"value": round(1.0 / cpu_step_s, 5), "unit": "steps/s", "cores": cpu_threads, "kind": "oracle",
                         "sample": cpu_desc},
    }
    print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


def run_reference(args, g, nl, B, P, G, T, Lb, params):
    """The CPU oracle, as it stands, on a bounded sample of the workload (host cores only)."""
    w = inputs.model_weights(g, seed=0, device="cpu", n_layers=min(2, nl))
    times = []
    desc, threads = "", 0
    for i in range(args.warmup + args.steps):
        step_s, desc, threads = time_oracle_sample(g, w, nl, B, P, G, Lb, params)
        if i >= args.warmup:
            times.append(step_s)
        if sum(times) > 90:          # keep the whole run within a few minutes
            break
    step = statistics.mean(times)
    line = {"impl": "reference", "metric": "denoising_steps_per_s", "value": round(1.0 / step, 5), "unit": "steps/s",
            "n_gpus": args.gpus, "steps": len(times), "warmup": args.warmup, "ms_per_step": round(step * 1e3, 2),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{args.workload}: CPU oracle on a bounded sample"},
            "cpu_baseline": {"value": round(1.0 / step, 5), "unit": "steps/s", "cores": threads, "kind": "oracle",
                             "sample": desc},
            "e2e": {"value": round(1.0 / step, 5), "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


if __name__ == "__main__":
    sys.exit(main())
