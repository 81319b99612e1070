#!/usr/bin/env python
"""Benchmark of the JoT denoising step on B200.

A step is one pass of the whole hot path over one batch: transformer forward over the canvas, LM head
fused with the online softmax statistics over the masked rows of the current block, acceptance /
freeze update.  Default workload: the LLaDA-8B-shaped random-init model, batch 1, prompt 128 + 256
masked tokens, semi-autoregressive blocks of 32 (seeded synthetic weights and tokens).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload llada8b|tiny|lmhead]

`--workload lmhead` times the fused LM-head + acceptance part alone on given hidden states
([8, 384, 4096] rows against a [126464, 4096] head, planted logit bump, half of the 256 generation
positions masked).

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

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/, keyed by kernel class and workload; removed (-> null) whenever the kernel changes afterwards.
NCU_TRAFFIC = {
    ("llada8b", "gemm_gate_up"): 216.7e6,     # profiles/gemm_llada8b_m384.md
    ("lmhead", "lm_head"): 1067.0e6,          # profiles/lm_head_pair_lmhead.md
}

WORKLOADS = {
    # name: (geometry, B, P, G, T, block_len, (tau_max, tau_min, gamma, D))
    "llada8b": (inputs.LLADA_8B, 1, 128, 256, 256, 32, (30.0, 1.0, 0.5, 8)),
    "tiny": (inputs.TINY, 1, 32, 64, 64, 64, (90.0, 1.0, 0.5, 8)),
    "lmhead": (inputs.LLADA_8B, 8, 128, 256, 1, 256, (30.0, 1.0, 0.5, 8)),
    # the two large-batch shapes: tensor-bound steps (parity-test shapes; here for their per-kernel rates)
    "dream7b": (inputs.DREAM_7B, 8, 256, 256, 256, 256, (90.0, 1.0, 0.5, 8)),
    "llada8b_b16": (inputs.LLADA_8B, 16, 192, 512, 512, 32, (30.0, 1.0, 0.5, 8)),
}
BIG = {"dream7b", "llada8b_b16"}


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
def dist_setup(world, dev):
    """One process per GPU; the process group only carries the timing barrier and the max over ranks
    (replicas are independent: there is no collective on the data path)."""
    if world > 1:
        import torch.distributed as dist
        if dev.type == "cuda":
            dist.init_process_group("nccl", device_id=dev)
        else:
            dist.init_process_group("gloo")


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def aggregate_rate(units_per_rank, world, ms_max):
    """Whole-job rate: what all ranks processed divided by the slowest rank's time."""
    return world * units_per_rank / (ms_max / 1e3)


def max_over_ranks(values, world, dev):
    t = torch.tensor(values, dtype=torch.float64, device=dev)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def timed_region(run_steps, fresh_state, steps, warmup, world, dev, model, jot):
    """W warm-up steps, then K steps timed with CUDA events on the launching stream (plain run: this is the
    reported value), then the same K steps once more with an event pair around every kernel launch (the
    per-kernel durations behind the roofline; the events cost host time, so that pass is not the value)."""
    run_steps(warmup, fresh_state())
    state = fresh_state()
    barrier(world)
    launches0 = jot.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(dev) as clocks:
        ev0.record()
        run_steps(steps, state)
        ev1.record()
        barrier(world)
    ms = ev0.elapsed_time(ev1)
    launches = jot.launch_count() - launches0
    state = fresh_state()
    torch.cuda.synchronize()
    model.profile(True)
    run_steps(steps, state)
    torch.cuda.synchronize()
    prof = model.profile_read()
    model.profile(False)
    return ms, launches, clocks.summary(), prof


def kernel_report(prof, steps, flops_per_launch, bytes_per_launch, peaks, peaks_kind, workload):
    total = sum(v[0] for v in prof.values()) or 1.0
    rep = {}
    for k, (ms, n) in prof.items():
        if not n:
            continue
        e = {"ms_per_step": round(ms / steps, 4), "share": round(ms / total, 4), "launches_per_step": round(n / steps, 2)}
        if k in flops_per_launch:
            e["tflops"] = round(flops_per_launch[k] / (ms / n * 1e-3) / 1e12, 1)
        if k in bytes_per_launch:
            e["gbs"] = round(bytes_per_launch[k] / (ms / n * 1e-3) / 1e9, 1)
        rep[k] = e
    dom = max(prof, key=lambda k: prof[k][0])
    ms, n = prof[dom]
    tensor_peak = peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"])
    hbm_peak = peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"])
    traffic = NCU_TRAFFIC.get((workload, dom))
    if dom in flops_per_launch:
        ach = flops_per_launch[dom] / (ms / n * 1e-3) / 1e12
        roof = {"kernel": dom, "bound": "tensor", "achieved": round(ach, 2), "peak": tensor_peak, "unit": "TFLOP/s",
                "frac": round(ach / tensor_peak, 4), "traffic": traffic,
                "peak_kind": f"cuBLAS bf16 sustained, of {peaks_kind}", "avg_launch_ms": round(ms / n, 4), "launches": n,
                "frac_of_nominal_2250": round(ach / 2250.0, 4)}
    else:
        b = bytes_per_launch.get(dom)
        ach = b / (ms / n * 1e-3) / 1e9 if b else None
        roof = {"kernel": dom, "bound": "hbm", "achieved": round(ach, 1) if ach else None, "peak": hbm_peak,
                "unit": "GB/s", "frac": round(ach / hbm_peak, 4) if ach else None, "traffic": traffic,
                "peak_kind": f"copy bandwidth, of {peaks_kind}", "avg_launch_ms": round(ms / n, 4), "launches": n}
    return rep, roof


def workload_config(args, g, nl, B, P, G, Lb, params, world):
    if args.workload == "lmhead":
        return {"workload": f"lmhead: hidden [{B},{P + G},{g.d_model}] x head [{g.vocab},{g.d_model}], planted bump, prompt {P} "
                            f"resolved + {G} positions masked with p=0.5, then acceptance; JoT ({params[0]:g},{params[1]:g},"
                            f"{params[2]:g},{params[3]})",
                "l2": "inputs exceed L2: the head alone is %.2f GB" % (g.vocab * g.d_model * 2 / 1e9),
                "parallelism": "independent replicas" if world > 1 else "single GPU"}
    return {"workload": f"{args.workload}: {nl} layers d={g.d_model} heads={g.n_q_heads}/{g.n_kv_heads}x{g.head_dim} "
                        f"ff={g.d_ff} vocab={g.vocab}; batch {B} per GPU, prompt {P} + {G} masked, blocks of {Lb}, "
                        f"JoT ({params[0]:g},{params[1]:g},{params[2]:g},{params[3]})",
            "l2": "inputs exceed L2: every step streams %.1f GB of weights" % (weight_bytes(g, nl) / 1e9),
            "parallelism": "independent replicas" if world > 1 else "single GPU"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llada8b", choices=sorted(WORKLOADS))
    ap.add_argument("--layers", type=int, default=None, help="override depth (profiling small cases; not a result)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    g, B, P, G, T, Lb, params = WORKLOADS[args.workload]
    nl = g.n_layers if args.layers is None else args.layers
    config = workload_config(args, g, nl, B, P, G, Lb, params, world)

    if args.impl == "reference":
        if rank != 0:
            return 0
        return run_reference(args, config, g, nl, B, P, G, T, Lb, params)

    from paper_2602_11133_b200 import jot
    jot._lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist_setup(world, dev)
    peaks, peaks_kind = load_peaks()
    runner = run_lmhead if args.workload == "lmhead" else run_model
    line = runner(args, jot, dev, world, rank, peaks, peaks_kind, config, g, nl, B, P, G, T, Lb, params)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


def base_line(args, world, metric, unit, value, ms_per_step, config, clocks, launches):
    return {"metric": metric, "value": round(value, 3), "unit": unit, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(ms_per_step, 4), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config, "clocks": clocks,
            "gpu_launches": int(launches)}


def run_model(args, jot, dev, world, rank, peaks, peaks_kind, config, g, nl, B, P, G, T, Lb, params):
    L = P + G
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

    ms, launches, clocks, prof = timed_region(run_steps, canvas0.clone, args.steps, args.warmup, world, dev, model, jot)

    # end to end through the public call: pinned host prompt -> jot_generate -> host tokens.  The large-batch
    # shapes would take minutes for a whole generation: they run the first `steps` iterations' worth instead
    # (generation length cut to steps tokens' blocks on the same prompt), flagged in the output.
    e2e_T, e2e_G = T, G
    if args.workload in BIG:
        e2e_G = max(Lb, min(G, (args.steps // Lb) * Lb)) if Lb < G else G
        e2e_T = min(T, max(args.steps, 1)) if Lb >= G else e2e_G
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    d_prompt = prompt_host.to(dev, non_blocking=True)
    out, used, passes = model.generate(d_prompt, e2e_G, e2e_T, jp, min(Lb, e2e_G))
    host_out = out.cpu()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    graph_ms = None
    if args.workload == "tiny":
        # launch-latency-bound shape: the same generation with the step replayed as a CUDA graph
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        model.generate(prompt_host.to(dev, non_blocking=True), e2e_G, e2e_T, jp, min(Lb, e2e_G), use_cuda_graph=True)[0].cpu()
        torch.cuda.synchronize()
        graph_ms = (time.perf_counter() - t0) * 1e3
    ms_max, e2e_ms_max = max_over_ranks([ms, e2e_s * 1e3], world, dev)
    if rank != 0:
        return None

    M = B * L
    flops = {"gemm_qkv": 2 * M * g.d_model * g.qkv_rows, "gemm_o": 2 * M * g.n_q_heads * g.head_dim * g.d_model,
             "gemm_gate_up": 2 * M * g.d_model * 2 * g.d_ff, "gemm_down": 2 * M * g.d_ff * g.d_model,
             "attention": 4 * B * g.n_q_heads * L * L * g.head_dim, "lm_head": 2 * B * Lb * g.d_model * g.vocab}
    nbytes = {"lm_head": g.vocab * g.d_model * 2, "rmsnorm": 2 * M * g.d_model * 2,
              "rope": M * g.qkv_rows * 2 * 2, "embed": 2 * M * g.d_model * 2}
    kernels, roofline = kernel_report(prof, args.steps, flops, nbytes, peaks, peaks_kind, args.workload)
    step_s = ms_max / 1e3 / args.steps
    body_flops, head_flops = step_flops(g, nl, B, L, B * Lb)
    tensor_peak = peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"])
    whole = {"step_tflops": round((body_flops + head_flops) / step_s / 1e12, 1),
             "tensor_frac": round((body_flops + head_flops) / step_s / 1e12 / tensor_peak, 4),
             "weight_stream_gbs": round(weight_bytes(g, nl) / step_s / 1e9, 1),
             "hbm_frac": round(weight_bytes(g, nl) / step_s / 1e9 / peaks.get("hbm_gbs", 6650.0), 4),
             "of": peaks_kind}
    line = base_line(args, world, "denoising_steps_per_s", "steps/s", aggregate_rate(args.steps, world, ms_max),
                     ms_max / args.steps, config, clocks, launches)
    line["generated_tokens_per_s"] = round(world * B * (host_out.shape[1] - P) / (e2e_ms_max / 1e3), 2)
    line["e2e"] = {"value": round(world * passes / (e2e_ms_max / 1e3), 3), "unit": "steps/s",
                   "h2d_bytes_per_step": round(prompt_host.numel() * 4 / max(passes, 1), 2),
                   "d2h_bytes_per_step": round(host_out.numel() * 4 / max(passes, 1) + 16, 2),
                   "call": "jot_generate: pinned host prompt in, host tokens out (whole generation)",
                   "forward_passes": passes, "steps_used": used,
                   "generation": f"{e2e_G} tokens, up to {e2e_T} steps" + (" (shortened)" if (e2e_G, e2e_T) != (G, T) else "")}
    if graph_ms is not None:
        line["e2e"]["us_per_step"] = round(e2e_ms_max * 1e3 / max(passes, 1), 1)
        line["e2e"]["us_per_step_with_cuda_graph"] = round(graph_ms * 1e3 / max(passes, 1), 1)
        line["e2e"]["kernels_per_step"] = round(launches / args.steps, 1)
    line["roofline"], line["step_roofline"], line["kernels"] = roofline, whole, kernels
    cpu_step_s, cpu_desc, cpu_threads = time_oracle_sample(g, weights, nl, B, P, G, Lb, params)
    line["cpu_baseline"] = {"value": round(1.0 / cpu_step_s, 5), "unit": "steps/s", "cores": cpu_threads,
                            "kind": "oracle", "sample": cpu_desc}
    return line


# ------------------------------------------------------------------------------------------------ LM head alone
def lmhead_setup(jot, g, B, P, G, dev):
    case = inputs.lm_head_case(0, B, P, G, g.d_model, g.vocab, g.mask_id, device=dev)
    gg = inputs.ModelGeometry(0, g.d_model, 1, 1, 64, 64, g.vocab, g.mask_id)
    weights = {"embed": case.w, "lm_head": case.w,
               "final_norm": torch.ones(g.d_model, dtype=torch.bfloat16, device=dev), "layers": []}
    return case, jot.Model(gg, weights, B, P + G)


def time_oracle_lmhead(case, params, sample_rows=48):
    """CPU oracle on a bounded sample: logits + statistics of `sample_rows` active rows (scaled to all active
    rows) plus the acceptance update of the whole batch."""
    from oracle import jot_oracle as jo
    from oracle import model_oracle as mo
    tok = case.tokens.cpu()
    B, L, P = case.B, case.L, case.P
    rows = [(b, i) for b in range(B) for i in range(P, L) if int(tok[b, i]) == case.mask_id]
    flat = torch.tensor([b * L + i for b, i in rows[:sample_rows]])
    hid, w = case.hidden.cpu(), case.w.cpu()
    bid, bval = case.bump_id.cpu().view(-1), case.bump_val.cpu().view(-1)
    t0 = time.perf_counter()
    logits = mo.lm_head_logits(hid[flat], w, bid[flat], bval[flat])
    st = [jo.row_stats(logits[r].numpy(), case.mask_id) for r in range(len(flat))]
    t1 = time.perf_counter()
    jp = jo.JotParams(*params)
    for b in range(B):
        xs = tok[b].tolist()
        stats = {i: st[(k % len(st))] for k, (bb, i) in enumerate(rows) if bb == b}
        jo.accept_freeze(xs, stats, jp, case.mask_id, P, L, 1)
    t2 = time.perf_counter()
    step_s = (t1 - t0) * len(rows) / len(flat) + (t2 - t1)
    desc = (f"LM-head logits and statistics of {len(flat)} of the {len(rows)} active rows (time scaled by "
            f"{len(rows)}/{len(flat)}) + acceptance of all {B} sequences; float64")
    return step_s, desc, torch.get_num_threads()


def run_lmhead(args, jot, dev, world, rank, peaks, peaks_kind, config, g, nl, B, P, G, T, Lb, params):
    L = P + G
    case, model = lmhead_setup(jot, g, B, P, G, dev)
    jp = jot.Params(*params)
    stats = jot.Stats.empty(B, L, dev)
    n_masked = torch.zeros(B, dtype=torch.int32, device=dev)
    R = int((case.tokens[:, P:] == g.mask_id).sum().item())

    def run_steps(n, tokens):
        for s in range(n):
            tokens.copy_(case.tokens)                     # same mask state every step: R stays fixed
            model.lm_head_stats(case.hidden, tokens, P, L, out=stats, bump_id=case.bump_id, bump_val=case.bump_val)
            jot.accept_freeze(jp, g.mask_id, tokens, P, L, 1, stats, n_masked, step_index=s + 1)

    ms, launches, clocks, prof = timed_region(run_steps, case.tokens.clone, args.steps, args.warmup, world, dev, model,
                                              jot)
    # end to end: hidden states, tokens and bump from pinned host memory; updated tokens and counts back
    h_hidden, h_tokens = case.hidden.cpu().pin_memory(), case.tokens.cpu().pin_memory()
    h_bid, h_bval = case.bump_id.cpu().pin_memory(), case.bump_val.cpu().pin_memory()
    e2e_steps = max(3, min(args.steps, 16))
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for s in range(e2e_steps):
        d_h, d_t = h_hidden.to(dev, non_blocking=True), h_tokens.to(dev, non_blocking=True)
        d_bi, d_bv = h_bid.to(dev, non_blocking=True), h_bval.to(dev, non_blocking=True)
        model.lm_head_stats(d_h, d_t, P, L, out=stats, bump_id=d_bi, bump_val=d_bv)
        jot.accept_freeze(jp, g.mask_id, d_t, P, L, 1, stats, n_masked, step_index=s + 1)
        out_t, out_n = d_t.cpu(), n_masked.cpu()
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / e2e_steps
    ms_max, e2e_ms_max = max_over_ranks([ms, e2e_s * 1e3], world, dev)
    if rank != 0:
        return None
    flops = {"lm_head": 2 * R * g.d_model * g.vocab}
    nbytes = {"rows": 2 * R * g.d_model * 2, "merge": R * 16 * 18, "accept": B * L * 20}
    kernels, roofline = kernel_report(prof, args.steps, flops, nbytes, peaks, peaks_kind, args.workload)
    roofline["active_rows"] = R
    roofline["frac_of_burst"] = round(roofline["achieved"] / peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"]), 4) \
        if roofline.get("bound") == "tensor" else None
    line = base_line(args, world, "lm_head_accept_steps_per_s", "steps/s", aggregate_rate(args.steps, world, ms_max),
                     ms_max / args.steps, config, clocks, launches)
    line["active_rows_per_s"] = round(world * R * args.steps / (ms_max / 1e3), 1)
    line["e2e"] = {"value": round(world / (e2e_ms_max / 1e3), 3), "unit": "steps/s",
                   "h2d_bytes_per_step": int(h_hidden.numel() * 2 + h_tokens.numel() * 4 + h_bid.numel() * 8),
                   "d2h_bytes_per_step": int(out_t.numel() * 4 + out_n.numel() * 4),
                   "call": "jot_lm_head_stats + jot_accept_freeze on pinned host inputs, host tokens out"}
    line["roofline"], line["kernels"] = roofline, kernels
    cpu_step_s, cpu_desc, cpu_threads = time_oracle_lmhead(case, params)
    line["cpu_baseline"] = {"value": round(1.0 / cpu_step_s, 5), "unit": "steps/s", "cores": cpu_threads,
                            "kind": "oracle", "sample": cpu_desc}
    return line


def run_reference(args, config, g, nl, B, P, G, T, Lb, params):
    """The CPU oracle, as it stands, on a bounded sample of the workload (host cores only)."""
    times, desc, threads = [], "", 0
    if args.workload == "lmhead":
        case = inputs.lm_head_case(0, B, P, G, g.d_model, g.vocab, g.mask_id, device="cpu")
        sample = lambda: time_oracle_lmhead(case, params)
        metric = "lm_head_accept_steps_per_s"
    else:
        w = inputs.model_weights(g, seed=0, device="cpu", n_layers=min(2, nl))
        sample = lambda: time_oracle_sample(g, w, nl, B, P, G, Lb, params)
        metric = "denoising_steps_per_s"
    for i in range(args.warmup + args.steps):
        step_s, desc, threads = sample()
        if i >= args.warmup:
            times.append(step_s)
        if sum(times) > 90:          # keep the whole run within a few minutes
            break
    step = statistics.mean(times)
    line = {"impl": "reference", "metric": metric, "value": round(1.0 / step, 5), "unit": "steps/s",
            "n_gpus": args.gpus, "steps": len(times), "warmup": args.warmup, "ms_per_step": round(step * 1e3, 2),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config,
            "cpu_baseline": {"value": round(1.0 / step, 5), "unit": "steps/s", "cores": threads, "kind": "oracle",
                             "sample": desc},
            "e2e": {"value": round(1.0 / step, 5), "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


if __name__ == "__main__":
    sys.exit(main())
