#!/usr/bin/env python
"""Benchmark of the JoT denoising step on B200.

A step is one pass of the whole hot path over one batch: transformer forward over the canvas, LM head
fused with the online softmax statistics over the masked rows of the current block, acceptance /
freeze update.  Default workload: the LLaDA-8B-shaped random-init model, batch 1, prompt 128 + 256
masked tokens, semi-autoregressive blocks of 32 (seeded synthetic weights and tokens).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME] [--no-workloads]

At one GPU the default run also measures, briefly, the other workload shapes (tiny model, fused LM head +
acceptance alone, the same LLaDA-shaped model decoding one block of 256, the Dream-7B shape at batch 8, the
LLaDA shape at batch 16 with a 704-token canvas) and reports them under "workloads"; the headline value stays
the default workload's.

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

NOMINAL_BF16_TFLOPS = 2250.0      # dense bf16 figure of the data sheet, for context beside the measured peaks

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from an ncu capture of this launch shape,
# keyed by (workload, kernel class); an entry is dropped (-> null) whenever its kernel changes afterwards.
NCU_TRAFFIC = {
    ("llada8b", "gemm_gate_up"): 214.1e6,     # 207.1 MB read + 5.9-8.0 MB written (two launches); algorithmic 213.8 MB
    ("llada8b_1block", "gemm_gate_up"): 214.1e6,
    ("lmhead", "lm_head"): 1191.5e6,          # mean of two captured launches; algorithmic 1044.6 MB
}

WORKLOADS = {
    # name: (geometry, B, P, G, T, block_len, (tau_max, tau_min, gamma, D))
    "llada8b": (inputs.LLADA_8B, 1, 128, 256, 256, 32, (30.0, 1.0, 0.5, 8)),
    "tiny": (inputs.TINY, 1, 32, 64, 64, 64, (90.0, 1.0, 0.5, 8)),
    "lmhead": (inputs.LLADA_8B, 8, 128, 256, 1, 256, (30.0, 1.0, 0.5, 8)),
    # the default model decoding its 256 tokens as ONE block (256 active rows in the first step)
    "llada8b_1block": (inputs.LLADA_8B, 1, 128, 256, 256, 256, (30.0, 1.0, 0.5, 8)),
    # the two large-batch shapes: tensor-bound steps (parity-test shapes; here for their per-kernel rates)
    "dream7b": (inputs.DREAM_7B, 8, 256, 256, 256, 256, (90.0, 1.0, 0.5, 8)),
    "llada8b_b16": (inputs.LLADA_8B, 16, 192, 512, 512, 32, (30.0, 1.0, 0.5, 8)),
}
BIG = {"dream7b", "llada8b_b16"}
BUMPED = {"llada8b_b16"}            # workloads defined with the planted logit bump on the LM head


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
def oracle_step(g, w_cpu, n_layers, x, P, Lb, params, bump=None):
    """One denoising step of the CPU oracle as it stands, on canvas x [B, L]: the body over the whole canvas, the LM
    head, the statistics and the acceptance over the first block's rows.  Returns seconds."""
    from oracle import jot_oracle as jo
    from oracle import model_oracle as mo
    B, L = x.shape
    rows = [(b, i) for b in range(B) for i in range(P, P + Lb)]
    jp = jo.JotParams(*params)
    t0 = time.perf_counter()
    h = mo.hidden_states(g, w_cpu, x, True, n_layers)
    sel = torch.stack([h[b, i] for b, i in rows])
    flat = torch.tensor([b * L + i for b, i in rows])
    logits = mo.lm_head_logits(sel, w_cpu["lm_head"], None if bump is None else bump[0].view(-1)[flat],
                               None if bump is None else bump[1].view(-1)[flat])
    for b in range(B):
        xs = x[b].tolist()
        st = {i: jo.row_stats(logits[r].numpy(), g.mask_id) for r, (bb, i) in enumerate(rows) if bb == b}
        jo.accept_freeze(xs, st, jp, g.mask_id, P, P + Lb, 1)
    return time.perf_counter() - t0


def oracle_sample(name, g, w_cpu, nl, B, P, G, Lb, params):
    """What the CPU oracle is timed on for workload `name`, and the factor from that sample to a whole step.
    The single-sequence workloads run one real step at full depth (factor 1).  The batched ones would take minutes per
    step, so they run ONE of the B independent sequences and scale by B.  Returns (seconds of the sample,
    factor, description)."""
    L = P + G
    Bs = 1 if name in BIG else B
    prompt = inputs.prompt(0, Bs, P, g.vocab, g.mask_id)
    x = torch.cat([prompt, torch.full((Bs, G), g.mask_id, dtype=torch.int32)], dim=1)
    bump = inputs.logit_bump(0, Bs, L, g.vocab, g.mask_id, 12.0) if name in BUMPED else None
    sec = oracle_step(g, w_cpu, nl, x, P, Lb, params, bump)
    desc = (f"one real oracle step: all {nl} layers over a {Bs}x{L} canvas, LM head + statistics + acceptance over the "
            f"{Bs * Lb} rows of the first block; float64")
    if Bs != B:
        desc += f"; 1 of the {B} independent sequences, time scaled by {B}"
    return sec, B / Bs, desc


def cpu_weights(g, nl, dev_weights=None):
    """bf16 weights on the host: copied from the device when the GPU arm already drew them, else drawn (on a GPU
    when there is one: the generator is a counter hash, far quicker there) and copied."""
    if dev_weights is not None:
        return inputs.weights_to(dev_weights, "cpu")
    if torch.cuda.is_available():
        return inputs.weights_to(inputs.model_weights(g, seed=0, device="cuda", n_layers=nl), "cpu")
    return inputs.model_weights(g, seed=0, device="cpu", n_layers=nl)


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
    per-kernel durations behind the roofline; the events cost host time, so that pass is not the value).
    The single-step calls only enqueue (jot_set_sync off): the status is read once, after the timed region."""
    model.set_sync(False)
    run_steps(warmup, fresh_state())
    model.read_status()
    state = fresh_state()
    barrier(world)
    launches0 = jot.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(dev) as clocks:
        ev0.record()
        run_steps(steps, state)
        ev1.record()
        barrier(world)
    model.read_status()
    ms = ev0.elapsed_time(ev1)
    launches = jot.launch_count() - launches0
    state = fresh_state()
    torch.cuda.synchronize()
    model.profile(True)
    run_steps(steps, state)
    model.read_status()
    prof = model.profile_read()
    model.profile(False)
    model.set_sync(True)
    return ms, launches, clocks.summary(), prof


def peak_set(peaks, peaks_kind, clocks):
    """The measured denominators and which of the two tensor figures the sampled clock belongs to: the burst figure was
    taken with the SM clock near its maximum, the sustained one under the power cap (about two thirds of it)."""
    burst = peaks.get("bf16_tflops", FALLBACK_PEAKS["bf16_tflops"])
    sustained = peaks.get("bf16_tflops_sustained", FALLBACK_PEAKS["bf16_tflops_sustained"])
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    regime = "burst" if (mhz and mx and mhz >= 0.9 * mx) else "between burst and sustained" if (
        mhz and mx and mhz >= 0.75 * mx) else "sustained" if mhz else "unknown"
    return {"burst": burst, "sustained": sustained, "hbm": peaks.get("hbm_gbs", FALLBACK_PEAKS["hbm_gbs"]),
            "kind": peaks_kind, "clock_regime": regime}


def tensor_fracs(tflops, pk):
    return {"frac_of_burst": round(tflops / pk["burst"], 4), "frac_of_sustained": round(tflops / pk["sustained"], 4),
            "frac_of_nominal_2250": round(tflops / NOMINAL_BF16_TFLOPS, 4)}


def kernel_report(prof, steps, flops_per_launch, bytes_per_launch, pk, workload, clocks):
    """Per kernel class: time per step, share, rate, and its fraction of every denominator; the dominant class as the
    roofline entry.  A tensor-bound class is held against the measured burst peak (the stricter measured figure;
    the sustained and the data-sheet figures are given beside it), an HBM-bound one against the measured copy
    bandwidth."""
    total = sum(v[0] for v in prof.values()) or 1.0
    mhz = clocks.get("sm_mhz")
    rep = {}
    for k, (ms, n) in prof.items():
        if not n:
            continue
        e = {"ms_per_step": round(ms / steps, 4), "share": round(ms / total, 4), "launches_per_step": round(n / steps, 2),
             "avg_launch_us": round(ms / n * 1e3, 2)}
        if mhz:
            e["avg_launch_us_x_ghz"] = round(ms / n * mhz, 2)          # clock-independent measure of the launch
        if k in flops_per_launch:
            e["tflops"] = round(flops_per_launch[k] / (ms / n * 1e-3) / 1e12, 1)
            e.update(tensor_fracs(e["tflops"], pk))
        if k in bytes_per_launch:
            e["gbs"] = round(bytes_per_launch[k] / (ms / n * 1e-3) / 1e9, 1)
            e["frac_of_hbm"] = round(e["gbs"] / pk["hbm"], 4)
        rep[k] = e
    dom = max(prof, key=lambda k: prof[k][0])
    ms, n = prof[dom]
    traffic = NCU_TRAFFIC.get((workload, dom))
    if dom in flops_per_launch:
        ach = flops_per_launch[dom] / (ms / n * 1e-3) / 1e12
        roof = {"kernel": dom, "bound": "tensor", "achieved": round(ach, 2), "peak": pk["burst"], "unit": "TFLOP/s",
                "frac": round(ach / pk["burst"], 4), "traffic": traffic,
                "peak_kind": f"cuBLAS bf16 burst, of {pk['kind']}; sampled clock regime: {pk['clock_regime']}",
                "avg_launch_ms": round(ms / n, 4), "launches": n}
        roof.update(tensor_fracs(ach, pk))
    else:
        b = bytes_per_launch.get(dom)
        ach = b / (ms / n * 1e-3) / 1e9 if b else None
        roof = {"kernel": dom, "bound": "hbm", "achieved": round(ach, 1) if ach else None, "peak": pk["hbm"],
                "unit": "GB/s", "frac": round(ach / pk["hbm"], 4) if ach else None, "traffic": traffic,
                "peak_kind": f"copy bandwidth, of {pk['kind']}", "avg_launch_ms": round(ms / n, 4), "launches": n}
    return rep, roof


def workload_config(name, g, nl, B, P, G, Lb, params, world):
    if name == "lmhead":
        return {"workload": f"lmhead: hidden [{B},{P + G},{g.d_model}] x head [{g.vocab},{g.d_model}], planted bump, prompt {P} "
                            f"resolved + {G} positions masked with p=0.5, then acceptance; JoT ({params[0]:g},{params[1]:g},"
                            f"{params[2]:g},{params[3]})",
                "l2": "inputs exceed L2: the head alone is %.2f GB" % (g.vocab * g.d_model * 2 / 1e9),
                "parallelism": "independent replicas" if world > 1 else "single GPU"}
    return {"workload": f"{name}: {nl} layers d={g.d_model} heads={g.n_q_heads}/{g.n_kv_heads}x{g.head_dim} "
                        f"ff={g.d_ff} vocab={g.vocab}; batch {B} per GPU, prompt {P} + {G} masked, blocks of {Lb}, "
                        f"JoT ({params[0]:g},{params[1]:g},{params[2]:g},{params[3]})"
                        + ("; planted logit bump on the LM head" if name in BUMPED else ""),
            "l2": ("inputs exceed L2: every step streams %.1f GB of weights" % (weight_bytes(g, nl) / 1e9))
                  if weight_bytes(g, nl) > 126e6 else
                  "weights (%.1f MB) stay in L2 and nothing is flushed: a launch-latency-bound shape, reported in "
                  "microseconds per step, not against a roofline" % (weight_bytes(g, nl) / 1e6),
            "parallelism": "independent replicas" if world > 1 else "single GPU"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llada8b", choices=sorted(WORKLOADS))
    ap.add_argument("--layers", type=int, default=None, help="override depth (profiling small cases; not a result)")
    ap.add_argument("--no-workloads", action="store_true", help="skip the brief runs of the other workload shapes")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    g, B, P, G, T, Lb, params = WORKLOADS[args.workload]
    nl = g.n_layers if args.layers is None else args.layers
    config = workload_config(args.workload, g, nl, B, P, G, Lb, params, world)

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
    if args.workload == "lmhead":
        line = run_lmhead(args, jot, dev, world, rank, peaks, peaks_kind, config, g, B, P, G, params, args.steps,
                          args.warmup, full=True)
    else:
        line = run_model(args, jot, dev, world, rank, peaks, peaks_kind, config, args.workload, g, nl, B, P, G, T, Lb,
                         params)
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


def model_flops_bytes(g, B, L, R):
    M = B * L
    flops = {"gemm_qkv": 2 * M * g.d_model * g.qkv_rows, "gemm_o": 2 * M * g.n_q_heads * g.head_dim * g.d_model,
             "gemm_gate_up": 2 * M * g.d_model * 2 * g.d_ff, "gemm_down": 2 * M * g.d_ff * g.d_model,
             "attention": 4 * B * g.n_q_heads * L * L * g.head_dim, "lm_head": 2 * R * g.d_model * g.vocab}
    nbytes = {"lm_head": g.vocab * g.d_model * 2, "rmsnorm": 2 * M * g.d_model * 2, "embed": 2 * M * g.d_model * 2}
    return flops, nbytes


def measure_model(jot, dev, world, peaks, peaks_kind, name, g, nl, weights, B, P, G, Lb, params, steps, warmup):
    """Device-timed steps of one model workload.  Returns (model, dict of everything measured)."""
    L = P + G
    model = jot.Model(g, weights, B, L)
    jp = jot.Params(*params)
    prompt_host = inputs.prompt(0, B, P, g.vocab, g.mask_id).pin_memory()
    canvas0 = torch.cat([prompt_host, torch.full((B, G), g.mask_id, dtype=torch.int32)], dim=1).to(dev)
    stats = jot.Stats.empty(B, L, dev)
    n_masked = torch.zeros(B, dtype=torch.int32, device=dev)
    bump = {}
    if name in BUMPED:
        bid, bval = inputs.logit_bump(0, B, L, g.vocab, g.mask_id, 12.0, device=dev)
        bump = dict(bump_id=bid, bump_val=bval)

    def run_steps(n, tokens):
        """n denoising steps of the block schedule (one token per step by the schedule, early exits on top)."""
        for s in range(n):
            blk = min(s // Lb, G // Lb - 1)
            lo = P + blk * Lb
            model.denoise_step(tokens, lo, lo + Lb, out=stats, **bump)
            jot.accept_freeze(jp, g.mask_id, tokens, lo, lo + Lb, 1, stats, n_masked, step_index=s + 1)

    ms, launches, clocks, prof = timed_region(run_steps, canvas0.clone, steps, warmup, world, dev, model, jot)
    pk = peak_set(peaks, peaks_kind, clocks)
    R = B * Lb
    flops, nbytes = model_flops_bytes(g, B, L, R)
    kernels, roofline = kernel_report(prof, steps, flops, nbytes, pk, name, clocks)
    gemm_ms = sum(prof[k][0] for k in ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down"))
    gemm_fl = sum(flops[k] * prof[k][1] for k in ("gemm_qkv", "gemm_o", "gemm_gate_up", "gemm_down"))
    gemms = {"tflops": round(gemm_fl / (gemm_ms * 1e-3) / 1e12, 1) if gemm_ms else None}
    if gemm_ms:
        gemms.update(tensor_fracs(gemms["tflops"], pk))
        gemms["note"] = "all four projections of every layer together, from the per-launch event timing"
    step_s = ms / 1e3 / steps
    body_flops, head_flops = step_flops(g, nl, B, L, R)
    whole = {"step_tflops": round((body_flops + head_flops) / step_s / 1e12, 1),
             "weight_stream_gbs": round(weight_bytes(g, nl) / step_s / 1e9, 1),
             "hbm_frac": round(weight_bytes(g, nl) / step_s / 1e9 / pk["hbm"], 4), "of": peaks_kind,
             "clock_regime": pk["clock_regime"]}
    whole.update(tensor_fracs(whole["step_tflops"], pk))
    return model, dict(ms=ms, launches=launches, clocks=clocks, kernels=kernels, roofline=roofline, gemms=gemms,
                       whole=whole, prompt_host=prompt_host, jp=jp, bump=bump)


def run_model(args, jot, dev, world, rank, peaks, peaks_kind, config, name, g, nl, B, P, G, T, Lb, params):
    L = P + G
    weights = inputs.model_weights(g, seed=0, device=dev, n_layers=nl)
    model, m = measure_model(jot, dev, world, peaks, peaks_kind, name, g, nl, weights, B, P, G, Lb, params, args.steps,
                             args.warmup)
    prompt_host, jp = m["prompt_host"], m["jp"]

    # end to end through the public call: pinned host prompt -> jot_generate -> host tokens.  The large-batch
    # shapes would take minutes for a whole generation: they run the first `steps` iterations' worth instead
    # (generation length cut to steps tokens' blocks on the same prompt), flagged in the output.
    e2e_T, e2e_G = T, G
    if name in BIG:
        e2e_G = max(Lb, min(G, (args.steps // Lb) * Lb)) if Lb < G else G
        e2e_T = min(T, max(args.steps, 1)) if Lb >= G else e2e_G
    e2e_bump = {k: v[:, :P + e2e_G].contiguous() for k, v in m["bump"].items()}
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    d_prompt = prompt_host.to(dev, non_blocking=True)
    out, used, passes = model.generate(d_prompt, e2e_G, e2e_T, jp, min(Lb, e2e_G), **e2e_bump)
    host_out = out.cpu()
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    graph_ms = None
    if name == "tiny":
        # launch-latency-bound shape: the same generation with the step replayed as a CUDA graph
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        model.generate(prompt_host.to(dev, non_blocking=True), e2e_G, e2e_T, jp, min(Lb, e2e_G), use_cuda_graph=True)[0].cpu()
        torch.cuda.synchronize()
        graph_ms = (time.perf_counter() - t0) * 1e3
    ms_max, e2e_ms_max = max_over_ranks([m["ms"], e2e_s * 1e3], world, dev)
    if rank != 0:
        return None
    line = base_line(args, world, "denoising_steps_per_s", "steps/s", aggregate_rate(args.steps, world, ms_max),
                     ms_max / args.steps, config, m["clocks"], m["launches"])
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
        line["e2e"]["kernels_per_step"] = round(m["launches"] / args.steps, 1)
    line["roofline"], line["step_roofline"], line["kernels"], line["gemms"] = m["roofline"], m["whole"], m["kernels"], m["gemms"]
    line["launches_per_step"] = round(m["launches"] / args.steps, 1)

    # the CPU oracle beside it: one real step at full depth on the host cores
    w_cpu = cpu_weights(g, nl, weights)
    sec, factor, desc = oracle_sample(name, g, w_cpu, nl, B, P, G, Lb, params)
    del w_cpu
    line["cpu_baseline"] = {"value": round(1.0 / (sec * factor), 5), "unit": "steps/s", "cores": torch.get_num_threads(),
                            "kind": "oracle", "sample": desc, "sample_seconds": round(sec, 2)}

    if world == 1 and name == "llada8b" and args.layers is None and not args.no_workloads:
        line["workloads"] = other_workloads(args, jot, dev, peaks, peaks_kind, model, weights)
    model.close()
    return line


def other_workloads(args, jot, dev, peaks, peaks_kind, model, weights):
    """Brief device-timed runs of the other workload shapes (one GPU): ms per step, the dominant kernel's roofline
    entry, every class's rate and fractions, the sampled clock.  The default workload's weights serve the two
    other LLaDA-shaped runs."""
    out = {}
    model.close()

    def brief(name, w, steps, warmup):
        g, B, P, G, T, Lb, params = WORKLOADS[name]
        nl = len(w["layers"])
        mdl, m = measure_model(jot, dev, 1, peaks, peaks_kind, name, g, nl, w, B, P, G, Lb, params, steps, warmup)
        e = {"config": workload_config(name, g, nl, B, P, G, Lb, params, 1)["workload"], "steps": steps, "warmup": warmup,
             "ms_per_step": round(m["ms"] / steps, 4), "steps_per_s": round(steps / (m["ms"] / 1e3), 3),
             "launches_per_step": round(m["launches"] / steps, 1), "clocks": m["clocks"], "roofline": m["roofline"],
             "step_roofline": m["whole"], "gemms": m["gemms"], "kernels": m["kernels"]}
        return mdl, m, e

    mdl, m, out["llada8b_1block"] = brief("llada8b_1block", weights, 16, 3)
    mdl.close()
    out["llada8b_kv_cache"] = kv_cache_generation(jot, dev, weights)
    mdl, m, out["llada8b_b16"] = brief("llada8b_b16", weights, 6, 3)
    mdl.close()
    del mdl, m, weights
    torch.cuda.empty_cache()
    gd = WORKLOADS["dream7b"][0]
    wd = inputs.model_weights(gd, seed=0, device=dev, n_layers=gd.n_layers)
    mdl, m, out["dream7b"] = brief("dream7b", wd, 8, 3)
    mdl.close()
    del mdl, m, wd
    torch.cuda.empty_cache()
    gt = WORKLOADS["tiny"][0]
    wt = inputs.model_weights(gt, seed=0, device=dev, n_layers=gt.n_layers)
    mdl, m, e = brief("tiny", wt, 64, 4)
    # launch-latency-bound: the whole generation through jot_generate, plain launches and CUDA-graph replay
    _, B, P, G, T, Lb, params = WORKLOADS["tiny"]
    for key, kw in (("us_per_step_generate", {}), ("us_per_step_generate_cuda_graph", {"use_cuda_graph": True})):
        mdl.generate(m["prompt_host"].to(dev), G, T, m["jp"], Lb, **kw)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        _, used, passes = mdl.generate(m["prompt_host"].to(dev), G, T, m["jp"], Lb, **kw)
        torch.cuda.synchronize()
        e[key] = round((time.perf_counter() - t0) * 1e6 / max(passes, 1), 1)
    e["note"] = "launch-latency-bound: microseconds per step and launches per step are the figures; no roofline fraction applies"
    out["tiny"] = e
    mdl.close()
    g8, B, P, G, T, Lb, params = WORKLOADS["lmhead"]
    cfg = workload_config("lmhead", g8, 0, B, P, G, Lb, params, 1)
    e = run_lmhead(args, jot, dev, 1, 0, peaks, peaks_kind, cfg, g8, B, P, G, params, 20, 3, full=False)
    out["lmhead"] = e
    return out


def kv_cache_generation(jot, dev, weights):
    """The default workload's generation (256 tokens in blocks of 32) decoded under the block-wise KV cache: the first
    step of a block runs the whole canvas, the others only the block's 32 rows against cached keys and values.
    Whole-call wall time from a pinned host prompt to host tokens, beside the same call without the cache."""
    g, B, P, G, T, Lb, params = WORKLOADS["llada8b"]
    model = jot.Model(g, weights, B, P + G)
    cache_bytes = model.attach_kv_cache()
    jp = jot.Params(*params)
    prompt_host = inputs.prompt(0, B, P, g.vocab, g.mask_id).pin_memory()
    res = {}
    for key, kw in (("plain", {}), ("kv_cache", {"kv_cache": True})):
        model.generate(prompt_host.to(dev), Lb, Lb, jp, Lb, **kw)                      # warm-up: one block
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        out, used, passes = model.generate(prompt_host.to(dev, non_blocking=True), G, T, jp, Lb, **kw)
        out.cpu()
        torch.cuda.synchronize()
        sec = time.perf_counter() - t0
        res[key] = {"seconds": round(sec, 4), "forward_passes": passes, "steps_used": used,
                    "ms_per_forward_pass": round(sec * 1e3 / max(passes, 1), 3),
                    "generated_tokens_per_s": round(B * G / sec, 1)}
    model.close()
    res["config"] = (f"llada8b weights, batch {B}, prompt {P} + {G} tokens in blocks of {Lb}: per block one full pass over the "
                     f"{P + G}-row canvas, then passes over the block's {Lb} rows; cache {cache_bytes / 1e6:.0f} MB (caller-owned)")
    res["note"] = ("random-init weights: early exits depend on the planted confidence, so the step counts of the two modes "
                   "are what they are; the per-pass time is the comparable figure")
    return res


# ------------------------------------------------------------------------------------------------ LM head alone
def lmhead_setup(jot, g, B, P, G, dev):
    case = inputs.lm_head_case(0, B, P, G, g.d_model, g.vocab, g.mask_id, device=dev)
    gg = inputs.ModelGeometry(0, g.d_model, 1, 1, 64, 64, g.vocab, g.mask_id)
    weights = {"embed": case.w, "lm_head": case.w,
               "final_norm": torch.ones(g.d_model, dtype=torch.bfloat16, device=dev), "layers": []}
    return case, jot.Model(gg, weights, B, P + G)


def time_oracle_lmhead(case, params):
    """The CPU oracle on the whole LM-head workload: logits and statistics of every active row, then the acceptance
    update of every sequence.  Returns (seconds, description)."""
    from oracle import jot_oracle as jo
    from oracle import model_oracle as mo
    tok = case.tokens.cpu()
    B, L, P = case.B, case.L, case.P
    rows = [(b, i) for b in range(B) for i in range(P, L) if int(tok[b, i]) == case.mask_id]
    flat = torch.tensor([b * L + i for b, i in rows])
    hid, w = case.hidden.cpu(), case.w.cpu()
    bid, bval = case.bump_id.cpu().view(-1), case.bump_val.cpu().view(-1)
    jp = jo.JotParams(*params)
    t0 = time.perf_counter()
    st = {}
    for c in range(0, len(rows), 128):                     # 128 rows of float64 logits at a time (130 MB)
        sel = flat[c:c + 128]
        logits = mo.lm_head_logits(hid[sel], w, bid[sel], bval[sel])
        for r in range(len(sel)):
            st[rows[c + r]] = jo.row_stats(logits[r].numpy(), case.mask_id)
    for b in range(B):
        xs = tok[b].tolist()
        jo.accept_freeze(xs, {i: s for (bb, i), s in st.items() if bb == b}, jp, case.mask_id, P, L, 1)
    sec = time.perf_counter() - t0
    return sec, (f"one real oracle step: LM-head logits and statistics of all {len(rows)} active rows + acceptance of all "
                 f"{B} sequences; float64")


def run_lmhead(args, jot, dev, world, rank, peaks, peaks_kind, config, g, B, P, G, params, steps, warmup, full):
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

    ms, launches, clocks, prof = timed_region(run_steps, case.tokens.clone, steps, warmup, world, dev, model, jot)
    pk = peak_set(peaks, peaks_kind, clocks)
    flops = {"lm_head": 2 * R * g.d_model * g.vocab}
    nbytes = {"rows": 2 * R * g.d_model * 2, "merge": R * 16 * 18, "accept": B * L * 20}
    kernels, roofline = kernel_report(prof, steps, flops, nbytes, pk, "lmhead", clocks)
    roofline["active_rows"] = R
    # the whole fused path (row list, head, merge, acceptance) against the head's own roofline
    path_tflops = flops["lm_head"] / (ms / 1e3 / steps) / 1e12
    path = {"tflops": round(path_tflops, 1), "note": "LM-head flops over the time of the WHOLE step (row gather, head, merge, "
            "acceptance, and the canvas reset of the benchmark loop)"}
    path.update(tensor_fracs(path_tflops, pk))
    if not full:
        model.close()
        return {"config": config["workload"], "steps": steps, "warmup": warmup, "ms_per_step": round(ms / steps, 4),
                "steps_per_s": round(steps / (ms / 1e3), 3), "launches_per_step": round(launches / steps, 1),
                "clocks": clocks, "roofline": roofline, "fused_path": path, "kernels": kernels}
    # end to end: hidden states, tokens and bump from pinned host memory; updated tokens and counts back
    h_hidden, h_tokens = case.hidden.cpu().pin_memory(), case.tokens.cpu().pin_memory()
    h_bid, h_bval = case.bump_id.cpu().pin_memory(), case.bump_val.cpu().pin_memory()
    e2e_steps = max(3, min(steps, 16))
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
    line = base_line(args, world, "lm_head_accept_steps_per_s", "steps/s", aggregate_rate(steps, world, ms_max),
                     ms_max / steps, config, clocks, launches)
    line["active_rows_per_s"] = round(world * R * steps / (ms_max / 1e3), 1)
    line["e2e"] = {"value": round(world / (e2e_ms_max / 1e3), 3), "unit": "steps/s",
                   "h2d_bytes_per_step": int(h_hidden.numel() * 2 + h_tokens.numel() * 4 + h_bid.numel() * 8),
                   "d2h_bytes_per_step": int(out_t.numel() * 4 + out_n.numel() * 4),
                   "call": "jot_lm_head_stats + jot_accept_freeze on pinned host inputs, host tokens out"}
    line["roofline"], line["kernels"], line["fused_path"] = roofline, kernels, path
    sec, desc = time_oracle_lmhead(case, params)
    line["cpu_baseline"] = {"value": round(1.0 / sec, 5), "unit": "steps/s", "cores": torch.get_num_threads(),
                            "kind": "oracle", "sample": desc, "sample_seconds": round(sec, 2)}
    model.close()
    return line


def run_reference(args, config, g, nl, B, P, G, T, Lb, params):
    """The CPU oracle, as it stands, on the host cores.  A timed "step" is one real oracle step of the workload (for
    the batched shapes: of one of their independent sequences); ms_per_step is its measured wall time.  The run is
    held to about two minutes: fewer steps than asked for are timed when a step takes long, and `steps` says how
    many were."""
    budget_s = 110.0
    name = args.workload
    if name == "lmhead":
        case = inputs.lm_head_case(0, B, P, G, g.d_model, g.vocab, g.mask_id,
                                   device="cuda" if torch.cuda.is_available() else "cpu")
        sample = lambda: time_oracle_lmhead(case, params) + (1.0,)
        metric = "lm_head_accept_steps_per_s"
        order = lambda r: (r[0], r[2], r[1])
    else:
        w = cpu_weights(g, nl)
        sample = lambda: oracle_sample(name, g, w, nl, B, P, G, Lb, params)
        metric = "denoising_steps_per_s"
        order = lambda r: r
    times, desc, factor, spent = [], "", 1.0, 0.0
    warm = 0
    for i in range(args.warmup + args.steps):
        sec, factor, desc = order(sample())
        spent += sec
        if i < args.warmup and spent + sec * 2 < budget_s * 0.4:
            warm += 1
            continue
        times.append(sec)
        if spent + sec > budget_s:
            break
    step = statistics.mean(times)
    line = {"impl": "reference", "metric": metric, "value": round(1.0 / (step * factor), 5), "unit": "steps/s",
            "n_gpus": args.gpus, "steps": len(times), "warmup": warm, "ms_per_step": round(step * 1e3, 2),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config,
            "cpu_baseline": {"value": round(1.0 / (step * factor), 5), "unit": "steps/s", "cores": torch.get_num_threads(),
                             "kind": "oracle", "sample": desc, "sample_seconds": round(step, 2)},
            "e2e": {"value": round(1.0 / (step * factor), 5), "unit": "steps/s", "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


if __name__ == "__main__":
    sys.exit(main())
