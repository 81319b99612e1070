"""ctypes binding of libjot.so: argument marshalling only.

Every step of the JoT denoising path runs inside the CUDA library; this module turns torch tensors
into raw device pointers, checks dtypes/shapes, and raises on any non-zero status.  There is no
fallback: if the library is missing or fails to load, importing the binding's functions raises.
"""
from __future__ import annotations

import ctypes as C
import dataclasses
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libjot.so")

EXPORTS = [
    "jot_status_string", "jot_last_cuda_error", "jot_workspace_bytes", "jot_init_model", "jot_free_model",
    "jot_denoise_step", "jot_lm_head_stats", "jot_accept_freeze", "jot_generate", "jot_gemm_bf16",
    "jot_launch_count", "jot_profile", "jot_profile_read", "jot_gemm_bf16_noalloc",
    "jot_selftest_wait_expiry", "jot_kv_cache_bytes", "jot_attach_kv_cache", "jot_denoise_step_cached",
    "jot_max_active_rows", "jot_lm_head_partition", "jot_set_sync", "jot_read_status",
    "jot_lm_head_stats_slice", "jot_merge_stats",
]

NOALLOC_SCRATCH_BYTES = 16 << 20

PROF_CLASSES = ["embed", "rmsnorm", "gemm_qkv", "rope", "attention", "gemm_o", "gemm_gate_up", "gemm_down", "rows",
                "lm_head", "merge", "accept"]


class JotError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib().jot_status_string(status).decode()
        cuda = _lib().jot_last_cuda_error()
        super().__init__(f"{where}: {msg} (status {status}, cuda error {cuda})")


GATE_RATIO, GATE_MAXPROB, GATE_GLOBAL_GAP = 0, 1, 2
SCHEDULE_FIXED, SCHEDULE_FRACTIONAL = 0, 1


class Params(C.Structure):
    """tau_max, tau_min, gamma, D of Algorithm 1; eps of Eq. 4."""
    _fields_ = [("tau_max", C.c_float), ("tau_min", C.c_float), ("gamma", C.c_float), ("D", C.c_int32),
                ("eps", C.c_float), ("schedule_after_exit", C.c_int32), ("gate", C.c_int32),
                ("prob_threshold", C.c_float), ("gap_threshold", C.c_float), ("schedule", C.c_int32)]

    def __init__(self, tau_max=90.0, tau_min=1.0, gamma=0.5, D=8, eps=1e-12, schedule_after_exit=0, gate=0,
                 prob_threshold=0.9, gap_threshold=5.0, schedule=0):
        super().__init__(tau_max, tau_min, gamma, D, eps, schedule_after_exit, gate, prob_threshold, gap_threshold,
                         schedule)


class ModelConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ff", C.c_int32), ("vocab", C.c_int32), ("mask_id", C.c_int32),
                ("rope_theta", C.c_float), ("rms_eps", C.c_float)]


class _Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("attn_norm", C.POINTER(C.c_void_p)), ("wqkv", C.POINTER(C.c_void_p)), ("wo", C.POINTER(C.c_void_p)),
                ("mlp_norm", C.POINTER(C.c_void_p)), ("w_gate_up", C.POINTER(C.c_void_p)),
                ("w_down", C.POINTER(C.c_void_p))]


class Sampling(C.Structure):
    """Sampling-based finalisation: temperature > 0 draws each active row's token from softmax(l / T)."""
    _fields_ = [("temperature", C.c_float), ("seed", C.c_uint64), ("step", C.c_int32)]


class GenConfig(C.Structure):
    _fields_ = [("gen_len", C.c_int32), ("steps", C.c_int32), ("block_len", C.c_int32),
                ("exclude_mask_token", C.c_int32), ("compact_finished", C.c_int32), ("use_cuda_graph", C.c_int32),
                ("temperature", C.c_float), ("seed_lo", C.c_uint32), ("seed_hi", C.c_uint32), ("kv_cache", C.c_int32)]


class _Trace(C.Structure):
    _fields_ = [("exit_step", C.c_void_p), ("exit_reason", C.c_void_p), ("mean_ratio", C.c_void_p),
                ("n_candidates", C.c_void_p)]


@dataclasses.dataclass
class Trace:
    """Optional per-position / per-step record of a generation (device tensors)."""
    exit_step: torch.Tensor        # [B, L] int16: 1-based step of the sequence that finalised the position
    exit_reason: torch.Tensor      # [B, L] uint8: bit 0 early exit, bit 1 transfer schedule
    mean_ratio: torch.Tensor       # [steps, B] float32: mean confidence ratio over the step's candidates
    n_candidates: torch.Tensor     # [steps, B] int32


_LIB = None


def _lib():
    global _LIB
    if _LIB is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_11133_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        lib = C.CDLL(LIB_PATH)
        lib.jot_status_string.restype = C.c_char_p
        lib.jot_status_string.argtypes = [C.c_int]
        lib.jot_last_cuda_error.restype = C.c_int
        lib.jot_workspace_bytes.restype = C.c_size_t
        lib.jot_workspace_bytes.argtypes = [C.POINTER(ModelConfig), C.c_int, C.c_int]
        lib.jot_init_model.argtypes = [C.POINTER(ModelConfig), C.POINTER(_Weights), C.c_int, C.c_int, C.c_void_p,
                                       C.c_size_t, C.POINTER(C.c_void_p)]
        lib.jot_free_model.argtypes = [C.c_void_p]
        step_args = [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                     C.c_void_p, C.c_void_p, C.POINTER(Sampling), C.c_void_p, C.c_void_p]
        lib.jot_denoise_step.argtypes = [C.c_void_p, C.c_void_p] + step_args
        lib.jot_lm_head_stats.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p] + step_args
        lib.jot_lm_head_stats_slice.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                                C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                                C.c_void_p, C.POINTER(Sampling), C.c_void_p, C.c_void_p]
        lib.jot_merge_stats.argtypes = [C.c_int] + [C.c_void_p] * 13
        lib.jot_kv_cache_bytes.restype = C.c_size_t
        lib.jot_kv_cache_bytes.argtypes = [C.POINTER(ModelConfig), C.c_int, C.c_int]
        lib.jot_attach_kv_cache.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t]
        lib.jot_denoise_step_cached.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                                C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                                C.c_void_p, C.POINTER(Sampling), C.c_void_p, C.c_void_p]
        lib.jot_accept_freeze.argtypes = [C.POINTER(Params), C.c_int, C.c_int32, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                          C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
        lib.jot_generate.argtypes = [C.c_void_p, C.POINTER(Params), C.c_int, C.POINTER(GenConfig), C.c_void_p, C.c_int,
                                     C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_int32),
                                     C.POINTER(C.c_int32), C.POINTER(_Trace), C.c_void_p]
        lib.jot_gemm_bf16.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                      C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        lib.jot_gemm_bf16_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                              C.c_void_p, C.c_void_p]
        lib.jot_launch_count.restype = C.c_int64
        lib.jot_selftest_wait_expiry.argtypes = [C.c_void_p, C.c_uint64, C.c_void_p]
        lib.jot_max_active_rows.argtypes = [C.c_int]
        lib.jot_lm_head_partition.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]
        lib.jot_set_sync.argtypes = [C.c_void_p, C.c_int]
        lib.jot_read_status.argtypes = [C.c_void_p, C.c_void_p]
        lib.jot_profile.argtypes = [C.c_void_p, C.c_int]
        lib.jot_profile_read.argtypes = [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int64), C.c_int]
        _LIB = lib
    return _LIB


def _check(status: int, where: str):
    if status != 0:
        raise JotError(status, where)


def _ptr(t: Optional[torch.Tensor], dtype, name: str) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of {dtype}, got {t.dtype} on {t.device}")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _sampling_args(sampling, out, B, L, device):
    """(pointer to the descriptor or None, device pointer of the sampled-token array or None)."""
    if sampling is None or not sampling.temperature > 0:
        return None, None
    if out.sampled is None:
        out.sampled = torch.zeros(B, L, dtype=torch.int32, device=device)
    return C.byref(sampling), _ptr(out.sampled, torch.int32, "sampled")


def max_active_rows(n_sms: int) -> int:
    return int(_lib().jot_max_active_rows(n_sms))


def lm_head_partition(active_rows: int, n_ctas: int, vocab_tiles: int, pair_mode: bool):
    """(row blocks, vocabulary chunks per row block) of the LM-head schedule; host arithmetic only."""
    n_rb, n_ch = C.c_int(0), C.c_int(0)
    _check(_lib().jot_lm_head_partition(active_rows, n_ctas, vocab_tiles, int(pair_mode), C.byref(n_rb), C.byref(n_ch)),
           "jot_lm_head_partition")
    return n_rb.value, n_ch.value


def launch_count() -> int:
    return int(_lib().jot_launch_count())


@dataclasses.dataclass
class Stats:
    """Per-position softmax statistics, each [B, L]; only active rows are written."""
    top1: torch.Tensor
    top2: torch.Tensor
    sumexp: torch.Tensor
    argmax: torch.Tensor
    sampled: Optional[torch.Tensor] = None      # [B, L] int32, written when sampling is on

    @staticmethod
    def empty(B: int, L: int, device) -> "Stats":
        return Stats(torch.zeros(B, L, dtype=torch.float32, device=device),
                     torch.zeros(B, L, dtype=torch.float32, device=device),
                     torch.ones(B, L, dtype=torch.float32, device=device),
                     torch.zeros(B, L, dtype=torch.int32, device=device))


class Model:
    """Owner of the device workspace and the library's model handle.  Weights are borrowed."""

    def __init__(self, geometry, weights: dict, max_batch: int, max_seq: int):
        g = geometry
        self.geometry = g
        self.cfg = ModelConfig(len(weights["layers"]), g.d_model, g.n_q_heads, g.n_kv_heads, g.head_dim, g.d_ff,
                               g.vocab, g.mask_id, g.rope_theta, g.rms_eps)
        self.weights = weights           # keep the tensors alive
        self.max_batch, self.max_seq = max_batch, max_seq
        lib = _lib()
        nbytes = lib.jot_workspace_bytes(C.byref(self.cfg), max_batch, max_seq)
        if nbytes == 0:
            raise JotError(-2, "jot_workspace_bytes")
        dev = weights["lm_head"].device
        self.workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device=dev)
        base = (self.workspace.data_ptr() + 1023) // 1024 * 1024
        nl = self.cfg.n_layers
        arr = lambda key: (C.c_void_p * max(nl, 1))(*[_ptr(lw[key], torch.bfloat16, key) for lw in weights["layers"]])
        self._arrays = [arr(k) for k in ("attn_norm", "wqkv", "wo", "mlp_norm", "w_gate_up", "w_down")]
        w = _Weights(_ptr(weights["embed"], torch.bfloat16, "embed"), _ptr(weights["lm_head"], torch.bfloat16, "lm_head"),
                     _ptr(weights["final_norm"], torch.bfloat16, "final_norm"),
                     *[C.cast(a, C.POINTER(C.c_void_p)) for a in self._arrays])
        handle = C.c_void_p()
        _check(lib.jot_init_model(C.byref(self.cfg), C.byref(w), max_batch, max_seq, base, nbytes, C.byref(handle)),
               "jot_init_model")
        self.handle = handle
        self.kv_cache = None

    def close(self):
        if getattr(self, "handle", None):
            _lib().jot_free_model(self.handle)
            self.handle = None
        self.kv_cache = None

    # ---- block-wise KV cache -----------------------------------------------------------------------
    def attach_kv_cache(self) -> int:
        """Allocate the cache for (max_batch, max_seq) and hand it to the library; returns its size in bytes."""
        nbytes = _lib().jot_kv_cache_bytes(C.byref(self.cfg), self.max_batch, self.max_seq)
        if nbytes == 0:
            raise JotError(-2, "jot_kv_cache_bytes")
        self.kv_cache = torch.empty(nbytes + 1024, dtype=torch.uint8, device=self.workspace.device)
        base = (self.kv_cache.data_ptr() + 1023) // 1024 * 1024
        _check(_lib().jot_attach_kv_cache(self.handle, base, nbytes), "jot_attach_kv_cache")
        return int(nbytes)

    def detach_kv_cache(self) -> None:
        _check(_lib().jot_attach_kv_cache(self.handle, None, 0), "jot_attach_kv_cache")
        self.kv_cache = None

    def denoise_step_cached(self, tokens: torch.Tensor, blk_lo: int, blk_hi: int, refresh: bool,
                            out: Optional["Stats"] = None, exclude_mask_token: bool = True,
                            bump_id: Optional[torch.Tensor] = None, bump_val: Optional[torch.Tensor] = None,
                            sampling: Optional[Sampling] = None) -> "Stats":
        B, L = tokens.shape
        out = out or Stats.empty(B, L, tokens.device)
        sp, d_sampled = _sampling_args(sampling, out, B, L, tokens.device)
        _check(_lib().jot_denoise_step_cached(self.handle, _ptr(tokens, torch.int32, "tokens"), B, L, blk_lo, blk_hi,
                                              int(refresh), int(exclude_mask_token), _ptr(bump_id, torch.int32, "bump_id"),
                                              _ptr(bump_val, torch.float32, "bump_val"), out.top1.data_ptr(),
                                              out.top2.data_ptr(), out.sumexp.data_ptr(), out.argmax.data_ptr(), sp,
                                              d_sampled, _stream()),
               "jot_denoise_step_cached")
        return out

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_sync(self, sync: bool) -> None:
        """sync=False: the single-step calls return once their kernels are enqueued; read_status() asks later."""
        _check(_lib().jot_set_sync(self.handle, int(sync)), "jot_set_sync")

    def read_status(self) -> None:
        """Synchronise the current stream and raise if a kernel reported a failure since the last read."""
        _check(_lib().jot_read_status(self.handle, _stream()), "jot_read_status")

    def profile(self, enable: bool) -> None:
        """Start (and clear) or stop per-kernel-class event timing."""
        _check(_lib().jot_profile(self.handle, int(enable)), "jot_profile")

    def profile_read(self) -> dict:
        """{class: (milliseconds, spans)} accumulated since profile(True)."""
        n = len(PROF_CLASSES)
        ms, cnt = (C.c_double * n)(), (C.c_int64 * n)()
        _check(_lib().jot_profile_read(self.handle, ms, cnt, n), "jot_profile_read")
        return {name: (ms[i], int(cnt[i])) for i, name in enumerate(PROF_CLASSES)}

    # ---- one step -------------------------------------------------------------------------------
    def denoise_step(self, tokens: torch.Tensor, blk_lo: int, blk_hi: int, out: Optional[Stats] = None,
                     exclude_mask_token: bool = True, bump_id: Optional[torch.Tensor] = None,
                     bump_val: Optional[torch.Tensor] = None, sampling: Optional[Sampling] = None) -> Stats:
        B, L = tokens.shape
        out = out or Stats.empty(B, L, tokens.device)
        sp, d_sampled = _sampling_args(sampling, out, B, L, tokens.device)
        _check(_lib().jot_denoise_step(self.handle, _ptr(tokens, torch.int32, "tokens"), B, L, blk_lo, blk_hi,
                                       int(exclude_mask_token), _ptr(bump_id, torch.int32, "bump_id"),
                                       _ptr(bump_val, torch.float32, "bump_val"), out.top1.data_ptr(),
                                       out.top2.data_ptr(), out.sumexp.data_ptr(), out.argmax.data_ptr(), sp,
                                       d_sampled, _stream()),
               "jot_denoise_step")
        return out

    def lm_head_stats(self, hidden: torch.Tensor, tokens: torch.Tensor, blk_lo: int, blk_hi: int,
                      out: Optional[Stats] = None, exclude_mask_token: bool = True,
                      bump_id: Optional[torch.Tensor] = None, bump_val: Optional[torch.Tensor] = None,
                      sampling: Optional[Sampling] = None) -> Stats:
        B, L = tokens.shape
        if hidden.shape != (B * L, self.cfg.d_model):
            raise ValueError("hidden must be [B*L, d_model]")
        out = out or Stats.empty(B, L, tokens.device)
        sp, d_sampled = _sampling_args(sampling, out, B, L, tokens.device)
        _check(_lib().jot_lm_head_stats(self.handle, _ptr(hidden, torch.bfloat16, "hidden"),
                                        _ptr(tokens, torch.int32, "tokens"), B, L, blk_lo, blk_hi,
                                        int(exclude_mask_token), _ptr(bump_id, torch.int32, "bump_id"),
                                        _ptr(bump_val, torch.float32, "bump_val"), out.top1.data_ptr(),
                                        out.top2.data_ptr(), out.sumexp.data_ptr(), out.argmax.data_ptr(), sp,
                                        d_sampled, _stream()),
               "jot_lm_head_stats")
        return out

    def lm_head_stats_slice(self, hidden: torch.Tensor, tokens: torch.Tensor, blk_lo: int, blk_hi: int, v_lo: int,
                            v_hi: int, out: Optional[Stats] = None, exclude_mask_token: bool = True,
                            bump_id: Optional[torch.Tensor] = None, bump_val: Optional[torch.Tensor] = None) -> Stats:
        """Statistics of the active rows over the vocabulary slice [v_lo, v_hi) only (one rank's share of a
        vocabulary-parallel head)."""
        B, L = tokens.shape
        if hidden.shape != (B * L, self.cfg.d_model):
            raise ValueError("hidden must be [B*L, d_model]")
        out = out or Stats.empty(B, L, tokens.device)
        _check(_lib().jot_lm_head_stats_slice(self.handle, _ptr(hidden, torch.bfloat16, "hidden"),
                                              _ptr(tokens, torch.int32, "tokens"), B, L, blk_lo, blk_hi,
                                              int(exclude_mask_token), _ptr(bump_id, torch.int32, "bump_id"),
                                              _ptr(bump_val, torch.float32, "bump_val"), v_lo, v_hi, out.top1.data_ptr(),
                                              out.top2.data_ptr(), out.sumexp.data_ptr(), out.argmax.data_ptr(), None,
                                              None, _stream()),
               "jot_lm_head_stats_slice")
        return out

    # ---- Algorithm 1 ----------------------------------------------------------------------------
    def generate(self, prompt: torch.Tensor, gen_len: int, steps: int, params, block_len: Optional[int] = None,
                 exclude_mask_token: bool = True, bump_id: Optional[torch.Tensor] = None,
                 bump_val: Optional[torch.Tensor] = None, compact_finished: bool = True, use_cuda_graph: bool = False,
                 temperature: float = 0.0, seed: int = 0, trace: bool = False, kv_cache: bool = False):
        """Returns (tokens [B, P+gen_len] int32 on device, steps_used list[int], forward_passes int), and a
        Trace as a fourth element when trace is set."""
        B, P = prompt.shape
        per_seq = isinstance(params, (list, tuple))
        if per_seq:
            if len(params) != B:
                raise ValueError("need one Params per sequence")
            parr = (Params * B)(*params)
        else:
            parr = (Params * 1)(params)
        gen = GenConfig(gen_len, steps, block_len or gen_len, int(exclude_mask_token), int(compact_finished),
                        int(use_cuda_graph), float(temperature), seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF,
                        int(kv_cache))
        out = torch.empty(B, P + gen_len, dtype=torch.int32, device=prompt.device)
        used = (C.c_int32 * B)()
        passes = C.c_int32(0)
        tr, tr_arg = None, None
        if trace:
            dev = prompt.device
            tr = Trace(torch.empty(B, P + gen_len, dtype=torch.int16, device=dev),
                       torch.empty(B, P + gen_len, dtype=torch.uint8, device=dev),
                       torch.empty(steps, B, dtype=torch.float32, device=dev),
                       torch.empty(steps, B, dtype=torch.int32, device=dev))
            tr_arg = C.byref(_Trace(tr.exit_step.data_ptr(), tr.exit_reason.data_ptr(), tr.mean_ratio.data_ptr(),
                                    tr.n_candidates.data_ptr()))
        _check(_lib().jot_generate(self.handle, parr, int(per_seq), C.byref(gen), _ptr(prompt, torch.int32, "prompt"), B,
                                   P, _ptr(bump_id, torch.int32, "bump_id"), _ptr(bump_val, torch.float32, "bump_val"),
                                   out.data_ptr(), used, C.byref(passes), tr_arg, _stream()), "jot_generate")
        if trace:
            return out, list(used), int(passes.value), tr
        return out, list(used), int(passes.value)


def accept_freeze(params, mask_id: int, tokens: torch.Tensor, blk_lo: int, blk_hi: int, k_transfer: int,
                  stats: Stats, n_masked: Optional[torch.Tensor] = None, exit_reason: Optional[torch.Tensor] = None,
                  exit_step: Optional[torch.Tensor] = None, step_index: int = 0) -> None:
    """In-place acceptance / freeze update of tokens [B, L] (Section 4.1, Algorithm 1).
    params: one Params for the whole batch, or a list of B (one per sequence)."""
    B, L = tokens.shape
    per_seq = isinstance(params, (list, tuple))
    if per_seq:
        if len(params) != B:
            raise ValueError("need one Params per sequence")
        parr = (Params * B)(*params)
    else:
        parr = (Params * 1)(params)
    _check(_lib().jot_accept_freeze(parr, int(per_seq), mask_id, _ptr(tokens, torch.int32, "tokens"), B, L, blk_lo,
                                    blk_hi, k_transfer, _ptr(stats.top1, torch.float32, "top1"),
                                    _ptr(stats.top2, torch.float32, "top2"), _ptr(stats.sumexp, torch.float32, "sumexp"),
                                    _ptr(stats.argmax, torch.int32, "argmax"), _ptr(n_masked, torch.int32, "n_masked"),
                                    _ptr(exit_reason, torch.uint8, "exit_reason"),
                                    _ptr(exit_step, torch.int16, "exit_step"), step_index, _stream()),
           "jot_accept_freeze")


def merge_stats(a: Stats, b: Stats, out: Optional[Stats] = None) -> Stats:
    """Statistics of the same positions over two disjoint vocabulary slices -> over their union (device kernel)."""
    out = out or Stats(torch.empty_like(a.top1), torch.empty_like(a.top2), torch.empty_like(a.sumexp),
                       torch.empty_like(a.argmax))
    n = a.top1.numel()
    args = []
    for s in (a, b, out):
        args += [_ptr(s.top1, torch.float32, "top1"), _ptr(s.top2, torch.float32, "top2"),
                 _ptr(s.sumexp, torch.float32, "sumexp"), _ptr(s.argmax, torch.int32, "argmax")]
    _check(_lib().jot_merge_stats(n, *args, _stream()), "jot_merge_stats")
    return out


def gemm_bf16(a: torch.Tensor, w: torch.Tensor, residual: Optional[torch.Tensor] = None,
              out: Optional[torch.Tensor] = None, scratch: Optional[torch.Tensor] = None) -> torch.Tensor:
    """out[M, N] = a[M, K] @ w[N, K]^T (+ residual), bf16 in/out, fp32 accumulate.
    scratch: optional float32 CUDA tensor the kernel may use for split-K partial sums."""
    M, K = a.shape
    N = w.shape[0]
    out = torch.empty(M, N, dtype=torch.bfloat16, device=a.device) if out is None else out
    status = torch.zeros(1, dtype=torch.int32, device=a.device)
    _check(_lib().jot_gemm_bf16(_ptr(a, torch.bfloat16, "a"), _ptr(w, torch.bfloat16, "w"),
                                _ptr(residual, torch.bfloat16, "residual"), _ptr(out, torch.bfloat16, "out"), M, N, K,
                                _ptr(scratch, torch.float32, "scratch"), scratch.numel() * 4 if scratch is not None else 0,
                                status.data_ptr(), _stream()), "jot_gemm_bf16")
    if int(status.item()) != 0:
        raise JotError(-5, "jot_gemm_bf16")
    return out


def gemm_bf16_noalloc(a: torch.Tensor, w: torch.Tensor, residual: Optional[torch.Tensor], out: torch.Tensor,
                      status: torch.Tensor) -> torch.Tensor:
    """out[M, N] = a[M, K] @ w[N, K]^T (+ residual) through the entry point that never allocates.

    For callers that may not create device memory (a serving loop with a fixed memory plan, a plugin that
    only gets buffers handed to it): the split-K scratch is a fixed 16 MiB array inside the library, so
    4 * M * N * 4 bytes must fit in it.  `out` and the int32 `status` word are the caller's, too; this
    wrapper creates no tensor.  Calls share the array: keep them on one stream."""
    M, K = a.shape
    N = w.shape[0]
    _check(_lib().jot_gemm_bf16_noalloc(_ptr(a, torch.bfloat16, "a"), _ptr(w, torch.bfloat16, "w"),
                                        _ptr(residual, torch.bfloat16, "residual"), _ptr(out, torch.bfloat16, "out"),
                                        M, N, K, _ptr(status, torch.int32, "status"), _stream()),
           "jot_gemm_bf16_noalloc")
    return out


def selftest_wait_expiry(limit_ns: int = 20_000_000) -> int:
    """Run the bounded-wait self test; returns the status word the kernel wrote (1 = the wait gave up)."""
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    _check(_lib().jot_selftest_wait_expiry(status.data_ptr(), limit_ns, _stream()), "jot_selftest_wait_expiry")
    return int(status.item())
