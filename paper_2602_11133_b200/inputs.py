"""Seeded synthetic inputs for JoT decoding workloads.

This module only *draws inputs*: model weights, prompts, hidden states, planted
logit bumps and mask states.  It contains none of the method's arithmetic (no
softmax, thresholds, acceptance, transformer math) and imports neither the CUDA
binding nor the CPU oracle, so both sides can consume the very same tensors.

Every value is a pure function of (seed, tensor name, flat index): a 64-bit
counter hash (splitmix64 finaliser) gives two 24-bit uniforms per element and
Box-Muller turns them into a normal deviate.  The integer part is exact on any
device; the float part (log/cos) may differ in the last bit between devices, so
a workload is drawn ONCE on one device and copied wherever else it is needed.
"""
from __future__ import annotations

import dataclasses
import math
import zlib
from typing import Dict, Optional

import torch

_MASK64 = (1 << 64) - 1


def _to_i64(v: int) -> int:
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


_GOLDEN = _to_i64(0x9E3779B97F4A7C15)
_MIX1 = _to_i64(0xBF58476D1CE4E5B9)
_MIX2 = _to_i64(0x94D049BB133111EB)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift on int64 (torch's >> is arithmetic)."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _splitmix(x: torch.Tensor) -> torch.Tensor:
    x = x + _GOLDEN
    x = (x ^ _lsr(x, 30)) * _MIX1
    x = (x ^ _lsr(x, 27)) * _MIX2
    return x ^ _lsr(x, 31)


def _stream_key(seed: int, name: str) -> int:
    """One 64-bit key per (seed, tensor name)."""
    h = zlib.crc32(name.encode()) & 0xFFFFFFFF
    k = (seed * 0x9E3779B97F4A7C15 + h * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & _MASK64
    # one scalar splitmix round so nearby seeds give unrelated streams
    k = (k + 0x9E3779B97F4A7C15) & _MASK64
    k = ((k ^ (k >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    k = ((k ^ (k >> 27)) * 0x94D049BB133111EB) & _MASK64
    return _to_i64(k ^ (k >> 31))


def hash_bits(seed: int, name: str, n: int, device="cpu", start: int = 0) -> torch.Tensor:
    """int64 tensor of n hashed 64-bit words for flat indices start..start+n-1."""
    idx = torch.arange(start, start + n, dtype=torch.int64, device=device)
    return _splitmix(idx ^ _stream_key(seed, name))


def uniform01(seed: int, name: str, n: int, device="cpu", start: int = 0) -> torch.Tensor:
    """float64 uniforms in (0,1) from the top 24 bits of the hash."""
    b = hash_bits(seed, name, n, device, start)
    return (_lsr(b, 40).to(torch.float64) + 0.5) / float(1 << 24)


def randint(seed: int, name: str, n: int, high: int, device="cpu") -> torch.Tensor:
    """int64 integers uniform on [0, high) (top 32 hash bits, multiply-shift)."""
    b = _lsr(hash_bits(seed, name, n, device), 32)
    return (b * high) >> 32


def normal(seed: int, name: str, shape, std: float = 1.0, mean: float = 0.0,
           dtype=torch.bfloat16, device="cpu", chunk: int = 1 << 26) -> torch.Tensor:
    """N(mean, std) tensor of the given shape, rounded (RNE) to `dtype`."""
    n = int(math.prod(shape))
    out = torch.empty(n, dtype=dtype, device=device)
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        b = hash_bits(seed, name, m, device, s)
        u1 = (_lsr(b, 40).to(torch.float32) + 0.5) / float(1 << 24)
        u2 = ((b & 0xFFFFFF).to(torch.float32) + 0.5) / float(1 << 24)
        z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
        out[s:s + m] = (z * std + mean).to(dtype)
    return out.view(*shape)


# ----------------------------------------------------------------------------
# model geometry + weights
# ----------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class ModelGeometry:
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab: int
    mask_id: int
    rope_theta: float = 10000.0
    rms_eps: float = 1e-5

    @property
    def qkv_rows(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim


TINY = ModelGeometry(2, 256, 4, 4, 64, 704, 4096, 4095, 10000.0)
LLADA_8B = ModelGeometry(32, 4096, 32, 32, 128, 12288, 126464, 126336, 500000.0)
DREAM_7B = ModelGeometry(28, 3584, 28, 4, 128, 18944, 152064, 151666, 1000000.0)


def model_weights(g: ModelGeometry, seed: int = 0, device="cpu", std: float = 0.02,
                  n_layers: Optional[int] = None) -> Dict[str, object]:
    """bf16 weights ~N(0, std); RMSNorm gains ~N(1, 0.1) so a dropped gain shows.

    Layout (all row-major, [out_features, in_features]):
      embed [V,d]; lm_head [V,d]; final_norm [d];
      per layer: attn_norm [d], wqkv [(nq+2nkv)*hd, d] (Q rows, then K, then V),
      wo [d, nq*hd], mlp_norm [d], w_gate_up [2*ff, d] (gate rows, then up rows),
      w_down [d, ff].
    """
    nl = g.n_layers if n_layers is None else n_layers
    d, ff = g.d_model, g.d_ff
    w: Dict[str, object] = {
        "embed": normal(seed, "embed", (g.vocab, d), std, device=device),
        "lm_head": normal(seed, "lm_head", (g.vocab, d), std, device=device),
        "final_norm": normal(seed, "final_norm", (d,), 0.1, 1.0, device=device),
        "layers": [],
    }
    for l in range(nl):
        w["layers"].append({
            "attn_norm": normal(seed, f"l{l}.attn_norm", (d,), 0.1, 1.0, device=device),
            "wqkv": normal(seed, f"l{l}.wqkv", (g.qkv_rows, d), std, device=device),
            "wo": normal(seed, f"l{l}.wo", (d, g.n_q_heads * g.head_dim), std, device=device),
            "mlp_norm": normal(seed, f"l{l}.mlp_norm", (d,), 0.1, 1.0, device=device),
            "w_gate_up": normal(seed, f"l{l}.w_gate_up", (2 * ff, d), std, device=device),
            "w_down": normal(seed, f"l{l}.w_down", (d, ff), std, device=device),
        })
    return w


def weights_to(w: Dict[str, object], device) -> Dict[str, object]:
    out = {k: (v.to(device) if torch.is_tensor(v) else v) for k, v in w.items() if k != "layers"}
    out["layers"] = [{k: v.to(device) for k, v in lw.items()} for lw in w["layers"]]
    return out


# ----------------------------------------------------------------------------
# token-side inputs
# ----------------------------------------------------------------------------
def token_ids(seed: int, name: str, n: int, vocab: int, mask_id: int, device="cpu") -> torch.Tensor:
    """int32 ids uniform on [0, vocab) without mask_id."""
    t = randint(seed, name, n, vocab - 1, device)
    t = t + (t >= mask_id).to(torch.int64)
    return t.to(torch.int32)


def prompt(seed: int, B: int, P: int, vocab: int, mask_id: int, device="cpu") -> torch.Tensor:
    return token_ids(seed, "prompt", B * P, vocab, mask_id, device).view(B, P)


def logit_bump(seed: int, B: int, L: int, vocab: int, mask_id: int, hi: float = 12.0, device="cpu"):
    """Planted bump: per canvas position one token id (never mask_id) and a value ~U(0, hi) (fp32)."""
    ids = token_ids(seed, "bump_id", B * L, vocab, mask_id, device).view(B, L)
    val = (uniform01(seed, "bump_val", B * L, device) * hi).to(torch.float32).view(B, L)
    return ids, val


def partially_masked_canvas(seed: int, B: int, P: int, G: int, vocab: int, mask_id: int,
                            p_mask: float = 0.5, device="cpu") -> torch.Tensor:
    """[B, P+G] int32: P resolved prompt ids, then G positions each masked with prob p_mask
    (resolved generation positions hold random ids)."""
    x = token_ids(seed, "canvas", B * (P + G), vocab, mask_id, device).view(B, P + G).clone()
    m = (uniform01(seed, "canvas_mask", B * G, device) < p_mask).view(B, G)
    x[:, P:][m] = mask_id
    return x


def hidden_states(seed: int, rows: int, d: int, device="cpu") -> torch.Tensor:
    return normal(seed, "hidden", (rows, d), 1.0, device=device)


@dataclasses.dataclass
class LMHeadCase:
    """Standalone fused LM-head + acceptance workload (hidden states given)."""
    hidden: torch.Tensor      # [B*L, d] bf16
    w: torch.Tensor           # [V, d] bf16
    tokens: torch.Tensor      # [B, L] int32
    bump_id: torch.Tensor     # [B, L] int32
    bump_val: torch.Tensor    # [B, L] fp32
    B: int
    L: int
    P: int
    vocab: int
    mask_id: int


def lm_head_case(seed: int = 0, B: int = 8, P: int = 128, G: int = 256, d: int = 4096,
                 vocab: int = 126464, mask_id: int = 126336, device="cpu") -> LMHeadCase:
    L = P + G
    ids, val = logit_bump(seed, B, L, vocab, mask_id, 12.0, device)
    return LMHeadCase(
        hidden=hidden_states(seed, B * L, d, device),
        w=normal(seed, "lm_head", (vocab, d), 0.02, device=device),
        tokens=partially_masked_canvas(seed, B, P, G, vocab, mask_id, 0.5, device),
        bump_id=ids, bump_val=val, B=B, L=L, P=P, vocab=vocab, mask_id=mask_id)
