"""CPU oracle for the denoiser f_theta of Algorithm 1 -- TEST INFRASTRUCTURE ONLY.

The paper treats the network as given ("Compute logits l <- f_theta(x)", Algorithm 1; "Reverse
process", Section 3.1): a bidirectional transformer that returns one logit row per canvas position.
The geometry used here is the Llama-style one the workloads name: RMSNorm, rotary position
embedding (rotate-half, absolute canvas positions), grouped-query softmax attention WITHOUT any
mask, SwiGLU MLP, untied LM head, no biases.

Plain PyTorch CPU ops in float64; library matmul/softmax serve as steps, nothing is blocked, fused
or reordered.  It shares no code with the CUDA library and is never imported by it.

Precision contract ("bf16 path"): weights are bf16 values; the activation tensors that the device
path keeps in bf16 are rounded to bf16 here at the same named points, and nowhere else:
  embedding rows; each RMSNorm output; the QKV projection; rotated q and k; the un-normalised
  attention probabilities exp(s - rowmax) (the row sum uses the unrounded values); the attention
  output; each residual sum (projection + residual, rounded once); silu(gate)*up (from unrounded
  gate and up); logits are float64 and never rounded.
`round_activations=False` drops every one of those roundings (pure float64 reference).

Pinned by tests against closed forms (RoPE rotation, attention row sums, permutation behaviour) and
against an independent restatement built from torch.nn.functional routines; the float64/bf16
contract itself is a reading of this build, not of the paper.
"""
from __future__ import annotations

import math
from typing import Dict, Optional, Sequence

import torch

F64 = torch.float64


def _r(t: torch.Tensor, on: bool) -> torch.Tensor:
    """Round to bf16 and come back to float64 (a named rounding point of the contract)."""
    return t.to(torch.bfloat16).to(F64) if on else t


def rmsnorm(h: torch.Tensor, gain: torch.Tensor, eps: float) -> torch.Tensor:
    return h * torch.rsqrt((h * h).mean(dim=-1, keepdim=True) + eps) * gain.to(F64)


def rope(t: torch.Tensor, theta: float) -> torch.Tensor:
    """t: [B, L, H, hd].  Rotate-half: pair (j, j + hd/2) turns by angle pos * theta^(-2j/hd)."""
    B, L, H, hd = t.shape
    half = hd // 2
    inv = theta ** (-torch.arange(half, dtype=F64) * 2.0 / hd)
    ang = torch.arange(L, dtype=F64)[:, None] * inv[None, :]          # [L, half]
    c, s = torch.cos(ang)[None, :, None, :], torch.sin(ang)[None, :, None, :]
    a, b = t[..., :half], t[..., half:]
    return torch.cat([a * c - b * s, b * c + a * s], dim=-1)


def attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, round_p: bool) -> torch.Tensor:
    """q: [B, L, Hq, hd]; k, v: [B, L, Hkv, hd]; every query sees every key (no mask)."""
    B, L, Hq, hd = q.shape
    group = Hq // k.shape[2]
    k = k.repeat_interleave(group, dim=2)
    v = v.repeat_interleave(group, dim=2)
    s = torch.einsum("blhd,bmhd->bhlm", q, k) / math.sqrt(hd)
    e = torch.exp(s - s.max(dim=-1, keepdim=True).values)
    denom = e.sum(dim=-1, keepdim=True)
    o = torch.einsum("bhlm,bmhd->blhd", _r(e, round_p), v) / denom.permute(0, 2, 1, 3)
    return o


def hidden_states(g, w: Dict[str, object], tokens: torch.Tensor, round_activations: bool = True,
                  n_layers: Optional[int] = None) -> torch.Tensor:
    """Final-normalised hidden states [B, L, d] (float64, bf16-valued when rounding is on)."""
    ra = round_activations
    B, L = tokens.shape
    nq, nkv, hd, d = g.n_q_heads, g.n_kv_heads, g.head_dim, g.d_model
    h = w["embed"][tokens.long()].to(F64)                               # [B, L, d]
    layers = w["layers"] if n_layers is None else w["layers"][:n_layers]
    for lw in layers:
        a = _r(rmsnorm(h, lw["attn_norm"], g.rms_eps), ra)
        qkv = _r(a @ lw["wqkv"].to(F64).T, ra)
        q = qkv[..., : nq * hd].reshape(B, L, nq, hd)
        k = qkv[..., nq * hd: (nq + nkv) * hd].reshape(B, L, nkv, hd)
        v = qkv[..., (nq + nkv) * hd:].reshape(B, L, nkv, hd)
        q = _r(rope(q, g.rope_theta), ra)
        k = _r(rope(k, g.rope_theta), ra)
        o = _r(attention(q, k, v, ra), ra).reshape(B, L, nq * hd)
        h = _r(h + o @ lw["wo"].to(F64).T, ra)
        a = _r(rmsnorm(h, lw["mlp_norm"], g.rms_eps), ra)
        gu = a @ lw["w_gate_up"].to(F64).T
        gate, up = gu[..., : g.d_ff], gu[..., g.d_ff:]
        act = _r(gate * torch.sigmoid(gate) * up, ra)
        h = _r(h + act @ lw["w_down"].to(F64).T, ra)
    return _r(rmsnorm(h, w["final_norm"], g.rms_eps), ra)


def lm_head_logits(hidden_rows: torch.Tensor, w_lm: torch.Tensor,
                   bump_id: Optional[torch.Tensor] = None,
                   bump_val: Optional[torch.Tensor] = None) -> torch.Tensor:
    """logits [R, V] = hidden_rows [R, d] @ w_lm[V, d]^T in float64, plus the planted bump."""
    l = hidden_rows.to(F64) @ w_lm.to(F64).T
    if bump_id is not None:
        rows = torch.arange(l.shape[0])
        l[rows, bump_id.long()] += bump_val.to(F64)
    return l


def logits(g, w: Dict[str, object], tokens: torch.Tensor, rows: Optional[Sequence] = None,
           round_activations: bool = True, n_layers: Optional[int] = None) -> torch.Tensor:
    """f_theta(x): logits for canvas positions.  rows = list of (b, i); None = every position."""
    h = hidden_states(g, w, tokens, round_activations, n_layers)
    B, L, d = h.shape
    if rows is None:
        return lm_head_logits(h.reshape(B * L, d), w["lm_head"]).reshape(B, L, -1)
    sel = torch.stack([h[b, i] for b, i in rows])
    return lm_head_logits(sel, w["lm_head"])
