"""Pins for the denoiser side of the CPU oracle: closed forms, invariants and an independent restatement
built from torch.nn.functional routines."""
import math

import pytest
import torch
import torch.nn.functional as F

from oracle import model_oracle as mo
from paper_2602_11133_b200 import inputs

G = inputs.ModelGeometry(n_layers=2, d_model=64, n_q_heads=4, n_kv_heads=2, head_dim=16, d_ff=96,
                         vocab=50, mask_id=49, rope_theta=10000.0)


def test_rope_closed_form():
    # one head, hd = 4: pairs (0,2) and (1,3); angles pos*1 and pos*theta^(-1/2)
    t = torch.zeros(1, 3, 1, 4, dtype=torch.float64)
    t[0, :, 0, 0] = 1.0          # unit vector in pair 0
    t[0, :, 0, 1] = 2.0          # length-2 vector in pair 1
    out = mo.rope(t, 100.0)
    for pos in range(3):
        assert out[0, pos, 0, 0].item() == pytest.approx(math.cos(pos))
        assert out[0, pos, 0, 2].item() == pytest.approx(math.sin(pos))
        assert out[0, pos, 0, 1].item() == pytest.approx(2 * math.cos(pos / 10.0))
        assert out[0, pos, 0, 3].item() == pytest.approx(2 * math.sin(pos / 10.0))
    # rotations preserve norms, and q.k depends only on the position difference
    q = torch.randn(1, 6, 1, 8, dtype=torch.float64).expand(1, 6, 1, 8)
    q = q[:, :1].expand(1, 6, 1, 8).contiguous()
    r = mo.rope(q, 10000.0)
    assert torch.allclose(r.norm(dim=-1), q.norm(dim=-1))
    d01 = (r[0, 0, 0] * r[0, 1, 0]).sum()
    d34 = (r[0, 3, 0] * r[0, 4, 0]).sum()
    assert d01.item() == pytest.approx(d34.item())


def test_rmsnorm_closed_form():
    h = torch.tensor([[3.0, -4.0, 0.0, 0.0]], dtype=torch.float64)
    g = torch.tensor([1.0, 2.0, 1.0, 1.0])
    out = mo.rmsnorm(h, g, 0.0)
    assert torch.allclose(out, torch.tensor([[3 / 2.5, -8 / 2.5, 0, 0]], dtype=torch.float64))


def test_attention_rows_average_values_and_see_everything():
    torch.manual_seed(0)
    q = torch.randn(2, 5, 4, 8, dtype=torch.float64)
    k = torch.randn(2, 5, 2, 8, dtype=torch.float64)
    v = torch.ones(2, 5, 2, 8, dtype=torch.float64)
    assert torch.allclose(mo.attention(q, k, v, False), torch.ones(2, 5, 4, 8, dtype=torch.float64))
    # q = 0 -> uniform weights -> mean of all values, including LATER positions (no causal mask)
    v = torch.randn(2, 5, 2, 8, dtype=torch.float64)
    o = mo.attention(torch.zeros_like(q), k, v, False)
    assert torch.allclose(o[:, 0, 0], v[:, :, 0].mean(dim=1))
    assert torch.allclose(o[:, 0, 3], v[:, :, 1].mean(dim=1))      # GQA: heads 2,3 read kv head 1


def independent_forward(g, w, tokens):
    """Same network from torch.nn.functional building blocks (float64, no activation rounding)."""
    B, L = tokens.shape
    hd, nq, nkv = g.head_dim, g.n_q_heads, g.n_kv_heads
    pos = torch.arange(L, dtype=torch.float64)
    inv = 1.0 / (g.rope_theta ** (torch.arange(0, hd, 2, dtype=torch.float64) / hd))
    fr = torch.outer(pos, inv)
    cos = torch.cat([fr.cos(), fr.cos()], -1)[None, None]
    sin = torch.cat([fr.sin(), fr.sin()], -1)[None, None]

    def rot(x):                                                      # [B, H, L, hd]
        x1, x2 = x[..., : hd // 2], x[..., hd // 2:]
        return x * cos + torch.cat([-x2, x1], -1) * sin

    h = F.embedding(tokens.long(), w["embed"].double())
    for lw in w["layers"]:
        a = F.rms_norm(h, (g.d_model,), lw["attn_norm"].double(), g.rms_eps)
        qkv = F.linear(a, lw["wqkv"].double())
        q, k, v = qkv.split([nq * hd, nkv * hd, nkv * hd], dim=-1)
        q = rot(q.view(B, L, nq, hd).transpose(1, 2))
        k = rot(k.view(B, L, nkv, hd).transpose(1, 2))
        v = v.view(B, L, nkv, hd).transpose(1, 2)
        o = F.scaled_dot_product_attention(q, k, v, is_causal=False, enable_gqa=True)
        h = h + F.linear(o.transpose(1, 2).reshape(B, L, nq * hd), lw["wo"].double())
        a = F.rms_norm(h, (g.d_model,), lw["mlp_norm"].double(), g.rms_eps)
        gate, up = F.linear(a, lw["w_gate_up"].double()).chunk(2, dim=-1)
        h = h + F.linear(F.silu(gate) * up, lw["w_down"].double())
    h = F.rms_norm(h, (g.d_model,), w["final_norm"].double(), g.rms_eps)
    return F.linear(h, w["lm_head"].double())


def test_forward_matches_independent_restatement():
    w = inputs.model_weights(G, seed=3, std=0.2)
    tokens = inputs.prompt(1, 2, 11, G.vocab, G.mask_id)
    want = independent_forward(G, w, tokens)
    got = mo.logits(G, w, tokens, round_activations=False)
    assert got.shape == (2, 11, G.vocab)
    assert torch.allclose(got, want, rtol=1e-10, atol=1e-10)
    rows = [(0, 3), (1, 10), (1, 0)]
    sel = mo.logits(G, w, tokens, rows=rows, round_activations=False)
    for r, (b, i) in enumerate(rows):
        assert torch.allclose(sel[r], want[b, i], rtol=1e-10, atol=1e-10)


def test_rounded_contract_stays_close_to_unrounded():
    w = inputs.model_weights(G, seed=3, std=0.2)
    tokens = inputs.prompt(1, 2, 11, G.vocab, G.mask_id)
    a = mo.logits(G, w, tokens, round_activations=True)
    b = mo.logits(G, w, tokens, round_activations=False)
    assert (a - b).abs().max().item() < 0.05 * b.abs().max().item()
    assert (a - b).abs().max().item() > 0.0


def test_bidirectional_not_causal():
    w = inputs.model_weights(G, seed=3, std=0.2)
    tokens = inputs.prompt(2, 1, 9, G.vocab, G.mask_id)
    t2 = tokens.clone()
    t2[0, 8] = (t2[0, 8] + 1) % (G.vocab - 1)
    a = mo.logits(G, w, tokens, round_activations=False)
    b = mo.logits(G, w, t2, round_activations=False)
    assert (a[0, 0] - b[0, 0]).abs().max().item() > 1e-6           # the first position sees the last one


def test_batch_rows_are_independent():
    w = inputs.model_weights(G, seed=3, std=0.2)
    tokens = inputs.prompt(4, 3, 7, G.vocab, G.mask_id)
    full = mo.logits(G, w, tokens)
    for b in range(3):
        one = mo.logits(G, w, tokens[b:b + 1])
        assert torch.allclose(full[b], one[0], rtol=1e-12, atol=1e-12)


def test_lm_head_bump():
    h = torch.randn(3, 8, dtype=torch.float64)
    wl = torch.randn(10, 8, dtype=torch.float64)
    ids = torch.tensor([2, 9, 0], dtype=torch.int32)
    val = torch.tensor([1.5, 0.25, 3.0])
    l = mo.lm_head_logits(h, wl, ids, val)
    base = h @ wl.T
    base[0, 2] += 1.5
    base[1, 9] += 0.25
    base[2, 0] += 3.0
    assert torch.allclose(l, base)


# ---------------------------------------------------------------- the input generators themselves
def test_inputs_are_seeded_and_well_formed():
    a = inputs.normal(0, "x", (1000, 64), 0.02)
    b = inputs.normal(0, "x", (1000, 64), 0.02)
    c = inputs.normal(1, "x", (1000, 64), 0.02)
    assert a.dtype == torch.bfloat16 and torch.equal(a, b) and not torch.equal(a, c)
    f = a.float()
    assert abs(f.mean().item()) < 5e-4 and f.std().item() == pytest.approx(0.02, rel=0.02)
    # chunked generation is index-addressed: same values whatever the chunk size
    d = inputs.normal(0, "x", (1000, 64), 0.02, chunk=777)
    assert torch.equal(a, d)
    p = inputs.prompt(0, 4, 100, 4096, 4095)
    assert p.dtype == torch.int32 and p.min() >= 0 and p.max() < 4095
    t = inputs.token_ids(0, "t", 50000, 17, 5)
    assert 5 not in set(t.tolist()) and set(t.tolist()) == set(range(17)) - {5}
    cv = inputs.partially_masked_canvas(0, 8, 128, 256, 126464, 126336)
    assert (cv[:, :128] != 126336).all()
    frac = (cv[:, 128:] == 126336).float().mean().item()
    assert 0.45 < frac < 0.55
    ids, val = inputs.logit_bump(0, 8, 384, 126464, 126336)
    assert (ids != 126336).all() and val.min() >= 0 and val.max() <= 12 and val.dtype == torch.float32
