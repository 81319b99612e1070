"""Pins for the denoiser side of the CPU oracle: closed forms, invariants and an independent restatement
built from torch.nn.functional routines."""
import math

import numpy as np
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


# ---------------------------------------------------------------- block-wise KV cache
def _tiny_case(seed=2, B=2, P=6, G=18):
    g = inputs.ModelGeometry(2, 64, 2, 1, 32, 96, 128, 127, 10000.0)
    w = inputs.model_weights(g, seed=seed)
    tokens = inputs.partially_masked_canvas(seed, B, P, G, g.vocab, g.mask_id, 0.6)
    return g, w, tokens


def test_cached_pass_with_block_equal_to_canvas_is_the_full_pass():
    g, w, tokens = _tiny_case()
    cache = []
    full = mo.hidden_states(g, w, tokens, cache_out=cache)
    assert len(cache) == g.n_layers and cache[0][0].shape == (2, 24, g.n_kv_heads, g.head_dim)
    # the cache's content is irrelevant when every position is recomputed
    junk = [(torch.full_like(k, 7.0), torch.full_like(v, -3.0)) for k, v in cache]
    got = mo.hidden_states_cached(g, w, tokens, junk, 0, tokens.shape[1])
    assert torch.equal(got, full)


@pytest.mark.parametrize("lo,hi", [(6, 12), (12, 24), (0, 6), (9, 10)])
def test_cached_pass_on_an_unchanged_canvas_gives_the_full_pass_rows(lo, hi):
    for ra in (True, False):
        g, w, tokens = _tiny_case()
        cache = []
        full = mo.hidden_states(g, w, tokens, round_activations=ra, cache_out=cache)
        got = mo.hidden_states_cached(g, w, tokens, cache, lo, hi, round_activations=ra)
        assert got.shape == (2, hi - lo, g.d_model)
        assert torch.allclose(got, full[:, lo:hi], rtol=0, atol=1e-12 if not ra else 0.0)


def test_cache_is_stale_outside_the_block_and_fresh_inside():
    g, w, tokens = _tiny_case()
    lo, hi = 12, 18
    cache = []
    mo.hidden_states(g, w, tokens, cache_out=cache)
    base = mo.hidden_states_cached(g, w, tokens, cache, lo, hi)
    outside = tokens.clone()
    outside[:, 3] = (outside[:, 3] + 5) % 100          # prefix token changes after the refresh
    outside[:, 20] = (outside[:, 20] + 9) % 100        # and a suffix token
    assert torch.equal(mo.hidden_states_cached(g, w, outside, cache, lo, hi), base)       # not seen
    assert not torch.equal(mo.hidden_states(g, w, outside)[:, lo:hi], base)               # the full pass sees it
    inside = tokens.clone()
    inside[:, 14] = (inside[:, 14] + 11) % 100
    got = mo.hidden_states_cached(g, w, inside, cache, lo, hi)
    assert not torch.equal(got, base)                                                     # seen by the block's rows
    # and it is an approximation of the full pass on the new canvas, not equal to it: positions outside the
    # block would have reacted to the new token
    full_new = mo.hidden_states(g, w, inside)[:, lo:hi]
    diff = (got - full_new).abs().max().item()
    assert 0 < diff < 0.5 * full_new.abs().max().item()
    # the cache itself is never written
    again = []
    mo.hidden_states(g, w, tokens, cache_out=again)
    assert all(torch.equal(a[0], b[0]) and torch.equal(a[1], b[1]) for a, b in zip(cache, again))


def test_cached_layer_against_loops():
    """One layer, one head, no rounding: attention of a block row written out with Python loops over keys,
    taking fresh keys / values inside the block and the cached ones outside."""
    g = inputs.ModelGeometry(1, 16, 1, 1, 16, 32, 64, 63, 10000.0)
    w = inputs.model_weights(g, seed=4)
    L, lo, hi = 10, 4, 7
    old = inputs.partially_masked_canvas(4, 1, 2, L - 2, g.vocab, g.mask_id, 0.5)
    new = old.clone()
    new[0, 5] = 17
    cache = []
    mo.hidden_states(g, w, old, round_activations=False, cache_out=cache)
    lw = w["layers"][0]
    h_new = w["embed"][new.long()].double()[0]                                 # [L, d]
    hd = g.head_dim

    def qkv_row(h_row, pos):
        a = h_row * (h_row.pow(2).mean() + g.rms_eps).rsqrt() * lw["attn_norm"].double()
        z = lw["wqkv"].double() @ a
        q, k, v = z[:hd], z[hd:2 * hd], z[2 * hd:]
        def rot(t):
            out = t.clone()
            for j in range(hd // 2):
                ang = pos * g.rope_theta ** (-2.0 * j / hd)
                out[j] = t[j] * math.cos(ang) - t[j + hd // 2] * math.sin(ang)
                out[j + hd // 2] = t[j + hd // 2] * math.cos(ang) + t[j] * math.sin(ang)
            return out
        return rot(q), rot(k), v

    fresh = {i: qkv_row(h_new[i], i) for i in range(lo, hi)}
    want = []
    for i in range(lo, hi):
        q = fresh[i][0]
        scores, vals = [], []
        for j in range(L):
            k_j = fresh[j][1] if lo <= j < hi else cache[0][0][0, j, 0]
            v_j = fresh[j][2] if lo <= j < hi else cache[0][1][0, j, 0]
            scores.append(float(q @ k_j) / math.sqrt(hd))
            vals.append(v_j)
        mx = max(scores)
        e = [math.exp(s - mx) for s in scores]
        o = sum(ei * vj for ei, vj in zip(e, vals)) / sum(e)
        h1 = h_new[i] + lw["wo"].double() @ o
        a = h1 * (h1.pow(2).mean() + g.rms_eps).rsqrt() * lw["mlp_norm"].double()
        gu = lw["w_gate_up"].double() @ a
        gate, up = gu[:g.d_ff], gu[g.d_ff:]
        h2 = h1 + lw["w_down"].double() @ (gate / (1 + torch.exp(-gate)) * up)
        want.append(h2 * (h2.pow(2).mean() + g.rms_eps).rsqrt() * w["final_norm"].double())
    got = mo.hidden_states_cached(g, w, new, cache, lo, hi, round_activations=False)[0]
    assert torch.allclose(got, torch.stack(want), rtol=1e-10, atol=1e-12)


def test_block_cached_denoiser_refreshes_on_block_change():
    g, w, _ = _tiny_case()
    P, G, Lb = 6, 18, 6
    x = inputs.prompt(1, 1, P, g.vocab, g.mask_id)[0].tolist() + [g.mask_id] * G
    den = mo.BlockCachedDenoiser(g, w, P, Lb)
    first = den(x, [6, 7, 8, 9, 10, 11])
    full = mo.logits(g, w, torch.tensor([x], dtype=torch.int32), rows=[(0, i) for i in range(6, 12)])
    assert all(np.array_equal(first[i], full[r].numpy()) for r, i in enumerate(range(6, 12)))   # refresh = full pass
    x[7] = 3
    den(x, [6, 8, 9])
    assert (den.full_passes, den.cached_passes) == (1, 1)
    x[6] = x[8] = x[9] = x[10] = x[11] = 5
    den(x, [12, 13])                                     # next block: refresh, again the full pass
    assert (den.full_passes, den.cached_passes) == (2, 1)
    full = mo.logits(g, w, torch.tensor([x], dtype=torch.int32), rows=[(0, 12), (0, 13)])
    again = den(x, [12, 13])                             # same canvas, now through the cache: same rows
    assert np.allclose(again[12], full[0].numpy(), rtol=0, atol=1e-9)
    assert (den.full_passes, den.cached_passes) == (2, 2)


def test_generation_under_the_block_cache():
    """Algorithm 1 over the cached denoiser: one full pass per block, every other step recomputes the block
    only; with a single block spanning the whole generation the first step equals the uncached run's."""
    from oracle import jot_oracle as jo
    g, w, _ = _tiny_case()
    P, G, Lb, T = 6, 18, 6, 18
    prompt = inputs.prompt(1, 1, P, g.vocab, g.mask_id)[0].tolist()
    bump = inputs.logit_bump(2, 1, P + G, g.vocab, g.mask_id, hi=10.0)
    bump = (bump[0][0], bump[1][0])
    den = mo.BlockCachedDenoiser(g, w, P, Lb, bump)
    tr = jo.generate(den, prompt, G, T, jo.JotParams(30, 1, 0.5, 4), g.mask_id, Lb)
    assert all(t != g.mask_id for t in tr.x)
    assert den.full_passes == G // Lb and den.full_passes + den.cached_passes == tr.steps_used
    plain = mo.BlockCachedDenoiser(g, w, P, G, bump)          # one block: first step is the plain full pass
    tr1 = jo.generate(plain, prompt, G, T, jo.JotParams(30, 1, 0.5, 4), g.mask_id, G)

    def uncached(x, rows):
        l = mo.logits(g, w, torch.tensor([x], dtype=torch.int32), rows=[(0, i) for i in rows])
        for r, i in enumerate(rows):
            l[r, int(bump[0][i])] += float(bump[1][i])
        return {i: l[r].numpy() for r, i in enumerate(rows)}
    tr2 = jo.generate(uncached, prompt, G, T, jo.JotParams(30, 1, 0.5, 4), g.mask_id, G)
    assert tr1.canvases[1] == tr2.canvases[1]
