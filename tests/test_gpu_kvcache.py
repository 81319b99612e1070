"""GPU parity of the block-wise KV cache composition (Section 6.2, "Composability with KV-cache
acceleration") against the CPU oracle: one cached step, the stale-cache property, and Algorithm 1 under the
cache."""
import math

import numpy as np
import pytest
import torch

from helpers import GAP_TOL, REL_TOL, compare_stats, oracle_stats_for_rows
from oracle import jot_oracle as jo
from oracle import model_oracle as mo
from paper_2602_11133_b200 import inputs

pytestmark = pytest.mark.gpu

GEOMS = {
    "tiny": inputs.TINY,
    "gqa": inputs.ModelGeometry(2, 256, 4, 2, 64, 320, 1032, 1000, 10000.0),
    "hd128": inputs.ModelGeometry(2, 256, 2, 1, 128, 704, 2048, 2047, 500000.0),
}


@pytest.fixture(scope="module")
def jot():
    from paper_2602_11133_b200 import jot as binding
    binding._lib()
    return binding


def fill_some(tokens, g, lo, hi, seed, inside=0.4, outside=0.3):
    """A later canvas of the same run: some masked positions inside and outside [lo, hi) now hold tokens."""
    rng = np.random.default_rng(seed)
    out = tokens.clone()
    B, L = tokens.shape
    for b in range(B):
        for i in range(L):
            if int(out[b, i]) == g.mask_id:
                p = inside if lo <= i < hi else outside
                if rng.random() < p:
                    out[b, i] = int(rng.integers(0, g.vocab - 1))
                    if int(out[b, i]) >= g.mask_id:
                        out[b, i] += 1
    return out


@pytest.mark.parametrize("name,B,P,G,lo,hi", [
    ("tiny", 1, 32, 64, 32, 64),         # block of 32 rows, one key block
    ("tiny", 2, 60, 140, 96, 112),       # block of 16 in the middle of L = 200: cached prefix and suffix
    ("gqa", 3, 17, 120, 41, 65),         # ragged: block of 24 starting at an odd position, L = 137
    ("hd128", 2, 128, 256, 256, 384),    # block of 128 at the end: no suffix, three key blocks
    ("hd128", 1, 64, 320, 64, 224),      # block of 160 rows: two query tiles
])
def test_cached_step_matches_oracle(jot, name, B, P, G, lo, hi):
    g = GEOMS[name]
    w_cpu = inputs.model_weights(g, seed=0)
    w_gpu = inputs.weights_to(w_cpu, "cuda")
    L = P + G
    canvas0 = inputs.partially_masked_canvas(1, B, P, G, g.vocab, g.mask_id, 0.8)
    canvas0[:, lo:hi] = g.mask_id                                  # a block starts fully masked
    canvas1 = fill_some(canvas0, g, lo, hi, seed=7)
    model = jot.Model(g, w_gpu, B, L)
    model.attach_kv_cache()
    plain = model.denoise_step(canvas0.cuda(), lo, hi)
    first = model.denoise_step_cached(canvas0.cuda(), lo, hi, refresh=True)
    for a, b in ((plain.top1, first.top1), (plain.top2, first.top2), (plain.sumexp, first.sumexp), (plain.argmax, first.argmax)):
        assert torch.equal(a, b)                                   # a refresh is the plain pass
    st = model.denoise_step_cached(canvas1.cuda(), lo, hi, refresh=False)
    torch.cuda.synchronize()
    cache = []
    mo.hidden_states(g, w_cpu, canvas0, cache_out=cache)
    h = mo.hidden_states_cached(g, w_cpu, canvas1, cache, lo, hi)
    rows = [(b, i) for b in range(B) for i in range(lo, hi) if int(canvas1[b, i]) == g.mask_id]
    assert len(rows) >= (hi - lo) // 3
    logits = mo.lm_head_logits(torch.stack([h[b, i - lo] for b, i in rows]), w_cpu["lm_head"])
    want = oracle_stats_for_rows(logits, g.mask_id)
    flat = torch.tensor([b * L + i for b, i in rows])
    pick = lambda t: t.cpu().view(-1)[flat].numpy()
    n, near = compare_stats(pick(st.top1), pick(st.top2), pick(st.sumexp), pick(st.argmax), want, rel=REL_TOL)
    err = max(abs(a - s.m1) for a, s in zip(pick(st.top1), want))
    # the cached step is an approximation of the full pass on the new canvas, and a different one from it
    full = model.denoise_step(canvas1.cuda(), lo, hi)
    drift = (full.top1.cpu().view(-1)[flat] - st.top1.cpu().view(-1)[flat]).abs().max().item()
    print(f"{name} [{lo},{hi}): {n} rows, {near} near ties, max |top1 err| {err:.2e}; cached vs full pass {drift:.2e}")
    assert near <= max(2, n // 20)
    # rows outside the active set are untouched
    untouched = torch.ones(B * L, dtype=torch.bool)
    untouched[flat] = False
    assert (st.sumexp.cpu().view(-1)[untouched] == 1.0).all()
    model.close()


def test_cache_is_stale_outside_the_block_on_the_gpu(jot):
    g = GEOMS["gqa"]
    B, P, G, lo, hi = 2, 20, 100, 52, 84
    L = P + G
    w_gpu = inputs.weights_to(inputs.model_weights(g, seed=0), "cuda")
    canvas0 = inputs.partially_masked_canvas(2, B, P, G, g.vocab, g.mask_id, 0.7)
    canvas0[:, lo:hi] = g.mask_id
    model = jot.Model(g, w_gpu, B, L)
    with pytest.raises(jot.JotError):
        model.denoise_step_cached(canvas0.cuda(), lo, hi, refresh=True)            # no cache attached
    model.attach_kv_cache()
    with pytest.raises(jot.JotError):
        model.denoise_step_cached(canvas0.cuda(), lo, hi, refresh=False)           # nothing cached yet
    model.denoise_step_cached(canvas0.cuda(), lo, hi, refresh=True)
    base = model.denoise_step_cached(canvas0.cuda(), lo, hi, refresh=False)
    outside = canvas0.clone()
    outside[:, 3] = (outside[:, 3] + 5) % 900
    outside[:, 100] = 77
    got = model.denoise_step_cached(outside.cuda(), lo, hi, refresh=False)
    for a, b in ((base.top1, got.top1), (base.top2, got.top2), (base.sumexp, got.sumexp), (base.argmax, got.argmax)):
        assert torch.equal(a, b)                                   # changes outside the block are not seen ...
    full = model.denoise_step(outside.cuda(), lo, hi)
    assert not torch.equal(full.top1, base.top1)                   # ... which the full pass does see
    inside = canvas0.clone()
    inside[:, 60] = 5
    got = model.denoise_step_cached(inside.cuda(), lo, hi, refresh=False)
    assert not torch.equal(got.top1[:, lo:hi], base.top1[:, lo:hi])                # changes inside are
    # the cached step on the unchanged canvas reproduces the refresh within rounding of the accumulation order
    first = model.denoise_step(canvas0.cuda(), lo, hi)
    assert (first.top1 - base.top1).abs().max().item() < 2e-2 and torch.equal(first.argmax[:, lo:hi][first.top1[:, lo:hi] - first.top2[:, lo:hi] > 0.1],
                                                                             base.argmax[:, lo:hi][first.top1[:, lo:hi] - first.top2[:, lo:hi] > 0.1])
    with pytest.raises(jot.JotError):
        model.denoise_step_cached(canvas0[:1].contiguous().cuda(), lo, hi, refresh=False)   # another batch size
    model.detach_kv_cache()
    with pytest.raises(jot.JotError):
        model.denoise_step_cached(canvas0.cuda(), lo, hi, refresh=False)
    model.close()


@pytest.mark.parametrize("params,block_len", [(jo.JotParams(30.0, 1.0, 0.5, 8), 16), (jo.JotParams(60.0, 1.0, 0.5, 8), 32),
                                              (jo.DREAM_DEFAULT, 64)])
def test_generation_under_the_cache_matches_oracle(jot, params, block_len):
    """Teacher-forced replay of the oracle's cached trajectory (refresh at the first step of every block, the
    block's rows afterwards), then the free-running loop."""
    g = inputs.TINY
    P, G, T = 32, 64, 64
    L = P + G
    w_cpu = inputs.model_weights(g, seed=0)
    w_gpu = inputs.weights_to(w_cpu, "cuda")
    prompt = inputs.prompt(0, 1, P, g.vocab, g.mask_id)
    bump = inputs.logit_bump(9, 1, L, g.vocab, g.mask_id, hi=12.0)
    den = mo.BlockCachedDenoiser(g, w_cpu, P, block_len, (bump[0][0], bump[1][0]))
    tr = jo.generate(den, prompt[0].tolist(), G, T, params, g.mask_id, block_len)
    assert den.full_passes == G // block_len and den.cached_passes == tr.steps_used - den.full_passes
    model = jot.Model(g, w_gpu, 1, L)
    model.attach_kv_cache()
    jp = jot.Params(params.tau_max, params.tau_min, params.gamma, params.D, params.eps)
    ks = jo.transfer_counts(block_len, T // (G // block_len))
    d_bump = dict(bump_id=bump[0].cuda(), bump_val=bump[1].cuda())
    excused, step_in_block = 0, {}
    for n, (cv, rep, (lo, hi)) in enumerate(zip(tr.canvases, tr.reports, tr.blocks)):
        s = step_in_block.get(lo, 0)
        step_in_block[lo] = s + 1
        x = torch.tensor([cv], dtype=torch.int32, device="cuda")
        st = model.denoise_step_cached(x, lo, hi, refresh=(s == 0), **d_bump)
        jot.accept_freeze(jp, g.mask_id, x, lo, hi, ks[s], st)
        got = x.cpu()[0].tolist()
        want = tr.canvases[n + 1] if n + 1 < len(tr.canvases) else tr.x
        if got == want:
            continue
        A = [i for i in range(lo, hi) if cv[i] == g.mask_id]
        sumexp = st.sumexp.cpu()[0]
        best = max(1.0 / float(sumexp[i]) for i in A)
        for i in A:
            if got[i] == want[i]:
                continue
            near_tau = i in rep.near_margin
            near_gap = float(st.top1[0, i] - st.top2[0, i]) < GAP_TOL
            near_rank = abs(1.0 / float(sumexp[i]) - best) <= REL_TOL * best
            assert near_tau or near_gap or near_rank, (n, i, got[i], want[i], rep.ratio.get(i), rep.tau.get(i))
            excused += 1
    print(f"cached, blocks of {block_len}: {len(tr.canvases)} steps ({den.full_passes} full), {excused} excused")
    assert excused <= 2
    out, used, passes = model.generate(prompt.cuda(), G, T, jp, block_len, kv_cache=True, **d_bump)
    got = out.cpu()[0].tolist()
    assert got[:P] == prompt[0].tolist() and all(t != g.mask_id for t in got) and passes == used[0]
    # always: the library's cached loop equals the host-driven loop over the single-step entry points
    x = torch.tensor([prompt[0].tolist() + [g.mask_id] * G], dtype=torch.int32, device="cuda")
    man_used = 0
    for blk in range(G // block_len):
        lo, hi = P + blk * block_len, P + (blk + 1) * block_len
        for s in range(T // (G // block_len)):
            if int((x[0, lo:hi] == g.mask_id).sum()) == 0:
                break
            st = model.denoise_step_cached(x, lo, hi, refresh=(s == 0), **d_bump)
            jot.accept_freeze(jp, g.mask_id, x, lo, hi, ks[s], st)
            man_used += 1
    assert got == x.cpu()[0].tolist() and used[0] == man_used
    if excused == 0:
        assert used[0] == tr.steps_used and got == tr.x
        print("free-running cached run equals the oracle")
    else:
        print(f"free-running equality with the oracle NOT asserted ({excused} excused decisions in the replay)")
    # without an attached cache the call is refused
    model.detach_kv_cache()
    with pytest.raises(jot.JotError):
        model.generate(prompt.cuda(), G, T, jp, block_len, kv_cache=True, **d_bump)
    model.close()


def test_cached_generation_batch_moves_block_by_block(jot):
    """Three sequences with different thresholds under the cache: each equals its own single-sequence run
    (waiting for the others at a block's end changes nothing), step counts differ, passes = the sum over blocks
    of the slowest sequence's steps; the trace rows are per sequence."""
    g = GEOMS["gqa"]
    P, G, T, B, Lb = 24, 64, 64, 3, 16
    L = P + G
    w_gpu = inputs.weights_to(inputs.model_weights(g, seed=0), "cuda")
    prompt = inputs.prompt(8, B, P, g.vocab, g.mask_id).cuda()
    ids, val = inputs.logit_bump(8, B, L, g.vocab, g.mask_id, hi=14.0, device="cuda")
    model = jot.Model(g, w_gpu, B, L)
    model.attach_kv_cache()
    pl = [jot.Params(0.0, 0.0, 0.5, 8), jot.Params(30.0, 1.0, 0.5, 8), jot.Params(float("inf"), float("inf"), 0.5, 8)]
    out, used, passes, tr = model.generate(prompt, G, T, pl, Lb, bump_id=ids, bump_val=val, kv_cache=True, trace=True)
    assert (out != g.mask_id).all() and torch.equal(out[:, :P], prompt)
    assert used[0] == G // Lb and used[2] == T and used[0] < used[1] < used[2] and passes == T
    for b in range(B):
        o1, u1, p1, t1 = model.generate(prompt[b:b + 1].contiguous(), G, T, pl[b], Lb, bump_id=ids[b:b + 1].contiguous(),
                                        bump_val=val[b:b + 1].contiguous(), kv_cache=True, trace=True)
        assert torch.equal(o1[0], out[b]) and u1[0] == used[b] and p1 == used[b]
        assert torch.equal(t1.exit_step[0], tr.exit_step[b]) and torch.equal(t1.exit_reason[0], tr.exit_reason[b])
        assert torch.equal(t1.n_candidates[:, 0], tr.n_candidates[:, b])
    # sampling under the cache: same call twice gives the same tokens, another seed other tokens
    a = model.generate(prompt, G, T, pl, Lb, bump_id=ids, bump_val=val, kv_cache=True, temperature=0.9, seed=5)
    b2 = model.generate(prompt, G, T, pl, Lb, bump_id=ids, bump_val=val, kv_cache=True, temperature=0.9, seed=5)
    c = model.generate(prompt, G, T, pl, Lb, bump_id=ids, bump_val=val, kv_cache=True, temperature=0.9, seed=6)
    assert torch.equal(a[0], b2[0]) and a[1] == b2[1] and not torch.equal(a[0], c[0])
    model.close()
