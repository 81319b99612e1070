"""GPU parity of the whole denoising step and of Algorithm 1 against the CPU oracle (small models)."""
import math

import numpy as np
import pytest
import torch

from helpers import (GAP_TOL, REL_TOL, assert_generate_matches, compare_stats, oracle_stats_for_rows,
                     replay_trajectory)
from oracle import jot_oracle as jo
from oracle import model_oracle as mo
from paper_2602_11133_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def jot():
    from paper_2602_11133_b200 import jot as binding
    binding._lib()
    return binding


GEOMS = {
    "tiny": inputs.TINY,                                                                  # hd 64, MHA
    "gqa": inputs.ModelGeometry(2, 256, 4, 2, 64, 320, 1032, 1000, 10000.0),              # hd 64, GQA 2:1, odd sizes
    "hd128": inputs.ModelGeometry(2, 256, 2, 1, 128, 704, 2048, 2047, 500000.0),          # hd 128, GQA 2:1
    # feed-forward widths whose gate/up weights form whole 256-row slabs: at 353 .. 384 canvas rows that projection
    # runs two units of work per CTA pair (8 slabs: every pair has a second unit; 9 slabs: one pair has none)
    "ff1024": inputs.ModelGeometry(2, 256, 2, 1, 128, 1024, 2048, 2047, 500000.0),
    "ff1152": inputs.ModelGeometry(2, 256, 4, 2, 64, 1152, 1032, 1000, 10000.0),
}


def masked_canvas(seed, B, P, G, g, p_mask):
    return inputs.partially_masked_canvas(seed, B, P, G, g.vocab, g.mask_id, p_mask)


@pytest.mark.parametrize("name,B,P,G,p_mask", [
    ("tiny", 1, 32, 64, 1.0),          # first step of the tiny workload: whole block masked, one key block
    ("tiny", 2, 60, 140, 0.5),         # L = 200: two key blocks with a ragged tail, two sequences
    ("gqa", 3, 17, 120, 0.7),          # L = 137
    ("hd128", 2, 128, 256, 0.5),       # L = 384: three key blocks
    # canvases of at most 256 rows run the slab projection kernel (weight rows as the MMA's M side)
    ("gqa", 1, 17, 120, 0.7),          # 137 rows: one accumulator of 160 columns, ragged everything
    ("hd128", 1, 64, 192, 0.5),        # 256 rows: the largest canvas on that path, one head per CTA
    ("tiny", 2, 30, 70, 0.6),          # 200 rows, two sequences in one token tile, two heads per CTA
    ("tiny", 1, 8, 24, 1.0),           # 32 rows: the smallest accumulator
    # gate/up as two units per pair (a whole slab, then a third of the tokens of another one)
    ("ff1024", 1, 128, 256, 0.5),      # 384 rows
    ("ff1152", 2, 60, 125, 0.6),       # 370 rows: ragged last token group, two sequences, a pair without a second unit
    ("ff1024", 1, 100, 253, 0.5),      # 353 rows: the smallest canvas on that path
])
def test_denoise_step_matches_oracle(jot, name, B, P, G, p_mask):
    g = GEOMS[name]
    w_cpu = inputs.model_weights(g, seed=0)
    w_gpu = inputs.weights_to(w_cpu, "cuda")
    L = P + G
    tokens = masked_canvas(1, B, P, G, g, p_mask)
    model = jot.Model(g, w_gpu, B, L)
    st = model.denoise_step(tokens.cuda(), P, L)
    torch.cuda.synchronize()
    rows = [(b, i) for b in range(B) for i in range(P, L) if int(tokens[b, i]) == g.mask_id]
    logits = mo.logits(g, w_cpu, tokens, rows=rows)
    want = oracle_stats_for_rows(logits, g.mask_id)
    flat = torch.tensor([b * L + i for b, i in rows])
    pick = lambda t: t.cpu().view(-1)[flat].numpy()
    # a model without the planted bump has many near-equal logits: the argmax must agree wherever the two largest are
    # further apart than twice the largest logit error of this very comparison (never less than the strict 1e-3)
    n, near = compare_stats(pick(st.top1), pick(st.top2), pick(st.sumexp), pick(st.argmax), want, rel=REL_TOL,
                            gap_from_error=True)
    print(f"{name}: {n} rows, {near} with a top-2 gap inside that margin, max |top1 err| "
          f"{max(abs(a - s.m1) for a, s in zip(pick(st.top1), want)):.2e}")
    import helpers
    # outside the margin the argmax was required to be equal; inside it a flip is legitimate, but a broken argmax
    # would flip most of those rows, not a fraction
    assert helpers.LAST_COMPARE["argmax_differs"] <= max(2, helpers.LAST_COMPARE["inside_margin"] // 4)
    # the same against the oracle without any bf16 rounding of activations: the plain float64 network
    plain = oracle_stats_for_rows(mo.logits(g, w_cpu, tokens, rows=rows, round_activations=False), g.mask_id)
    n2, near2 = compare_stats(pick(st.top1), pick(st.top2), pick(st.sumexp), pick(st.argmax), plain, rel=REL_TOL,
                              gap_from_tolerance=True)
    err = max(abs(a - s.m1) / max(abs(s.m1), 1.0) for a, s in zip(pick(st.top1), plain))
    print(f"{name}: against the unrounded float64 oracle: max relative top-1 logit error {err:.2e} (tolerance {REL_TOL:g}), "
          f"{near2} of {n2} rows inside the argmax margin")
    model.close()


@pytest.mark.parametrize("name,B,L", [("tiny", 1, 384), ("hd128", 2, 300), ("gqa", 1, 137)])
def test_attention_with_scores_that_keep_rising(jot, name, B, L):
    """Attention keeps a lazy reference maximum per half row and rescales its accumulator in tensor memory when a
    later key block tops it by more than 2^8.  Ordinary random-init weights never get there, so this model has
    query / key projections 50 times larger: the scores spread over hundreds, every row raises its reference
    several times, and the softmax is nearly one-hot.  Hidden states after one layer against the oracle."""
    g = GEOMS[name]
    w_cpu = inputs.model_weights(g, seed=0, n_layers=1)
    qk_rows = (g.n_q_heads + g.n_kv_heads) * g.head_dim
    big = inputs.normal(11, "big_qk", (qk_rows, g.d_model), 1.0)
    w_cpu["layers"][0]["wqkv"] = torch.cat([big, w_cpu["layers"][0]["wqkv"][qk_rows:]]).contiguous()
    w_gpu = inputs.weights_to(w_cpu, "cuda")
    tokens = inputs.partially_masked_canvas(2, B, L // 3, L - L // 3, g.vocab, g.mask_id, 0.5)
    model = jot.Model(g, w_gpu, B, L)
    st = model.denoise_step(tokens.cuda(), L // 3, L)
    torch.cuda.synchronize()
    rows = [(b, i) for b in range(B) for i in range(L // 3, L) if int(tokens[b, i]) == g.mask_id]
    # how far the scores rise from one key block of 128 to a later one (oracle side, first head)
    lw = w_cpu["layers"][0]
    a = mo._r(mo.rmsnorm(w_cpu["embed"][tokens.long()].double(), lw["attn_norm"], g.rms_eps), True)
    qkv = mo._r(a @ lw["wqkv"].double().T, True)
    q = mo.rope(qkv[..., :g.head_dim].reshape(B, L, 1, g.head_dim), g.rope_theta)
    k = mo.rope(qkv[..., g.n_q_heads * g.head_dim: g.n_q_heads * g.head_dim + g.head_dim].reshape(B, L, 1, g.head_dim), g.rope_theta)
    s = torch.einsum("blhd,bmhd->blm", q, k) / math.sqrt(g.head_dim) * math.log2(math.e)
    if L > 128:
        rise = (s[:, :, 128:].max(dim=-1).values - s[:, :, :128].max(dim=-1).values)
        assert int((rise > 8).sum()) > (L // 4 if L >= 256 else 0), "the case must make the reference maximum move"
    logits = mo.logits(g, w_cpu, tokens, rows=rows)
    want = oracle_stats_for_rows(logits, g.mask_id)
    flat = torch.tensor([b * L + i for b, i in rows])
    pick = lambda t: t.cpu().view(-1)[flat].numpy()
    n, near = compare_stats(pick(st.top1), pick(st.top2), pick(st.sumexp), pick(st.argmax), want, rel=REL_TOL,
                            gap_from_tolerance=True)
    print(f"{name} with rising scores: {n} rows checked, max |top1 err| "
          f"{max(abs(x - w.m1) for x, w in zip(pick(st.top1), want)):.2e}")
    model.close()


def oracle_trajectory(g, w_cpu, prompt_row, G, T, params, block_len, bump=None):
    def logits_fn(x, rows):
        t = torch.tensor([x], dtype=torch.int32)
        l = mo.logits(g, w_cpu, t, rows=[(0, i) for i in rows])
        if bump is not None:
            for r, i in enumerate(rows):
                l[r, int(bump[0][0, i])] += float(bump[1][0, i])
        return {i: l[r].numpy() for r, i in enumerate(rows)}
    return jo.generate(logits_fn, prompt_row, G, T, params, g.mask_id, block_len)


@pytest.mark.parametrize("params,block_len,bumped", [
    (jo.DREAM_DEFAULT, None, False), (jo.LLADA_DEFAULT, 16, False), (jo.JotParams(3.0, 1.0, 0.5, 8), None, False),
    (jo.DREAM_DEFAULT, None, True), (jo.LLADA_DEFAULT, 16, True), (jo.JotParams(60.0, 1.0, 0.7, 8), 32, True)])
def test_tiny_generation_teacher_forced_and_free_running(jot, params, block_len, bumped):
    """Tiny workload: 2 layers, d 256, vocab 4096, prompt 32, 64 masked tokens, up to 64 steps.
    Every step of the oracle's trajectory is replayed on the GPU from the oracle's canvas.

    Without the planted bump a random-init model is almost equally (un)sure everywhere: the masked
    positions' max-probabilities agree to a fraction of a percent, so which ONE the schedule reveals is
    decided below the stated tolerance of the confidences; any pick within that tolerance of the best is
    valid and is counted.  With the bump confidences are spread out and decisions must agree exactly."""
    g = inputs.TINY
    P, G, T = 32, 64, 64
    w_cpu = inputs.model_weights(g, seed=0)
    w_gpu = inputs.weights_to(w_cpu, "cuda")
    prompt = inputs.prompt(0, 1, P, g.vocab, g.mask_id)
    bump = inputs.logit_bump(9, 1, P + G, g.vocab, g.mask_id, hi=12.0) if bumped else None
    tr = oracle_trajectory(g, w_cpu, prompt[0].tolist(), G, T, params, block_len, bump)
    d_bump = dict(bump_id=bump[0].cuda(), bump_val=bump[1].cuda()) if bumped else {}
    model = jot.Model(g, w_gpu, 1, P + G)
    jp = jot.Params(params.tau_max, params.tau_min, params.gamma, params.D, params.eps)
    Lb = block_len or G
    ks = jo.transfer_counts(Lb, T // (G // Lb))
    _, excused = replay_trajectory(jot, model, tr, params, g.mask_id, ks, bump)
    print(f"teacher-forced: {len(tr.canvases)} steps, {excused} excused near-margin differences")
    if bumped:
        assert excused <= 2
        assert tr.steps_used < T          # the bump makes positions exit early
    else:
        # positions are counted, two per swapped pick: at most half of the steps may pick another of the near-equal
        # candidates (measured: 19-28 of 63 steps, depending on the rounding pattern of the attention kernel)
        assert excused <= len(tr.canvases)

    out, used, passes = model.generate(prompt.cuda(), G, T, jp, block_len, **d_bump)
    got = out.cpu()[0].tolist()
    assert got[:P] == prompt[0].tolist() and all(t != g.mask_id for t in got)
    assert 1 <= used[0] <= T and passes == used[0]
    assert_generate_matches(jot, model, prompt, G, T, jp, block_len, g.mask_id, bump, out, used, tr, excused)
    model.close()


def test_generate_batch_equals_separate_runs(jot):
    g = inputs.TINY
    P, G, T, B = 16, 32, 32, 3
    w_gpu = inputs.weights_to(inputs.model_weights(g, seed=0), "cuda")
    prompt = inputs.prompt(5, B, P, g.vocab, g.mask_id).cuda()
    ids, val = inputs.logit_bump(5, B, P + G, g.vocab, g.mask_id, hi=14.0, device="cuda")
    model = jot.Model(g, w_gpu, B, P + G)
    jp = jot.Params(30.0, 1.0, 0.5, 8)
    out, used, passes = model.generate(prompt, G, T, jp, 8, bump_id=ids, bump_val=val)
    assert passes == max(used) or passes >= max(used)
    assert (out != g.mask_id).all() and torch.equal(out[:, :P], prompt)
    for b in range(B):
        o1, u1, _ = model.generate(prompt[b:b + 1].contiguous(), G, T, jp, 8, bump_id=ids[b:b + 1].contiguous(),
                                   bump_val=val[b:b + 1].contiguous())
        assert torch.equal(o1[0], out[b]) and u1[0] == used[b]
    # the planted bump makes sequences stop early at different steps
    assert min(used) < T
    # finished sequences dropping out of the forward pass changes nothing but the work done
    out_nc, used_nc, passes_nc = model.generate(prompt, G, T, jp, 8, bump_id=ids, bump_val=val, compact_finished=False)
    assert torch.equal(out, out_nc) and used == used_nc and passes == passes_nc
    # replaying the step as a CUDA graph changes nothing either
    out_g, used_g, passes_g = model.generate(prompt, G, T, jp, 8, bump_id=ids, bump_val=val, use_cuda_graph=True)
    assert torch.equal(out, out_g) and used == used_g and passes == passes_g
    # same call twice: identical result
    out2, used2, _ = model.generate(prompt, G, T, jp, 8, bump_id=ids, bump_val=val)
    assert torch.equal(out, out2) and used == used2
    # per-sequence parameters: threshold 0 finishes in one step per block, threshold inf takes every step
    pl = [jot.Params(0.0, 0.0, 0.5, 8), jot.Params(float("inf"), float("inf"), 0.5, 8), jp]
    out3, used3, _ = model.generate(prompt, G, T, pl, 8, bump_id=ids, bump_val=val)
    assert used3[0] == G // 8 and used3[1] == T and used3[2] == used[2]
    assert torch.equal(out3[2], out[2])
    model.close()


def test_finished_sequences_drop_out_of_the_batch(jot):
    """Five sequences with very different thresholds finish at different steps; compacting the batch to the
    live sequences must not change any token or step count (rows of a projection do not depend on which
    other rows share the launch)."""
    g = GEOMS["gqa"]
    P, G, T, B = 24, 64, 64, 5
    w_gpu = inputs.weights_to(inputs.model_weights(g, seed=0), "cuda")
    prompt = inputs.prompt(8, B, P, g.vocab, g.mask_id).cuda()
    ids, val = inputs.logit_bump(8, B, P + G, g.vocab, g.mask_id, hi=14.0, device="cuda")
    model = jot.Model(g, w_gpu, B, P + G)
    pl = [jot.Params(0.0, 0.0, 0.5, 8), jot.Params(30.0, 1.0, 0.5, 8), jot.Params(float("inf"), float("inf"), 0.5, 8),
          jot.Params(5.0, 1.0, 0.9, 16), jot.Params(90.0, 1.0, 0.5, 8)]
    on = model.generate(prompt, G, T, pl, 16, bump_id=ids, bump_val=val, compact_finished=True)
    off = model.generate(prompt, G, T, pl, 16, bump_id=ids, bump_val=val, compact_finished=False)
    assert torch.equal(on[0], off[0]) and on[1] == off[1] and on[2] == off[2]
    used = on[1]
    assert used[0] == G // 16 and used[2] == T and len(set(used)) >= 3 and (on[0] != g.mask_id).all()
    model.close()


def test_argument_validation(jot):
    g = inputs.TINY
    w_gpu = inputs.weights_to(inputs.model_weights(g, seed=0, n_layers=1), "cuda")
    model = jot.Model(g, w_gpu, 2, 64)
    tok = torch.zeros(2, 64, dtype=torch.int32, device="cuda")
    with pytest.raises(jot.JotError):
        model.denoise_step(torch.zeros(3, 64, dtype=torch.int32, device="cuda"), 0, 64)     # batch too large
    with pytest.raises(jot.JotError):
        model.denoise_step(torch.zeros(2, 65, dtype=torch.int32, device="cuda"), 0, 65)     # canvas too long
    with pytest.raises(jot.JotError):
        model.denoise_step(tok, 10, 5)
    with pytest.raises(jot.JotError):
        model.generate(tok[:, :8].contiguous(), 30, 30, jot.Params(), 8)                    # block does not divide
    with pytest.raises(TypeError):
        model.denoise_step(tok.cpu(), 0, 64)
    bad = inputs.ModelGeometry(1, 250, 4, 4, 64, 704, 4096, 4095)
    with pytest.raises(jot.JotError):
        jot.Model(bad, w_gpu, 1, 8)
    model.close()


@pytest.mark.parametrize("block_len,T", [(16, 32), (None, 16), (32, 64)])
def test_generation_under_the_fractional_schedule(jot, block_len, T):
    """The adaptive transfer schedule (ceil of what is still masked over the steps the block has left) inside
    jot_generate on the tiny model with the planted bump: teacher-forced replay of the oracle's trajectory, the
    library's loop against the host-driven loop (always), against the oracle when nothing was excused; and the
    runs under the two schedules really differ."""
    g = inputs.TINY
    P, G = 32, 64
    params = jo.LLADA_DEFAULT
    w_cpu = inputs.model_weights(g, seed=0)
    w_gpu = inputs.weights_to(w_cpu, "cuda")
    prompt = inputs.prompt(0, 1, P, g.vocab, g.mask_id)
    bump = inputs.logit_bump(9, 1, P + G, g.vocab, g.mask_id, hi=12.0)

    def logits_fn(x, rows):
        l = mo.logits(g, w_cpu, torch.tensor([x], dtype=torch.int32), rows=[(0, i) for i in rows])
        for r, i in enumerate(rows):
            l[r, int(bump[0][0, i])] += float(bump[1][0, i])
        return {i: l[r].numpy() for r, i in enumerate(rows)}
    tr = jo.generate(logits_fn, prompt[0].tolist(), G, T, params, g.mask_id, block_len, schedule="fractional")
    tr_fixed = jo.generate(logits_fn, prompt[0].tolist(), G, T, params, g.mask_id, block_len)
    Lb = block_len or G
    Tb = T // (G // Lb)
    model = jot.Model(g, w_gpu, 1, P + G)
    rule = lambda cv, lo, hi, s: jo.fractional_transfer_count(sum(1 for i in range(lo, hi) if cv[i] == g.mask_id), Tb - s)
    steps, excused = replay_trajectory(jot, model, tr, params, g.mask_id, rule, bump)
    assert excused <= 2
    jp = jot.Params(params.tau_max, params.tau_min, params.gamma, params.D, params.eps, schedule=jot.SCHEDULE_FRACTIONAL)
    d_bump = dict(bump_id=bump[0].cuda(), bump_val=bump[1].cuda())
    out, used, passes = model.generate(prompt.cuda(), G, T, jp, block_len, **d_bump)
    got = out.cpu()[0].tolist()
    assert all(t != g.mask_id for t in got) and used[0] <= T
    from helpers import manual_generate
    man, man_used = manual_generate(jot, model, prompt[0].tolist(), G, T, jp, block_len, g.mask_id, bump, fractional=True)
    assert got == man and used[0] == man_used
    if excused == 0:
        assert used[0] == tr.steps_used and got == tr.x
    print(f"fractional schedule, blocks of {Lb}, {Tb} steps each: {tr.steps_used} steps (fixed table: {tr_fixed.steps_used}), "
          f"{excused} excused; oracle equality {'asserted' if excused == 0 else 'NOT asserted'}")
    assert tr.steps_used != tr_fixed.steps_used or tr.x != tr_fixed.x or T == G      # the schedules differ once exits run ahead
    with pytest.raises(jot.JotError):
        model.generate(prompt.cuda(), G, T, jot.Params(schedule=7), block_len)
    # under the block-wise KV cache (all sequences in lock-step) the same rule applies
    model.attach_kv_cache()
    o1 = model.generate(prompt.cuda(), G, T, jp, block_len, kv_cache=True, **d_bump)
    assert (o1[0] != g.mask_id).all() and o1[1][0] <= T
    model.close()


def test_token_id_outside_the_vocabulary_is_reported_not_read(jot):
    """A token id outside [0, vocab) must come back as an argument error: the row is embedded as token 0 (no read
    leaves the embedding matrix), the status word records it, and the model works again on corrected input."""
    g = inputs.TINY
    w_gpu = inputs.weights_to(inputs.model_weights(g, seed=0, n_layers=1), "cuda")
    model = jot.Model(g, w_gpu, 2, 64)
    good = inputs.partially_masked_canvas(3, 2, 16, 48, g.vocab, g.mask_id, 0.5).cuda()
    ref = model.denoise_step(good, 16, 64)
    for bad_id in (g.vocab, g.vocab + 12345, -1, -2 ** 31):
        bad = good.clone()
        bad[1, 3] = bad_id
        with pytest.raises(jot.JotError) as e:
            model.denoise_step(bad, 16, 64)
        assert e.value.status == -1
        again = model.denoise_step(good, 16, 64)                   # the report was cleared; same result as before
        assert torch.equal(again.top1, ref.top1) and torch.equal(again.argmax, ref.argmax)
    with pytest.raises(jot.JotError) as e:                         # the generate loop reports it the same way
        model.generate(torch.full((1, 8), g.vocab, dtype=torch.int32, device="cuda"), 8, 8, jot.Params())
    assert e.value.status == -1
    out, used, _ = model.generate(good[:1, :16].contiguous(), 16, 16, jot.Params())
    assert (out != g.mask_id).all()
    model.close()


def test_steps_without_a_synchronisation_per_call(jot):
    """jot_set_sync(0): the single-step calls only enqueue; the status is read when the caller asks.  Results are
    those of the synchronous calls, and a failure that happened in between is still reported by jot_read_status."""
    g = inputs.TINY
    w_gpu = inputs.weights_to(inputs.model_weights(g, seed=0), "cuda")
    model = jot.Model(g, w_gpu, 1, 96)
    x = inputs.partially_masked_canvas(4, 1, 32, 64, g.vocab, g.mask_id, 0.6).cuda()
    ref = model.denoise_step(x, 32, 96)
    model.set_sync(False)
    outs = [model.denoise_step(x, 32, 96) for _ in range(5)]       # five steps in flight, no host round trip
    model.read_status()
    for o in outs:
        assert torch.equal(o.top1, ref.top1) and torch.equal(o.sumexp, ref.sumexp) and torch.equal(o.argmax, ref.argmax)
    bad = x.clone()
    bad[0, 0] = g.vocab
    model.denoise_step(bad, 32, 96)                                # returns ok: nothing has been read yet
    with pytest.raises(jot.JotError) as e:
        model.read_status()
    assert e.value.status == -1
    model.read_status()                                            # cleared
    model.set_sync(True)
    model.close()


# ---------------------------------------------------------------- sampling-based finalisation (Section 4.1)
def sampled_oracle_trajectory(g, w_cpu, prompt_row, G, T, params, block_len, bump, temperature, seed, seq_index=0,
                              bump_row=0):
    """Oracle run with sampled finalisation; also returns the logits rows of every step, for the draw margins."""
    seen = []

    def logits_fn(x, rows):
        t = torch.tensor([x], dtype=torch.int32)
        l = mo.logits(g, w_cpu, t, rows=[(0, i) for i in rows])
        for r, i in enumerate(rows):
            l[r, int(bump[0][bump_row, i])] += float(bump[1][bump_row, i])
        out = {i: l[r].numpy() for r, i in enumerate(rows)}
        seen.append(out)
        return out
    tr = jo.generate(logits_fn, prompt_row, G, T, params, g.mask_id, block_len, sampling=(temperature, seed),
                     seq_index=seq_index)
    return tr, seen


@pytest.mark.parametrize("params,block_len,temperature", [
    (jo.LLADA_DEFAULT, 16, 0.7), (jo.DREAM_DEFAULT, None, 1.0), (jo.JotParams(60.0, 1.0, 0.7, 8), 32, 1.5)])
def test_tiny_generation_with_sampled_finalisation(jot, params, block_len, temperature):
    """Teacher-forced replay of the oracle's sampled trajectory (each step: denoise with the step's stream,
    acceptance writes the drawn tokens), then the free-running loop with the same seed."""
    g = inputs.TINY
    P, G, T, seed = 32, 64, 64, 0xC0FFEE1234
    L = P + G
    w_cpu = inputs.model_weights(g, seed=0)
    w_gpu = inputs.weights_to(w_cpu, "cuda")
    prompt = inputs.prompt(0, 1, P, g.vocab, g.mask_id)
    bump = inputs.logit_bump(9, 1, L, g.vocab, g.mask_id, hi=12.0)
    tr, seen = sampled_oracle_trajectory(g, w_cpu, prompt[0].tolist(), G, T, params, block_len, bump, temperature, seed)
    d_bump = dict(bump_id=bump[0].cuda(), bump_val=bump[1].cuda())
    model = jot.Model(g, w_gpu, 1, L)
    jp = jot.Params(params.tau_max, params.tau_min, params.gamma, params.D, params.eps)
    Lb = block_len or G
    ks = jo.transfer_counts(Lb, T // (G // Lb))
    excused = sampled_not_argmax = 0
    step_in_block = {}
    for n, (cv, rep, (lo, hi)) in enumerate(zip(tr.canvases, tr.reports, tr.blocks)):
        s = step_in_block.get(lo, 0)
        step_in_block[lo] = s + 1
        x = torch.tensor([cv], dtype=torch.int32, device="cuda")
        st = model.denoise_step(x, lo, hi, sampling=jot.Sampling(temperature, seed, n), **d_bump)
        jot.accept_freeze(jp, g.mask_id, x, lo, hi, ks[s], jot.Stats(st.top1, st.top2, st.sumexp, st.sampled))
        got = x.cpu()[0].tolist()
        want = tr.canvases[n + 1] if n + 1 < len(tr.canvases) else tr.x
        sumexp = st.sumexp.cpu()[0]
        A = [i for i in range(lo, hi) if cv[i] == g.mask_id]
        best = max(1.0 / float(sumexp[i]) for i in A)
        am = st.argmax.cpu()[0]
        for i in A:
            if want[i] != g.mask_id:
                sampled_not_argmax += int(want[i] != int(am[i]))
            if got[i] == want[i]:
                continue
            scale = max(abs(float(st.top1[0, i])), 1.0)
            if got[i] != g.mask_id and want[i] != g.mask_id:          # both finalised it: the draw differs
                _, gap = jo.sample_tokens_fast(seen[n][i], g.mask_id, temperature, seed, n, i)
                assert gap <= 2 * REL_TOL * scale / temperature, (n, i, got[i], want[i], gap)
            else:                                                      # the decision differs
                near_tau = i in rep.near_margin
                near_rank = abs(1.0 / float(sumexp[i]) - best) <= REL_TOL * best
                assert near_tau or near_rank, (n, i, got[i], want[i], rep.ratio.get(i), rep.tau.get(i))
            excused += 1
    print(f"sampled, T={temperature}: {len(tr.canvases)} steps, {excused} excused, "
          f"{sampled_not_argmax} finalised tokens differ from the argmax")
    assert excused <= 2
    out, used, passes = model.generate(prompt.cuda(), G, T, jp, block_len, temperature=temperature, seed=seed, **d_bump)
    got = out.cpu()[0].tolist()
    assert got[:P] == prompt[0].tolist() and all(t != g.mask_id for t in got) and passes == used[0]
    assert_generate_matches(jot, model, prompt, G, T, jp, block_len, g.mask_id, bump, out, used, tr, excused,
                            label="sampled: ", sampling=(temperature, seed))
    # temperature 0 is the argmax path whatever the seed
    o0, u0, _ = model.generate(prompt.cuda(), G, T, jp, block_len, temperature=0.0, seed=seed, **d_bump)
    o1, u1, _ = model.generate(prompt.cuda(), G, T, jp, block_len, **d_bump)
    assert torch.equal(o0, o1) and u0 == u1
    model.close()


def test_sampled_generation_batch_graph_and_compaction(jot):
    """Under sampling each sequence's stream is keyed by its own flat canvas positions and the number of
    forward passes so far: batch row b equals the oracle run with seq_index = b, and neither the CUDA-graph
    replay nor dropping finished sequences out of the batch changes a token."""
    g = inputs.TINY
    P, G, T, B, seed, temperature = 16, 32, 32, 3, 777, 0.8
    L = P + G
    w_cpu = inputs.model_weights(g, seed=0)
    w_gpu = inputs.weights_to(w_cpu, "cuda")
    prompt = inputs.prompt(5, B, P, g.vocab, g.mask_id)
    bump = inputs.logit_bump(5, B, L, g.vocab, g.mask_id, hi=14.0)
    d_bump = dict(bump_id=bump[0].cuda(), bump_val=bump[1].cuda())
    model = jot.Model(g, w_gpu, B, L)
    params = jo.JotParams(30.0, 1.0, 0.5, 8)
    jp = jot.Params(30.0, 1.0, 0.5, 8)
    out, used, passes = model.generate(prompt.cuda(), G, T, jp, 8, temperature=temperature, seed=seed, **d_bump)
    assert (out != g.mask_id).all() and len(set(used)) >= 1 and passes == max(used)
    for kw in (dict(compact_finished=False), dict(use_cuda_graph=True), dict(use_cuda_graph=True, compact_finished=False)):
        o, u, p = model.generate(prompt.cuda(), G, T, jp, 8, temperature=temperature, seed=seed, **d_bump, **kw)
        assert torch.equal(o, out) and u == used and p == passes, kw
    o2, _, _ = model.generate(prompt.cuda(), G, T, jp, 8, temperature=temperature, seed=seed + 1, **d_bump)
    assert not torch.equal(o2, out)
    o_arg, _, _ = model.generate(prompt.cuda(), G, T, jp, 8, **d_bump)
    assert not torch.equal(o_arg, out)
    agree = 0
    for b in range(B):
        tr, seen = sampled_oracle_trajectory(g, w_cpu, prompt[b].tolist(), G, T, params, 8, bump, temperature, seed,
                                             seq_index=b, bump_row=b)
        # the smallest margin of anything that decided this run: if none is tight the runs must be identical
        tight = any(rep.near_margin for rep in tr.reports)
        for n, rep in enumerate(tr.reports):
            for i in set(rep.exited) | set(rep.scheduled):
                _, gap = jo.sample_tokens_fast(seen[n][i], g.mask_id, temperature, seed, n, b * L + i)
                tight = tight or gap < 0.05
            p1 = sorted((jo.row_stats(seen[n][i], g.mask_id).p1 for i in seen[n]), reverse=True)
            tight = tight or (len(p1) > 1 and p1[0] - p1[1] < 2e-2 * p1[0])
        same = out.cpu()[b].tolist() == tr.x and used[b] == tr.steps_used
        agree += int(same)
        assert same or tight, b
    print(f"sampled batch: {agree} of {B} sequences agree with the oracle token for token")
    model.close()


def test_generation_trace_matches_oracle(jot):
    """Exit step and exit reason of every position, and the mean confidence ratio of every step (the
    quantities behind the paper's confidence-dynamics plots), against the oracle's trajectory."""
    g = inputs.TINY
    P, G, T, block_len = 32, 64, 64, 16
    L = P + G
    params = jo.LLADA_DEFAULT
    w_cpu = inputs.model_weights(g, seed=0)
    w_gpu = inputs.weights_to(w_cpu, "cuda")
    prompt = inputs.prompt(0, 1, P, g.vocab, g.mask_id)
    bump = inputs.logit_bump(9, 1, L, g.vocab, g.mask_id, hi=12.0)
    tr = oracle_trajectory(g, w_cpu, prompt[0].tolist(), G, T, params, block_len, bump)
    model = jot.Model(g, w_gpu, 2, L)
    jp = jot.Params(params.tau_max, params.tau_min, params.gamma, params.D, params.eps)
    ks = jo.transfer_counts(block_len, T // (G // block_len))
    _, excused = replay_trajectory(jot, model, tr, params, g.mask_id, ks, bump)
    out, used, passes, trace = model.generate(prompt.cuda(), G, T, jp, block_len, bump_id=bump[0].cuda(),
                                              bump_val=bump[1].cuda(), trace=True)
    es, er = trace.exit_step.cpu()[0].tolist(), trace.exit_reason.cpu()[0].tolist()
    mr, nc = trace.mean_ratio.cpu()[:, 0].tolist(), trace.n_candidates.cpu()[:, 0].tolist()
    # invariants that hold whatever the trajectory
    assert all(e == 0 and r == 0 for e, r in zip(es[:P], er[:P]))
    assert all(1 <= e <= used[0] and r in (1, 2, 3) for e, r in zip(es[P:], er[P:]))
    assert all(n == 0 and m == 0.0 for n, m in zip(nc[used[0]:], mr[used[0]:])) and all(n > 0 for n in nc[:used[0]])
    assert sum(1 for r in er[P:] if r & 2) >= used[0] - (G // block_len)      # the schedule reveals one per step
    assert_generate_matches(jot, model, prompt, G, T, jp, block_len, g.mask_id, bump, out, used, tr, excused,
                            label="trace: ")
    if excused == 0:
        assert es == tr.exit_step
        want_reason = [0] * L
        for rep in tr.reports:
            for i in rep.exited:
                want_reason[i] |= 1
            for i in rep.scheduled:
                want_reason[i] |= 2
        assert er == want_reason
        for n, rep in enumerate(tr.reports):
            assert nc[n] == len(rep.ratio)
            want = sum(rep.ratio.values()) / len(rep.ratio)
            # r = 1 / (exp(m2 - m1) + eps S): a logit error e changes ln r by up to ~e * r / (r + 1) per term
            scale = 12.0                      # magnitude of the logits with the planted bump
            assert abs(math.log(mr[n]) - math.log(want)) <= 2 * REL_TOL * scale, (n, mr[n], want)
    print(f"trace: {used[0]} steps, {excused} excused; mean r first/last step {mr[0]:.3g} / {mr[used[0] - 1]:.3g}")
    # the trace does not depend on batch neighbours, compaction or graph replay
    prompt2 = torch.cat([prompt, inputs.prompt(3, 1, P, g.vocab, g.mask_id)]).cuda()
    bid2 = torch.cat([bump[0], bump[0]]).cuda()
    bval2 = torch.cat([bump[1], bump[1] * 0.5]).cuda()
    for kw in (dict(), dict(compact_finished=False), dict(use_cuda_graph=True)):
        o2, u2, _, t2 = model.generate(prompt2, G, T, jp, block_len, bump_id=bid2, bump_val=bval2, trace=True, **kw)
        assert torch.equal(o2[0], out[0]) and u2[0] == used[0]
        assert torch.equal(t2.exit_step[0], trace.exit_step[0]) and torch.equal(t2.exit_reason[0], trace.exit_reason[0])
        assert torch.equal(t2.mean_ratio[:, 0], trace.mean_ratio[:, 0])
        assert torch.equal(t2.n_candidates[:, 0], trace.n_candidates[:, 0])
    model.close()


def test_generation_under_the_global_early_commit_gate(jot):
    """The global early-commit rule (Section 2) inside Algorithm 1 on the tiny model with the planted bump:
    a threshold nothing clears gives plain schedule decoding (T steps), one everything clears commits a block
    per step, and a threshold in between reproduces the oracle's trajectory (tokens and step count)."""
    g = inputs.TINY
    P, G, T, Lb = 32, 64, 64, 16
    w_cpu = inputs.model_weights(g, seed=0)
    w_gpu = inputs.weights_to(w_cpu, "cuda")
    prompt = inputs.prompt(0, 1, P, g.vocab, g.mask_id)
    bump = inputs.logit_bump(9, 1, P + G, g.vocab, g.mask_id, hi=12.0)
    d_bump = dict(bump_id=bump[0].cuda(), bump_val=bump[1].cuda())
    model = jot.Model(g, w_gpu, 1, P + G)
    _, used, _ = model.generate(prompt.cuda(), G, T, jot.Params(gate=jot.GATE_GLOBAL_GAP, gap_threshold=1e30), Lb, **d_bump)
    assert used[0] == T
    out, used, _ = model.generate(prompt.cuda(), G, T, jot.Params(gate=jot.GATE_GLOBAL_GAP, gap_threshold=-1e30), Lb, **d_bump)
    assert used[0] == G // Lb and (out != g.mask_id).all()
    # the blocks' mean gaps differ (random bumps): a threshold between them commits some blocks at once and leaves
    # the others to the schedule
    for thr in (4.0, 4.5, 5.0, 5.5, 6.0, 6.5, 7.0, 8.0):
        tr = oracle_trajectory(g, w_cpu, prompt[0].tolist(), G, T, jo.JotParams(gate="globalgap", gap_threshold=thr), Lb, bump)
        if G // Lb < tr.steps_used < T:
            break
    assert G // Lb < tr.steps_used < T                      # the gate fired somewhere, but not everywhere
    out, used, _ = model.generate(prompt.cuda(), G, T, jot.Params(gate=jot.GATE_GLOBAL_GAP, gap_threshold=thr), Lb, **d_bump)
    # the mean gap of a step is within the logit tolerance of the oracle's; a step whose mean sits that close to
    # the threshold may legitimately go either way, every other step must agree
    # (2-layer model: the measured logit error is ~2e-3, so 0.02 on a mean of gaps is a wide berth)
    margins = [abs(float(np.mean(gaps)) - thr) for gaps in step_gaps(tr, g, w_cpu, bump)]
    print(f"threshold {thr}: oracle used {tr.steps_used} steps, smallest |mean gap - threshold| {min(margins):.3f}")
    from helpers import manual_generate
    jp_gap = jot.Params(gate=jot.GATE_GLOBAL_GAP, gap_threshold=thr)
    man, man_used = manual_generate(jot, model, prompt[0].tolist(), G, T, jp_gap, Lb, g.mask_id, bump)
    assert out.cpu()[0].tolist() == man and used[0] == man_used        # always: library loop == host-driven loop
    if min(margins) >= 0.02:
        assert used[0] == tr.steps_used and out.cpu()[0].tolist() == tr.x
        print("free-running run equals the oracle")
    else:
        print("free-running equality with the oracle NOT asserted: a step's mean gap sits within 0.02 of the threshold")
    model.close()


def step_gaps(tr, g, w_cpu, bump):
    """Top-2 logit gaps of the candidates at every step of an oracle trajectory."""
    out = []
    for x, (lo, hi) in zip(tr.canvases, tr.blocks):
        rows = [i for i in range(lo, hi) if x[i] == g.mask_id]
        l = mo.logits(g, w_cpu, torch.tensor([x], dtype=torch.int32), rows=[(0, i) for i in rows])
        for r, i in enumerate(rows):
            l[r, int(bump[0][0, i])] += float(bump[1][0, i])
        out.append([float(st.m1 - st.m2) for st in (jo.row_stats(l[r].numpy(), g.mask_id) for r in range(len(rows)))])
    return out
