"""Parity on the other workload shapes (reduced depth, full widths): Dream-7B geometry (28 query / 4 KV heads,
d 3584, ff 18944, vocab 152064, batch 8, canvas 512) and LLaDA-8B geometry decoded block-semi-autoregressively
with the planted bump (batch > 1, per-sequence block pointers)."""
import pytest
import torch

import helpers
from helpers import GAP_TOL, REL_TOL, compare_stats, oracle_stats_for_rows, replay_trajectory
from oracle import jot_oracle as jo
from oracle import model_oracle as mo
from paper_2602_11133_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def jot():
    from paper_2602_11133_b200 import jot as binding
    binding._lib()
    return binding


def test_dream_shape_step_two_layers(jot):
    g = inputs.DREAM_7B
    B, P, G = 8, 256, 256
    L = P + G
    w_gpu = inputs.model_weights(g, seed=0, device="cuda", n_layers=2)
    model = jot.Model(g, w_gpu, B, L)
    tokens = inputs.partially_masked_canvas(2, B, P, G, g.vocab, g.mask_id, 0.5, device="cuda")
    bid, bval = inputs.logit_bump(2, B, L, g.vocab, g.mask_id, 12.0, device="cuda")
    st = model.denoise_step(tokens, P, L, bump_id=bid, bump_val=bval)
    torch.cuda.synchronize()
    tok = tokens.cpu()
    rows = [(b, i) for b in range(B) for i in range(P, L) if int(tok[b, i]) == g.mask_id]
    assert 900 < len(rows) < 1150
    # the oracle runs the body on sequences 0 and 7 only (sequences are independent) and the head on 24 rows
    w_cpu = inputs.weights_to(w_gpu, "cpu")
    picks = []
    for b in (0, B - 1):
        h = mo.hidden_states(g, w_cpu, tok[b:b + 1])
        mine = [i for bb, i in rows if bb == b]
        sel = mine[:: max(1, len(mine) // 12)][:12]
        flat = torch.tensor([b * L + i for i in sel])
        logits = mo.lm_head_logits(h[0, torch.tensor(sel)], w_cpu["lm_head"], bid.cpu().view(-1)[flat],
                                   bval.cpu().view(-1)[flat])
        picks.append((flat, oracle_stats_for_rows(logits, g.mask_id)))
    for flat, want in picks:
        pick = lambda t: t.cpu().view(-1)[flat].numpy()
        n, near = compare_stats(pick(st.top1), pick(st.top2), pick(st.sumexp), pick(st.argmax), want, rel=REL_TOL)
        assert n == 12 and near <= 1
    check_against_unrounded_oracle(g, w_cpu, tok, 0, P, L, rows, bid, bval, st, "dream shape, 2 layers")
    model.close()


def check_against_unrounded_oracle(g, w_cpu, tok, b, P, L, rows, bid, bval, st, label):
    """The same statistics against the oracle WITHOUT any bf16 rounding of activations (the plain float64
    definition of the network), at the stated 2e-2 of the logit scale: shows what the rounding contract of the
    other comparison does and does not absorb."""
    h = mo.hidden_states(g, w_cpu, tok[b:b + 1], round_activations=False)
    mine = [i for bb, i in rows if bb == b]
    sel = mine[:: max(1, len(mine) // 12)][:12]
    flat = torch.tensor([b * L + i for i in sel])
    logits = mo.lm_head_logits(h[0, torch.tensor(sel)], w_cpu["lm_head"], bid.cpu().view(-1)[flat], bval.cpu().view(-1)[flat])
    want = oracle_stats_for_rows(logits, g.mask_id)
    pick = lambda t: t.cpu().view(-1)[flat].numpy()
    n, near = compare_stats(pick(st.top1), pick(st.top2), pick(st.sumexp), pick(st.argmax), want, rel=REL_TOL,
                            gap_from_tolerance=True)
    err = max(abs(a - s.m1) / max(abs(s.m1), 1.0) for a, s in zip(pick(st.top1), want))
    print(f"{label}: against the unrounded float64 oracle, max relative top-1 logit error {err:.2e} over {n} rows "
          f"(tolerance {REL_TOL:g}); {near} rows inside the argmax margin")


def test_llada_long_generation_shape_step_two_layers(jot):
    """The long-generation workload's launch shape at reduced depth: LLaDA-8B widths, batch 16, prompt 192 + 512
    masked tokens (canvas 704, 11264 rows through the CTA-pair projections), statistics for the first block of
    32 of every sequence (512 active rows), planted bump.  The oracle runs sequences 0, 7 and 15."""
    g = inputs.LLADA_8B
    B, P, G, Lb = 16, 192, 512, 32
    L = P + G
    w_gpu = inputs.model_weights(g, seed=0, device="cuda", n_layers=2)
    model = jot.Model(g, w_gpu, B, L)
    prompt = inputs.prompt(5, B, P, g.vocab, g.mask_id)
    tokens = torch.cat([prompt, torch.full((B, G), g.mask_id, dtype=torch.int32)], dim=1).cuda()
    bid, bval = inputs.logit_bump(5, B, L, g.vocab, g.mask_id, 12.0, device="cuda")
    st = model.denoise_step(tokens, P, P + Lb, bump_id=bid, bump_val=bval)
    torch.cuda.synchronize()
    w_cpu = inputs.weights_to(w_gpu, "cpu")
    tok = tokens.cpu()
    n_near = n_differ = 0
    for b in (0, 7, B - 1):
        h = mo.hidden_states(g, w_cpu, tok[b:b + 1])
        sel = list(range(P, P + Lb, 3))                                    # 11 of the block's 32 rows
        flat = torch.tensor([b * L + i for i in sel])
        logits = mo.lm_head_logits(h[0, torch.tensor(sel)], w_cpu["lm_head"], bid.cpu().view(-1)[flat],
                                   bval.cpu().view(-1)[flat])
        want = oracle_stats_for_rows(logits, g.mask_id)
        pick = lambda t: t.cpu().view(-1)[flat].numpy()
        # two layers at these widths leave ~0.02 of bf16 noise on a logit: values are held to half the stated
        # tolerance, and two logits closer than twice that may swap places (counted)
        n, near = compare_stats(pick(st.top1), pick(st.top2), pick(st.sumexp), pick(st.argmax), want, rel=REL_TOL / 2,
                                gap_from_tolerance=True)
        assert n == len(sel)
        n_near += near
        n_differ += helpers.LAST_COMPARE["argmax_differs"]
    # What the arithmetic predicts: the margin is 2 * 0.01 * 5.6 = 0.11 logits; where the planted bump loses (about
    # half of the rows) the two largest of 126k Gaussian logits (sigma 1.28) lie ~0.26 apart on average, so about
    # 0.5 * (1 - exp(-0.11 / 0.26)) = 17 % of the rows, 5-6 of 33, fall inside it.  Inside the margin the argmax only
    # flips when the noise (~0.02) exceeds the actual gap: a fifth of those.  Caps at twice the prediction.
    print(f"{n_near} of 33 sampled rows had a top-2 gap inside the margin; argmax actually differed on {n_differ}")
    assert n_near <= 11 and n_differ <= 3
    rows = [(0, i) for i in range(P, P + Lb)]
    check_against_unrounded_oracle(g, w_cpu, tok, 0, P, L, rows, bid, bval, st, "LLaDA shape, batch 16, 2 layers")
    model.close()


def test_llada_shape_block_generation_with_bump(jot):
    """Sixteen sequences (the long-generation workload's batch), prompt 64 + 96 masked tokens in 3 blocks of 32,
    LLaDA defaults, planted bump; sequences 0 and 15 are replayed against the oracle.
    Each sequence's oracle trajectory (Algorithm 1) is replayed step by step on the GPU; then the GPU's
    free-running batched jot_generate is checked for the loop invariants and compared with the oracle's
    step counts (two bf16 layers at these widths move logits by ~1e-2, so a free run may part ways with the
    oracle at a decision inside that margin; the replay is the exact comparison)."""
    g = inputs.LLADA_8B
    B, P, G, Lb, T = 16, 64, 96, 32, 96
    L = P + G
    w_gpu = inputs.model_weights(g, seed=0, device="cuda", n_layers=2)
    w_cpu = inputs.weights_to(w_gpu, "cpu")
    model = jot.Model(g, w_gpu, B, L)
    prompt = inputs.prompt(3, B, P, g.vocab, g.mask_id)
    bid, bval = inputs.logit_bump(3, B, L, g.vocab, g.mask_id, 12.0)
    params = jo.LLADA_DEFAULT
    jp = jot.Params(params.tau_max, params.tau_min, params.gamma, params.D, params.eps)
    out, used, passes = model.generate(prompt.cuda(), G, T, jp, Lb, bump_id=bid.cuda(), bump_val=bval.cuda())
    out = out.cpu()
    assert (out != g.mask_id).all() and torch.equal(out[:, :P], prompt) and passes == max(used)
    w_lm = w_cpu["lm_head"].double()
    ks = jo.transfer_counts(Lb, T // (G // Lb))
    assert len(set(used)) >= 4                       # the bump staggers the sequences: per-sequence block pointers at work
    for b in (0, B - 1):
        def logits_fn(x, rows, b=b):
            h = mo.hidden_states(g, w_cpu, torch.tensor([x], dtype=torch.int32))
            l = h[0, torch.tensor(rows)] @ w_lm.T
            for r, i in enumerate(rows):
                l[r, int(bid[b, i])] += float(bval[b, i])
            return {i: l[r].numpy() for r, i in enumerate(rows)}
        tr = jo.generate(logits_fn, prompt[b].tolist(), G, T, params, g.mask_id, Lb)
        assert tr.steps_used < T            # the bump makes positions exit early, at staggered steps
        steps, excused = replay_trajectory(jot, model, tr, params, g.mask_id, ks,
                                           (bid[b:b + 1].contiguous(), bval[b:b + 1].contiguous()), from_tolerance=True)
        same = sum(int(out[b, i]) == tr.x[i] for i in range(L))
        print(f"sequence {b}: oracle {tr.steps_used} steps, free-running GPU {used[b]} steps, {same}/{L} final tokens "
              f"equal; replay of {steps} steps: {excused} differences, all inside the tolerance margin")
        assert excused <= max(3, steps // 5)        # positions, and a swapped pick of the schedule counts twice
        assert abs(used[b] - tr.steps_used) <= 6       # once one token differs the free runs are different samples
    model.close()


def test_dream_shape_generation_with_a_sweep_setting(jot):
    """Algorithm 1 at Dream widths (2 layers, GQA 28 / 4, vocabulary 152064) under one setting of the paper's
    hyper-parameter sweep, (tau_max, gamma, D) = (120, 0.3, 8): two sequences, prompt 32 + 32 masked tokens in one
    block, planted bump; sequence 0 is replayed against the oracle and the library's loop is held against the
    host-driven loop."""
    from helpers import manual_generate
    g = inputs.DREAM_7B
    B, P, G, T = 2, 32, 32, 32
    L = P + G
    w_gpu = inputs.model_weights(g, seed=0, device="cuda", n_layers=2)
    w_cpu = inputs.weights_to(w_gpu, "cpu")
    model = jot.Model(g, w_gpu, B, L)
    prompt = inputs.prompt(4, B, P, g.vocab, g.mask_id)
    bid, bval = inputs.logit_bump(4, B, L, g.vocab, g.mask_id, 12.0)
    params = jo.JotParams(120.0, 1.0, 0.3, 8)
    jp = jot.Params(params.tau_max, params.tau_min, params.gamma, params.D, params.eps)
    out, used, passes = model.generate(prompt.cuda(), G, T, jp, None, bump_id=bid.cuda(), bump_val=bval.cuda())
    out = out.cpu()
    assert (out != g.mask_id).all() and torch.equal(out[:, :P], prompt) and passes == max(used)
    w_lm = w_cpu["lm_head"].double()

    def logits_fn(x, rows):
        h = mo.hidden_states(g, w_cpu, torch.tensor([x], dtype=torch.int32))
        l = h[0, torch.tensor(rows)] @ w_lm.T
        for r, i in enumerate(rows):
            l[r, int(bid[0, i])] += float(bval[0, i])
        return {i: l[r].numpy() for r, i in enumerate(rows)}
    tr = jo.generate(logits_fn, prompt[0].tolist(), G, T, params, g.mask_id, None)
    assert tr.steps_used < T
    ks = jo.transfer_counts(G, T)
    bump0 = (bid[:1].contiguous(), bval[:1].contiguous())
    steps, excused = replay_trajectory(jot, model, tr, params, g.mask_id, ks, bump0, from_tolerance=True)
    assert excused <= max(2, steps // 5)
    man, man_used = manual_generate(jot, model, prompt[0].tolist(), G, T, jp, None, g.mask_id, bump0)
    one, used1, _ = model.generate(prompt[:1].contiguous().cuda(), G, T, jp, None, bump_id=bump0[0].cuda(),
                                   bump_val=bump0[1].cuda())
    assert one.cpu()[0].tolist() == man and used1[0] == man_used           # always
    same = sum(int(a == b) for a, b in zip(man, tr.x))
    print(f"dream widths, (120, 0.3, 8): oracle {tr.steps_used} steps, GPU {man_used}; replay of {steps} steps: {excused} "
          f"excused; {same}/{L} final tokens equal; oracle equality {'asserted' if excused == 0 else 'NOT asserted'}")
    if excused == 0:
        assert man == tr.x and man_used == tr.steps_used
    model.close()


@pytest.mark.parametrize("name,B,L", [("dream", 8, 512), ("dream", 8, 256), ("dream", 3, 512), ("llada", 16, 704)])
def test_copies_of_one_sequence_get_identical_statistics(jot, name, B, L):
    """Sequences are independent, so B copies of one canvas must come out bit for bit alike, run after run.  With
    several work items per attention CTA (896 / 448 / 336 / 3072 items on 148 CTAs here) any hand-over between
    items that goes wrong shows up as a copy that differs; it needs no oracle and covers every row of every copy."""
    g = inputs.DREAM_7B if name == "dream" else inputs.LLADA_8B
    P = L // 2
    w_gpu = inputs.model_weights(g, seed=0, device="cuda", n_layers=1)
    model = jot.Model(g, w_gpu, B, L)
    one = inputs.partially_masked_canvas(5, 1, P, L - P, g.vocab, g.mask_id, 0.5, device="cuda")
    tokens = one.repeat(B, 1).contiguous()
    first = None
    for rep in range(3):
        st = model.denoise_step(tokens, P, L)
        torch.cuda.synchronize()
        active = tokens[0] == g.mask_id
        active[:P] = False
        assert int(active.sum()) > 20
        got = [t[:, active].clone() for t in (st.top1, st.top2, st.sumexp, st.argmax)]
        assert all(torch.isfinite(t).all() for t in got[:3])
        for t in got:
            assert (t == t[0:1]).all(), f"{name} B={B} L={L} run {rep}: a copy differs from copy 0"
        if first is None:
            first = got
        else:
            assert all((a == b).all() for a, b in zip(got, first)), f"{name} B={B} L={L}: run {rep} differs from run 0"
    model.close()
