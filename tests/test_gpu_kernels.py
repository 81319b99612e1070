"""GPU parity tests of the individual kernels against the CPU oracle, through the C ABI."""
import math
import random

import numpy as np
import pytest
import torch

from helpers import (GAP_TOL, bf16_matmul_oracle, compare_stats, oracle_accept_batch, oracle_stats_for_rows)
from oracle import jot_oracle as jo
from oracle import model_oracle as mo
from paper_2602_11133_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def jot():
    from paper_2602_11133_b200 import jot as binding
    binding._lib()          # fail loudly if the library is missing
    return binding


# ---------------------------------------------------------------- projection GEMM
@pytest.mark.parametrize("M,N,K", [
    (128, 256, 64), (96, 768, 256), (96, 256, 704), (384, 4096, 4096), (200, 1408, 256),
    (384, 12288, 4096), (1000, 3584, 1024), (130, 136, 72),
    (1024, 4096, 1024), (640, 1024, 512), (2048, 8192, 512), (300, 520, 200),      # CTA-pair tiles, odd row-block counts
])
@pytest.mark.parametrize("with_res", [False, True])
def test_gemm_matches_float64_definition(jot, M, N, K, with_res):
    check_gemm(jot, M, N, K, with_res)


# canvases of at most 512 rows without scratch run the slab kernel: one or two accumulators, K cut over the CTA pairs
# of a cluster (2, 3 or 4 ranges, reduce-scatter through distributed shared memory) when there are few slabs
@pytest.mark.parametrize("M,N,K", [
    (1, 256, 64), (31, 136, 72), (255, 520, 1096), (257, 264, 200), (512, 1024, 512), (448, 4096, 1024),
    (96, 512, 4096), (200, 2048, 2048), (384, 1032, 12288), (320, 256, 8192),
])
@pytest.mark.parametrize("with_res", [False, True])
def test_gemm_small_canvas_shapes(jot, M, N, K, with_res):
    check_gemm(jot, M, N, K, with_res)


def check_gemm(jot, M, N, K, with_res):
    a = inputs.normal(1, "a", (M, K), 1.0).cuda()
    w = inputs.normal(1, "w", (N, K), 0.05).cuda()
    res = inputs.normal(1, "r", (M, N), 1.0).cuda() if with_res else None
    out = jot.gemm_bf16(a, w, res)
    torch.cuda.synchronize()
    want = bf16_matmul_oracle(a.cpu(), w.cpu(), None if res is None else res.cpu())
    got = out.cpu().double()
    # one bf16 rounding of an fp32-accumulated value: half an ulp (2^-9 relative) plus accumulation noise
    err = (got - want).abs()
    tol = 2.0 ** -8 * want.abs() + 1e-3 * want.abs().max()
    assert (err <= tol).all(), f"max err {err.max().item()} at {torch.nonzero(err > tol)[:4].tolist()}"
    # and it is not trivially zero
    assert got.abs().max().item() > 0.1


@pytest.mark.parametrize("M,N,K", [(384, 4096, 4096), (384, 4096, 12288), (200, 512, 2048), (96, 264, 1096)])
@pytest.mark.parametrize("with_res", [False, True])
def test_gemm_split_k_matches_float64_definition(jot, M, N, K, with_res):
    """Few output tiles and a long K: the kernel cuts K into ranges and a second kernel adds them."""
    a = inputs.normal(4, "a", (M, K), 1.0).cuda()
    w = inputs.normal(4, "w", (N, K), 0.03).cuda()
    res = inputs.normal(4, "r", (M, N), 1.0).cuda() if with_res else None
    scratch = torch.empty(4 * M * N, dtype=torch.float32, device="cuda")
    n0 = jot.launch_count()
    out = jot.gemm_bf16(a, w, res, scratch=scratch)
    assert jot.launch_count() - n0 == 2          # partial-sum kernel + reduction: the split path really ran
    want = bf16_matmul_oracle(a.cpu(), w.cpu(), None if res is None else res.cpu())
    err = (out.cpu().double() - want).abs()
    tol = 2.0 ** -8 * want.abs() + 1e-3 * want.abs().max()
    assert (err <= tol).all(), f"max err {err.max().item()}"


def test_gemm_residual_in_place(jot):
    a = inputs.normal(2, "a", (384, 512), 1.0).cuda()
    w = inputs.normal(2, "w", (1024, 512), 0.05).cuda()
    h = inputs.normal(2, "h", (384, 1024), 1.0).cuda()
    want = bf16_matmul_oracle(a.cpu(), w.cpu(), h.cpu())
    jot.gemm_bf16(a, w, h, out=h)
    torch.cuda.synchronize()
    err = (h.cpu().double() - want).abs()
    assert (err <= 2.0 ** -8 * want.abs() + 1e-3 * want.abs().max()).all()


def test_bounded_wait_gives_up_and_leaves_the_context_usable(jot):
    """A wait on a barrier that nothing signals ends after its time limit with a status, not a hang."""
    import time
    t0 = time.perf_counter()
    assert jot.selftest_wait_expiry(20_000_000) == 1
    assert time.perf_counter() - t0 < 2.0
    a = inputs.normal(1, "a", (128, 64), 1.0).cuda()
    w = inputs.normal(1, "w", (256, 64), 0.05).cuda()
    out = jot.gemm_bf16(a, w)                      # the context is still healthy
    assert torch.isfinite(out.float()).all()


# ---------------------------------------------------------------- acceptance / freeze
def random_accept_case(seed, B, L, P, mask_id, V, hot=0.3):
    rng = np.random.default_rng(seed)
    tokens = rng.integers(0, V - 1, size=(B, L)).astype(np.int32)
    tokens[tokens >= mask_id] += 1
    masked = rng.random((B, L)) < 0.55
    masked[:, :P] = False
    tokens[masked] = mask_id
    gap = rng.random((B, L)) * np.where(rng.random((B, L)) < hot, 9.0, 0.6)
    top1 = (rng.standard_normal((B, L)) * 2 + 4).astype(np.float32)
    top2 = (top1 - gap).astype(np.float32)
    sumexp = (1.0 + np.exp(top2.astype(np.float64) - top1) + rng.random((B, L)) * 5).astype(np.float32)
    argmax = rng.integers(0, V - 1, size=(B, L)).astype(np.int32)
    argmax[argmax >= mask_id] += 1
    return tokens, top1, top2, sumexp, argmax


@pytest.mark.parametrize("B,L,P,lo,hi,k", [
    (1, 96, 32, 32, 96, 1), (8, 384, 128, 128, 384, 1), (3, 704, 192, 224, 256, 1), (4, 100, 0, 0, 100, 3),
    (2, 1000, 10, 10, 1000, 7), (16, 704, 192, 192, 704, 2), (2, 33, 5, 5, 33, 40),
])
@pytest.mark.parametrize("params", [jo.DREAM_DEFAULT, jo.LLADA_DEFAULT, jo.JotParams(60, 1, 0.7, 8),
                                    jo.JotParams(90, 30, 0.9, 16), jo.JotParams(120, 1, 0.3, 32)])
def test_accept_freeze_matches_oracle(jot, B, L, P, lo, hi, k, params):
    V, mask_id = 5000, 4321
    tokens, top1, top2, sumexp, argmax = random_accept_case(B * 1000 + L, B, L, P, mask_id, V)
    want, reps = oracle_accept_batch(torch.from_numpy(tokens), top1, top2, sumexp, argmax, params, mask_id, lo, hi, k)
    d_tok = torch.from_numpy(tokens).cuda()
    st = jot.Stats(torch.from_numpy(top1).cuda(), torch.from_numpy(top2).cuda(), torch.from_numpy(sumexp).cuda(),
                   torch.from_numpy(argmax).cuda())
    n_masked = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    reason = torch.zeros(B, L, dtype=torch.uint8, device="cuda")
    estep = torch.zeros(B, L, dtype=torch.int16, device="cuda")
    jot.accept_freeze(jot.Params(params.tau_max, params.tau_min, params.gamma, params.D, params.eps), mask_id, d_tok,
                      lo, hi, k, st, n_masked, reason, estep, step_index=7)
    torch.cuda.synchronize()
    got = d_tok.cpu()
    near = 0
    for b in range(B):
        nm = set(reps[b].near_margin)
        near += len(nm)
        for i in range(L):
            if i in nm:
                # the early-exit decision may legitimately differ; either outcome must be a valid one
                assert int(got[b, i]) in (mask_id, int(argmax[b, i]))
                continue
            assert int(got[b, i]) == int(want[b, i]), (b, i, reps[b].ratio.get(i), reps[b].tau.get(i))
        if not nm:
            assert int(n_masked[b]) == int((want[b, lo:hi] == mask_id).sum())
            exp_reason = np.zeros(L, dtype=np.uint8)
            for i in reps[b].exited:
                exp_reason[i] |= 1
            for i in reps[b].scheduled:
                exp_reason[i] |= 2
            assert np.array_equal(reason[b].cpu().numpy(), exp_reason)
            assert np.array_equal(estep[b].cpu().numpy(), np.where(exp_reason > 0, 7, 0).astype(np.int16))
    assert near <= max(2, B * L // 200)
    # untouched outside the block, prompt never changes, frozen tokens never change
    assert torch.equal(got[:, :lo], torch.from_numpy(tokens)[:, :lo])
    assert torch.equal(got[:, hi:], torch.from_numpy(tokens)[:, hi:])
    keep = torch.from_numpy(tokens) != mask_id
    assert torch.equal(got[keep], torch.from_numpy(tokens)[keep])


# the hyper-parameter sweep of the paper's Dream runs (Appendix, "Hyperparameter sweep" table): tau_max x (gamma, D)
SWEEP = [jo.JotParams(float(t), 1.0, g, D) for t in (60, 90, 120) for g, D in ((0.3, 8), (0.5, 8), (0.5, 16), (0.7, 8))]


@pytest.mark.parametrize("B,L,P,lo,hi,k", [(8, 512, 256, 256, 512, 1), (3, 704, 192, 224, 256, 1)])
@pytest.mark.parametrize("params", SWEEP, ids=lambda p: f"tau{p.tau_max:g}-g{p.gamma:g}-D{p.D}")
def test_accept_freeze_sweep_settings(jot, B, L, P, lo, hi, k, params):
    """Every one of the 12 sweep settings, on the Dream-shaped canvas (batch 8, 256 + 256) and on a block of a
    long canvas: canvas, masked count and exit reasons equal to the oracle's outside its near-margin list."""
    V, mask_id = 152064, 151666
    tokens, top1, top2, sumexp, argmax = random_accept_case(77 * B + params.D, B, L, P, mask_id, V)
    want, reps = oracle_accept_batch(torch.from_numpy(tokens), top1, top2, sumexp, argmax, params, mask_id, lo, hi, k)
    d_tok = torch.from_numpy(tokens).cuda()
    st = jot.Stats(*[torch.from_numpy(t).cuda() for t in (top1, top2, sumexp, argmax)])
    n_masked = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    reason = torch.zeros(B, L, dtype=torch.uint8, device="cuda")
    jot.accept_freeze(jot.Params(params.tau_max, params.tau_min, params.gamma, params.D, params.eps), mask_id, d_tok,
                      lo, hi, k, st, n_masked, reason)
    got, reason = d_tok.cpu(), reason.cpu().numpy()
    n_exit = 0
    for b in range(B):
        nm = set(reps[b].near_margin)
        assert len(nm) <= 2
        for i in range(L):
            if i not in nm:
                assert int(got[b, i]) == int(want[b, i]), (b, i, reps[b].ratio.get(i), reps[b].tau.get(i))
        if not nm:
            assert int(n_masked[b]) == int((want[b, lo:hi] == mask_id).sum())
            assert sorted(np.nonzero(reason[b] & 1)[0].tolist()) == sorted(reps[b].exited)
            assert sorted(np.nonzero(reason[b] & 2)[0].tolist()) == sorted(reps[b].scheduled)
        n_exit += len(reps[b].exited)
    assert n_exit > 0                      # the setting decides something on this input


def test_accept_freeze_per_sequence_parameters(jot):
    """One call, a different parameter set for every sequence: each sequence must come out as the oracle run
    with ITS set, and at least two sequences must differ from what a shared set would have given them."""
    V, mask_id, B, L, P = 5000, 4321, 6, 384, 128
    tokens, top1, top2, sumexp, argmax = random_accept_case(4242, B, L, P, mask_id, V)
    sets = [jo.DREAM_DEFAULT, jo.LLADA_DEFAULT, jo.JotParams(60, 1, 0.7, 8), jo.JotParams(120, 1, 0.3, 32),
            jo.JotParams(5, 5, 0.5, 8), jo.JotParams(90, 30, 0.9, 16)]
    d_tok = torch.from_numpy(tokens).cuda()
    st = jot.Stats(*[torch.from_numpy(t).cuda() for t in (top1, top2, sumexp, argmax)])
    n_masked = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    jot.accept_freeze([jot.Params(p.tau_max, p.tau_min, p.gamma, p.D, p.eps) for p in sets], mask_id, d_tok, P, L, 2,
                      st, n_masked)
    got = d_tok.cpu()
    differs_from_shared = 0
    for b, prm in enumerate(sets):
        sl = slice(b, b + 1)
        want, reps = oracle_accept_batch(torch.from_numpy(tokens[sl]), top1[sl], top2[sl], sumexp[sl], argmax[sl], prm,
                                         mask_id, P, L, 2)
        nm = set(reps[0].near_margin)
        assert len(nm) <= 2
        for i in range(L):
            if i not in nm:
                assert int(got[b, i]) == int(want[0, i]), (b, i)
        shared, _ = oracle_accept_batch(torch.from_numpy(tokens[sl]), top1[sl], top2[sl], sumexp[sl], argmax[sl], sets[0],
                                        mask_id, P, L, 2)
        differs_from_shared += int(not torch.equal(shared, want))
    assert differs_from_shared >= 2
    with pytest.raises(jot.JotError) as e:       # more sequences than parameter sets fit into one launch
        big = torch.from_numpy(np.repeat(tokens[:1], 65, axis=0).copy()).cuda()
        st65 = jot.Stats(*[torch.from_numpy(np.repeat(t[:1], 65, axis=0).copy()).cuda() for t in (top1, top2, sumexp, argmax)])
        jot.accept_freeze([jot.Params()] * 65, mask_id, big, P, L, 1, st65)
    assert e.value.status == -2


def test_accept_freeze_degenerate_cases(jot):
    V, mask_id, B, L = 100, 99, 2, 64
    tokens, top1, top2, sumexp, argmax = random_accept_case(5, B, L, 8, mask_id, V)
    st = jot.Stats(*[torch.from_numpy(t).cuda() for t in (top1, top2, sumexp, argmax)])
    # nothing masked in the block: no change, zero left
    t0 = torch.from_numpy(tokens).cuda()
    t0[:, 8:16] = 5
    before = t0.clone()
    n = torch.full((B,), -1, dtype=torch.int32, device="cuda")
    jot.accept_freeze(jot.Params(), mask_id, t0, 8, 16, 1, st, n)
    assert torch.equal(t0, before) and n.tolist() == [0, 0]
    # empty range
    jot.accept_freeze(jot.Params(), mask_id, t0, 20, 20, 1, st, n)
    assert torch.equal(t0, before) and n.tolist() == [0, 0]
    # threshold 0: everything in the block is finalised at once (uncapped), k = 0
    t1 = torch.from_numpy(tokens).cuda()
    jot.accept_freeze(jot.Params(0.0, 0.0, 0.5, 8), mask_id, t1, 8, L, 0, st, n)
    assert (t1[:, 8:] != mask_id).all() and n.tolist() == [0, 0]
    # threshold +inf and k = 0: nothing happens
    t2 = torch.from_numpy(tokens).cuda()
    jot.accept_freeze(jot.Params(float("inf"), float("inf"), 0.5, 8), mask_id, t2, 8, L, 0, st, n)
    assert torch.equal(t2.cpu(), torch.from_numpy(tokens))
    # invalid arguments are refused on the host
    with pytest.raises(jot.JotError):
        jot.accept_freeze(jot.Params(D=0), mask_id, t2, 8, L, 1, st, n)
    with pytest.raises(jot.JotError):
        jot.accept_freeze(jot.Params(D=33), mask_id, t2, 8, L, 1, st, n)
    with pytest.raises(jot.JotError):
        jot.accept_freeze(jot.Params(), mask_id, t2, 8, L + 1, 1, st, n)


# ---------------------------------------------------------------- fused LM head + statistics
def lm_head_model(jot, d, V, mask_id, w_lm, max_batch, max_seq):
    g = inputs.ModelGeometry(0, d, 1, 1, 64, 64, V, mask_id)
    weights = {"embed": w_lm, "lm_head": w_lm, "final_norm": torch.ones(d, dtype=torch.bfloat16, device="cuda"),
               "layers": []}
    return jot.Model(g, weights, max_batch, max_seq)


@pytest.mark.parametrize("B,P,G,d,V,bump", [
    (1, 32, 64, 256, 4096, False),        # tiny model's head
    (2, 40, 200, 512, 5000, True),        # ragged vocabulary tail (5000 = 19.5 tiles of 256), 2 row blocks
    (3, 100, 284, 256, 1032, True),       # several row blocks, vocabulary smaller than the grid
    (8, 128, 256, 1024, 12800, True),     # > 1024 active rows: wide-tile path
])
def test_lm_head_stats_match_oracle(jot, B, P, G, d, V, bump):
    mask_id = V - 7
    case = inputs.lm_head_case(3, B, P, G, d, V, mask_id, device="cuda")
    model = lm_head_model(jot, d, V, mask_id, case.w, B, P + G)
    L = P + G
    st = model.lm_head_stats(case.hidden, case.tokens, P, L, exclude_mask_token=True,
                             bump_id=case.bump_id if bump else None, bump_val=case.bump_val if bump else None)
    torch.cuda.synchronize()
    tok = case.tokens.cpu()
    rows = [(b, i) for b in range(B) for i in range(P, L) if int(tok[b, i]) == mask_id]
    assert len(rows) > 0
    flat = torch.tensor([b * L + i for b, i in rows])
    logits = mo.lm_head_logits(case.hidden.cpu()[flat], case.w.cpu(),
                               case.bump_id.cpu().view(-1)[flat] if bump else None,
                               case.bump_val.cpu().view(-1)[flat] if bump else None)
    want = oracle_stats_for_rows(logits, mask_id)
    pick = lambda t: t.cpu().view(-1)[flat].numpy()
    n, near = compare_stats(pick(st.top1), pick(st.top2), pick(st.sumexp), pick(st.argmax), want, rel=1e-3)
    assert near <= max(1, n // 100)
    # rows that are not active are left untouched
    untouched = torch.ones(B * L, dtype=torch.bool)
    untouched[flat] = False
    assert (st.sumexp.cpu().view(-1)[untouched] == 1.0).all() and (st.argmax.cpu().view(-1)[untouched] == 0).all()
    model.close()


def test_lm_head_mask_token_and_ties(jot):
    # hidden = one-hot rows and a crafted head make exact ties and a dominant mask column
    d, V, mask_id, B, L = 64, 512, 100, 1, 128
    w = torch.zeros(V, d, dtype=torch.bfloat16)
    w[100, 0] = 8.0          # mask column would win
    w[7, 0] = 2.0
    w[300, 0] = 2.0          # exact tie with column 7 -> argmax 7, top2 == top1
    w[450, 0] = 1.0
    hidden = torch.zeros(B * L, d, dtype=torch.bfloat16)
    hidden[:, 0] = 1.0
    tokens = torch.full((B, L), mask_id, dtype=torch.int32)
    model = lm_head_model(jot, d, V, mask_id, w.cuda(), B, L)
    st = model.lm_head_stats(hidden.cuda(), tokens.cuda(), 0, L, exclude_mask_token=True)
    assert (st.argmax.cpu() == 7).all() and (st.top1.cpu() == 2.0).all() and (st.top2.cpu() == 2.0).all()
    S = 2.0 + math.exp(-1.0) + (V - 4) * math.exp(-2.0)
    assert torch.allclose(st.sumexp.cpu(), torch.full((B, L), S), rtol=1e-5)
    st = model.lm_head_stats(hidden.cuda(), tokens.cuda(), 0, L, exclude_mask_token=False)
    assert (st.argmax.cpu() == 100).all() and (st.top1.cpu() == 8.0).all() and (st.top2.cpu() == 2.0).all()
    # no active rows at all: a no-op
    tokens[:] = 3
    out = jot.Stats.empty(B, L, "cuda")
    model.lm_head_stats(hidden.cuda(), tokens.cuda(), 0, L, out=out)
    assert (out.sumexp == 1.0).all()
    model.close()


# ---------------------------------------------------------------- vocabulary slices (one rank's share of the head)
@pytest.mark.parametrize("B,P,G,d,V,cuts", [
    (1, 32, 64, 256, 4096, (2048,)),                    # two equal slices, narrow-tile schedule
    (2, 40, 200, 512, 5000, (1280, 2560, 3840)),        # four slices, ragged vocabulary tail, two row blocks
    (8, 128, 256, 1024, 12800, (6400,)),                # CTA-pair schedule
    (2, 16, 100, 256, 4096, (1000, 3001)),              # cuts that are not tile multiples
])
def test_vocabulary_slices_merge_to_the_full_head(jot, B, P, G, d, V, cuts):
    """The head over disjoint vocabulary slices, merged on the device by the head's own rule, equals the head over
    the whole vocabulary: top-1, runner-up and argmax exactly, the sum to fp32 rounding; each slice equals the
    oracle's statistics of that slice."""
    from paper_2602_11133_b200 import vocab_parallel as vp
    mask_id = V - 7
    case = inputs.lm_head_case(6, B, P, G, d, V, mask_id, device="cuda")
    model = lm_head_model(jot, d, V, mask_id, case.w, B, P + G)
    L = P + G
    kw = dict(bump_id=case.bump_id, bump_val=case.bump_val)
    full = model.lm_head_stats(case.hidden, case.tokens, P, L, **kw)
    bounds = [0] + list(cuts) + [V]
    parts = [model.lm_head_stats_slice(case.hidden, case.tokens, P, L, a, b, **kw) for a, b in zip(bounds, bounds[1:])]
    acc = parts[0]
    for nxt in parts[1:]:
        acc = jot.merge_stats(acc, nxt)
    tok = case.tokens.cpu()
    active = (tok == mask_id)
    active[:, :P] = False
    assert int(active.sum()) > 0
    a = active.cuda()
    assert torch.equal(acc.top1[a], full.top1[a]) and torch.equal(acc.top2[a], full.top2[a])
    assert torch.equal(acc.argmax[a], full.argmax[a])
    assert torch.allclose(acc.sumexp[a], full.sumexp[a], rtol=3e-5, atol=0)      # fp32 sums of approximate exponentials in another order
    # the packed 16-byte tuples survive the round trip of the exchange format
    t = vp.unpack_tuples(vp.pack_tuples(acc.top1, acc.top2, acc.sumexp, acc.argmax))
    assert torch.equal(t[0], acc.top1) and torch.equal(t[3], acc.argmax)
    # a few rows of every slice against the oracle's slice statistics
    rows = [(b, i) for b in range(B) for i in range(P, L) if bool(active[b, i])][:: max(1, int(active.sum()) // 6)][:6]
    flat = torch.tensor([b * L + i for b, i in rows])
    logits = mo.lm_head_logits(case.hidden.cpu()[flat], case.w.cpu(), case.bump_id.cpu().view(-1)[flat],
                               case.bump_val.cpu().view(-1)[flat])
    for (lo, hi), st in zip(zip(bounds, bounds[1:]), parts):
        want = [jo.row_stats_slice(logits[r].numpy(), lo, hi, mask_id) for r in range(len(rows))]
        pick = lambda t: t.cpu().view(-1)[flat].numpy()
        compare_stats(pick(st.top1), pick(st.top2), pick(st.sumexp), pick(st.argmax), want, rel=1e-3)
    with pytest.raises(jot.JotError):
        model.lm_head_stats_slice(case.hidden, case.tokens, P, L, 10, 10, **kw)
    with pytest.raises(jot.JotError):
        model.lm_head_stats_slice(case.hidden, case.tokens, P, L, 0, V + 1, **kw)
    model.close()


def test_vocabulary_slice_with_nothing_but_the_mask_token(jot):
    d, V, mask_id, B, L = 64, 512, 100, 1, 128
    w = (torch.randn(V, d) * 0.1).bfloat16()
    hidden = torch.randn(B * L, d).bfloat16()
    tokens = torch.full((B, L), mask_id, dtype=torch.int32)
    model = lm_head_model(jot, d, V, mask_id, w.cuda(), B, L)
    e = model.lm_head_stats_slice(hidden.cuda(), tokens.cuda(), 0, L, 100, 101)
    assert (e.top1 == -float("inf")).all() and (e.sumexp == 0).all() and (e.argmax == 2 ** 31 - 1).all()
    rest_a = model.lm_head_stats_slice(hidden.cuda(), tokens.cuda(), 0, L, 0, 100)
    rest_b = model.lm_head_stats_slice(hidden.cuda(), tokens.cuda(), 0, L, 101, V)
    full = model.lm_head_stats(hidden.cuda(), tokens.cuda(), 0, L)
    acc = jot.merge_stats(jot.merge_stats(rest_a, e), rest_b)
    assert torch.equal(acc.top1, full.top1) and torch.equal(acc.argmax, full.argmax) and torch.equal(acc.top2, full.top2)
    assert torch.allclose(acc.sumexp, full.sumexp, rtol=3e-5)
    model.close()


# ---------------------------------------------------------------- sampling-based finalisation (Section 4.1)
@pytest.mark.parametrize("B,P,G,d,V,T", [
    (1, 32, 64, 256, 4096, 1.0),          # one narrow-tile chunk schedule
    (2, 40, 200, 512, 5000, 0.7),         # ragged vocabulary tail, two row blocks
    (8, 128, 256, 1024, 12800, 1.3),      # CTA-pair path
])
def test_lm_head_sampled_tokens_match_oracle(jot, B, P, G, d, V, T):
    """The token drawn in the head's epilogue is the oracle's Gumbel-max draw from the same counter stream,
    row by row; the unperturbed statistics do not depend on whether sampling is on."""
    mask_id = V - 7
    seed, step = 0x1234_5678_9ABC_DEF1, 5
    case = inputs.lm_head_case(4, B, P, G, d, V, mask_id, device="cuda")
    model = lm_head_model(jot, d, V, mask_id, case.w, B, P + G)
    L = P + G
    plain = model.lm_head_stats(case.hidden, case.tokens, P, L, bump_id=case.bump_id, bump_val=case.bump_val)
    st = model.lm_head_stats(case.hidden, case.tokens, P, L, bump_id=case.bump_id, bump_val=case.bump_val,
                             sampling=jot.Sampling(T, seed, step))
    torch.cuda.synchronize()
    for a, b in ((plain.top1, st.top1), (plain.top2, st.top2), (plain.sumexp, st.sumexp), (plain.argmax, st.argmax)):
        assert torch.equal(a, b)
    tok = case.tokens.cpu()
    rows = [(b, i) for b in range(B) for i in range(P, L) if int(tok[b, i]) == mask_id]
    if len(rows) > 160:                     # the oracle's draw costs a pass over V per row
        rows = rows[:40] + rows[len(rows) // 2 - 40:len(rows) // 2 + 40] + rows[-40:]
    flat = torch.tensor([b * L + i for b, i in rows])
    logits = mo.lm_head_logits(case.hidden.cpu()[flat], case.w.cpu(), case.bump_id.cpu().view(-1)[flat],
                               case.bump_val.cpu().view(-1)[flat]).numpy()
    got = st.sampled.cpu().view(-1)[flat].tolist()
    am = st.argmax.cpu().view(-1)[flat].tolist()
    near = differs_from_argmax = 0
    for r, f in enumerate(flat.tolist()):
        want, gap = jo.sample_tokens_fast(logits[r], mask_id, T, seed, step, f)
        scale = max(float(np.abs(np.delete(logits[r], mask_id)).max()), 1.0)
        if gap < 2 * 1e-3 * scale / T:      # the two best perturbed scores are closer than the logit tolerance
            near += 1
            assert 0 <= got[r] < V and got[r] != mask_id
            continue
        assert got[r] == want, (r, f, got[r], want, gap)
        differs_from_argmax += int(want != am[r])
    assert near <= max(1, len(rows) // 50)
    assert differs_from_argmax > len(rows) // 10          # a real draw, not the argmax in disguise
    # another step index or seed gives another stream
    st2 = model.lm_head_stats(case.hidden, case.tokens, P, L, bump_id=case.bump_id, bump_val=case.bump_val,
                              sampling=jot.Sampling(T, seed, step + 1))
    st3 = model.lm_head_stats(case.hidden, case.tokens, P, L, bump_id=case.bump_id, bump_val=case.bump_val,
                              sampling=jot.Sampling(T, seed + 1, step))
    a = st.sampled.view(-1)[flat.cuda()]
    assert (st2.sampled.view(-1)[flat.cuda()] != a).float().mean() > 0.1
    assert (st3.sampled.view(-1)[flat.cuda()] != a).float().mean() > 0.1
    model.close()


def test_lm_head_sampling_low_temperature_is_argmax(jot):
    """T -> 0 makes the Gumbel term negligible: the draw equals the argmax wherever the top-2 gap is clear."""
    d, V, B, P, G = 256, 4096, 2, 16, 112
    mask_id = V - 7
    case = inputs.lm_head_case(5, B, P, G, d, V, mask_id, device="cuda")
    model = lm_head_model(jot, d, V, mask_id, case.w, B, P + G)
    st = model.lm_head_stats(case.hidden, case.tokens, P, P + G, bump_id=case.bump_id, bump_val=case.bump_val,
                             sampling=jot.Sampling(1e-3, 99, 0))
    active = (case.tokens == mask_id)
    active[:, :P] = False
    clear = active & ((st.top1 - st.top2) > 0.05)           # Gumbel differences stay below ~30 * T
    assert clear.sum() > 20 and torch.equal(st.sampled[clear], st.argmax[clear])
    with pytest.raises(jot.JotError):
        model.lm_head_stats(case.hidden, case.tokens, P, P + G, sampling=jot.Sampling(1.0, 1, -1))
    model.close()


@pytest.mark.parametrize("B,L,P,lo,hi,k", [(4, 384, 128, 128, 384, 1), (2, 1000, 10, 10, 1000, 7), (6, 704, 192, 224, 256, 1)])
def test_accept_freeze_global_gap_gate_matches_oracle(jot, B, L, P, lo, hi, k):
    """The global early-commit rule the paper contrasts JoT with (Section 2): per sequence, all candidates exit
    when their mean top-2 logit gap clears the threshold, else none; schedule and OR unchanged.  The threshold is
    set at the median of the sequences' mean gaps so that both outcomes occur."""
    V, mask_id = 5000, 4321
    tokens, top1, top2, sumexp, argmax = random_accept_case(B * 31 + L, B, L, P, mask_id, V)
    means = []
    for b in range(B):
        c = [i for i in range(lo, hi) if tokens[b, i] == mask_id]
        means.append(float(np.mean([float(top1[b, i]) - float(top2[b, i]) for i in c])))
    thr = float(np.median(means)) * 1.0001 + 1e-4
    params = jo.JotParams(gate="globalgap", gap_threshold=thr)
    want, reps = oracle_accept_batch(torch.from_numpy(tokens), top1, top2, sumexp, argmax, params, mask_id, lo, hi, k)
    d_tok = torch.from_numpy(tokens).cuda()
    st = jot.Stats(*[torch.from_numpy(t).cuda() for t in (top1, top2, sumexp, argmax)])
    reason = torch.zeros(B, L, dtype=torch.uint8, device="cuda")
    jot.accept_freeze(jot.Params(gate=jot.GATE_GLOBAL_GAP, gap_threshold=thr), mask_id, d_tok, lo, hi, k, st, exit_reason=reason)
    got = d_tok.cpu()
    outcomes = set()
    for b in range(B):
        assert not reps[b].near_margin, "the case should not sit on the threshold"
        outcomes.add(len(reps[b].exited) > 0)
        assert torch.equal(got[b], want[b]), b
        n_cand = sum(1 for i in range(lo, hi) if tokens[b, i] == mask_id)
        assert len(reps[b].exited) in (0, n_cand)                 # everything or nothing
        flagged = int((reason[b].cpu() & 1).sum())
        assert flagged == len(reps[b].exited)
    assert outcomes == {True, False}
    with pytest.raises(jot.JotError):
        jot.accept_freeze(jot.Params(gate=jot.GATE_GLOBAL_GAP, gap_threshold=float("nan")), mask_id, d_tok, lo, hi, k, st)


@pytest.mark.parametrize("B,L,P,lo,hi,k", [(4, 384, 128, 128, 384, 1), (2, 1000, 10, 10, 1000, 7), (3, 704, 192, 224, 256, 1)])
@pytest.mark.parametrize("pth", [0.5, 0.9])
def test_accept_freeze_probability_gate_matches_oracle(jot, B, L, P, lo, hi, k, pth):
    """The fixed gate p1 >= threshold that the paper contrasts the ratio test with (Section 2): same kernel,
    same schedule and OR, no spatial modulation."""
    V, mask_id = 5000, 4321
    tokens, top1, top2, sumexp, argmax = random_accept_case(B * 77 + L, B, L, P, mask_id, V)
    sumexp = (1.0 + (sumexp - 1.0) * 0.2).astype(np.float32)          # p1 spread on both sides of the gate
    params = jo.JotParams(90, 1, 0.5, 8, gate="maxprob", prob_threshold=pth)
    want, reps = oracle_accept_batch(torch.from_numpy(tokens), top1, top2, sumexp, argmax, params, mask_id, lo, hi, k)
    d_tok = torch.from_numpy(tokens).cuda()
    st = jot.Stats(*[torch.from_numpy(t).cuda() for t in (top1, top2, sumexp, argmax)])
    reason = torch.zeros(B, L, dtype=torch.uint8, device="cuda")
    jot.accept_freeze(jot.Params(90, 1, 0.5, 8, gate=jot.GATE_MAXPROB, prob_threshold=pth), mask_id, d_tok, lo, hi, k, st,
                      exit_reason=reason)
    got = d_tok.cpu()
    n_exit = 0
    for b in range(B):
        nm = set(reps[b].near_margin)
        n_exit += len(reps[b].exited)
        for i in range(L):
            if i in nm:
                assert int(got[b, i]) in (mask_id, int(argmax[b, i]))
            else:
                assert int(got[b, i]) == int(want[b, i]), (b, i, 1.0 / sumexp[b, i])
    assert n_exit > 0
    # the ratio gate on the same statistics decides differently somewhere: the switch is really read
    t2 = torch.from_numpy(tokens).cuda()
    jot.accept_freeze(jot.Params(90, 1, 0.5, 8), mask_id, t2, lo, hi, k, st)
    assert not torch.equal(t2, d_tok)
    with pytest.raises(jot.JotError):
        jot.accept_freeze(jot.Params(gate=3), mask_id, t2, lo, hi, k, st)
    with pytest.raises(jot.JotError):
        jot.accept_freeze(jot.Params(gate=jot.GATE_MAXPROB, prob_threshold=0.0), mask_id, t2, lo, hi, k, st)
