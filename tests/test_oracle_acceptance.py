"""Pins for the acceptance side of the CPU oracle (Section 4.1, Algorithm 1) against what the paper and
plain mathematics fix: printed constants, hand-worked closed forms, brute force, invariants."""
import math
import random

import numpy as np
import pytest

from conftest import read_table
from oracle import jot_oracle as jo

M = 99  # a mask id for toy canvases


def canvas(pattern):
    """'r' resolved, 'm' masked."""
    return [M if c == "m" else 7 for c in pattern]


# ---------------------------------------------------------------- Eq. 5-7: printed / hand-worked values
def test_w_max_closed_forms():
    for gamma, D, want in read_table("w_max.txt"):
        assert jo.w_max(gamma, int(D)) == pytest.approx(want, rel=1e-9)
    assert jo.w_max(0.5, 8) == 255.0 / 128.0


def test_threshold_table_next_to_prompt():
    x = canvas("r" * 12 + "m" * 40)
    for k, w, phi, t90, t30 in read_table("threshold_table.txt"):
        i = 11 + int(k)
        assert jo.spatial_weight(x, i, M, 0.5, 8) == pytest.approx(w, abs=1e-15)
        assert jo.softening(w, 0.5, 8) == pytest.approx(phi, rel=1e-14, abs=1e-16)
        assert jo.position_threshold(x, i, M, jo.DREAM_DEFAULT) == pytest.approx(t90, rel=1e-14)
        assert jo.position_threshold(x, i, M, jo.LLADA_DEFAULT) == pytest.approx(t30, rel=1e-14)


def test_threshold_endpoints_and_single_neighbour():
    # interior of a masked region keeps tau_max; fully resolved window gives tau_min (text after Eq. 7)
    x = canvas("m" * 30)
    assert jo.position_threshold(x, 15, M, jo.DREAM_DEFAULT) == 90.0
    x = canvas("r" * 10 + "m" + "r" * 10)
    assert jo.position_threshold(x, 10, M, jo.DREAM_DEFAULT) == pytest.approx(1.0, abs=1e-12)
    # one resolved neighbour at distance 1 only: phi = 0.5 / (255/128) = 64/255
    x = canvas("m" * 10 + "r" + "m" * 10)
    assert jo.softening(jo.spatial_weight(x, 11, M, 0.5, 8), 0.5, 8) == pytest.approx(64 / 255)
    assert jo.position_threshold(x, 11, M, jo.DREAM_DEFAULT) == pytest.approx(90 - 89 * 64 / 255)
    assert jo.position_threshold(x, 9, M, jo.DREAM_DEFAULT) == pytest.approx(90 - 89 * 64 / 255)


def test_window_radius_and_edges():
    # a resolved token at distance D counts, at D+1 it does not; outside the canvas nothing counts
    x = canvas("r" + "m" * 9)
    assert jo.spatial_weight(x, 8, M, 0.5, 8) == 0.5 ** 8
    assert jo.spatial_weight(x, 9, M, 0.5, 8) == 0.0
    x = canvas("m" + "r" * 3)
    assert jo.spatial_weight(x, 0, M, 0.5, 8) == 0.5 + 0.25 + 0.125
    # asymmetric: the position itself (j = i) is never counted even when resolved elsewhere
    x = canvas("rrmrr")
    assert jo.spatial_weight(x, 2, M, 0.3, 1) == pytest.approx(0.6)


def test_no_spatial_special_case():
    # tau_max == tau_min: the threshold is the same everywhere (Section 6.3 "Threshold Ablation")
    p = jo.JotParams(90.0, 90.0, 0.5, 8)
    x = canvas("rrrrmmmmmmmmrmmmrr")
    assert {jo.position_threshold(x, i, M, p) for i in range(len(x)) if x[i] == M} == {90.0}


def test_spatial_weight_is_a_1d_convolution():
    # Section 4.2 "Computational overhead": the weight is a 1-D convolution with a fixed kernel
    rng = random.Random(3)
    for gamma, D in [(0.5, 8), (0.3, 8), (0.7, 8), (0.9, 16), (0.5, 4)]:
        x = [M if rng.random() < 0.6 else 5 for _ in range(57)]
        res = np.array([0.0 if t == M else 1.0 for t in x])
        ker = np.array([gamma ** abs(d) if d != 0 else 0.0 for d in range(-D, D + 1)])
        conv = np.convolve(res, ker, mode="same")
        for i in range(len(x)):
            if x[i] == M:
                assert jo.spatial_weight(x, i, M, gamma, D) == pytest.approx(conv[i], rel=1e-12, abs=1e-15)
                assert 0.0 <= jo.softening(conv[i], gamma, D) <= 1.0


# ---------------------------------------------------------------- Eq. 4: confidence ratio
def test_ratio_is_a_logit_margin():
    # Section 4.1: r >= tau asks for a top-2 logit gap of ln(tau): "about 4.5 for tau = 90 and 3.4 for 30"
    assert math.log(90) == pytest.approx(4.5, abs=0.01)
    assert math.log(30) == pytest.approx(3.4, abs=0.01)
    for tau in (90.0, 30.0):
        for delta, expect in ((+1e-6, True), (-1e-6, False)):
            l = np.full(50, -3.0)
            l[17] = 2.0
            l[31] = 2.0 - math.log(tau) - delta
            st = jo.row_stats(l)
            r = jo.confidence_ratio(st.p1, st.p2, 1e-12)
            assert (r >= tau) == expect
            assert r == pytest.approx(math.exp(st.m1 - st.m2), rel=1e-9)
            assert st.i1 == 17


def test_row_stats_brute_force_tiny_vocab():
    rng = random.Random(0)
    for trial in range(200):
        V = rng.randint(3, 16)
        l = [rng.choice([-2.0, -1.0, 0.0, 0.5, 1.0, 3.0]) + (rng.random() if trial % 2 else 0.0) for _ in range(V)]
        mid = rng.randrange(V) if trial % 3 == 0 else None
        st = jo.row_stats(np.array(l), mid)
        cand = [(v, i) for i, v in enumerate(l) if i != mid]
        z = sum(math.exp(v) for v, _ in cand)
        probs = sorted(((math.exp(v) / z, i) for v, i in cand), key=lambda t: (-t[0], t[1]))
        best = max(v for v, _ in cand)
        assert st.i1 == min(i for v, i in cand if v == best)
        assert st.p1 == pytest.approx(probs[0][0], rel=1e-12)
        assert st.p2 == pytest.approx(probs[1][0], rel=1e-12)
        assert st.p1 >= st.p2
        if sum(1 for v, _ in cand if v == best) > 1:       # exact tie: p2 = p1, r < 1
            assert st.m2 == st.m1
            assert jo.confidence_ratio(st.p1, st.p2) < 1.0


def test_slice_statistics_merge_to_the_whole_row():
    # brute force on tiny vocabularies with ties and an excluded column: any cut into 1..4 slices, merged in any
    # order and association, gives the single-pass statistics (top-1, runner-up and argmax exactly, the sum to
    # rounding)
    rng = random.Random(7)
    for trial in range(300):
        V = rng.randrange(2, 14)
        l = np.array([rng.choice([-1.0, 0.0, 0.5, 2.0, 2.0, 3.25]) for _ in range(V)])
        mask = rng.choice([None, rng.randrange(V)])
        if mask is not None and V == 2:
            continue
        want = jo.row_stats(l, mask)
        cuts = sorted(rng.sample(range(1, V), min(rng.randrange(0, 4), V - 1)))
        parts = [jo.row_stats_slice(l, a, b, mask) for a, b in zip([0] + cuts, cuts + [V])]
        rng.shuffle(parts)
        while len(parts) > 1:                                    # random association
            k = rng.randrange(len(parts) - 1)
            parts[k:k + 2] = [jo.merge_row_stats(parts[k], parts[k + 1])]
        got = parts[0]
        assert (got.m1, got.i1, got.m2) == (want.m1, want.i1, want.m2), (l, mask, cuts)
        assert got.S == pytest.approx(want.S, rel=1e-12)
    # the neutral element: a slice that holds only the excluded token changes nothing
    e = jo.row_stats_slice(np.array([1.0, 5.0, 2.0]), 1, 2, mask_id=1)
    a = jo.row_stats_slice(np.array([1.0, 5.0, 2.0]), 0, 1)
    assert e.m1 == -math.inf and e.S == 0.0
    m = jo.merge_row_stats(a, e)
    assert (m.m1, m.i1, m.m2, m.S) == (a.m1, a.i1, a.m2, a.S) and jo.merge_row_stats(e, a).i1 == a.i1


def test_ratio_temperature_invariance_of_the_definition():
    # r uses un-tempered logits, so it is exp(gap) whatever else is in the row
    l = np.array([0.3, 5.0, 1.0, -2.0])
    st = jo.row_stats(l)
    assert jo.confidence_ratio(st.p1, st.p2, 0.0) == pytest.approx(math.exp(4.0), rel=1e-12)


def test_ratio_finite_when_p2_underflows():
    l = np.array([0.0, 1000.0, -1000.0])
    st = jo.row_stats(l)
    r = jo.confidence_ratio(st.p1, st.p2, 1e-12)
    assert math.isfinite(r) and r == pytest.approx(1e12, rel=1e-9)


# ---------------------------------------------------------------- transfer schedule
def test_transfer_counts():
    assert jo.transfer_counts(64, 64) == [1] * 64
    assert jo.transfer_counts(32, 32) == [1] * 32
    assert jo.transfer_counts(10, 4) == [3, 3, 2, 2]
    for L, T in [(256, 256), (7, 3), (5, 5), (3, 3), (100, 7)]:
        ks = jo.transfer_counts(L, T)
        assert sum(ks) == L and len(ks) == T and max(ks) - min(ks) <= 1


# ---------------------------------------------------------------- accept / freeze on one step
def stats_from_gap(i1, gap, p1=None):
    """RowStats with a chosen top-2 gap; S chosen so p1 is as requested."""
    S = (1.0 + math.exp(-gap)) if p1 is None else 1.0 / p1
    return jo.RowStats(m1=1.0, i1=i1, m2=1.0 - gap, S=S)


def test_accept_or_with_schedule_uncapped():
    x = canvas("rrrr" + "mmmmmm")
    lo, hi = 4, 10
    # position 4 sits next to the prompt: tau = 90 - 89*phi with w = .5+.25+.125+.0625
    stats = {i: stats_from_gap(100 + i, 0.1, p1=0.2) for i in range(lo, hi)}
    stats[4] = stats_from_gap(104, math.log(20.0), p1=0.3)     # r = 20 >= tau(4)?
    w4 = 0.5 + 0.25 + 0.125 + 0.0625
    tau4 = 90 - 89 * w4 / (255 / 128)
    assert tau4 == pytest.approx(90 - 89 * 8 / 17)          # 0.9375 / 1.9921875 = 8/17 -> 48.1176
    stats[7] = stats_from_gap(107, 0.1, p1=0.9)                # schedule picks the max-prob row
    rep = jo.accept_freeze(x, stats, jo.DREAM_DEFAULT, M, lo, hi, 1)
    assert rep.exited == [] and rep.scheduled == [7]
    assert x == [7, 7, 7, 7, M, M, M, 107, M, M]
    # now make 4 clear its (softened) gate and 9 clear tau_max: both exit in the same step, plus schedule
    x = canvas("rrrr" + "mmmmmm")
    stats[4] = stats_from_gap(104, math.log(49.0), p1=0.3)
    stats[9] = stats_from_gap(109, math.log(90.0) + 1e-9, p1=0.1)
    rep = jo.accept_freeze(x, stats, jo.DREAM_DEFAULT, M, lo, hi, 1)
    assert rep.exited == [4, 9] and rep.scheduled == [7]
    assert x == [7, 7, 7, 7, 104, M, M, 107, M, 109]
    # every position clears the gate: all finalised at once (Section 4.2 "uncapped")
    x = canvas("rrrr" + "mmmmmm")
    big = {i: stats_from_gap(200 + i, 10.0) for i in range(lo, hi)}
    rep = jo.accept_freeze(x, big, jo.DREAM_DEFAULT, M, lo, hi, 1)
    assert x == [7, 7, 7, 7, 204, 205, 206, 207, 208, 209] and len(rep.exited) == 6


def test_decision_is_inclusive():
    # Eq. 8 is r >= tau: a ratio exactly on the threshold exits
    st = jo.RowStats(m1=0.0, i1=5, m2=math.log(0.5), S=2.0)           # p1 = 0.5, p2 = 0.25, r = 2 exactly
    assert jo.confidence_ratio(st.p1, st.p2, 0.0) == 2.0
    x = canvas("mm")
    rep = jo.accept_freeze(x, {0: st, 1: st}, jo.JotParams(2.0, 2.0, 0.5, 8, eps=0.0), M, 0, 2, 0)
    assert rep.exited == [0, 1] and x == [5, 5]
    x = canvas("mm")
    rep = jo.accept_freeze(x, {0: st, 1: st}, jo.JotParams(2.0000002, 2.0000002, 0.5, 8, eps=0.0), M, 0, 2, 0)
    assert rep.exited == [] and x == [M, M]


def test_schedule_ties_and_alternative_reading():
    x = canvas("mmmm")
    stats = {i: stats_from_gap(50 + i, 0.1, p1=0.5) for i in range(4)}
    rep = jo.accept_freeze(x, stats, jo.JotParams(1e30, 1e30, 0.5, 8), M, 0, 4, 2)
    assert rep.scheduled == [0, 1]                              # equal p1 -> lower positions
    # OR reading: schedule ranks all of M_n, so it may coincide with an early exit ...
    x = canvas("mmmm")
    stats[2] = stats_from_gap(52, 20.0, p1=0.99)
    rep = jo.accept_freeze(x, stats, jo.DREAM_DEFAULT, M, 0, 4, 1)
    assert rep.exited == [2] and rep.scheduled == [2] and x.count(M) == 3
    # ... while "schedule on the remaining positions" reveals one more
    x = canvas("mmmm")
    rep = jo.accept_freeze(x, stats, jo.DREAM_DEFAULT, M, 0, 4, 1, schedule_after_exit=True)
    assert rep.exited == [2] and rep.scheduled == [0] and x.count(M) == 2


def test_block_restriction_sees_full_canvas():
    # candidates only inside [lo, hi); the window still sees resolved tokens outside the block
    x = canvas("rrrr" + "mmmm" + "mmmm")
    stats = {i: stats_from_gap(300 + i, 10.0) for i in range(4, 8)}
    jo.accept_freeze(x, stats, jo.DREAM_DEFAULT, M, 4, 8, 1)
    assert x[4:8] == [304, 305, 306, 307] and x[8:] == [M] * 4
    p = jo.DREAM_DEFAULT
    assert jo.position_threshold(x, 8, M, p) < 90.0            # neighbours in the earlier block count


# ---------------------------------------------------------------- Algorithm 1: invariants + special cases
def random_stats_fn(seed, V=1000, hot=0.3):
    def fn(x, rows):
        out = {}
        for i in rows:
            rng = random.Random(hash((seed, i, x.count(M))) & 0xFFFFFFFF)
            gap = rng.random() * (8.0 if rng.random() < hot else 0.5)
            out[i] = jo.RowStats(m1=2.0, i1=rng.randrange(V - 1), m2=2.0 - gap, S=1.0 + math.exp(-gap) + rng.random() * 3)
        return out
    return fn


@pytest.mark.parametrize("block_len", [None, 8])
@pytest.mark.parametrize("params", [jo.DREAM_DEFAULT, jo.LLADA_DEFAULT, jo.JotParams(60, 1, 0.7, 8), jo.JotParams(90, 30, 0.9, 16)])
def test_generate_invariants(params, block_len):
    rng = random.Random(1)
    prompt = [rng.randrange(900) for _ in range(12)]
    G, T = 32, 32
    tr = jo.generate(None, prompt, G, T, params, M, block_len, stats_fn=random_stats_fn(5))
    assert tr.x[:12] == prompt                                   # the prompt never changes
    assert all(t != M for t in tr.x)                             # everything finalised
    assert 1 <= tr.steps_used <= T
    prev = None
    for cv, rep in zip(tr.canvases, tr.reports):
        if prev is not None:
            assert cv.count(M) < prev.count(M)                   # at least one position per step
            for a, b in zip(prev, cv):
                assert a == M or a == b                          # frozen tokens never change
        prev = cv
    for a, b in zip(tr.canvases[-1], tr.x):
        assert a == M or a == b
    for i in range(12, 12 + G):                                  # exit_step agrees with the canvas history
        s = tr.exit_step[i]
        assert 1 <= s <= tr.steps_used
        assert tr.canvases[s - 1][i] == M and (s == tr.steps_used or tr.canvases[s][i] != M)


def test_generate_threshold_infinite_is_plain_topk_decoding():
    # nothing clears the gate: exactly T steps of ordinary max-prob decoding (Section 4.2)
    prompt = [1, 2, 3]
    G = T = 10
    fn = random_stats_fn(11)
    tr = jo.generate(None, prompt, G, T, jo.JotParams(float("inf"), float("inf"), 0.5, 8), M, stats_fn=fn)
    assert tr.steps_used == T and all(r.exited == [] for r in tr.reports)
    x = prompt + [M] * G                                         # independent restatement of the baseline
    for _ in range(T):
        A = [i for i in range(len(x)) if x[i] == M]
        st = fn(x, A)
        best = min(A, key=lambda i: (-st[i].p1, i))
        x[best] = st[best].i1
    assert x == tr.x


def test_generate_threshold_zero_finishes_one_step_per_block():
    prompt = [1, 2, 3, 4]
    tr = jo.generate(None, prompt, 32, 32, jo.JotParams(0.0, 0.0, 0.5, 8), M, None, stats_fn=random_stats_fn(2))
    assert tr.steps_used == 1
    tr = jo.generate(None, prompt, 32, 32, jo.JotParams(0.0, 0.0, 0.5, 8), M, 8, stats_fn=random_stats_fn(2))
    assert tr.steps_used == 4
    # step-speedup = configured / actual steps (Section 6.1 "Experimental Setup")
    assert 32 / tr.steps_used == 8.0


def test_generate_decodes_blocks_left_to_right():
    # Semi-autoregressive decoding (Appendix "Experimental Configuration": the canvas is generated "in fixed-size
    # blocks", each block only after the ones before it): a stub model that writes, for every position, whether the
    # position one block to its LEFT was already resolved when it was asked.  Left to right, every block after
    # the first sees a resolved left neighbour and a masked right one; any other order changes the tokens.
    P, Lb, nb = 4, 4, 4
    G = Lb * nb
    asked = []

    def stats_fn(x, A):
        asked.append((min(A), max(A)))
        out = {}
        for i in A:
            left_resolved = x[i - Lb] != M                       # prompt or an earlier block
            right_masked = i + Lb >= len(x) or x[i + Lb] == M
            tok = 100 + (1 if left_resolved else 0) + (2 if right_masked else 0)
            out[i] = jo.RowStats(5.0, tok, 0.0, 1.5)
        return out
    tr = jo.generate(None, [1, 2, 3, 4], G, G, jo.JotParams(0.0, 0.0, 0.5, 8), M, Lb, stats_fn=stats_fn)
    assert tr.x[P:] == [103] * G                                 # left resolved AND right still masked, everywhere
    assert tr.blocks == [(P + b * Lb, P + (b + 1) * Lb) for b in range(nb)]
    assert asked == [(P + b * Lb, P + (b + 1) * Lb - 1) for b in range(nb)]
    # one block at a time: a step never touches a position outside the block it was run for
    for cv, nxt, (lo, hi) in zip(tr.canvases, tr.canvases[1:] + [tr.x], tr.blocks):
        assert all(a == b for i, (a, b) in enumerate(zip(cv, nxt)) if not lo <= i < hi)


def test_generate_schedule_table_restarts_in_every_block():
    # Nothing clears the gate, so each step finalises exactly what the schedule reveals: 6 positions over the 4
    # steps of a block are 2, 2, 1, 1 (the remainder goes to the earliest steps), and the next block starts over.
    inf = float("inf")
    tr = jo.generate(None, [7, 8], 12, 8, jo.JotParams(inf, inf, 0.5, 8), M, 6, stats_fn=random_stats_fn(3))
    assert tr.steps_used == 8
    assert [len(r.scheduled) for r in tr.reports] == [2, 2, 1, 1, 2, 2, 1, 1]
    assert [cv.count(M) for cv in tr.canvases] == [12, 10, 8, 7, 6, 4, 2, 1]


def test_fractional_schedule_counts():
    # hand-worked: ceil(remaining / steps left)
    assert jo.fractional_transfer_count(6, 4) == 2 and jo.fractional_transfer_count(4, 3) == 2
    assert jo.fractional_transfer_count(2, 2) == 1 and jo.fractional_transfer_count(1, 1) == 1
    assert jo.fractional_transfer_count(7, 1) == 7 and jo.fractional_transfer_count(0, 3) == 0
    assert jo.fractional_transfer_count(1, 9) == 1                       # progress while anything is masked
    # without early exits it walks down exactly the fixed table, for every block length and step count
    for Lb in range(1, 40):
        for Tb in range(1, Lb + 1):
            left, got = Lb, []
            for s in range(Tb):
                k = jo.fractional_transfer_count(left, Tb - s)
                got.append(k)
                left -= k
            assert left == 0 and got == jo.transfer_counts(Lb, Tb), (Lb, Tb)


def test_fractional_schedule_in_the_loop():
    inf = float("inf")
    # nothing clears the gate: same steps and same counts as the fixed table
    fn = random_stats_fn(3)
    a = jo.generate(None, [7, 8], 12, 8, jo.JotParams(inf, inf, 0.5, 8), M, 6, stats_fn=fn, schedule="fractional")
    b = jo.generate(None, [7, 8], 12, 8, jo.JotParams(inf, inf, 0.5, 8), M, 6, stats_fn=fn)
    assert a.x == b.x and [len(r.scheduled) for r in a.reports] == [2, 2, 1, 1, 2, 2, 1, 1]
    # early exits run ahead of the pace: a hand-made model in which canvas positions 4..11 of the 12-token block
    # 2..13 clear the threshold at the first step and also hold the highest max-probabilities.  Step 1 reveals 3
    # (all among the 8 exits): 4 left.  The fixed table (3 per step) then reveals 3 and 1: three steps.  The
    # fractional schedule re-divides what is still masked over the steps left: ceil(4 / 3) = 2, ceil(2 / 2) = 1,
    # ceil(1 / 1) = 1: four steps, never more than the pace needs.
    def stats_fn(x, A):
        out = {}
        for i in A:
            sure = 4 <= i <= 11
            out[i] = jo.RowStats(20.0 if sure else 1.0, 50 + i, 0.0, 1.0 + i * 1e-3 + (0.0 if sure else 5.0))
        return out
    fr = jo.generate(None, [1, 2], 12, 4, jo.JotParams(50.0, 50.0, 0.5, 8), M, None, stats_fn=stats_fn, schedule="fractional")
    fx = jo.generate(None, [1, 2], 12, 4, jo.JotParams(50.0, 50.0, 0.5, 8), M, None, stats_fn=stats_fn)
    assert sorted(fr.reports[0].exited) == list(range(4, 12)) and fr.reports[0].scheduled == [4, 5, 6]
    assert [len(r.scheduled) for r in fr.reports] == [3, 2, 1, 1] and fr.steps_used == 4
    assert [cv.count(M) for cv in fr.canvases] == [12, 4, 2, 1]
    assert [len(r.scheduled) for r in fx.reports] == [3, 3, 1] and fx.steps_used == 3
    # invariants under the adaptive schedule with random statistics: ends within its steps, one or more per step
    for Lb in (None, 8):
        tr = jo.generate(None, [5] * 6, 32, 16, jo.DREAM_DEFAULT, M, Lb, stats_fn=random_stats_fn(9), schedule="fractional")
        assert all(t != M for t in tr.x) and tr.steps_used <= 16
        assert all(len(r.scheduled) >= 1 for r in tr.reports)


def test_generate_with_logits_fn_excludes_mask_token():
    V = 12
    mid = V - 1

    def logits_fn(x, rows):
        out = {}
        for i in rows:
            l = np.linspace(-1, 1, V) * ((i % 3) - 1.0)
            l[mid] = 50.0                                        # the model "predicts" the mask token
            out[i] = l
        return out
    tr = jo.generate(logits_fn, [0, 1], 6, 6, jo.DREAM_DEFAULT, mid)
    assert all(t != mid for t in tr.x)


def test_reversal_budget_number():
    # Section 5 "Why Early Exit Preserves Quality": 2 * 256 / (1 + 90) is "about 5.6"
    assert 2 * 256 / 91 == pytest.approx(5.6, abs=0.05)


# ---------------------------------------------------------------- sampling-based finalisation, probability gate
def test_counter_generator_matches_published_splitmix64_vectors():
    # first outputs of the reference implementation for seed 1234567
    want = [6457827717110365317, 3203168211198807973, 9817491932198370423, 4593380528125082431, 16408922859458223821]
    assert [jo.splitmix64_output(1234567, n) for n in range(1, 6)] == want


def test_gumbel_max_draws_follow_the_softmax():
    # chi-square of 20000 draws against softmax(l / T) on a 6-token vocabulary (mask column excluded)
    l = np.array([1.0, 0.2, -0.5, 2.0, 50.0, 0.0])
    mask = 4
    for T in (1.0, 0.5):
        p = np.exp(np.delete(l, mask) / T)
        p /= p.sum()
        counts = np.zeros(6)
        n = 20000
        for step in range(n):
            counts[jo.sample_token(l, mask, T, seed=7, step=step, flat_pos=3)] += 1
        assert counts[mask] == 0
        c = np.delete(counts, mask)
        chi2 = float(((c - n * p) ** 2 / (n * p)).sum())
        assert chi2 < 20.5, (T, chi2)             # 4 degrees of freedom: P(chi2 > 20.5) < 4e-4
    # the fast version is the same draw
    for step in range(200):
        assert jo.sample_tokens_fast(l, mask, 0.7, 11, step, 5)[0] == jo.sample_token(l, mask, 0.7, 11, step, 5)
    # temperature -> 0 recovers the argmax; different positions and steps get different streams
    assert all(jo.sample_token(l, mask, 1e-3, 1, s, 0) == 3 for s in range(50))
    assert len({jo.gumbel_key(1, s, q) for s in range(20) for q in range(20)}) == 400


def test_sampled_token_is_what_a_finalised_position_receives():
    x = canvas("rrmm")
    stats = {2: stats_from_gap(50, 10.0), 3: stats_from_gap(51, 0.01, p1=0.1)}
    rep = jo.accept_freeze(x, stats, jo.DREAM_DEFAULT, M, 2, 4, 0, tokens={2: 77, 3: 78})
    assert rep.exited == [2] and x == [7, 7, 77, M]            # decisions unchanged, token replaced


def test_probability_gate():
    x = canvas("rrmmm")
    stats = {2: stats_from_gap(60, 0.1, p1=0.95), 3: stats_from_gap(61, 9.0, p1=0.5), 4: stats_from_gap(62, 0.1, p1=0.9)}
    p = jo.JotParams(gate="maxprob", prob_threshold=0.9)
    rep = jo.accept_freeze(x, stats, p, M, 2, 5, 0)
    assert rep.exited == [2, 4] and x == [7, 7, 60, M, 62]      # inclusive; a large ratio alone does not pass


def test_global_gap_gate_commits_everything_or_nothing():
    """Section 2: the global early-commit rule finalises all remaining masked positions at once when the top-2
    gap clears a threshold.  Read as the mean logit gap of the candidates; hand-computed cases."""
    # gaps 6, 2, 4 -> mean 4.0
    mk = lambda: {2: stats_from_gap(60, 6.0, p1=0.5), 3: stats_from_gap(61, 2.0, p1=0.9), 4: stats_from_gap(62, 4.0, p1=0.2)}
    x = canvas("rrmmm")
    rep = jo.accept_freeze(x, mk(), jo.JotParams(gate="globalgap", gap_threshold=4.0), M, 2, 5, 0)
    assert rep.exited == [2, 3, 4] and x == [7, 7, 60, 61, 62]          # inclusive, and uncapped
    x = canvas("rrmmm")
    rep = jo.accept_freeze(x, mk(), jo.JotParams(gate="globalgap", gap_threshold=4.5), M, 2, 5, 1)
    assert rep.exited == [] and rep.scheduled == [3] and x == [7, 7, M, 61, M]   # below: plain schedule step
    # only the candidates of the current block count: position 4 (gap 1) lies outside it -> mean (6 + 2) / 2 = 4,
    # where the mean over all three masked positions would be 3
    x = canvas("rrmmm")
    st3 = mk()
    st3[4] = stats_from_gap(62, 1.0, p1=0.2)
    rep = jo.accept_freeze(x, st3, jo.JotParams(gate="globalgap", gap_threshold=4.0), M, 2, 4, 0)
    assert rep.exited == [2, 3] and x == [7, 7, 60, 61, M]
    # a single very confident position does not commit the rest (the per-token ratio gate would exit it)
    st = {2: stats_from_gap(60, 12.0), 3: stats_from_gap(61, 0.0), 4: stats_from_gap(62, 0.0)}
    x = canvas("rrmmm")
    assert jo.accept_freeze(x, st, jo.JotParams(gate="globalgap", gap_threshold=5.0), M, 2, 5, 0).exited == []
    x = canvas("rrmmm")
    assert jo.accept_freeze(x, st, jo.DREAM_DEFAULT, M, 2, 5, 0).exited == [2]
    # near the threshold every candidate is reported
    x = canvas("rrmmm")
    rep = jo.accept_freeze(x, mk(), jo.JotParams(gate="globalgap", gap_threshold=4.0 * (1 + 5e-4)), M, 2, 5, 0)
    assert rep.near_margin == [2, 3, 4]


def test_global_gap_gate_in_the_loop():
    """Threshold -inf-like: the first step commits the whole block (steps_used = number of blocks);
    threshold +inf-like: plain schedule decoding, exactly T steps."""
    prompt = [7] * 4
    def stats_fn(x, rows):
        return {i: stats_from_gap(100 + i, 3.0, p1=0.5 + 0.001 * i) for i in rows}
    t = jo.generate(None, prompt, 8, 8, jo.JotParams(gate="globalgap", gap_threshold=-1e30), M, block_len=4, stats_fn=stats_fn)
    assert t.steps_used == 2 and t.x[4:] == [104 + j for j in range(8)]
    t = jo.generate(None, prompt, 8, 8, jo.JotParams(gate="globalgap", gap_threshold=1e30), M, block_len=4, stats_fn=stats_fn)
    assert t.steps_used == 8 and all(len(r.exited) == 0 and len(r.scheduled) == 1 for r in t.reports)
