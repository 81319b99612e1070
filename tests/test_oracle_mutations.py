"""Do the pins bite?  Each case plants one plausible mistake in the CPU oracle (a dropped term, a wrong sign
or index, a transposed operand, a swapped tie rule) and checks that at least one of the pin tests then fails.
The mistakes are planted in the oracle only, on the CPU; the CUDA path is not involved."""
import math

import numpy as np
import pytest
import torch

import test_oracle_acceptance as pins_a
import test_oracle_model as pins_m
from oracle import jot_oracle as jo
from oracle import model_oracle as mo

# the pins of the global early-commit gate are checked against their own planted mistakes below: the
# rewritten decision rules of accept_variant() do not know that gate, so those pins would "notice" anything
ACCEPT_PINS = [getattr(pins_a, n) for n in dir(pins_a) if n.startswith("test_") and not n.startswith("test_global_gap")]
GAP_PINS = [getattr(pins_a, n) for n in dir(pins_a) if n.startswith("test_global_gap")]
MODEL_PINS = [pins_m.test_rope_closed_form, pins_m.test_rmsnorm_closed_form,
              pins_m.test_attention_rows_average_values_and_see_everything,
              pins_m.test_forward_matches_independent_restatement, pins_m.test_bidirectional_not_causal,
              pins_m.test_lm_head_bump]


def some_pin_fails(pins):
    for t in pins:
        marks = [m for m in getattr(t, "pytestmark", []) if m.name == "parametrize"]
        try:
            if marks:
                run_parametrized(t, marks)
            else:
                t()
        except Exception:          # an assertion, or the mistake breaking the code outright
            return True
    return False


def run_parametrized(t, marks):
    # cartesian product of the parametrize marks (single-name or comma-separated names)
    combos = [{}]
    for m in marks:
        names = [n.strip() for n in m.args[0].split(",")]
        new = []
        for c in combos:
            for v in m.args[1]:
                vals = v if len(names) > 1 else (v,)
                d = dict(c)
                d.update(dict(zip(names, vals)))
                new.append(d)
        combos = new
    for c in combos:
        t(**c)


def test_pins_pass_on_the_unmodified_oracle():
    assert not some_pin_fails(ACCEPT_PINS)
    assert not some_pin_fails(MODEL_PINS)


# ---------------------------------------------------------------- acceptance side
def mut_spatial_left_only(x, i, mask_id, gamma, D):
    return sum(gamma ** (i - j) for j in range(len(x)) if 0 < i - j <= D and x[j] != mask_id)


def mut_spatial_radius_off_by_one(x, i, mask_id, gamma, D):
    return sum(gamma ** abs(i - j) for j in range(len(x)) if j != i and abs(i - j) <= D - 1 and x[j] != mask_id)


def mut_spatial_counts_self_and_masked(x, i, mask_id, gamma, D):
    return sum(gamma ** abs(i - j) for j in range(len(x)) if j != i and abs(i - j) <= D and x[j] == mask_id)


def mut_spatial_linear_kernel(x, i, mask_id, gamma, D):
    return sum(gamma * abs(i - j) for j in range(len(x)) if j != i and abs(i - j) <= D and x[j] != mask_id)


def mut_row_stats_highest_index(logits, mask_id=None):
    l = np.asarray(logits, dtype=np.float64).copy()
    if mask_id is not None:
        l[mask_id] = -np.inf
    order = np.argsort(l, kind="stable")[::-1]
    return jo.RowStats(float(l[order[0]]), int(order[0]), float(l[order[1]]), float(np.sum(np.exp(l - l[order[0]]))))


def mut_row_stats_keeps_mask_column(logits, mask_id=None):
    return ORIG["row_stats"](logits, None)


def mut_row_stats_distinct_runner_up(logits, mask_id=None):
    st = ORIG["row_stats"](logits, mask_id)
    l = np.asarray(logits, dtype=np.float64).copy()
    if mask_id is not None:
        l[mask_id] = -np.inf
    lower = l[l < st.m1]
    return jo.RowStats(st.m1, st.i1, float(lower.max()) if lower.size else st.m1, st.S)


ORIG = {n: getattr(jo, n) for n in ("spatial_weight", "w_max", "softening", "threshold", "confidence_ratio", "row_stats",
                                     "transfer_counts", "accept_freeze")}

ACCEPT_MUTATIONS = {
    "w_max without the factor 2": ("w_max", lambda g, D: sum(g ** d for d in range(1, D + 1))),
    "w_max sums d = 0..D": ("w_max", lambda g, D: 2.0 * sum(g ** d for d in range(0, D + 1))),
    "spatial weight: left side only": ("spatial_weight", mut_spatial_left_only),
    "spatial weight: radius D - 1": ("spatial_weight", mut_spatial_radius_off_by_one),
    "spatial weight: counts masked instead of resolved": ("spatial_weight", mut_spatial_counts_self_and_masked),
    "spatial weight: gamma * d instead of gamma ** d": ("spatial_weight", mut_spatial_linear_kernel),
    "softening without the clamp and inverted": ("softening", lambda w, g, D: 1.0 - min(1.0, w / ORIG["w_max"](g, D))),
    "threshold: interpolates the wrong way": ("threshold", lambda phi, tmax, tmin: tmin + (tmax - tmin) * phi),
    "threshold: ignores tau_min": ("threshold", lambda phi, tmax, tmin: tmax - tmax * phi),
    "ratio: p2 / p1": ("confidence_ratio", lambda p1, p2, eps=1e-12: p2 / (p1 + eps)),
    "ratio: difference instead of quotient": ("confidence_ratio", lambda p1, p2, eps=1e-12: p1 - p2),
    "argmax ties to the highest index": ("row_stats", mut_row_stats_highest_index),
    "mask column not excluded": ("row_stats", mut_row_stats_keeps_mask_column),
    "runner-up skips exact ties": ("row_stats", mut_row_stats_distinct_runner_up),
    "merge: runner-up forgets the smaller maximum": (
        "merge_row_stats", lambda a, b: jo.RowStats(max(a.m1, b.m1), b.i1 if (b.m1 > a.m1 or (b.m1 == a.m1 and b.i1 < a.i1)) else a.i1,
                                                    max(a.m2, b.m2),
                                                    (0.0 if a.m1 == -math.inf else a.S * math.exp(a.m1 - max(a.m1, b.m1))) +
                                                    (0.0 if b.m1 == -math.inf else b.S * math.exp(b.m1 - max(a.m1, b.m1))))),
    "merge: sums added without rescaling": (
        "merge_row_stats", lambda a, b: jo.RowStats(max(a.m1, b.m1), b.i1 if (b.m1 > a.m1 or (b.m1 == a.m1 and b.i1 < a.i1)) else a.i1,
                                                    max(a.m2, b.m2, min(a.m1, b.m1)), a.S + b.S)),
    "merge: equal maxima resolve to the later slice": (
        "merge_row_stats", lambda a, b: jo.RowStats(max(a.m1, b.m1), b.i1 if b.m1 >= a.m1 else a.i1,
                                                    max(a.m2, b.m2, min(a.m1, b.m1)),
                                                    (0.0 if a.m1 == -math.inf else a.S * math.exp(a.m1 - max(a.m1, b.m1))) +
                                                    (0.0 if b.m1 == -math.inf else b.S * math.exp(b.m1 - max(a.m1, b.m1))))),
    "fractional schedule rounds down": ("fractional_transfer_count", lambda n, t: n // t),
    "fractional schedule divides by one step too many": ("fractional_transfer_count", lambda n, t: -(-n // (t + 1))),
    "fractional schedule ignores what is left": ("fractional_transfer_count", lambda n, t: 1),
    "transfer counts: remainder to the last steps": (
        "transfer_counts", lambda L, T: [L // T + (1 if s >= T - L % T else 0) for s in range(T)]),
}


@pytest.mark.parametrize("name", sorted(ACCEPT_MUTATIONS))
def test_acceptance_pins_catch(name, monkeypatch):
    attr, fn = ACCEPT_MUTATIONS[name]
    monkeypatch.setattr(jo, attr, fn)
    assert some_pin_fails(ACCEPT_PINS), f"no pin noticed: {name}"


def accept_variant(**kw):
    """accept_freeze with one decision rule changed (rewritten here from the paper with the change planted)."""
    def fn(x, stats, p, mask_id, blk_lo, blk_hi, k_transfer, schedule_after_exit=False):
        x0 = list(x)
        A = [i for i in range(blk_lo, blk_hi) if x0[i] == mask_id]
        ratio, tau, E = {}, {}, []
        for i in A:
            r = jo.confidence_ratio(stats[i].p1, stats[i].p2, p.eps)
            t = jo.position_threshold(x if kw.get("live_canvas") else x0, i, mask_id, p)
            ratio[i], tau[i] = r, t
            ok = (r > t) if kw.get("strict") else (r >= t)
            if ok:
                E.append(i)
                if kw.get("live_canvas"):
                    x[i] = stats[i].i1
        cand = [i for i in A if i not in E] if (schedule_after_exit or kw.get("always_after_exit")) else A
        k = min(k_transfer, len(cand))
        key = (lambda i: (-stats[i].p1, -i)) if kw.get("tie_high") else (lambda i: (-stats[i].p1, i))
        if kw.get("rank_by_ratio"):
            key = lambda i: (-ratio[i], i)
        U = sorted(sorted(cand, key=key)[:k])
        chosen = (set(E) & set(U)) if kw.get("and_masks") else (set(E) | set(U))
        for i in chosen:
            x[i] = stats[i].i1
        return jo.StepReport(E, U, [], ratio, tau)
    return fn


DECISION_MUTATIONS = {
    "strict inequality": dict(strict=True),
    "schedule ties to the higher position": dict(tie_high=True),
    "schedule ranks by the ratio instead of max-prob": dict(rank_by_ratio=True),
    "AND of the two masks": dict(and_masks=True),
    "schedule always ranks what early exit left": dict(always_after_exit=True),
}


@pytest.mark.parametrize("name", sorted(DECISION_MUTATIONS))
def test_decision_pins_catch(name, monkeypatch):
    monkeypatch.setattr(jo, "accept_freeze", accept_variant(**DECISION_MUTATIONS[name]))
    assert some_pin_fails(ACCEPT_PINS), f"no pin noticed: {name}"


def generate_variant(old, new):
    """jo.generate with one line of its source replaced (the planted mistake), compiled in the oracle's namespace."""
    import inspect
    src = inspect.getsource(jo.generate)
    assert src.count(old) == 1, old
    ns = dict(vars(jo))
    exec(src.replace(old, new), ns)
    return ns["generate"]


LOOP_MUTATIONS = {
    "blocks decoded right to left": ("for blk in range(nb):", "for blk in reversed(range(nb)):"),
    "blocks decoded from the second one on, the first last": (
        "for blk in range(nb):", "for blk in list(range(1, nb)) + [0]:"),
    "candidates are every masked position, not the current block's": (
        "A = [i for i in range(lo, hi) if x[i] == mask_id]             # M_n",
        "A = [i for i in range(P, len(x)) if x[i] == mask_id]"),
    "the schedule table restarts only once": ('k = ks[s] if schedule == "fixed"',
                                              'k = ks[min(traj.steps_used, Tb - 1)] if schedule == "fixed"'),
    "the fractional schedule counts the steps of the whole run": (
        "fractional_transfer_count(len(A), Tb - s)", "fractional_transfer_count(len(A), steps - traj.steps_used)"),
}


@pytest.mark.parametrize("name", sorted(LOOP_MUTATIONS))
def test_loop_pins_catch(name, monkeypatch):
    old, new = LOOP_MUTATIONS[name]
    monkeypatch.setattr(jo, "generate", generate_variant(old, new))
    assert some_pin_fails(ACCEPT_PINS), f"no pin noticed: {name}"


def gap_variant(kind):
    """accept_freeze whose global early-commit branch carries one planted mistake."""
    orig = jo.accept_freeze

    def fn(x, stats, p, mask_id, blk_lo, blk_hi, k_transfer, schedule_after_exit=False, tokens=None):
        if p.gate != "globalgap":
            return orig(x, stats, p, mask_id, blk_lo, blk_hi, k_transfer, schedule_after_exit, tokens)
        A = [i for i in range(blk_lo, blk_hi) if x[i] == mask_id]
        pool = [i for i in range(len(x)) if x[i] == mask_id and i in stats] if kind == "whole canvas" else A
        gaps = [stats[i].m1 - stats[i].m2 for i in pool]
        if kind == "probability gap":
            gaps = [stats[i].p1 - stats[i].p2 for i in pool]
        stat = {"max": max, "min": min}.get(kind, lambda g: sum(g) / len(g))(gaps) if gaps else 0.0
        ok = stat > p.gap_threshold if kind == "strict" else stat >= p.gap_threshold
        E = list(A) if (A and ok) else []
        if kind == "per token":
            E = [i for i in A if stats[i].m1 - stats[i].m2 >= p.gap_threshold]
        near = list(A) if A and abs(stat - p.gap_threshold) <= 1e-3 * abs(p.gap_threshold) else []
        k = min(k_transfer, len(A))
        U = sorted(sorted(A, key=lambda i: (-stats[i].p1, i))[:k])
        for i in set(E) | set(U):
            x[i] = stats[i].i1
        return jo.StepReport(E, U, near, {}, {})
    return fn


GAP_MUTATIONS = ["max", "min", "strict", "whole canvas", "per token", "probability gap"]


def test_gap_variant_without_a_mistake_passes():
    import unittest.mock as um
    with um.patch.object(jo, "accept_freeze", gap_variant("none")):
        assert not some_pin_fails(GAP_PINS)


@pytest.mark.parametrize("kind", GAP_MUTATIONS)
def test_global_gap_pins_catch(kind, monkeypatch):
    monkeypatch.setattr(jo, "accept_freeze", gap_variant(kind))
    assert some_pin_fails(GAP_PINS), f"no pin noticed: {kind}"


# ---------------------------------------------------------------- denoiser side
def mut_rope_wrong_sign(t, theta, pos0=0):
    out = ORIG_M["rope"](t, theta, pos0)
    half = t.shape[-1] // 2
    return torch.cat([out[..., :half], -out[..., half:]], dim=-1)


def mut_rope_interleaved(t, theta, pos0=0):
    B, L, H, hd = t.shape
    inv = theta ** (-torch.arange(hd // 2, dtype=torch.float64) * 2.0 / hd)
    ang = torch.arange(pos0, pos0 + L, dtype=torch.float64)[:, None] * inv[None, :]
    c, s = torch.cos(ang)[None, :, None, :], torch.sin(ang)[None, :, None, :]
    a, b = t[..., 0::2], t[..., 1::2]
    out = torch.empty_like(t)
    out[..., 0::2] = a * c - b * s
    out[..., 1::2] = b * c + a * s
    return out


def mut_attention_causal(q, k, v, round_p):
    B, L, Hq, hd = q.shape
    g = Hq // k.shape[2]
    k, v = k.repeat_interleave(g, dim=2), v.repeat_interleave(g, dim=2)
    s = torch.einsum("blhd,bmhd->bhlm", q, k) / math.sqrt(hd)
    s = s + torch.triu(torch.full((L, L), float("-inf"), dtype=s.dtype), 1)
    return torch.einsum("bhlm,bmhd->blhd", torch.softmax(s, -1), v)


def mut_attention_no_scale(q, k, v, round_p):
    return ORIG_M["attention"](q * math.sqrt(q.shape[-1]), k, v, round_p)


def mut_attention_wrong_gqa(q, k, v, round_p):
    g = q.shape[2] // k.shape[2]
    return ORIG_M["attention"](q, k.repeat(1, 1, g, 1), v.repeat(1, 1, g, 1), round_p)   # tiles instead of interleaving


def mut_rmsnorm_mean_subtracted(h, gain, eps):
    hc = h - h.mean(dim=-1, keepdim=True)
    return hc * torch.rsqrt((hc * hc).mean(dim=-1, keepdim=True) + eps) * gain.to(torch.float64)


def mut_rmsnorm_no_gain(h, gain, eps):
    return h * torch.rsqrt((h * h).mean(dim=-1, keepdim=True) + eps)


def mut_lm_head_bump_everywhere(hidden_rows, w_lm, bump_id=None, bump_val=None):
    l = hidden_rows.to(torch.float64) @ w_lm.to(torch.float64).T
    if bump_id is not None:
        l += bump_val.to(torch.float64)[:, None]
    return l


def mut_rope_block_rows_start_at_zero(t, theta, pos0=0):
    return ORIG_M["rope"](t, theta, 0)


def mut_layer_cache_drops_the_suffix(g, lw, h, ra, pos0=0, context=None):
    if context is not None:                       # a prefix-only cache: nothing after the block is attended to
        end = pos0 + h.shape[1]
        context = (context[0][:, :end], context[1][:, :end])
    return ORIG_M["layer"](g, lw, h, ra, pos0, context)


def mut_layer_cache_ignored(g, lw, h, ra, pos0=0, context=None):
    return ORIG_M["layer"](g, lw, h, ra, pos0, None)      # the block attends only to itself


ORIG_M = {n: getattr(mo, n) for n in ("rope", "attention", "rmsnorm", "lm_head_logits", "layer")}
CACHE_PINS = [pins_m.test_cached_pass_with_block_equal_to_canvas_is_the_full_pass,
              pins_m.test_cached_pass_on_an_unchanged_canvas_gives_the_full_pass_rows,
              pins_m.test_cache_is_stale_outside_the_block_and_fresh_inside, pins_m.test_cached_layer_against_loops]
CACHE_MUTATIONS = {
    "cache: block rows rotated as if they sat at position 0": ("rope", mut_rope_block_rows_start_at_zero),
    "cache: keys and values after the block dropped": ("layer", mut_layer_cache_drops_the_suffix),
    "cache: context ignored": ("layer", mut_layer_cache_ignored),
}


@pytest.mark.parametrize("name", sorted(CACHE_MUTATIONS))
def test_cache_pins_catch(name, monkeypatch):
    assert not some_pin_fails(CACHE_PINS)
    attr, fn = CACHE_MUTATIONS[name]
    monkeypatch.setattr(mo, attr, fn)
    assert some_pin_fails(CACHE_PINS), f"no pin noticed: {name}"


MODEL_MUTATIONS = {
    "rope: rotation in the wrong direction on one half": ("rope", mut_rope_wrong_sign),
    "rope: interleaved pairs instead of rotate-half": ("rope", mut_rope_interleaved),
    "attention: causal mask": ("attention", mut_attention_causal),
    "attention: missing 1/sqrt(hd)": ("attention", mut_attention_no_scale),
    "attention: KV heads tiled instead of repeated": ("attention", mut_attention_wrong_gqa),
    "rmsnorm: subtracts the mean (LayerNorm)": ("rmsnorm", mut_rmsnorm_mean_subtracted),
    "rmsnorm: gain dropped": ("rmsnorm", mut_rmsnorm_no_gain),
    "lm head: bump added to every column": ("lm_head_logits", mut_lm_head_bump_everywhere),
}


@pytest.mark.parametrize("name", sorted(MODEL_MUTATIONS))
def test_model_pins_catch(name, monkeypatch):
    attr, fn = MODEL_MUTATIONS[name]
    monkeypatch.setattr(mo, attr, fn)
    assert some_pin_fails(MODEL_PINS), f"no pin noticed: {name}"
