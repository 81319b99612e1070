"""CPU oracle for JoT token-level early stopping -- TEST INFRASTRUCTURE ONLY.

A plain, slow restatement of the method in the paper's own order and notation
(Section 4.1 and Algorithm 1 of "Just on Time: Token-Level Early Stopping for
Diffusion Language Models").  It shares no code with the CUDA library, is never
imported by it, and exists only so that tests, the smoke check and the
benchmark's CPU-baseline leg have something independent to compare against.

All floating point is float64.  Where floating point decides an integer (the
test r >= tau of Eq. 8), both operands are first rounded to float32 -- the
precision the device kernel takes the decision in -- and `near_margin` reports
the positions whose decision is within 1e-3 (relative) of flipping.

Readings taken where the paper is silent (each is a keyword argument so the
choice is visible at the call site):
  * the mask token itself is not a candidate prediction (`exclude_mask_token`);
  * argmax ties resolve to the lowest token id; on an exact tie of the two
    largest logits p2 = p1;
  * the window sum of Eq. 5 skips j = i (i is masked) and positions outside the
    canvas contribute nothing; w_max is not adjusted at the canvas edges;
  * the transfer schedule is "k highest max-probability positions", with k from
    a fixed per-block table (or, as an option, the share of what is still
    masked that keeps the block on pace: fractional_transfer_count), and it
    ranks ALL currently masked candidates; its
    mask is OR-ed with the early-exit mask (Section 4.2 "Implementation
    details"); `schedule_after_exit=True` gives the other reading of
    Algorithm 1 (schedule ranks only what early exit left masked);
  * in block mode candidates are restricted to the current block while the
    spatial window still sees the whole canvas;
  * the "global early-commit rule" of the related work is read as: mean top-2
    logit gap of the candidates >= one threshold (see JotParams).

Parity unpinned: the choice among those readings (no printed output of the
paper distinguishes them).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Callable, List, Optional, Sequence, Tuple

import numpy as np


@dataclasses.dataclass(frozen=True)
class JotParams:
    """tau_max, tau_min, gamma, D of Algorithm 1; eps of Eq. 4 (1e-12, Section 4.2).

    gate = "ratio" is the paper's test r >= tau (Eq. 8).  gate = "maxprob" is the fixed probability gate the
    paper contrasts it with (Section 2: a position is finalised when its max probability clears a threshold,
    0.9 in the compared system): p1 >= prob_threshold, no spatial modulation.  gate = "globalgap" is the
    global early-commit rule the paper contrasts it with (Section 2: "once the top-2 confidence gap exceeds a
    threshold, all remaining masked positions are finalized simultaneously"): the mean over the candidates of
    the top-2 logit gap m1 - m2 is tested against gap_threshold and either every candidate exits or none does.
    The compared system stages three thresholds over decoding progress (7.5 / 5.0 / 2.5, Section 6.1 "Experimental Setup"); here
    the threshold is one input that a caller may change from step to step."""
    tau_max: float = 90.0
    tau_min: float = 1.0
    gamma: float = 0.5
    D: int = 8
    eps: float = 1e-12
    gate: str = "ratio"
    prob_threshold: float = 0.9
    gap_threshold: float = 5.0


DREAM_DEFAULT = JotParams(90.0, 1.0, 0.5, 8)   # Table 1 caption
LLADA_DEFAULT = JotParams(30.0, 1.0, 0.5, 8)   # Table 1 caption


# ----------------------------------------------------------------------------
# Eq. 4: confidence ratio from one row of logits
# ----------------------------------------------------------------------------
@dataclasses.dataclass
class RowStats:
    m1: float      # largest logit
    i1: int        # its index (lowest index among maxima)
    m2: float      # second-largest logit as an order statistic (== m1 on an exact tie)
    S: float       # sum_v exp(l_v - m1)

    @property
    def p1(self) -> float:
        return 1.0 / self.S

    @property
    def p2(self) -> float:
        return math.exp(self.m2 - self.m1) / self.S


def row_stats(logits: np.ndarray, mask_id: Optional[int] = None) -> RowStats:
    """Softmax without temperature over one row of logits; top-2 by a full sort (Section 4.1,
    "Confidence Metric").  If mask_id is given that column is not a candidate."""
    l = np.asarray(logits, dtype=np.float64).copy()
    if mask_id is not None:
        l[mask_id] = -np.inf
    order = np.argsort(-l, kind="stable")      # stable: lowest index first among equals
    i1 = int(order[0])
    m1 = float(l[i1])
    m2 = float(l[order[1]])
    S = float(np.sum(np.exp(l - m1)))
    return RowStats(m1, i1, m2, S)


def row_stats_slice(logits: np.ndarray, v_lo: int, v_hi: int, mask_id: Optional[int] = None) -> RowStats:
    """row_stats over the token ids [v_lo, v_hi) only; i1 stays a global token id.  A slice with no candidate
    (nothing but the excluded mask token) gives the neutral element (-inf, 2^31 - 1, -inf, 0)."""
    l = np.asarray(logits, dtype=np.float64)[v_lo:v_hi].copy()
    if mask_id is not None and v_lo <= mask_id < v_hi:
        l[mask_id - v_lo] = -np.inf
    if l.size == 0 or not np.isfinite(l.max()):
        return RowStats(-math.inf, 2 ** 31 - 1, -math.inf, 0.0)
    order = np.argsort(-l, kind="stable")
    m1 = float(l[order[0]])
    m2 = float(l[order[1]]) if l.size > 1 else -math.inf
    return RowStats(m1, v_lo + int(order[0]), m2, float(np.sum(np.exp(l - m1))))


def merge_row_stats(a: RowStats, b: RowStats) -> RowStats:
    """Statistics of one row over two disjoint sets of token ids -> over their union (what a vocabulary-parallel
    head does with its ranks' results).  The largest logit is the larger of the two; the runner-up is the
    largest of the two runner-ups and the smaller of the two maxima; the sums are brought to the new maximum;
    equal maxima resolve to the lower token id."""
    m1 = max(a.m1, b.m1)
    m2 = max(a.m2, b.m2, min(a.m1, b.m1))
    S = (0.0 if a.m1 == -math.inf else a.S * math.exp(a.m1 - m1)) + (0.0 if b.m1 == -math.inf else b.S * math.exp(b.m1 - m1))
    i1 = b.i1 if (b.m1 > a.m1 or (b.m1 == a.m1 and b.i1 < a.i1)) else a.i1
    return RowStats(m1, i1, m2, S)


def confidence_ratio(p1: float, p2: float, eps: float = 1e-12) -> float:
    """Eq. 4: r = p1 / (p2 + eps)."""
    return p1 / (p2 + eps)


# ----------------------------------------------------------------------------
# Section 4.1, "Early-Exit Decision": the finalised token may be sampled from pi instead of argmax
# ----------------------------------------------------------------------------
_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15


def _mix64(z: int) -> int:
    """Output function of splitmix64 (Steele, Lea, Flood 2014; Vigna's reference implementation)."""
    z &= _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def splitmix64_output(state0: int, n: int) -> int:
    """n-th output (n >= 1) of the splitmix64 stream whose state starts at state0."""
    return _mix64(state0 + n * _GOLDEN)


def gumbel_key(seed: int, step: int, flat_pos: int) -> int:
    """Start state of the stream that serves one (step, canvas position): a mix of the three numbers."""
    return _mix64((seed ^ (step << 40) ^ flat_pos) & _M64)


def sample_token(logits: np.ndarray, mask_id: Optional[int], temperature: float, seed: int, step: int,
                 flat_pos: int) -> int:
    """Draw from softmax(l / temperature) by the Gumbel-max identity: argmax_v (l_v / T + G_v), G_v = -ln(-ln u_v).

    u_v comes from a counter-based generator so that any implementation can reproduce the draw: the top 23
    bits k of output number v + 1 of the splitmix64 stream keyed by (seed, step, position) give
    u = (k + 0.5) / 2^23.  Ties resolve to the lowest token id; the mask column is not a candidate."""
    l = np.asarray(logits, dtype=np.float64)
    key = gumbel_key(seed, step, flat_pos)
    best, best_v = -math.inf, -1
    inv_t = 1.0 / temperature
    for v in range(l.shape[0]):
        if v == mask_id:
            continue
        k = splitmix64_output(key, v + 1) >> 41
        u = (k + 0.5) / float(1 << 23)
        score = l[v] * inv_t - math.log(-math.log(u))
        if score > best:
            best, best_v = score, v
    return best_v


def sample_tokens_fast(logits: np.ndarray, mask_id: Optional[int], temperature: float, seed: int, step: int,
                       flat_pos: int) -> Tuple[int, float]:
    """Same draw as sample_token with numpy integer arithmetic (for vocabularies of 1e5 entries); also returns
    the gap between the two largest perturbed scores (a draw decided by less than rounding noise is a tie)."""
    l = np.asarray(logits, dtype=np.float64)
    key = np.uint64(gumbel_key(seed, step, flat_pos))
    with np.errstate(over="ignore"):
        z = key + (np.arange(1, l.shape[0] + 1, dtype=np.uint64)) * np.uint64(_GOLDEN)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    u = ((z >> np.uint64(41)).astype(np.float64) + 0.5) / float(1 << 23)
    score = l / temperature - np.log(-np.log(u))
    if mask_id is not None:
        score[mask_id] = -np.inf
    order = np.argsort(-score, kind="stable")
    return int(order[0]), float(score[order[0]] - score[order[1]])


# ----------------------------------------------------------------------------
# Eq. 5-7: spatial weight, softening factor, adaptive threshold
# ----------------------------------------------------------------------------
def w_max(gamma: float, D: int) -> float:
    """Eq. 6 text: w_max = 2 * sum_{d=1..D} gamma^d."""
    return 2.0 * sum(gamma ** d for d in range(1, D + 1))


def spatial_weight(x: Sequence[int], i: int, mask_id: int, gamma: float, D: int) -> float:
    """Eq. 5: sum of gamma^|i-j| over unmasked j with |i-j| <= D, written as the double loop it is.
    j ranges over the whole canvas (prompt tokens count as unmasked)."""
    w = 0.0
    for j in range(len(x)):
        if j == i:
            continue
        if abs(i - j) <= D and x[j] != mask_id:
            w += gamma ** abs(i - j)
    return w


def softening(w: float, gamma: float, D: int) -> float:
    """Eq. 6: phi = min(1, w / w_max)."""
    return min(1.0, w / w_max(gamma, D))


def threshold(phi: float, tau_max: float, tau_min: float) -> float:
    """Eq. 7: tau = tau_max - (tau_max - tau_min) * phi."""
    return tau_max - (tau_max - tau_min) * phi


def position_threshold(x: Sequence[int], i: int, mask_id: int, p: JotParams) -> float:
    return threshold(softening(spatial_weight(x, i, mask_id, p.gamma, p.D), p.gamma, p.D),
                     p.tau_max, p.tau_min)


# ----------------------------------------------------------------------------
# transfer schedule (Section 3.2; Section 4.2 "Interaction with transfer schedules")
# ----------------------------------------------------------------------------
def transfer_counts(block_len: int, steps_per_block: int) -> List[int]:
    """How many positions the schedule reveals at each step of a block: block_len spread evenly over
    the steps, the remainder going to the earliest steps."""
    base, rem = divmod(block_len, steps_per_block)
    return [base + (1 if s < rem else 0) for s in range(steps_per_block)]


def fractional_transfer_count(n_masked: int, steps_left: int) -> int:
    """The adaptive alternative to the fixed table: with `steps_left` steps of the block still to run (this one
    included), reveal the share of what is STILL masked that keeps the block on pace to end with its last step:
    ceil(n_masked / steps_left).  The paper leaves the schedule to "the model's default unmasking schedule"
    (Section 4.2, "Interaction with transfer schedules"); samplers of the Dream family reveal a fraction of the
    remaining masked positions per step, which is this rule up to how the fraction is rounded.  Rounding up is this
    build's reading: it reveals at least one position while any is masked (every step makes progress, the block
    ends within its steps), and without early exits it reproduces transfer_counts exactly."""
    assert steps_left >= 1
    return -(-n_masked // steps_left)


# ----------------------------------------------------------------------------
# one acceptance / freeze update (inner part of Algorithm 1)
# ----------------------------------------------------------------------------
@dataclasses.dataclass
class StepReport:
    exited: List[int]          # E: positions finalised by the early-exit test
    scheduled: List[int]       # U: positions chosen by the transfer schedule
    near_margin: List[int]     # |r - tau| <= 1e-3 * tau : decision may legitimately differ in fp32
    ratio: dict                # position -> r
    tau: dict                  # position -> tau


def accept_freeze(x: List[int], stats: dict, p: JotParams, mask_id: int, blk_lo: int, blk_hi: int,
                  k_transfer: int, schedule_after_exit: bool = False, tokens: Optional[dict] = None) -> StepReport:
    """Update one sequence in place.  `stats[i]` is a RowStats for every masked i in [blk_lo, blk_hi).

    All decisions use the canvas and the statistics as they were at the start of the step.  `tokens[i]`, when
    given, is the token a finalised position receives (a sample from pi) instead of its argmax.
    """
    x0 = list(x)
    A = [i for i in range(blk_lo, blk_hi) if x0[i] == mask_id]          # Algorithm 1: M_n (in block)
    ratio, tau, near = {}, {}, []
    E = []
    if p.gate == "globalgap" and A:                                       # global early commit (Section 2)
        mean_gap = sum(stats[i].m1 - stats[i].m2 for i in A) / len(A)
        if abs(mean_gap - p.gap_threshold) <= 1e-3 * abs(p.gap_threshold):
            near = list(A)
        if np.float32(mean_gap) >= np.float32(p.gap_threshold):           # decided in float32
            E = list(A)
    for i in A:
        st = stats[i]
        r = confidence_ratio(st.p1, st.p2, p.eps)                         # Eq. 4
        t = position_threshold(x0, i, mask_id, p)                         # Eq. 5-7
        ratio[i], tau[i] = r, t
        if p.gate == "globalgap":
            continue
        if p.gate == "maxprob":                                           # fixed probability gate (Section 2)
            if abs(st.p1 - p.prob_threshold) <= 1e-3 * p.prob_threshold:
                near.append(i)
            if np.float32(st.p1) >= np.float32(p.prob_threshold):
                E.append(i)
            continue
        if abs(r - t) <= 1e-3 * abs(t):
            near.append(i)
        if np.float32(r) >= np.float32(t):                                # Eq. 8, decided in float32
            E.append(i)
    cand = [i for i in A if i not in E] if schedule_after_exit else A
    k = min(k_transfer, len(cand))
    ranked = sorted(cand, key=lambda i: (-stats[i].p1, i))                # highest max-prob, ties -> lower i
    U = sorted(ranked[:k])
    for i in set(E) | set(U):                                             # logical OR, uncapped
        x[i] = stats[i].i1 if tokens is None else tokens[i]               # finalise by argmax (or by the sample)
    return StepReport(E, U, near, ratio, tau)


# ----------------------------------------------------------------------------
# Algorithm 1 (with semi-autoregressive blocks for block_len < gen_len)
# ----------------------------------------------------------------------------
@dataclasses.dataclass
class Trajectory:
    x: List[int]
    steps_used: int
    canvases: List[List[int]]        # canvas BEFORE each step that ran
    reports: List[StepReport]
    exit_step: List[int]             # per position: 1-based step that finalised it, 0 if never masked
    blocks: List[Tuple[int, int]]    # (blk_lo, blk_hi) of each step that ran


def generate(logits_fn: Callable[[List[int], List[int]], dict], prompt: Sequence[int], gen_len: int,
             steps: int, p: JotParams, mask_id: int, block_len: Optional[int] = None,
             exclude_mask_token: bool = True, schedule_after_exit: bool = False,
             stats_fn: Optional[Callable[[List[int], List[int]], dict]] = None,
             sampling: Optional[Tuple[float, int]] = None, seq_index: int = 0,
             schedule: str = "fixed") -> Trajectory:
    """Algorithm 1 for one sequence.

    logits_fn(x, rows) returns {i: logits row (length K)} for the requested masked positions;
    alternatively stats_fn(x, rows) returns {i: RowStats} directly (for stub models in tests).
    sampling = (temperature, seed): finalised positions receive a sample from softmax(l / temperature) drawn
    with sample_tokens_fast, keyed by the 0-based index of the forward pass and the position's flat canvas
    index seq_index * L + i; the acceptance decisions themselves do not change.
    schedule = "fixed": the per-block table of transfer_counts; "fractional": fractional_transfer_count of what
    is still masked in the block and the steps the block has left.
    """
    assert schedule in ("fixed", "fractional")
    P = len(prompt)
    Lb = gen_len if block_len is None else block_len
    assert gen_len % Lb == 0
    nb = gen_len // Lb
    assert steps % nb == 0
    Tb = steps // nb
    ks = transfer_counts(Lb, Tb)
    x = list(prompt) + [mask_id] * gen_len                                # initialise canvas
    traj = Trajectory(x, 0, [], [], [0] * (P + gen_len), [])
    for blk in range(nb):
        lo, hi = P + blk * Lb, P + (blk + 1) * Lb
        for s in range(Tb):
            A = [i for i in range(lo, hi) if x[i] == mask_id]             # M_n
            if not A:                                                     # break when nothing is masked
                break
            drawn = None
            if stats_fn is not None:
                stats = stats_fn(x, A)
            else:
                rows = logits_fn(x, A)
                stats = {i: row_stats(rows[i], mask_id if exclude_mask_token else None) for i in A}
                if sampling is not None:
                    drawn = {i: sample_tokens_fast(rows[i], mask_id if exclude_mask_token else None, sampling[0],
                                                   sampling[1], traj.steps_used, seq_index * len(x) + i)[0] for i in A}
            traj.canvases.append(list(x))
            traj.blocks.append((lo, hi))
            k = ks[s] if schedule == "fixed" else fractional_transfer_count(len(A), Tb - s)
            rep = accept_freeze(x, stats, p, mask_id, lo, hi, k, schedule_after_exit, drawn)
            traj.reports.append(rep)
            traj.steps_used += 1
            for i in set(rep.exited) | set(rep.scheduled):
                traj.exit_step[i] = traj.steps_used
        assert all(x[i] != mask_id for i in range(lo, hi)), "block not finished within its steps"
    return traj
