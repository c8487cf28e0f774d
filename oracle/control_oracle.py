"""Oracle for the host-side decisions of the A/F data plane and the decode DVFS controller.
TEST INFRASTRUCTURE ONLY: imported by ``tests/`` alone; shares nothing with the library.

Plain Python restatements, in the paper's order and notation, of

* Eq. 2 (Section 4.3): layer time of the interleaved A/F pipeline;
* the interleaved schedule itself (Section 4.3: a microbatch proceeds as soon as its dependencies
  are satisfied; A of layer l+1 starts for microbatch i when F of layer l has returned it), as the
  longest path through the dependency graph of its stages;
* the choice of microbatch depth M and of the request split with the lowest predicted latency
  (Section 4.3, "Dynamic microbatch depth", "Adaptive request batching"), by exhaustive search;
* Algorithm 1 (window-based decode DVFS), the window-size rule that precedes it, and the prefill
  frequency-pair choice of Section 4.4.

Where the paper is silent the reading is stated at the function.
"""
from __future__ import annotations

import itertools
import math
from typing import Callable, List, Optional, Sequence, Tuple


# --------------------------------------------------------------------------- Eq. 2
def eq2_layer_time(t_a: float, t_f: float, t_comm: float, M: int) -> float:
    """Eq. 2: M = 1 -> t_A + t_F + t_comm;  M >= 2 -> max(t_A, t_F) + t_comm / M."""
    if M == 1:
        return t_a + t_f + t_comm
    return max(t_a, t_f) + t_comm / M


# --------------------------------------------------------------------------- profiled curves
def curve_eval(xs: Sequence[float], ys: Sequence[float], x: float) -> float:
    """Piecewise-linear interpolation through the profiled points (xs ascending); outside the
    profiled range the nearest segment is extended (a single point is a constant)."""
    n = len(xs)
    if n == 1:
        return ys[0]
    k = 0
    while k < n - 2 and x > xs[k + 1]:
        k += 1
    t = (x - xs[k]) / (xs[k + 1] - xs[k])
    return ys[k] + t * (ys[k + 1] - ys[k])


class Model:
    """Predicted stage times of one microbatch (microseconds).
    t_A = attn_tokens(sum of its context lengths) + attn_rows(rows);  t_F = ffn_rows(rows);
    one hidden-state transfer (either direction) = comm_fixed + comm_per_row * rows.
    shared = True: both sides run on one GPU and share its memory system; stages then do not
    overlap (reading: the measured one-GPU step times add up), and transfers cost nothing.
    A curve extended below zero predicts no time at all: stage times are clamped at zero."""

    def __init__(self, attn_tokens, attn_rows, ffn_rows, comm_fixed=0.0, comm_per_row=0.0, shared=False):
        self.attn_tokens, self.attn_rows, self.ffn_rows = attn_tokens, attn_rows, ffn_rows
        self.comm_fixed, self.comm_per_row, self.shared = comm_fixed, comm_per_row, shared

    def t_a(self, lens: Sequence[int]) -> float:
        return max(0.0, curve_eval(*self.attn_tokens, float(sum(lens))) + curve_eval(*self.attn_rows, float(len(lens))))

    def t_f(self, rows: int) -> float:
        return max(0.0, curve_eval(*self.ffn_rows, float(rows)))

    def t_x(self, rows: int) -> float:
        return 0.0 if self.shared else self.comm_fixed + self.comm_per_row * rows


# --------------------------------------------------------------------------- the interleaved schedule
def pipeline_makespan(model: Model, seq_lens: Sequence[int], offsets: Sequence[int], layers: int) -> float:
    """Longest path through the stage graph of `layers` layers x M microbatches.

    Stages of (l, i): A (attention side), X (transfer A -> F), F (FFN side), Y (transfer F -> A).
    Data edges: A -> X -> F -> Y -> A of (l+1, i).  Resource edges: each of the four engines (A GPUs,
    F GPUs, the two link directions) serves its stages one at a time in (l, i) order.  With
    model.shared all stages use one engine, in the order A(l,0) F(l,0) A(l,1) F(l,1) ...
    (reading: on one GPU the sides do not overlap)."""
    M = len(offsets) - 1
    dur = {}
    for i in range(M):
        rows = offsets[i + 1] - offsets[i]
        lens = seq_lens[offsets[i]:offsets[i + 1]]
        dur["A", i], dur["F", i], dur["X", i], dur["Y", i] = model.t_a(lens), model.t_f(rows), model.t_x(rows), model.t_x(rows)
    nodes = [(l, i, s) for l in range(layers) for i in range(M) for s in "AXFY"]
    preds = {n: [] for n in nodes}
    for l in range(layers):
        for i in range(M):
            preds[l, i, "X"].append((l, i, "A"))
            preds[l, i, "F"].append((l, i, "X"))
            preds[l, i, "Y"].append((l, i, "F"))
            if l + 1 < layers:
                preds[l + 1, i, "A"].append((l, i, "Y"))
    if model.shared:
        order = [(l, i, s) for l in range(layers) for i in range(M) for s in "AXFY"]
        for a, b in zip(order, order[1:]):
            preds[b].append(a)
    else:
        for s in "AXFY":
            order = [(l, i, s) for l in range(layers) for i in range(M)]
            for a, b in zip(order, order[1:]):
                preds[b].append(a)
    finish = {}

    def done(n):                      # memoised longest path to the end of stage n
        if n not in finish:
            start = max((done(p) for p in preds[n]), default=0.0)
            finish[n] = start + dur[n[2], n[1]]
        return finish[n]

    # iterate in an order that keeps the recursion shallow
    for n in nodes:
        done(n)
    return max(finish.values())


def plan_microbatches(model: Model, seq_lens: Sequence[int], layers: int, depths: Sequence[int],
                      granularity: int = 1) -> Tuple[int, List[int], float]:
    """Depth and contiguous split with the lowest predicted makespan, by exhaustive search over
    boundaries that are multiples of `granularity`.  Ties: the smaller depth, then the
    lexicographically smaller offsets (reading: the paper does not say)."""
    B = len(seq_lens)
    best = None
    for M in sorted(depths):
        if M < 1 or M > B:
            continue
        cuts = [c for c in range(granularity, B, granularity)]
        for inner in itertools.combinations(cuts, M - 1):
            offs = [0, *inner, B]
            t = pipeline_makespan(model, seq_lens, offs, layers)
            if best is None or t < best[2] - 1e-12:
                best = (M, offs, t)
    return best


# --------------------------------------------------------------------------- decode DVFS (Algorithm 1)
def dvfs_window(w_min: int, kappa: float, t_switch: float, t_iter: float) -> int:
    """W = max(W_min, round(kappa * T_switch / t_iter)) (Section 4.4, before Algorithm 1).
    Reading: round half away from zero."""
    return max(w_min, int(math.floor(kappa * t_switch / t_iter + 0.5)))


def dvfs_decode_step(f: Tuple[int, int], w: int, b_last: int, b_now: int, t_iter: float, tau: float, delta_b: float,
                     W: int, t_switch: float, t_hat: Sequence[Sequence[float]], e_hat: Sequence[Sequence[float]]):
    """Algorithm 1.  Frequencies are indices into the ascending DA / DF lists, so f_max is the last
    index of each; t_hat[a][f] / e_hat[a][f] are the predictions for the current decode state and
    depth.  Returns the new (f, w, b_last).  Reading: among equal-energy feasible pairs the first
    in (DA index, DF index) order wins."""
    w = w + 1
    delta = abs(b_now - b_last) / max(b_last, 1)
    if t_iter < tau and delta < delta_b and w < W:
        return f, w, b_last
    n_a, n_f = len(t_hat), len(t_hat[0])
    feasible = [(a, g) for a in range(n_a) for g in range(n_f) if t_hat[a][g] <= tau]
    if not feasible:
        return (n_a - 1, n_f - 1), 0, b_now
    star = min(feasible, key=lambda p: (e_hat[p[0]][p[1]], p[0], p[1]))
    if t_hat[f[0]][f[1]] > tau:
        f = star
    elif t_hat[star[0]][star[1]] + t_switch / W <= tau:
        f = star
    return f, 0, b_now


def dvfs_prefill_pair(t_hat, e_hat, budget: float, t_switch: float, current: Tuple[int, int], base: Tuple[int, int]):
    """Prefill pair (Section 4.4): among the pairs whose predicted time for the remaining layers,
    plus the switching overhead when the pair differs from the current one, fits the tightest
    remaining TTFT budget, the one with the lowest predicted energy.  Returns (pair, escalated,
    infeasible): escalated when the chosen pair exceeds the global plan's baseline in either
    domain; with no feasible pair, (f_max, f_max) and infeasible."""
    n_a, n_f = len(t_hat), len(t_hat[0])
    feasible = []
    for a in range(n_a):
        for g in range(n_f):
            cost = t_hat[a][g] + (t_switch if (a, g) != tuple(current) else 0.0)
            if cost <= budget:
                feasible.append((a, g))
    infeasible = not feasible
    if infeasible:
        star = (n_a - 1, n_f - 1)
    else:
        star = min(feasible, key=lambda p: (e_hat[p[0]][p[1]], p[0], p[1]))
    return star, (star[0] > base[0] or star[1] > base[1]), infeasible
