"""The library's host-side decisions (Eq. 2, interleaved-schedule makespan, depth / split choice,
Algorithm 1, prefill pair) against the control oracle, through the C ABI.  Host code only: runs
without a GPU."""
import math

import numpy as np
import pytest

from oracle import control_oracle as C
from paper_2608_01891_b200 import aflex as AF


def random_curve(rng, x_hi, y_hi, n=None):
    n = int(rng.integers(1, 5)) if n is None else n
    xs = np.sort(rng.choice(np.arange(0, x_hi + 1), size=n, replace=False)).astype(float).tolist()
    ys = np.sort(rng.uniform(0.0, y_hi, size=n)).tolist()
    return xs, ys


def random_model(rng, shared=None):
    shared = bool(rng.integers(2)) if shared is None else shared
    at, ar, fr = random_curve(rng, 4000, 300.0), random_curve(rng, 32, 20.0), random_curve(rng, 32, 300.0)
    cf, cr = float(rng.uniform(0, 5)), float(rng.uniform(0, 1))
    return (C.Model(at, ar, fr, cf, cr, shared), AF.pipeline_model(at, ar, fr, cf, cr, shared))


def test_eq2_and_curves_match_the_oracle():
    rng = np.random.default_rng(0)
    for _ in range(50):
        a, f, c = rng.uniform(0, 100, 3)
        for M in (1, 2, 3, 8):
            assert AF.eq2_layer_time(a, f, c, M) == pytest.approx(C.eq2_layer_time(a, f, c, M), rel=1e-15)
        xs, ys = random_curve(rng, 100, 50.0)
        cv = AF.curve(xs, ys)
        for x in rng.uniform(-20, 150, 10):
            assert AF.curve_eval(cv, x) == pytest.approx(C.curve_eval(xs, ys, x), rel=1e-12, abs=1e-12)
    assert math.isnan(AF.curve_eval(AF.curve([1.0, 1.0], [0.0, 1.0]), 0.5))      # x not strictly ascending


def test_makespan_matches_the_longest_path_oracle():
    rng = np.random.default_rng(1)
    for _ in range(200):
        om, lm = random_model(rng)
        B = int(rng.integers(1, 20))
        lens = rng.integers(1, 400, size=B).tolist()
        M = int(rng.integers(1, min(B, 5) + 1))
        cuts = sorted(rng.choice(np.arange(1, B), size=M - 1, replace=False).tolist()) if M > 1 else []
        offs = [0, *cuts, B]
        L = int(rng.integers(1, 6))
        assert AF.pipeline_makespan(lm, lens, offs, L) == pytest.approx(C.pipeline_makespan(om, lens, offs, L), rel=1e-12)


def test_library_clamps_the_stage_time_as_a_whole():
    # the hand-computed cases that pin the oracle's reading (a stage's time, i.e. the SUM of the token term and the
    # row term, is clamped at zero; the curves themselves are not), here against the library
    tokens = ([100.0, 200.0], [10.0, 30.0])                    # 20 tokens -> -6
    const = lambda v: ([0.0], [v])
    m = AF.pipeline_model(tokens, const(4.0), const(3.0), 0.0, 0.0, True)
    assert AF.pipeline_makespan(m, [20], [0, 1], 1) == pytest.approx(3.0)            # t_A = max(0, -6 + 4) = 0
    m = AF.pipeline_model(tokens, const(10.0), const(3.0), 0.0, 0.0, True)
    assert AF.pipeline_makespan(m, [20], [0, 1], 2) == pytest.approx(14.0)           # t_A = -6 + 10 = 4, not 0 + 10
    m = AF.pipeline_model(tokens, const(10.0), ([10.0, 20.0], [5.0, 25.0]), 0.0, 0.0, True)
    assert AF.pipeline_makespan(m, [20], [0, 1], 1) == pytest.approx(4.0)            # t_F(1 row) = max(0, -13) = 0


def test_makespan_rejects_bad_arguments():
    _, lm = random_model(np.random.default_rng(2))
    assert math.isnan(AF.pipeline_makespan(lm, [5, 5], [0, 1], 1))          # offsets do not end at the batch
    assert math.isnan(AF.pipeline_makespan(lm, [5, 5], [0, 2, 2], 1))       # empty microbatch
    assert math.isnan(AF.pipeline_makespan(lm, [5, 5], [0, 2], 0))          # no layers


def test_plan_matches_exhaustive_oracle():
    rng = np.random.default_rng(3)
    for _ in range(60):
        om, lm = random_model(rng)
        B = int(rng.integers(1, 13))
        lens = rng.integers(1, 400, size=B).tolist()
        L = int(rng.integers(1, 5))
        depths = [int(d) for d in rng.choice([1, 2, 3, 4], size=int(rng.integers(1, 4)), replace=False)]
        g = int(rng.integers(1, 4))
        want = C.plan_microbatches(om, lens, L, depths, g)
        if want is None:
            with pytest.raises(AF.AflexError):
                AF.plan_microbatches(lm, lens, L, depths, g)
            continue
        M, offs, t = AF.plan_microbatches(lm, lens, L, depths, g)
        assert t == pytest.approx(want[2], rel=1e-12)
        assert (M, offs) == (want[0], want[1])


def test_plan_on_one_gpu_keeps_depth_one_and_separate_pools_split():
    # curves shaped like the measured ones of configuration 2: weight-streaming F (flat in rows),
    # attention proportional to context tokens, a fixed cost per stage
    lens = [2300] * 32
    at, ar, fr = ([0.0, 73600.0], [8.0, 58.0]), ([0.0, 32.0], [20.0, 24.0]), ([1.0, 32.0], [128.0, 132.0])
    one_gpu = AF.pipeline_model(at, ar, fr, shared_memory_system=True)
    assert AF.plan_microbatches(one_gpu, lens, 4, [1, 2, 4], 4)[0] == 1
    # separate A and F pools, F compute-bound (cost proportional to rows), cheap transfer: overlap pays
    pools = AF.pipeline_model(at, ar, ([0.0, 32.0], [0.0, 130.0]), comm_fixed=2.0, comm_per_row=0.02)
    M, offs, t = AF.plan_microbatches(pools, lens, 8, [1, 2], 4)
    assert M == 2 and t < 0.75 * AF.pipeline_makespan(pools, lens, [0, 32], 8)


def test_plan_refuses_an_oversized_search():
    _, lm = random_model(np.random.default_rng(4))
    with pytest.raises(AF.AflexError) as ei:
        AF.plan_microbatches(lm, [10] * 256, 2, [6], 1)
    assert ei.value.status == AF.ERR_UNSUPPORTED
    assert AF.plan_microbatches(lm, [10] * 256, 2, [4], 32)[0] == 4          # a coarser grid is fine


# --------------------------------------------------------------------------- DVFS
def test_window_rule_matches_oracle():
    rng = np.random.default_rng(5)
    for _ in range(200):
        w_min, kappa = int(rng.integers(1, 20)), float(rng.uniform(0.5, 20))
        ts, ti = float(rng.uniform(0.1, 50)), float(rng.uniform(0.5, 30))
        assert AF.dvfs_window(w_min, kappa, ts, ti) == C.dvfs_window(w_min, kappa, ts, ti)
    assert AF.dvfs_window(1, 1.0, 5.0, 2.0) == 3


def test_algorithm1_random_walk_matches_oracle():
    rng = np.random.default_rng(6)
    for trial in range(40):
        n_a, n_f = int(rng.integers(1, 5)), int(rng.integers(1, 5))
        W, tau = int(rng.integers(1, 8)), float(rng.uniform(3, 8))
        delta_b, t_switch = float(rng.uniform(0.05, 0.5)), float(rng.uniform(0, 10))
        params = AF.DvfsParams(n_a, n_f, tau, delta_b, W, t_switch)
        f = (int(rng.integers(n_a)), int(rng.integers(n_f)))
        state = AF.DvfsState(f[0], f[1], 0, 50)
        w, b_last, b = 0, 50, 50
        for it in range(60):
            # predictions: faster and costlier with higher indices, jittered per iteration
            base = rng.uniform(6, 10)
            t_hat = [[base - 0.8 * a - 0.6 * g + rng.uniform(0, 0.3) for g in range(n_f)] for a in range(n_a)]
            e_hat = [[round(1 + 0.3 * a + 0.2 * g + rng.choice([0.0, 0.1]), 1) for g in range(n_f)] for a in range(n_a)]
            b = max(0, b + int(rng.integers(-12, 13)))
            t_iter = float(rng.uniform(2, 9))
            f_new, w, b_last = C.dvfs_decode_step(f, w, b_last, b, t_iter, tau, delta_b, W, t_switch, t_hat, e_hat)
            code = AF.dvfs_decode_step(params, t_hat, e_hat, b, t_iter, state)
            assert (state.i_da, state.i_df, state.w, state.b_last) == (f_new[0], f_new[1], w, b_last), (trial, it)
            assert code == (0 if w != 0 else (2 if f_new != f else 1))
            f = f_new


def test_algorithm1_rejects_bad_state():
    params = AF.DvfsParams(2, 2, 5.0, 0.2, 4, 1.0)
    assert AF.dvfs_decode_step(params, [[1, 1], [1, 1]], [[1, 1], [1, 1]], 4, 1.0, AF.DvfsState(2, 0, 0, 4)) == -1
    assert AF.dvfs_decode_step(AF.DvfsParams(2, 2, 5.0, 0.2, 0, 1.0), [[1, 1], [1, 1]], [[1, 1], [1, 1]], 4, 1.0,
                               AF.DvfsState(0, 0, 0, 4)) == -1


def test_prefill_pair_matches_oracle():
    rng = np.random.default_rng(7)
    for _ in range(200):
        n_a, n_f = int(rng.integers(1, 5)), int(rng.integers(1, 5))
        t_hat = [[float(rng.uniform(2, 10)) for _ in range(n_f)] for _ in range(n_a)]
        e_hat = [[float(rng.integers(1, 6)) for _ in range(n_f)] for _ in range(n_a)]
        cur = (int(rng.integers(n_a)), int(rng.integers(n_f)))
        base = (int(rng.integers(n_a)), int(rng.integers(n_f)))
        budget, ts = float(rng.uniform(1, 12)), float(rng.uniform(0, 2))
        pair, esc, inf = C.dvfs_prefill_pair(t_hat, e_hat, budget, ts, cur, base)
        got_pair, flags = AF.dvfs_prefill_pair(t_hat, e_hat, budget, ts, cur, base)
        assert got_pair == pair
        assert bool(flags & AF.DVFS_ESCALATED) == esc and bool(flags & AF.DVFS_INFEASIBLE) == inf
