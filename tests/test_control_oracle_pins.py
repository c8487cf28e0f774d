"""Pins for the control-side oracle (Eq. 2, the interleaved schedule, the depth / split choice,
Algorithm 1): hand-walked timelines, closed forms and the paper's own limits.  No GPU needed."""
import itertools

import numpy as np
import pytest

from oracle import control_oracle as C

CONST = lambda v: ([0.0], [v])


def const_model(a, f, x=0.0, per_row=0.0, shared=False):
    """Every microbatch costs a on the A side and f on the F side, whatever its size."""
    return C.Model(CONST(a), CONST(0.0), CONST(f), comm_fixed=x, comm_per_row=per_row, shared=shared)


def test_eq2_values():
    assert C.eq2_layer_time(3.0, 5.0, 2.0, 1) == 10.0
    assert C.eq2_layer_time(3.0, 5.0, 2.0, 2) == 6.0
    assert C.eq2_layer_time(7.0, 5.0, 2.0, 4) == 7.5


def test_curve_eval():
    xs, ys = [1.0, 2.0, 4.0], [10.0, 20.0, 30.0]
    assert C.curve_eval(xs, ys, 1.0) == 10.0 and C.curve_eval(xs, ys, 4.0) == 30.0
    assert C.curve_eval(xs, ys, 1.5) == 15.0 and C.curve_eval(xs, ys, 3.0) == 25.0
    assert C.curve_eval(xs, ys, 0.0) == 0.0          # first segment extended
    assert C.curve_eval(xs, ys, 6.0) == 40.0         # last segment extended
    assert C.curve_eval([5.0], [7.0], 100.0) == 7.0


def test_makespan_depth_one_is_eq2_first_case():
    m = const_model(3.0, 5.0, x=1.0)
    for L in (1, 2, 7):
        want = L * C.eq2_layer_time(3.0, 5.0, 2.0, 1)      # t_comm = one transfer each way
        assert C.pipeline_makespan(m, [10] * 6, [0, 6], L) == pytest.approx(want)


def test_makespan_hand_walked_timeline():
    # a = 3, f = 5, x = 1, M = 2, one layer:
    # A0 0-3, X0 3-4, F0 4-9, Y0 9-10; A1 3-6, X1 6-7, F1 9-14, Y1 14-15
    m = const_model(3.0, 5.0, x=1.0)
    assert C.pipeline_makespan(m, [10] * 4, [0, 2, 4], 1) == pytest.approx(15.0)


@pytest.mark.parametrize("a,f", [(4.0, 3.0), (2.0, 5.0), (3.0, 3.0)])
def test_makespan_two_microbatches_no_transfer_closed_form(a, f):
    m = const_model(a, f)
    for L in (1, 3, 10):
        got = C.pipeline_makespan(m, [8] * 4, [0, 2, 4], L)
        want = 2 * a * L + f if a >= f else a + 2 * f * L
        assert got == pytest.approx(want)


def test_steady_state_layer_time_is_eq2_second_case():
    # balanced sides, transfer proportional to rows: every extra layer costs max(t_A, t_F) + t_comm / M
    B, M = 8, 2
    a = f = 6.0                                            # per microbatch; per layer t_A = t_F = M * a
    per_row = 0.25                                         # one direction; whole batch both ways: t_comm = 2 * B * per_row
    m = const_model(a, f, per_row=per_row)
    offs = [0, 4, 8]
    t9, t10 = (C.pipeline_makespan(m, [5] * B, offs, L) for L in (9, 10))
    assert t10 - t9 == pytest.approx(C.eq2_layer_time(M * a, M * f, 2 * B * per_row, M))


def test_shared_memory_system_adds_every_stage():
    m = const_model(3.0, 5.0, x=9.0, shared=True)
    assert C.pipeline_makespan(m, [1] * 6, [0, 2, 4, 6], 4) == pytest.approx(4 * 3 * (3.0 + 5.0))


def test_stage_times_follow_the_curves():
    m = C.Model(([0.0, 100.0], [1.0, 11.0]), ([0.0, 10.0], [0.0, 5.0]), ([0.0, 10.0], [2.0, 12.0]), shared=True)
    # microbatch 0: lens 10+30 = 40 tokens, 2 rows: t_A = 5 + 1 = 6, t_F = 4; microbatch 1: 60 tokens, 1 row: 7 + .5, 3
    assert C.pipeline_makespan(m, [10, 30, 60], [0, 2, 3], 1) == pytest.approx(6.0 + 4.0 + 7.5 + 3.0)


def test_stage_time_is_clamped_at_zero_as_a_whole_not_curve_by_curve():
    # Reading (the paper's "profiled Attention/FFN latency curves" says nothing about extrapolation): a stage's
    # duration is the physical quantity and cannot be negative, while the two terms of t_A are only a fit whose
    # parts may have either sign (a negative token-term offset by a positive row-term is a legitimate fit).  So the
    # SUM is clamped, not each curve.  Numbers by hand: the token curve through (100, 10), (200, 30) has slope 0.2,
    # so 20 tokens give 10 - 80 * 0.2 = -6.
    tokens = ([100.0, 200.0], [10.0, 30.0])
    assert C.curve_eval(*tokens, 20.0) == pytest.approx(-6.0)
    # (a) row term +4: -6 + 4 = -2 -> the stage takes 0 (unclamped: -2; clamped curve by curve: 0 + 4 = 4)
    m = C.Model(tokens, CONST(4.0), CONST(3.0), shared=True)
    assert m.t_a([20]) == 0.0
    assert C.pipeline_makespan(m, [20], [0, 1], 1) == pytest.approx(0.0 + 3.0)
    # (b) row term +10: -6 + 10 = 4 stays 4 (clamped curve by curve: 0 + 10 = 10)
    m = C.Model(tokens, CONST(10.0), CONST(3.0), shared=True)
    assert m.t_a([20]) == pytest.approx(4.0)
    assert C.pipeline_makespan(m, [20], [0, 1], 2) == pytest.approx(2 * (4.0 + 3.0))
    # (c) the FFN curve through (10, 5), (20, 25) has slope 2: one row gives 5 - 18 = -13 -> 0 (unclamped: 4 - 13 = -9)
    m = C.Model(tokens, CONST(10.0), ([10.0, 20.0], [5.0, 25.0]), shared=True)
    assert m.t_f(1) == 0.0 and m.t_f(15) == pytest.approx(15.0)
    assert C.pipeline_makespan(m, [20], [0, 1], 1) == pytest.approx(4.0)
    # separate pools: the clamped stage still occupies no time on its engine (A0 0-0, F0 0-3, A1 0-0, F1 3-6)
    m = C.Model(tokens, CONST(4.0), CONST(3.0))
    assert C.pipeline_makespan(m, [20, 20], [0, 1, 2], 1) == pytest.approx(6.0)


def test_plan_prefers_depth_one_on_a_shared_memory_system():
    # fixed cost per stage launch (curves with an intercept): splitting only adds cost
    m = C.Model(([0.0, 1000.0], [10.0, 110.0]), CONST(5.0), ([0.0, 64.0], [100.0, 110.0]), shared=True)
    M, offs, t = C.plan_microbatches(m, [100] * 16, 4, [1, 2, 4])
    assert M == 1 and offs == [0, 16]
    assert t == pytest.approx(4 * (10 + 160 + 5 + 102.5))


def test_plan_prefers_two_microbatches_on_separate_pools_at_high_load():
    # costs proportional to the work, no intercepts, cheap transfer: overlap wins
    m = C.Model(([0.0, 1000.0], [0.0, 100.0]), CONST(0.0), ([0.0, 64.0], [0.0, 640.0]), comm_per_row=0.01)
    lens = [100] * 16
    M, offs, t = C.plan_microbatches(m, lens, 8, [1, 2])
    assert M == 2
    t1 = C.pipeline_makespan(m, lens, [0, 16], 8)
    assert t < 0.6 * t1           # balanced sides: close to half


def test_plan_adaptive_split_beats_equal_split_and_is_the_exhaustive_optimum():
    # one layer, F twice as slow as A, costs proportional to the work: with a share r of the rows in the
    # first microbatch the makespan is r a + max((1 - r) a, r f) + (1 - r) f, least at r = 1/3
    lens = [100] * 12
    a, f = 120.0, 240.0
    m = C.Model(([0.0, 1200.0], [0.0, a]), CONST(0.0), ([0.0, 12.0], [0.0, f]))
    M, offs, t = C.plan_microbatches(m, lens, 1, [2])
    assert offs == [0, 4, 12] and t == pytest.approx(280.0)
    assert C.pipeline_makespan(m, lens, [0, 6, 12], 1) == pytest.approx(300.0)
    for c in range(1, 12):
        r = c / 12.0
        assert C.pipeline_makespan(m, lens, [0, c, 12], 1) == pytest.approx(r * a + max((1 - r) * a, r * f) + (1 - r) * f)
    # granularity restricts the boundaries
    M3, offs3, t3 = C.plan_microbatches(m, lens, 1, [2], granularity=3)
    assert offs3[1] % 3 == 0 and t3 >= t
    # depth and split together
    M, offs, t2 = C.plan_microbatches(m, lens, 1, [1, 2, 3])
    every = {(M_,) + inner: C.pipeline_makespan(m, lens, [0, *inner, 12], 1)
             for M_ in (1, 2, 3) for inner in itertools.combinations(range(1, 12), M_ - 1)}
    assert t2 == pytest.approx(min(every.values())) and M == 3


# --------------------------------------------------------------------------- Algorithm 1
T_HAT = [[9.0, 7.0, 6.0], [8.0, 6.0, 5.0], [7.5, 5.5, 4.5]]      # rows: DA index, columns: DF index
E_HAT = [[1.0, 1.4, 2.0], [1.2, 1.6, 2.2], [1.5, 1.9, 2.6]]


def step(f, w, b_last, b_now, t_iter, tau, W=10, delta_b=0.2, t_switch=5.0):
    return C.dvfs_decode_step(f, w, b_last, b_now, t_iter, tau, delta_b, W, t_switch, T_HAT, E_HAT)


def test_alg1_keeps_the_pair_inside_a_quiet_window():
    assert step((1, 1), 3, 100, 105, 5.0, 6.5) == ((1, 1), 4, 100)


def test_alg1_triggers_on_window_end_batch_change_or_slow_iteration():
    # feasible pairs for tau = 6.5: t_hat <= 6.5 -> (0,2) e=2.0, (1,1) 1.6, (1,2) 2.2, (2,1) 1.9, (2,2) 2.6: f* = (1,1)
    assert step((1, 1), 9, 100, 100, 5.0, 6.5) == ((1, 1), 0, 100)               # w reaches W
    assert step((1, 2), 0, 100, 130, 5.0, 6.5)[1:] == (0, 130)                    # batch changed by 30 %
    assert step((1, 2), 0, 100, 100, 6.5, 6.5)[1:] == (0, 100)                    # t_iter not below tau


def test_alg1_switches_at_once_when_the_current_pair_misses_tau():
    # current (0,0): t_hat 9.0 > tau -> f* immediately, even if the lazy rule would refuse
    assert step((0, 0), 9, 100, 100, 9.0, 6.5, t_switch=1000.0) == ((1, 1), 0, 100)


def test_alg1_lazy_switch_counts_the_amortised_switching_time():
    # current (2,2) is feasible (4.5); f* = (1,1) with t_hat 6.0: switch only if 6.0 + T_switch / W <= 6.5
    assert step((2, 2), 9, 100, 100, 4.0, 6.5, W=10, t_switch=5.0) == ((1, 1), 0, 100)     # 6.0 + 0.5 <= 6.5
    assert step((2, 2), 9, 100, 100, 4.0, 6.5, W=10, t_switch=5.1) == ((2, 2), 0, 100)     # 6.51 > 6.5


def test_alg1_falls_back_to_maximum_frequencies():
    assert step((0, 1), 9, 100, 100, 9.0, 4.0) == ((2, 2), 0, 100)                # nothing reaches tau = 4.0


def test_alg1_energy_ties_take_the_first_pair():
    t = [[1.0, 1.0], [1.0, 1.0]]
    e = [[2.0, 1.0], [1.0, 1.0]]
    assert C.dvfs_decode_step((1, 1), 9, 4, 4, 0.5, 2.0, 0.5, 10, 0.0, t, e)[0] == (0, 1)


def test_window_rule():
    assert C.dvfs_window(8, 10.0, 2.0, 4.0) == 8            # round(5) = 5 < W_min
    assert C.dvfs_window(8, 10.0, 20.0, 4.0) == 50
    assert C.dvfs_window(1, 1.0, 5.0, 2.0) == 3             # 2.5 rounds away from zero


def test_prefill_pair():
    # budget 7.0, switching costs 0.5 unless the pair is the current one (1,2)
    pair, esc, inf = C.dvfs_prefill_pair(T_HAT, E_HAT, 7.0, 0.5, (1, 2), (1, 1))
    # feasible: (0,2) 6.5, (1,1) 6.5, (1,2) 5.0, (2,1) 6.0, (2,2) 5.0 -> lowest energy (1,1) = 1.6
    assert (pair, esc, inf) == ((1, 1), False, False)
    pair, esc, inf = C.dvfs_prefill_pair(T_HAT, E_HAT, 5.2, 0.5, (1, 2), (1, 1))
    assert (pair, esc, inf) == ((1, 2), True, False)         # (2,2) needs 4.5 + 0.5 too, but costs more energy
    pair, esc, inf = C.dvfs_prefill_pair(T_HAT, E_HAT, 1.0, 0.5, (1, 2), (1, 1))
    assert (pair, esc, inf) == ((2, 2), True, True)
