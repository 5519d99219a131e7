"""Pins of Algorithm 2 (slope-based per-class thresholds, Sec. 3.2) as the oracle reads it."""
import itertools

import numpy as np

import oracle
from oracle.calibrate import per_class_slopes, per_class_thresholds


def test_one_class_reduces_to_algorithm_1():
    rng = np.random.default_rng(1)
    U = rng.permutation(1000).astype(np.float32) / 1000
    pred = np.zeros(1000, np.uint8)
    correct = rng.integers(0, 2, 1000)
    tau, assigned, _ = per_class_thresholds(U, pred, correct, 1, 100, 24, 100)
    assert tau[0] == oracle.universal_thresholds(U, [76])[0]          # assigned portion 0.24 <-> q = 0.76
    assert assigned == 240 == int(np.count_nonzero(U > tau[0]))


def test_hand_example_the_class_with_wrong_uncertain_flows_goes_first():
    # class 0: scores .1 .2 .3 .4, the two most uncertain are wrong; class 1: scores .5 .6 .7 .8, all right.
    U = np.array([.1, .2, .3, .4, .5, .6, .7, .8], np.float32)
    pred = np.array([0, 0, 0, 0, 1, 1, 1, 1])
    correct = np.array([1, 1, 0, 0, 1, 1, 1, 1])
    R, tmax = per_class_slopes(U, pred, correct, 2, 4)
    # quantiles 3/4, 2/4, 1/4, 0 of 4 sorted scores -> thresholds U[3], U[2], U[1], U[1] (1-based)
    assert [float(t) for t, _, _ in R[0]] == [np.float32(.3), np.float32(.2), np.float32(.1)]
    assert [(dI, dA) for _, dI, dA in R[0]] == [(1, 1), (1, 1), (0, 1)]      # .4 wrong, .3 wrong, .2 right
    assert [(dI, dA) for _, dI, dA in R[1]] == [(0, 1), (0, 1), (0, 1)]
    assert tmax == [np.float32(.4), np.float32(.8)]
    tau, assigned, taken = per_class_thresholds(U, pred, correct, 2, 4, 1, 4)    # assign 2 of 8
    assert taken == [0, 0] and assigned == 2
    assert tau[0] == np.float32(.2) and tau[1] == np.float32(.8)                # class 1 untouched: nothing above its maximum
    tau, assigned, taken = per_class_thresholds(U, pred, correct, 2, 4, 1, 2)    # 4 of 8: slopes 1,1 then ties 0 -> lower class
    assert taken == [0, 0, 0, 1] and assigned == 4


def test_assigned_count_equals_a_direct_count_and_absent_class_keeps_global_max():
    rng = np.random.default_rng(2)
    n, C = 5000, 6
    U = rng.random(n).astype(np.float32)
    pred = rng.integers(0, C - 1, n)             # class C-1 never predicted
    correct = rng.random(n) > U * 0.8            # uncertain flows are wrong more often
    for a in (5, 24, 60, 100):
        tau, assigned, _ = per_class_thresholds(U, pred, correct, C, 50, a, 100)
        assert assigned == int(np.count_nonzero(U > tau[pred]))
        assert tau[C - 1] == U.max()
        if a < 100:
            assert assigned >= a * n // 100 and assigned - a * n // 100 <= n // 50 // (C - 1) + 50   # overshoot < one step
    tau, assigned, _ = per_class_thresholds(U, pred, correct, C, 50, 0, 100)
    assert assigned == 0 and all(tau[L] == U[pred == L].max() for L in range(C - 1))


def test_greedy_is_optimal_when_slopes_fall_brute_force():
    # With per-class slopes that do not rise, taking the steepest step first captures the most
    # wrong predictions for the number assigned; compare with every combination of per-class steps.
    rng = np.random.default_rng(3)
    checked = 0
    for trial in range(20):
        C, Q, per = 3, 4, 8
        U, pred, correct = [], [], []
        for L in range(C):
            u = np.sort(rng.random(per).astype(np.float32))
            wrong_p = np.linspace(0.05, 0.95, per) ** rng.uniform(0.5, 2)
            # make the number of wrong flows per quantile step non-increasing from the top down
            steps = np.array_split(np.arange(per)[::-1], Q)
            w = np.sort(rng.integers(0, 3, Q))[::-1]
            ok = np.ones(per, bool)
            for s, k in zip(steps, w):
                ok[s[:min(k, len(s))]] = False
            U += list(u); pred += [L] * per; correct += list(ok)
        U = np.array(U, np.float32); pred = np.array(pred); correct = np.array(correct)
        R, _ = per_class_slopes(U, pred, correct, C, Q)
        if any(R[L][j][1] * R[L][j + 1][2] < R[L][j + 1][1] * R[L][j][2] for L in range(C) for j in range(len(R[L]) - 1)):
            continue                                   # a rising slope: the premise does not hold for this draw
        checked += 1
        for a in (10, 30, 50):
            tau, assigned, taken = per_class_thresholds(U, pred, correct, C, Q, a, 100)
            got_wrong = int(np.count_nonzero((U > tau[pred]) & ~correct))
            best = 0
            for combo in itertools.product(*[range(len(R[L]) + 1) for L in range(C)]):
                A = sum(sum(x[2] for x in R[L][:combo[L]]) for L in range(C))
                I = sum(sum(x[1] for x in R[L][:combo[L]]) for L in range(C))
                if A <= assigned:
                    best = max(best, I)
            assert got_wrong == best
    assert checked >= 5
