"""Pins for the oracle's median-of-trials speedup (CPU only)."""
import os
import statistics

import numpy as np

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "median_cases.txt")


def test_hand_worked_medians():
    n = 0
    for line in open(GOLDEN):
        if not line.strip() or line.startswith("#"):
            continue
        lhs, rhs = line.split("|")
        cand, base = [[float(x) for x in part.split()] for part in lhs.split(";")]
        median, speedup = [float(x) for x in rhs.split()]
        fit = oracle.fitness(np.array([cand], np.float32), np.array(base, np.float32))[0]
        assert fit["median_ms"] == np.float32(median) and fit["speedup"] == np.float32(speedup)
        assert fit["valid"] == 1 and fit["status"] == 0
        n += 1
    assert n == 6


def test_against_statistics_module_and_numpy():
    rng = np.random.default_rng(4)
    for trials in (1, 2, 5, 100, 101, 128, 129, 1000):
        t = (1 + rng.random((7, trials))).astype(np.float32)
        t[3] = t[3, 0]                       # all equal
        t[4, : trials // 2] = t[4, 0]        # ties
        base = (2 + rng.random(trials)).astype(np.float32)
        fit = oracle.fitness(t, base)
        bm = np.float32(statistics.median([np.float32(x) for x in base]))
        for i in range(7):
            m = statistics.median([np.float32(x) for x in t[i]])     # binary32 arithmetic on the two middles
            assert fit["median_ms"][i] == np.float32(m)
            assert fit["median_ms"][i] == np.median(t[i]).astype(np.float32) or trials % 2 == 0
            assert fit["speedup"][i] == bm / np.float32(m)
        # permutation invariance
        p = rng.permutation(trials)
        assert np.array_equal(oracle.fitness(t[:, p], base[rng.permutation(trials)]), fit)


def test_same_times_give_speedup_one():
    t = np.array([[3.0, 1.5, 2.25, 9.0]], np.float32)
    assert oracle.fitness(t, t[0])[0]["speedup"] == 1.0


def test_failed_and_invalid_rows():
    t = np.array([[1, 2, 3], [1, np.nan, 3], [1, -2, 3], [0, 2, 3], [np.inf, 2, 3], [4, 5, 6]], np.float32)
    fit = oracle.fitness(t, np.array([2, 2, 2], np.float32), passed=[1, 1, 1, 1, 1, 0])
    assert fit["valid"].tolist() == [1, 0, 0, 0, 0, 0]
    assert fit["status"].tolist() == [0, 1, 1, 1, 1, 0]
    assert fit["speedup"].tolist() == [1.0, 0, 0, 0, 0, 0]
    assert fit["median_ms"][5] == 5.0       # the median of a failed candidate is still reported
    bad_base = oracle.fitness(t[:1], np.array([1, 0, 2], np.float32))
    assert bad_base["status"][0] == 2 and bad_base["valid"][0] == 0
