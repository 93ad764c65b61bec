"""Pins for the oracle's other run-time statistics (mean, min, trimmed mean, warm-up) and for the
population summary (CPU only)."""
import os
import statistics
from fractions import Fraction

import numpy as np
import pytest
import scipy.stats

import oracle

HERE = os.path.dirname(__file__)


def _f32(fr):
    """Nearest binary32 to an exact rational."""
    return np.float32(float(fr))


def test_hand_worked_statistics():
    n = 0
    for line in open(os.path.join(HERE, "golden", "statistic_cases.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        lhs, rhs = line.split("|")
        head, cand, base = [part.split() for part in lhs.split(";")]
        stat, warmup, trim = [int(x) for x in head]
        want, speedup = [float(x) for x in rhs.split()]
        fit = oracle.fitness_ex(np.array([cand], np.float32), np.array(base, np.float32), stat=stat, warmup=warmup, trim=trim)[0]
        assert fit["median_ms"] == np.float32(want) and fit["speedup"] == np.float32(speedup), line
        assert fit["valid"] == 1 and fit["status"] == 0
        n += 1
    assert n == 7


def test_mean_min_trimmed_against_exact_rationals_numpy_and_scipy():
    rng = np.random.default_rng(8)
    for trials in (1, 2, 3, 10, 100, 101, 1000):
        t = (10.0 ** rng.uniform(-2, 2, (6, trials))).astype(np.float32)
        base = (1 + rng.random(trials)).astype(np.float32)
        for warmup in (0, min(3, trials - 1)):
            kept, bkept = t[:, warmup:], base[warmup:]
            m = kept.shape[1]
            mean = oracle.fitness_ex(t, base, stat=oracle.STAT_MEAN, warmup=warmup)
            low = oracle.fitness_ex(t, base, stat=oracle.STAT_MIN, warmup=warmup)
            med = oracle.fitness_ex(t, base, stat=oracle.STAT_MEDIAN, warmup=warmup)
            assert np.array_equal(med, oracle.fitness(kept, bkept))
            b_mean = _f32(sum(Fraction(float(x)) for x in bkept) / m)
            for i in range(6):
                exact = sum(Fraction(float(x)) for x in kept[i]) / m
                assert mean["median_ms"][i] == _f32(exact)
                assert mean["speedup"][i] == b_mean / mean["median_ms"][i]
                assert low["median_ms"][i] == kept[i].min()
                assert low["speedup"][i] == bkept.min() / kept[i].min()
            for trim in (0, 1, m // 10, (m - 1) // 2):
                if 2 * trim >= m:
                    continue
                tm = oracle.fitness_ex(t, base, stat=oracle.STAT_TRIMMED_MEAN, warmup=warmup, trim=trim)
                for i in range(6):
                    srt = sorted(Fraction(float(x)) for x in kept[i])
                    exact = sum(srt[trim:m - trim]) / (m - 2 * trim)
                    assert tm["median_ms"][i] == _f32(exact)
                    if trim:
                        sp = scipy.stats.trim_mean(kept[i].astype(np.float64), trim / m + 1e-12)
                        assert abs(float(tm["median_ms"][i]) - sp) <= 1e-6 * sp
                if trim == 0:
                    assert np.array_equal(tm, mean)


def test_statistics_reject_bad_rows_and_arguments():
    t = np.array([[1, 2, 3, 4], [1, np.nan, 3, 4], [np.nan, 2, 3, 4]], np.float32)
    base = np.array([2, 2, 2, 2], np.float32)
    fit = oracle.fitness_ex(t, base, stat=oracle.STAT_MEAN, warmup=1, passed=[1, 1, 0])
    assert fit["status"].tolist() == [0, 1, 0] and fit["valid"].tolist() == [1, 0, 0]   # a bad warm-up run is ignored
    assert fit["median_ms"][2] == 3.0 and fit["speedup"][2] == 0.0
    for kw in (dict(stat=7), dict(stat=1, warmup=4), dict(stat=3, trim=2), dict(stat=3, warmup=2, trim=1)):
        with pytest.raises(ValueError):
            oracle.fitness_ex(t, base, **kw)


def _fits(valid, speedup):
    f = np.zeros(len(valid), oracle.FIT_DTYPE)
    f["valid"], f["speedup"] = valid, speedup
    f["median_ms"] = 1.0
    return f


def test_hand_worked_summary():
    runs, kernels, valid, speed, want = [], [], [], [], {}
    for line in open(os.path.join(HERE, "golden", "summary_case.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        w = line.split()
        if w[0][0].isdigit():
            runs.append(int(w[0])); kernels.append(int(w[1])); valid.append(int(w[2])); speed.append(float(w[3]))
        else:
            want[w[0]] = [float(x) for x in w[1:]]
    s, best, med = oracle.summary(_fits(valid, speed), kernels, 4, run_of=runs, n_run=2)
    assert best[0].tolist() == want["best0"] and best[1].tolist() == want["best1"]
    assert med.tolist() == want["run_median"] and s["median_speedup"] == want["median_speedup"][0]
    assert s["n_valid"] == want["n_valid"][0] and s["n_cand"] == 11 and s["validity"] == np.float32(9 / 11)
    assert s["speedup_count"] == want["speedup_count"][0] and s["hist"].tolist() == want["hist"]
    assert s["n_kernel"] == 4 and s["n_run"] == 2


def test_summary_against_python_statistics_and_numpy_histogram():
    rng = np.random.default_rng(21)
    for n_kernel, n_run, per in [(1, 1, 3), (6, 1, 45), (91, 3, 45), (10, 2, 1)]:
        n = n_kernel * n_run * per
        kernel_of = rng.integers(0, n_kernel, n)
        run_of = rng.integers(0, n_run, n)
        valid = (rng.random(n) < 0.6).astype(np.uint32)
        speed = np.where(valid == 1, 10.0 ** rng.uniform(-0.7, 1.3, n), 0.0).astype(np.float32)
        s, best, med = oracle.summary(_fits(valid, speed), kernel_of, n_kernel, run_of=run_of, n_run=n_run)
        want_best = np.zeros((n_run, n_kernel), np.float32)
        for i in range(n):
            if valid[i]:
                want_best[run_of[i], kernel_of[i]] = max(want_best[run_of[i], kernel_of[i]], speed[i])
        assert np.array_equal(best, want_best)
        want_med = [np.float32(statistics.median([np.float32(max(x, 1.0)) for x in row])) for row in want_best]
        assert med.tolist() == want_med
        assert s["median_speedup"] == _f32(sum(Fraction(float(x)) for x in want_med) / n_run)
        top = want_best.max(axis=0)
        assert s["hist"].tolist() == np.histogram(top, bins=[-np.inf, 1, 2, 5, 10, np.inf])[0].tolist()
        assert s["speedup_count"] == int((top > 1).sum()) and s["n_valid"] == int(valid.sum())
        assert s["validity"] == _f32(Fraction(int(valid.sum()), n))
        # the order of the candidates does not matter
        p = rng.permutation(n)
        s2, best2, med2 = oracle.summary(_fits(valid[p], speed[p]), kernel_of[p], n_kernel, run_of=run_of[p], n_run=n_run)
        assert s2 == s and np.array_equal(best2, best) and np.array_equal(med2, med)


def test_summary_floor_boundaries_and_errors():
    # no valid candidate at all: every kernel reports 1.0
    s, best, med = oracle.summary(_fits([0, 0, 0], [5, 6, 7]), [0, 1, 2], 3)
    assert s["median_speedup"] == 1.0 and s["hist"].tolist() == [3, 0, 0, 0, 0] and s["speedup_count"] == 0
    assert s["validity"] == 0.0 and not best.any()
    # range boundaries belong to the range above; exactly 1.0 is not a speed-up
    s, _, _ = oracle.summary(_fits([1] * 6, [1.0, 2.0, 5.0, 10.0, np.nextafter(np.float32(1), np.float32(0)), 0.25]),
                             [0, 1, 2, 3, 4, 4], 5)
    assert s["hist"].tolist() == [1, 1, 1, 1, 1] and s["speedup_count"] == 3
    # a kernel nobody tried counts as 1.0 too
    s, _, med = oracle.summary(_fits([1], [8.0]), [0], 3)
    assert med.tolist() == [1.0] and s["hist"].tolist() == [2, 0, 0, 1, 0]
    with pytest.raises(ValueError):
        oracle.summary(_fits([1], [1.0]), [3], 3)
    with pytest.raises(ValueError):
        oracle.summary(_fits([1], [1.0]), [0], 3, run_of=[1], n_run=1)


def test_elite_selection_against_lexsort_argmax_and_brute_force():
    rng = np.random.default_rng(33)
    for n in (0, 1, 2, 17, 450, 4095):
        valid = (rng.random(n) < 0.6).astype(np.uint32)
        speed = np.where(valid == 1, np.round(10.0 ** rng.uniform(-0.7, 1.3, n), 1), 7.0).astype(np.float32)   # many ties
        fits = _fits(valid, speed)
        vi = np.nonzero(valid)[0]
        order = vi[np.lexsort((vi, -speed[vi].astype(np.float64)))]        # speedup descending, then index ascending
        for k in (1, 4, 10, n + 3):
            idx, count = oracle.select_elite(fits, k)
            m = min(k, len(vi))
            assert count == m and idx[:m].tolist() == order[:m].tolist() and (idx[m:] == 0xFFFFFFFF).all()
        if len(vi):
            idx, _ = oracle.select_elite(fits, 1)                           # the single-solution strategy: the best one
            assert speed[idx[0]] == speed[vi].max() and idx[0] == vi[np.argmax(speed[vi])]
        # brute force: entry j beats exactly j valid candidates' worth of (speedup, -index) pairs
        idx, count = oracle.select_elite(fits, n)
        for j in range(count):
            i = idx[j]
            ahead = sum(1 for q in vi if speed[q] > speed[i] or (speed[q] == speed[i] and q < i))
            assert ahead == j
    # invalid candidates never appear, whatever their speedup field holds
    idx, count = oracle.select_elite(_fits([0, 1, 0], [99.0, 0.5, 98.0]), 3)
    assert count == 1 and idx.tolist() == [1, 0xFFFFFFFF, 0xFFFFFFFF]
