"""evo_fitness on the GPU against the oracle: bit-exact."""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def evo():
    import paper_2510_03760_b200 as evo
    return evo


def _check(evo, times, base, passed=None):
    t = torch.from_numpy(np.ascontiguousarray(times, dtype=np.float32)).cuda()
    b = torch.from_numpy(np.ascontiguousarray(base, dtype=np.float32)).cuda()
    p = torch.from_numpy(np.asarray(passed, dtype=np.int32)).cuda() if passed is not None else None
    got = evo.fits_to_numpy(evo.evo_fitness(t, b, p))
    want = oracle.fitness(times, base, passed)
    assert got.tobytes() == want.tobytes()
    got_h = evo.evo_fitness_host(times, base, passed)
    assert got_h.tobytes() == want.tobytes()


@pytest.mark.parametrize("trials", [1, 2, 5, 31, 32, 33, 100, 128, 129, 1000, 4096])
def test_medians_and_speedups(evo, trials):
    rng = np.random.default_rng(trials)
    n = 37 if trials < 1000 else 5
    times = (1 + rng.random((n, trials))).astype(np.float32) * (10.0 ** rng.uniform(-2, 2, (n, 1))).astype(np.float32)
    times[1] = times[1, 0]
    times[2, : trials // 2] = times[2, 0]
    base = (1 + rng.random(max(1, trials // 2))).astype(np.float32)
    _check(evo, times, base)
    _check(evo, times, base, passed=rng.integers(0, 2, n))


def test_invalid_times(evo):
    t = np.array([[1, 2, 3], [1, np.nan, 3], [1, -2, 3], [0, 2, 3], [np.inf, 2, 3], [4, 5, 6]], np.float32)
    _check(evo, t, np.array([2, 2, 2], np.float32), passed=[1, 1, 1, 1, 1, 0])
    _check(evo, t, np.array([2, 0, 2], np.float32))


def test_population_times(evo):
    for pop in (workloads.config1("cpu"), workloads.config5("cpu", n_cand=64, log2_max=11)):
        _check(evo, pop.times.numpy(), pop.base_times.numpy())


def test_argument_errors(evo):
    L, ctx = evo.load_library(), evo.default_context(0)
    t = torch.ones(8, dtype=torch.float32, device="cuda")
    o = torch.zeros(64, dtype=torch.uint8, device="cuda")
    assert L.evo_fitness(ctx._h, t.data_ptr(), 2, 0, t.data_ptr(), 4, None, o.data_ptr(), None) == -1
    assert L.evo_fitness(ctx._h, t.data_ptr(), 2, 4, t.data_ptr(), 5000, None, o.data_ptr(), None) == -1
    assert L.evo_fitness(ctx._h, None, 2, 4, t.data_ptr(), 4, None, o.data_ptr(), None) == -1
    assert L.evo_fitness(ctx._h, t.data_ptr(), 0, 4, t.data_ptr(), 4, None, None, None) == 0


@pytest.mark.parametrize("stat", [0, 1, 2, 3])
@pytest.mark.parametrize("trials", [1, 2, 7, 100, 129, 1000, 4096])
def test_other_statistics_and_warmup(evo, stat, trials):
    rng = np.random.default_rng(100 * stat + trials)
    n = 19 if trials < 1000 else 4
    times = (10.0 ** rng.uniform(-2, 2, (n, trials))).astype(np.float32)
    times[1] = times[1, 0]
    times[2, : trials // 2] = times[2, 0]
    base_trials = max(1, trials // 2) if trials > 7 else trials
    base = (1 + rng.random(base_trials)).astype(np.float32)
    passed = rng.integers(0, 2, n)
    for warmup in sorted({0, min(3, base_trials - 1)}):
        kept = min(trials, base_trials) - warmup
        for trim in sorted({0, (kept - 1) // 2, kept // 10}) if stat == 3 else [0]:
            t = torch.from_numpy(times).cuda()
            b = torch.from_numpy(base).cuda()
            p = torch.from_numpy(passed.astype(np.int32)).cuda()
            got = evo.fits_to_numpy(evo.evo_fitness(t, b, p, stat=stat, warmup=warmup, trim=trim))
            want = oracle.fitness_ex(times, base, passed, stat=stat, warmup=warmup, trim=trim)
            assert got.tobytes() == want.tobytes(), (stat, trials, warmup, trim)


def test_statistics_with_bad_runs_and_bad_arguments(evo):
    t = np.array([[1, 2, 3, 4], [1, np.nan, 3, 4], [np.nan, 2, 3, 4]], np.float32)
    base = np.array([2, 2, 2, 2], np.float32)
    got = evo.fits_to_numpy(evo.evo_fitness(torch.from_numpy(t).cuda(), torch.from_numpy(base).cuda(), stat=1, warmup=1))
    assert got.tobytes() == oracle.fitness_ex(t, base, stat=1, warmup=1).tobytes()
    for kw in (dict(stat=7), dict(stat=1, warmup=4), dict(stat=3, trim=2), dict(stat=3, warmup=2, trim=1)):
        with pytest.raises(evo.EvoError):
            evo.evo_fitness(torch.from_numpy(t).cuda(), torch.from_numpy(base).cuda(), **kw)
