"""evo_summary on the GPU against the oracle: every field bit-exact."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def evo():
    import paper_2510_03760_b200 as evo
    return evo


def _fits(valid, speedup):
    f = np.zeros(len(valid), oracle.FIT_DTYPE)
    f["valid"], f["speedup"] = valid, speedup
    f["median_ms"] = 1.0
    return f


def _check(evo, fits, kernel_of, n_kernel, run_of=None, n_run=1):
    d_fits = torch.from_numpy(fits.view(np.uint8).reshape(-1, 16).copy()).cuda() if len(fits) else \
        torch.empty((0, 16), dtype=torch.uint8, device="cuda")
    d_k = torch.from_numpy(np.asarray(kernel_of, dtype=np.int32)).cuda()
    d_r = torch.from_numpy(np.asarray(run_of, dtype=np.int32)).cuda() if run_of is not None else None
    s, best, med = evo.evo_summary(d_fits, d_k, n_kernel, run_of=d_r, n_run=n_run)
    got = evo.summary_to_numpy(s)
    want, want_best, want_med = oracle.summary(fits, kernel_of, n_kernel, run_of=run_of, n_run=n_run)
    assert got.tobytes() == want.tobytes(), (got, want)
    assert best.cpu().numpy().tobytes() == want_best.tobytes()
    assert med.cpu().numpy().tobytes() == want_med.tobytes()
    return got


@pytest.mark.parametrize("n_kernel,n_run,per", [(1, 1, 3), (2, 1, 1), (6, 1, 45), (91, 3, 45), (10, 2, 1), (1500, 2, 3),
                                                 (8192, 1, 1)])
def test_random_populations(evo, n_kernel, n_run, per):
    rng = np.random.default_rng(n_kernel + 7 * n_run)
    n = n_kernel * n_run * per
    kernel_of = rng.integers(0, n_kernel, n)
    run_of = rng.integers(0, n_run, n)
    valid = (rng.random(n) < 0.6).astype(np.uint32)
    speed = np.where(valid == 1, 10.0 ** rng.uniform(-0.7, 1.3, n), 0.0).astype(np.float32)
    speed[rng.integers(0, n, n // 5)] = 1.0         # ties and exact boundaries
    speed[rng.integers(0, n, n // 7)] = 2.0
    got = _check(evo, _fits(valid, speed), kernel_of, n_kernel, run_of, n_run)
    assert got["n_cand"] == n


def test_from_the_fitness_records_of_a_population(evo):
    # the records evo_fitness wrote are used as they are, on the device
    rng = np.random.default_rng(5)
    n, trials, n_kernel = 450, 20, 10
    times = (10.0 ** rng.uniform(-1, 1, (n, 1)) * (1 + rng.random((n, trials)))).astype(np.float32)
    base = (1 + rng.random(trials)).astype(np.float32)
    passed = (rng.random(n) < 0.7).astype(np.int32)
    kernel_of = (np.arange(n) // 45).astype(np.int32)
    fits = evo.evo_fitness(torch.from_numpy(times).cuda(), torch.from_numpy(base).cuda(), torch.from_numpy(passed).cuda())
    s, best, med = evo.evo_summary(fits, torch.from_numpy(kernel_of).cuda(), n_kernel)
    want, want_best, want_med = oracle.summary(oracle.fitness(times, base, passed), kernel_of, n_kernel)
    assert evo.summary_to_numpy(s).tobytes() == want.tobytes()
    assert best.cpu().numpy().tobytes() == want_best.tobytes() and med.cpu().numpy().tobytes() == want_med.tobytes()


def test_edge_cases(evo):
    _check(evo, _fits([0, 0, 0], [5, 6, 7]), [0, 1, 2], 3)                      # nobody valid: all 1.0
    _check(evo, _fits([1] * 6, [1.0, 2.0, 5.0, 10.0, np.nextafter(np.float32(1), np.float32(0)), 0.25]),
           [0, 1, 2, 3, 4, 4], 5)                                              # range boundaries
    _check(evo, _fits([1], [8.0]), [0], 3)                                     # kernels nobody tried
    _check(evo, _fits([], []), [], 4, n_run=2)                                 # no candidates at all
    _check(evo, _fits([1, 1], [np.inf, 3.0]), [0, 0], 1)                       # an infinite speedup is the largest


def test_ids_out_of_range_are_reported_and_skipped(evo):
    ctx = evo.Context(0)
    fits = torch.from_numpy(_fits([1, 1], [2.0, 3.0]).view(np.uint8).reshape(-1, 16).copy()).cuda()
    s, best, _ = evo.evo_summary(fits, torch.tensor([0, 9], dtype=torch.int32, device="cuda"), 2, ctx=ctx)
    with pytest.raises(evo.EvoError) as e:
        ctx.synchronize()
    assert e.value.status == -1
    assert best.cpu().numpy().tolist() == [[2.0, 0.0]]
    ctx.synchronize()
    L = evo.load_library()
    assert L.evo_summary(ctx._h, fits.data_ptr(), fits.data_ptr(), None, 2, 0, 1, fits.data_ptr(), fits.data_ptr(), None, None) == -1
    assert L.evo_summary(ctx._h, fits.data_ptr(), fits.data_ptr(), None, 2, 9000, 1, fits.data_ptr(), fits.data_ptr(), None, None) == -1


@pytest.mark.parametrize("n", [0, 1, 2, 255, 256, 257, 4095, 20000])
def test_elite_selection(evo, n):
    rng = np.random.default_rng(n)
    valid = (rng.random(n) < 0.6).astype(np.uint32)
    speed = np.where(valid == 1, np.round(10.0 ** rng.uniform(-0.7, 1.3, n), 1), 7.0).astype(np.float32)   # many ties
    fits = _fits(valid, speed)
    d_fits = torch.from_numpy(fits.view(np.uint8).reshape(-1, 16).copy()).cuda() if n else \
        torch.empty((0, 16), dtype=torch.uint8, device="cuda")
    for k in (1, 4, 45, n + 3):
        idx, count = evo.evo_select_elite(d_fits, k)
        want_idx, want_count = oracle.select_elite(fits, k)
        assert count.cpu().item() == want_count
        assert np.array_equal(idx.cpu().numpy().view(np.uint32), want_idx)
