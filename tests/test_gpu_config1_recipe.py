"""The smallest synthetic configuration built exactly from the seeded stream: reference = standard normals of Philox
seed 0, candidate = reference + 1e-4 * normals of seed 1, seven elements (the first seven distinct words of seed 2
mod 4096) off by 1.0, atol = rtol = 1e-2, five run times 1 + (word >> 8) / 2^24 ms from seeds 3 (candidate) and 4
(baseline).  The stream comes from the oracle's generator on the host, so the oracle and the GPU judge the same
bytes; what must come out is known by construction: exactly seven mismatches, largest difference about 1."""
import numpy as np
import pytest
import torch

import oracle
from parity import assert_results_equal, ordered

pytestmark = pytest.mark.gpu


def _config1_from_the_stream():
    n = 64 * 64
    ref = oracle.gen_inputs(0, 0, oracle.F32, n)
    cand = (ref + np.float32(1e-4) * oracle.gen_inputs(1, 0, oracle.F32, n)).astype(np.float32)
    pos = []
    for w in oracle.gen_u32(2, 0, 64):
        p = int(w) % n
        if p not in pos:
            pos.append(p)
        if len(pos) == 7:
            break
    cand[pos] = ref[pos] + np.float32(1.0)
    times = (1.0 + (oracle.gen_u32(3, 0, 5) >> 8).astype(np.float64) * 2.0 ** -24).astype(np.float32).reshape(1, 5)
    base = (1.0 + (oracle.gen_u32(4, 0, 5) >> 8).astype(np.float64) * 2.0 ** -24).astype(np.float32)
    return ref, cand, pos, times, base


def test_config1_from_the_philox_stream():
    import paper_2510_03760_b200 as evo
    ref, cand, pos, times, base = _config1_from_the_stream()
    # the library's own generator yields the same reference (to 4 ulp) from the same seed
    dev_ref = torch.empty(ref.size, dtype=torch.float32, device="cuda")
    evo.evo_gen_inputs(0, 0, evo.EVO_F32, ref.size, dev_ref)
    assert np.abs(ordered(dev_ref.cpu().numpy()) - ordered(ref)).max() <= 4
    # the check, on the oracle's bytes
    res, gp = evo.evo_validate([torch.from_numpy(cand).cuda()], [torch.from_numpy(ref).cuda()], 1e-2, 1e-2, groups=[0], n_group=1)
    got = evo.results_to_numpy(res)
    want = oracle.validate(cand, ref, oracle.F32, 1e-2, 1e-2)
    assert_results_equal(got, np.array([want]))
    assert got["n_mismatch"][0] == 7 and got["pass"][0] == 0 and gp.cpu().item() == 0
    assert abs(got["max_abs"][0] - 1.0) < 1e-3 and got["n_nonfinite"][0] == 0
    # the objective: the candidate is invalid, so no speedup; with a passing verdict the medians' quotient
    fit = evo.fits_to_numpy(evo.evo_fitness(torch.from_numpy(times).cuda(), torch.from_numpy(base).cuda(), gp))
    assert fit.tobytes() == oracle.fitness(times, base, np.array([0], np.uint32)).tobytes() and fit["valid"][0] == 0
    fit = evo.fits_to_numpy(evo.evo_fitness(torch.from_numpy(times).cuda(), torch.from_numpy(base).cuda()))
    want_fit = oracle.fitness(times, base)
    assert fit.tobytes() == want_fit.tobytes() and 0.5 < fit["speedup"][0] < 2.0 and 1.0 <= fit["median_ms"][0] < 2.0
