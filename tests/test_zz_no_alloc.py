"""evo_validate_static: the allocation-free variant of evo_validate, for callers that cannot
call cudaMalloc (their allocator owns the device, or they run under a no-allocation rule).
Its scratch is a fixed array inside the library that every call shares and that keeps the last
call's contents, so the check runs different populations back to back through the C ABI and
compares each with what evo_validate returns for the same tensors (same kernels: equal byte for
byte) and with the CPU oracle (the bars of every other parity test).  This file sorts last on
purpose: a run that stops at the first failure has then already run every other test."""
import numpy as np
import pytest
import torch

import workloads
from parity import assert_results_equal, oracle_population

pytestmark = pytest.mark.gpu


def _device_population(pop):
    dev_refs = [r.cuda() for r in pop.refs]
    cands = [t.cand.cuda() for t in pop.tensors]
    refs = [dev_refs[t.ref_index] for t in pop.tensors]
    groups = [t.group for t in pop.tensors]
    return cands, refs, groups


def _both_ways(evo, pop):
    cands, refs, groups = _device_population(pop)
    want_res, want_gp = evo.evo_validate(cands, refs, pop.atol, pop.rtol, groups=groups, n_group=pop.n_group)
    want_res, want_gp = evo.results_to_numpy(want_res), want_gp.cpu().numpy()
    # outputs are allocated by the caller, before the call; poison them so stale data would show
    res = torch.full((len(cands), 40), 0xAB, dtype=torch.uint8, device="cuda")
    gp = torch.full((pop.n_group,), -7, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    # free device memory as the driver counts it: a cudaMalloc inside the library would lower it,
    # whichever allocator the rest of the process uses
    free_before = torch.cuda.mem_get_info()[0]
    torch_before = torch.cuda.memory_allocated()
    evo.evo_validate_static(cands, refs, pop.atol, pop.rtol, res, groups=groups, n_group=pop.n_group, group_pass=gp)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free_before, "device memory was allocated during the call"
    assert torch.cuda.memory_allocated() == torch_before
    got = evo.results_to_numpy(res)
    assert got.tobytes() == want_res.tobytes(), pop.name + ": differs from evo_validate"
    assert np.array_equal(gp.cpu().numpy(), want_gp)
    oracle_res, oracle_gp = oracle_population(pop)
    assert_results_equal(got, oracle_res, pop.name + " (static scratch, against the oracle)")
    assert np.array_equal(gp.cpu().numpy().view(np.uint32), oracle_gp)


def test_static_scratch_matches_evo_validate_and_the_oracle_on_calls_in_a_row():
    import paper_2510_03760_b200 as evo
    # first call: ragged, mixed dtypes, many sets, and a schedule longer than one 16 KiB piece; second call:
    # fewer, larger tensors sharing one reference, so the scratch still holds the first call's longer schedule
    # when it starts; third: a single small tensor
    _both_ways(evo, workloads.config5("cpu", n_cand=120, log2_min=2.0, log2_max=16.0, trials=4))
    _both_ways(evo, workloads.config2("cpu", n=(1 << 17) + 33, k=6, trials=4))
    _both_ways(evo, workloads.config1("cpu"))


def test_population_beyond_the_fixed_scratch_is_refused():
    import paper_2510_03760_b200 as evo
    n_desc = 30000
    ref = torch.zeros(8, device="cuda")
    cands = [ref] * n_desc
    res = torch.zeros((n_desc, 40), dtype=torch.uint8, device="cuda")
    with pytest.raises(evo.EvoError) as e:
        evo.evo_validate_static(cands, ref, 0.1, 0.1, res)
    assert e.value.status == -5 and "scratch" in str(e.value)
    # and the entry point still works afterwards
    _both_ways(evo, workloads.config1("cpu"))
