"""The device-side waits of the checking kernel are bounded.  A wait that can never complete
(a barrier that nothing arrives on) must run out, raise the context's status word and return:
no trap, no hang, and the context keeps working afterwards."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from parity import assert_results_equal

pytestmark = pytest.mark.gpu


def test_a_wait_that_nothing_completes_runs_out_and_is_reported_once():
    import paper_2510_03760_b200 as evo
    ctx = evo.Context(0)
    ctx.synchronize()                              # nothing pending: no error
    ctx.selftest_wait(limit_us=2000)
    with pytest.raises(evo.EvoError) as e:
        ctx.synchronize()
    assert e.value.status == -6                    # EVO_ERR_TIMEOUT
    ctx.synchronize()                              # reported once, then cleared

    # the context is still usable and right
    g = torch.Generator().manual_seed(3)
    r = torch.randn(3 * 4096 + 11, generator=g)
    c = r + 0.004 * torch.randn(r.numel(), generator=g)
    res, _ = evo.evo_validate([c.cuda()], [r.cuda()], 0.005, 0.005, ctx=ctx)
    want = oracle.validate(workloads.to_host_bits(c), workloads.to_host_bits(r), workloads.F32, 0.005, 0.005)
    assert_results_equal(evo.results_to_numpy(res), np.array([want]))
    ctx.synchronize()


def test_results_of_a_run_that_gave_up_are_marked_incomplete():
    import paper_2510_03760_b200 as evo
    ctx = evo.Context(0)
    g = torch.Generator().manual_seed(4)
    r = torch.randn(4096, generator=g).cuda()
    # raise the status word first (the self-test's wait runs out), then validate on the same
    # context without clearing it: the second pass must refuse to report numbers
    ctx.selftest_wait(limit_us=1000)
    res, gp = evo.evo_validate([r.clone()], [r], 0.0, 0.0, groups=[0], n_group=1, ctx=ctx)
    got = evo.results_to_numpy(res)
    assert got["pass"][0] == 0 and got["flags"][0] == evo.EVO_FLAG_INCOMPLETE and gp.cpu().item() == 0
    with pytest.raises(evo.EvoError):
        ctx.synchronize()
    res, gp = evo.evo_validate([r.clone()], [r], 0.0, 0.0, groups=[0], n_group=1, ctx=ctx)
    assert evo.results_to_numpy(res)["pass"][0] == 1 and gp.cpu().item() == 1
