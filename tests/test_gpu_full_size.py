"""Parity at the full size of the roofline workload (16 x 2^28 fp32 candidates against one
1 GiB reference), in the launch configuration the benchmark times.  Every candidate is
checked by the oracle (about a second each)."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from parity import assert_results_equal

pytestmark = pytest.mark.gpu


def test_config4_full_size():
    import paper_2510_03760_b200 as evo
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs 40 GiB of device memory")
    pop = workloads.config4("cuda")
    cands = [t.cand for t in pop.tensors]
    res, gp = evo.evo_validate(cands, pop.refs[0], pop.atol, pop.rtol, groups=list(range(16)), n_group=16)
    got = evo.results_to_numpy(res)
    ref_host = pop.refs[0].cpu().numpy()
    want = np.zeros(16, dtype=oracle.RESULT_DTYPE)
    for i, c in enumerate(cands):
        want[i] = oracle.validate(c.cpu().numpy(), ref_host, oracle.F32, pop.atol, pop.rtol)
    assert_results_equal(got, want, "config4 full size")
    wrong = pop.facts["wrong"]
    assert got["pass"].sum() == 15 and got["pass"][wrong] == 0 and got["n_mismatch"][wrong] > 0.99 * (1 << 28)
    assert gp.cpu().tolist() == got["pass"].tolist()
