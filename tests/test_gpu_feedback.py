"""evo_mismatch_sample on the GPU against the oracle: indices, values and the total, exactly."""
import numpy as np
import pytest
import torch

import oracle
import workloads

pytestmark = pytest.mark.gpu
TORCH = {workloads.F32: torch.float32, workloads.F16: torch.float16, workloads.BF16: torch.bfloat16}


@pytest.fixture(scope="module")
def evo():
    import paper_2510_03760_b200 as evo
    return evo


def _same(got, want):
    """Indices exact; values bit for bit, except that a NaN only has to be a NaN (the payload of
    a widened 16-bit NaN is not part of the contract)."""
    assert got["index"].tolist() == want["index"].tolist()
    for k in ("cand", "ref"):
        g, w = got[k], want[k]
        assert np.array_equal(np.isnan(g), np.isnan(w))
        keep = ~np.isnan(w)
        assert g[keep].tobytes() == w[keep].tobytes()


def _check(evo, c, r, dtype, atol, rtol, max_out):
    got, found = evo.evo_mismatch_sample(c.cuda(), r.cuda(), atol, rtol, max_out)
    want, want_found = oracle.mismatch_sample(workloads.to_host_bits(c), workloads.to_host_bits(r), dtype, atol, rtol, max_out)
    assert found == want_found
    _same(got, want)
    return found


@pytest.mark.parametrize("dtype", [workloads.F32, workloads.F16, workloads.BF16])
def test_samples_at_various_sizes_rates_and_limits(evo, dtype):
    g = torch.Generator().manual_seed(7 + dtype)
    for n in (1, 255, 2048, 2049, 5 * 2048 + 77, 300000):
        for rate in (0.0, 1e-3, 0.3, 1.0):
            r = torch.randn(n, generator=g).to(TORCH[dtype])
            c32 = r.float() + 1e-4 * torch.randn(n, generator=g)
            hit = torch.rand(n, generator=g) < rate
            c32 = torch.where(hit, r.float() + 1.0, c32)
            c = c32.to(TORCH[dtype])
            if n > 300 and rate > 0:
                c[5] = float("nan"); c[n - 1] = float("inf"); r[200] = float("nan")
            for max_out in (0, 1, 64, 5000):
                _check(evo, c, r, dtype, 0.01, 0.01, max_out)


def test_unaligned_views(evo):
    g = torch.Generator().manual_seed(2)
    store_r = torch.randn(10000, generator=g)
    store_c = store_r + torch.where(torch.rand(10000, generator=g) < 0.05, 1.0, 0.0)
    for off in (0, 1, 3):
        _check(evo, store_c[off:off + 9000].contiguous()[:], store_r[off:off + 9000].contiguous()[:], workloads.F32, 0.01, 0.01, 100)
        c, r = store_c.cuda()[off:off + 9000], store_r.cuda()[off:off + 9000]       # device views at odd offsets
        got, found = evo.evo_mismatch_sample(c, r, 0.01, 0.01, 100)
        want, want_found = oracle.mismatch_sample(store_c[off:off + 9000].numpy(), store_r[off:off + 9000].numpy(), oracle.F32,
                                                  0.01, 0.01, 100)
        assert found == want_found
        _same(got, want)


def test_agrees_with_evo_validate_on_a_failed_candidate(evo):
    pop = workloads.config4("cpu", n=1 << 22, k=4)
    wrong = pop.facts["wrong"]
    ref = pop.refs[0].cuda()
    res, _ = evo.evo_validate([t.cand.cuda() for t in pop.tensors], [ref] * 4, pop.atol, pop.rtol)
    res = evo.results_to_numpy(res)
    for i, t in enumerate(pop.tensors):
        got, found = evo.evo_mismatch_sample(t.cand.cuda(), ref, pop.atol, pop.rtol, 16)
        assert found == res["n_mismatch"][i]
        assert (found > 0) == (i == wrong)
    _check(evo, pop.tensors[wrong].cand, pop.refs[0], workloads.F32, pop.atol, pop.rtol, 1000)


def test_empty_tensor_and_bad_arguments(evo):
    e = torch.empty(0, device="cuda")
    got, found = evo.evo_mismatch_sample(e, e, 0.1, 0.1, 4)
    assert found == 0 and len(got) == 0
    x = torch.ones(8, device="cuda")
    with pytest.raises(evo.EvoError):
        evo.evo_mismatch_sample(x, x, -1.0, 0.0, 4)
    with pytest.raises(ValueError):
        evo.evo_mismatch_sample(x, x.half(), 0.1, 0.1, 4)
