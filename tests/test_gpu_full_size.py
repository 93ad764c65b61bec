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


def test_config3_full_size():
    """128 candidates x 2^20 fp16/bf16 elements with NaN/Inf and boundary values: every tensor by the oracle."""
    import paper_2510_03760_b200 as evo
    pop = workloads.config3("cuda")
    cands = [t.cand for t in pop.tensors]
    refs = [pop.refs[t.ref_index] for t in pop.tensors]
    groups = [t.group for t in pop.tensors]
    res, gp = evo.evo_validate(cands, refs, pop.atol, pop.rtol, groups=groups, n_group=pop.n_group)
    got = evo.results_to_numpy(res)
    host_refs = [workloads.to_host_bits(r) for r in pop.refs]
    want = np.zeros(len(cands), dtype=oracle.RESULT_DTYPE)
    for i, t in enumerate(pop.tensors):
        want[i] = oracle.validate(workloads.to_host_bits(t.cand), host_refs[t.ref_index], t.dtype, pop.atol, pop.rtol)
    assert_results_equal(got, want, "config3 full size")
    assert want["n_nonfinite"].sum() > 50 and (want["flags"] != 0).sum() > 30        # the specials are really there
    assert np.array_equal(gp.cpu().numpy().view(np.uint32), oracle.group_pass(want, groups, pop.n_group))


def test_config5_full_size_sampled():
    """The ragged population at full size (1024 candidates, about 2000 tensors, 22 GB): a seeded sample of tensors
    by the oracle element by element, and for all of them what holds by construction."""
    import paper_2510_03760_b200 as evo
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * (1 << 30):
        pytest.skip("needs 60 GiB of device memory")
    pop = workloads.config5("cuda")
    cands = [t.cand for t in pop.tensors]
    refs = [pop.refs[t.ref_index] for t in pop.tensors]
    groups = [t.group for t in pop.tensors]
    res, gp = evo.evo_validate(cands, refs, pop.atol, pop.rtol, groups=groups, n_group=pop.n_group)
    got = evo.results_to_numpy(res)
    gp = gp.cpu().numpy()
    # by construction: candidates without injected elements pass; no NaN/Inf anywhere; errors below the tolerance scale
    rates = pop.facts["rates"]
    for i, t in enumerate(pop.tensors):
        if rates[t.group] == 0.0:
            assert got["pass"][i] == 1 and got["n_mismatch"][i] == 0, i
        assert got["n_nonfinite"][i] == 0 and got["flags"][i] == 0
        assert got["n_mismatch"][i] <= t.cand.numel()
    for g in range(pop.n_group):
        mine = [i for i, t in enumerate(pop.tensors) if t.group == g]
        assert gp[g] == int(all(got["pass"][i] for i in mine))
    # a seeded sample, biased to cover the largest and the smallest tensors and every dtype
    rng = np.random.default_rng(55)
    order = np.argsort([t.cand.numel() for t in pop.tensors])
    sample = set(order[:8].tolist()) | set(order[-6:].tolist()) | set(rng.choice(len(cands), 40, replace=False).tolist())
    for i in sorted(sample):
        t = pop.tensors[i]
        want = oracle.validate(workloads.to_host_bits(t.cand), workloads.to_host_bits(pop.refs[t.ref_index]), t.dtype,
                               pop.atol, pop.rtol)
        assert_results_equal(got[i:i + 1], np.array([want]), "config5 tensor %d (n=%d, dtype=%d)" % (i, t.cand.numel(), t.dtype))


def test_tensor_beyond_2_to_32_elements():
    """One bf16 tensor of 2^32 + 12293 elements (8 GiB each for candidate and reference): indices and counts past
    32 bits.  The candidate equals the reference except at planted positions around 2^31, 2^32 and the very end, so
    every statistic is known by construction; windows around the planted positions also go through the oracle."""
    import paper_2510_03760_b200 as evo
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * (1 << 30):
        pytest.skip("needs 40 GiB of device memory")
    n = (1 << 32) + 3 * 4096 + 5
    g = torch.Generator(device="cuda").manual_seed(99)
    ref = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    step = 1 << 28
    for lo in range(0, n, step):                                   # in slices: the generator's fp32 temporaries stay small
        hi = min(n, lo + step)
        ref[lo:hi] = torch.randn(hi - lo, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    cand = ref.clone()
    planted = [0, 4095, (1 << 31) - 1, 1 << 31, (1 << 32) - 1, 1 << 32, (1 << 32) + 4096, n - 6, n - 1]
    for p in planted:
        cand[p] = ref[p].float() + 1.0
    nan_at = (1 << 32) + 7
    cand[nan_at] = float("nan")
    atol = rtol = 0.01
    res, _ = evo.evo_validate([cand], [ref], atol, rtol)
    got = evo.results_to_numpy(res)[0]
    d = np.array([abs(np.float32(cand[p].float().item()) - np.float32(ref[p].float().item())) for p in planted], np.float32)
    rr = np.array([abs(np.float32(ref[p].float().item())) for p in planted], np.float32)
    assert (d > np.float32(atol) + np.float32(rtol) * rr).all()
    assert got["n_mismatch"] == len(planted) + 1 and got["n_nonfinite"] == 1 and got["flags"] == 1 and got["pass"] == 0
    assert got["max_abs"] == d.max() and got["max_rel"] == (d / rr).max()
    want_sse = float(np.sum(d.astype(np.float64) ** 2))
    assert abs(got["sse"] - want_sse) <= 1e-5 * want_sse
    # the offenders, with 64-bit indices
    recs, found = evo.evo_mismatch_sample(cand, ref, atol, rtol, 64)
    assert found == len(planted) + 1
    assert recs["index"].tolist() == sorted(planted + [nan_at])
    # windows around the planted positions through the oracle
    for p in (1 << 31, 1 << 32, n - 1):
        lo, hi = max(0, p - 5000), min(n, p + 5000)
        w_res, _ = evo.evo_validate([cand[lo:hi]], [ref[lo:hi]], atol, rtol)
        want = oracle.validate(workloads.to_host_bits(cand[lo:hi]), workloads.to_host_bits(ref[lo:hi]), oracle.BF16, atol, rtol)
        assert_results_equal(evo.results_to_numpy(w_res), np.array([want]), "window at %d" % p)
