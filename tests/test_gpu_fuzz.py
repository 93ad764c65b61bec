"""Seeded random populations through evo_validate against the oracle: shared and own references, all three
types, sizes around tile and vector boundaries, odd alignments, zeros, NaN/Inf, values on the tolerance
boundary, huge and tiny magnitudes.  Every field under the usual bars."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from parity import assert_results_equal

pytestmark = pytest.mark.gpu
TORCH = {workloads.F32: torch.float32, workloads.F16: torch.float16, workloads.BF16: torch.bfloat16}
SIZES = [0, 1, 2, 3, 4, 5, 7, 8, 9, 15, 16, 17, 255, 256, 1023, 4095, 4096, 4097, 4100, 4104, 8191, 8192, 8200,
         3 * 4096 + 1, 5 * 4096 + 2047, 40000, 150001]


def _population(rng, seed, sizes=SIZES, n_refs=None):
    g = torch.Generator().manual_seed(seed)
    n_refs = int(rng.integers(1, 5)) if n_refs is None else n_refs
    refs, tensors, gid = [], [], 0
    atol, rtol = [(0.01, 0.01), (0.0, 0.0), (1e-3, 0.0), (0.0, 1e-3), (0.25, 0.25)][int(rng.integers(0, 5))]
    for _ in range(n_refs):
        dtype = int(rng.choice([workloads.F32, workloads.F16, workloads.BF16]))
        tdt = TORCH[dtype]
        n = int(rng.choice(sizes))
        off = int(rng.choice([0, 0, 0, 1, 2, 3, 4, 8]))
        scale = float(rng.choice([1.0, 1.0, 1e-3, 30.0, 1e30 if dtype != workloads.F16 else 100.0, 1e-30 if dtype == workloads.F32 else 1e-3]))
        store = (torch.randn(n + off, generator=g) * scale).to(tdt)
        kind = int(rng.integers(0, 4))
        if kind == 1:
            store = torch.relu(store)                                  # many exact zeros
        ref = store[off:]
        refs.append(ref)
        k = int(rng.choice([1, 1, 2, 3, 8, 33, 40]))
        for _ in range(k):
            c_off = int(rng.choice([0, 0, 0, 1, 3, 8]))
            r32 = ref.float()
            mode = int(rng.integers(0, 6))
            if mode == 0:
                c32 = r32.clone()                                      # identical
            elif mode == 1:
                c32 = r32 + (atol + rtol * r32.abs()) * (torch.rand(n, generator=g) * 2.2 - 1.1)   # around the boundary
            elif mode == 2:
                c32 = r32 * (1 + 1e-3 * torch.randn(n, generator=g))
            elif mode == 3:
                c32 = torch.randn(n, generator=g) * scale             # unrelated
            elif mode == 4:
                c32 = r32 + 1e-6 * scale * torch.randn(n, generator=g)
            else:
                c32 = r32 * 1.5 if scale < 1e20 else r32 * -1.0       # may overflow in the difference
            if n and rng.random() < 0.5:
                idx = torch.randint(0, n, (max(1, n // 500),), generator=g)
                vals = torch.tensor([float("nan"), float("inf"), float("-inf")])[torch.randint(0, 3, idx.shape, generator=g)]
                c32[idx] = vals
            c_store = torch.zeros(n + c_off, dtype=tdt)
            c_store[c_off:] = c32.to(tdt)
            tensors.append(workloads.Tensor(c_store[c_off:], len(refs) - 1, gid % 7, dtype))
            gid += 1
        if n and rng.random() < 0.3:
            ref[int(rng.integers(0, n))] = float("nan")                # a NaN in the reference itself (after the candidates were derived)
    return workloads.Population("fuzz %d" % seed, refs, tensors, 7, atol, rtol, torch.ones(7, 1), torch.ones(1))


def _run(pop):
    import paper_2510_03760_b200 as evo
    # device copies keep each tensor's offset inside its allocation (odd alignments reach the kernel)
    def to_dev(t):
        base = t._base if t._base is not None else t
        d = base.cuda()
        return d[t.storage_offset():t.storage_offset() + t.numel()]
    dev_refs = [to_dev(r) for r in pop.refs]
    cands = [to_dev(t.cand) for t in pop.tensors]
    refs = [dev_refs[t.ref_index] for t in pop.tensors]
    groups = [t.group for t in pop.tensors]
    res, gp = evo.evo_validate(cands, refs, pop.atol, pop.rtol, groups=groups, n_group=pop.n_group)
    got = evo.results_to_numpy(res)
    host_refs = [workloads.to_host_bits(r) for r in pop.refs]
    want = np.zeros(len(cands), dtype=oracle.RESULT_DTYPE)
    for i, t in enumerate(pop.tensors):
        want[i] = oracle.validate(workloads.to_host_bits(t.cand), host_refs[t.ref_index], t.dtype, pop.atol, pop.rtol)
    assert_results_equal(got, want, pop.name)
    assert np.array_equal(gp.cpu().numpy().view(np.uint32), oracle.group_pass(want, groups, pop.n_group)), pop.name


@pytest.mark.parametrize("chunk", range(6))
def test_random_populations(chunk):
    rng = np.random.default_rng(1000 + chunk)
    for j in range(8):
        _run(_population(rng, 100 * chunk + j))


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_populations_with_a_few_tiles_per_cta(seed):
    """Enough tiles to fill every CTA but only a few each: the regime in which the filter of max d/|r| is seeded from
    each tensor's first tile."""
    rng = np.random.default_rng(7000 + seed)
    _run(_population(rng, 9000 + seed, sizes=[150001, 200000, 131072, 99999], n_refs=14))


def _from_bits32(bits):
    return torch.from_numpy(np.asarray(bits, dtype=np.uint32).view(np.float32).copy())


def _adversarial(dtype, k, seed, filler_tensors=0):
    """Full tiles whose quotients d/|r| live where the division-free filter of max d/|r| is most exposed:
    subnormal references with differences of the same order (products and quotients under- and overflow),
    a few normal elements mixed in so that the running maximum crosses the range where the approximate first-tile
    quotients are trusted, and the largest quotient placed in the last lane of the first tile.
    With `filler_tensors` the population has enough tiles for the seed pass to run."""
    rng = np.random.default_rng(seed)
    g = torch.Generator().manual_seed(seed)
    tdt = TORCH[dtype]
    n = 3 * 4096 + 777
    if dtype == workloads.F32:
        ref = _from_bits32(rng.integers(1, 1 << 14, n)) * torch.where(torch.rand(n, generator=g) < 0.5, -1.0, 1.0)   # 1e-45 .. 2e-41
        tiny = lambda m: _from_bits32(rng.integers(0, 1 << 14, m))
    else:
        sub = torch.finfo(tdt).smallest_normal / (1 << (10 if dtype == workloads.F16 else 7))     # smallest subnormal
        ref = (torch.from_numpy(rng.integers(1, 64, n)).float() * sub) * torch.where(torch.rand(n, generator=g) < 0.5, -1.0, 1.0)
        tiny = lambda m: torch.from_numpy(rng.integers(0, 64, m)).float() * sub
    ref = ref.to(tdt)
    refs, tensors = [ref], []
    for i in range(k):
        c = ref.float() + tiny(n) * torch.where(torch.rand(n, generator=g) < 0.5, -1.0, 1.0)
        if i % 3 == 1:                       # a few normal-range elements: quotients of order 1 among subnormal ones
            idx = torch.randint(0, n, (5,), generator=g)
            c[idx] = ref.float()[idx] * 3.0
        if i % 3 == 2:                       # the largest quotient in the last element of the first tile
            c[4095] = ref.float()[4095] * 40.0
        if i % 4 == 3:                       # zeros in the candidate: d == |r|, quotient exactly 1
            c[torch.randint(0, n, (50,), generator=g)] = 0.0
        tensors.append(workloads.Tensor(c.to(tdt), 0, i % 7, dtype))
    for j in range(filler_tensors):          # ordinary tensors that only add tiles
        r = torch.randn(60000, generator=g).to(tdt)
        refs.append(r)
        tensors.append(workloads.Tensor((r.float() * (1 + 1e-3 * torch.randn(60000, generator=g))).to(tdt), len(refs) - 1, j % 7, dtype))
    return workloads.Population("adversarial dtype %d k %d" % (dtype, k), refs, tensors, 7, 0.0, 1e-3,
                                torch.ones(7, 1), torch.ones(1))


@pytest.mark.parametrize("dtype", [workloads.F32, workloads.F16, workloads.BF16])
@pytest.mark.parametrize("k", [1, 2, 33])
def test_max_rel_filter_on_subnormal_references(dtype, k):
    _run(_adversarial(dtype, k, 50 + k))


@pytest.mark.parametrize("dtype", [workloads.F32, workloads.BF16])
def test_max_rel_filter_on_subnormal_references_with_the_seed_pass(dtype):
    """Same data inside a population large enough (at least as many tiles as CTAs, few tiles each) for the filter to be
    seeded from every tensor's first tile."""
    _run(_adversarial(dtype, 5, 91, filler_tensors=40))


def test_max_rel_filter_when_the_tolerance_product_overflows():
    """References of half the largest binary32 value with rtol large enough that rtol * |r| overflows to +Inf (every finite
    difference is then within tolerance), candidates at all distances up to an overflowing difference."""
    g = torch.Generator().manual_seed(5)
    n = 3 * 4096 + 99
    big = torch.finfo(torch.float32).max / 2
    ref = torch.where(torch.rand(n, generator=g) < 0.5, -big, big)
    cands = []
    for i in range(3):
        c = ref * (1 + (torch.rand(n, generator=g) - 0.5) * [1e-6, 1.0, 3.9][i])       # the last one overflows where signs flip
        cands.append(c)
    tensors = [workloads.Tensor(c, 0, i, workloads.F32) for i, c in enumerate(cands)]
    pop = workloads.Population("tolerance overflow", [ref], tensors, 7, 0.0, 3.0, torch.ones(7, 1), torch.ones(1))
    _run(pop)
