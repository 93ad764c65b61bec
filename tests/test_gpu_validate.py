"""evo_validate on the GPU against the oracle, on the same seeded tensors: counts, flags,
verdicts, max_abs and max_rel bit-exact; SSE within 1e-5 relative."""
import os

import numpy as np
import pytest
import torch

import oracle
import workloads
from parity import assert_results_equal, oracle_population

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "closeness_cases.txt")


@pytest.fixture(scope="module")
def evo():
    import paper_2510_03760_b200 as evo
    return evo


def run_gpu(evo, pop, host=False):
    cands = [t.cand for t in pop.tensors]
    refs = [pop.refs[t.ref_index] for t in pop.tensors]
    groups = [t.group for t in pop.tensors]
    if host:
        return evo.evo_validate_host(cands, refs, pop.atol, pop.rtol, groups=groups, n_group=pop.n_group)
    cands = [c.cuda() for c in cands]
    dev_refs = [r.cuda() for r in pop.refs]
    refs = [dev_refs[t.ref_index] for t in pop.tensors]
    res, gp = evo.evo_validate(cands, refs, pop.atol, pop.rtol, groups=groups, n_group=pop.n_group)
    return evo.results_to_numpy(res), gp.cpu().numpy().view(np.uint32)


def check(evo, pop, host=False):
    want, want_gp = oracle_population(pop)
    got, got_gp = run_gpu(evo, pop, host=host)
    assert_results_equal(got, want, pop.name)
    assert np.array_equal(got_gp, want_gp), pop.name
    return got


def test_config1_small_case(evo):
    got = check(evo, workloads.config1("cpu"))
    assert got["n_mismatch"][0] == 7


def test_config2_shared_reference(evo):
    pop = workloads.config2("cpu")
    got = check(evo, pop)
    assert got["n_mismatch"].tolist() == pop.facts["n_mismatch"]
    check(evo, pop, host=True)


def test_config3_sixteen_bit_with_specials(evo):
    # 2^18 elements per tensor: several tiles and a ragged tail (not a multiple of the tile),
    # rates raised so that NaN/Inf and boundary values occur in every tensor
    pop = workloads.config3("cpu", n=(1 << 18) + 1000, k_per_dtype=5, special_rate=2e-5, boundary_rate=1e-3)
    got = check(evo, pop)
    assert (got["n_nonfinite"] > 0).all() and (got["flags"] != 0).all()


def test_config3_more_members_than_one_set_holds(evo):
    pop = workloads.config3("cpu", n=20000, k_per_dtype=40, special_rate=1e-4)
    check(evo, pop)


def test_config4_scaled_one_fully_wrong_candidate(evo):
    pop = workloads.config4("cpu", n=(1 << 20) + 12, k=16)
    got = check(evo, pop)
    assert got["pass"].sum() == 15 and got["pass"][pop.facts["wrong"]] == 0


def test_config5_scaled_ragged_mixed(evo):
    pop = workloads.config5("cpu", n_cand=96, log2_min=0.0, log2_max=17.0, trials=4)
    check(evo, pop)
    check(evo, pop, host=True)


@pytest.mark.parametrize("dtype", [workloads.F32, workloads.F16, workloads.BF16])
def test_special_value_pairs(evo, dtype):
    pop = workloads.special_values(dtype)
    for atol, rtol in [(0.25, 0.25), (0.01, 0.01), (0.0, 0.5), (0.0, 0.0)]:
        pop.atol, pop.rtol = atol, rtol
        check(evo, pop)
    # the same pairs repeated to fill several full tiles (exercises the vector path)
    reps = 3 * 8192 // pop.refs[0].numel() + 1
    pop.refs[0] = pop.refs[0].repeat(reps)
    pop.tensors[0].cand = pop.tensors[0].cand.repeat(reps)
    pop.atol, pop.rtol = 0.25, 0.25
    check(evo, pop)


def test_hand_worked_cases(evo):
    def bits(h):
        return np.array([int(h, 16)], dtype=np.uint32).view(np.float32)[0]
    for line in open(GOLDEN):
        if not line.strip() or line.startswith("#"):
            continue
        a, b, note = line.split("|", 2)
        atol, rtol, r, c = [bits(x) for x in a.split()]
        mism, flags, nonfin = [int(x) for x in b.split()]
        for n in (1, 5000):           # alone (scalar path) and filling a tile (vector path)
            ct = torch.full((n,), float(c), dtype=torch.float32).cuda()
            rt = torch.full((n,), float(r), dtype=torch.float32).cuda()
            ct.view(torch.int32).fill_(int(np.float32(c).view(np.int32)))
            rt.view(torch.int32).fill_(int(np.float32(r).view(np.int32)))
            res, _ = evo.evo_validate([ct], [rt], float(atol), float(rtol))
            got = evo.results_to_numpy(res)[0]
            assert got["n_mismatch"] == mism * n and got["flags"] == flags and got["n_nonfinite"] == nonfin * n, note
            want = oracle.validate(ct.cpu().numpy(), rt.cpu().numpy(), oracle.F32, atol, rtol)
            assert_results_equal(np.array([got]), np.array([want]), note)


def _pop(refs, pairs, atol, rtol, dtype=workloads.F32):
    tensors = [workloads.Tensor(c, ri, g, dtype) for g, (c, ri) in enumerate(pairs)]
    return workloads.Population("adhoc", refs, tensors, len(pairs), atol, rtol, torch.ones(1, 1), torch.ones(1))


def test_unaligned_views_and_ragged_sizes(evo):
    g = torch.Generator().manual_seed(5)
    for dtype, tdt in [(workloads.F32, torch.float32), (workloads.F16, torch.float16), (workloads.BF16, torch.bfloat16)]:
        for n in (0, 1, 3, 255, 4095, 4096, 4097, 8192 + 5, 3 * 8192 + 4001):
            ref_store = torch.randn(n + 16, generator=g).to(tdt).cuda()
            cand_store = (ref_store.float() + 0.004 * torch.randn(n + 16, generator=g).cuda()).to(tdt)
            for ro, co in [(0, 0), (1, 1), (0, 3), (5, 2)]:
                r, c = ref_store[ro:ro + n], cand_store[co:co + n]
                res, _ = evo.evo_validate([c], [r], 0.005, 0.005)
                want = oracle.validate(workloads.to_host_bits(c), workloads.to_host_bits(r), dtype, 0.005, 0.005)
                assert_results_equal(evo.results_to_numpy(res), np.array([want]), "n=%d offs=%d,%d dt=%d" % (n, ro, co, dtype))


def test_ragged_tail_of_a_shared_reference_with_specials(evo):
    # several members per reference (also more than one set holds), a last tile that is ragged
    # down to a few elements past a 16-byte vector, and NaN/Inf planted in that tail
    g = torch.Generator().manual_seed(17)
    for tdt, dtype in [(torch.float32, workloads.F32), (torch.float16, workloads.F16), (torch.bfloat16, workloads.BF16)]:
        for n, k in [(3 * 4096 + 8 * 5 + 3, 5), (4096 + 7, 34), (2, 3), (9, 1), (2 * 4096 + 16, 2)]:
            ref = torch.randn(n, generator=g).to(tdt)
            tensors = []
            for i in range(k):
                c = (ref.float() + 0.004 * torch.randn(n, generator=g)).to(tdt)
                if i % 2 == 0:
                    c[n - 1] = float("nan")
                if i % 3 == 0 and n > 12:
                    c[n - 12] = float("inf")
                tensors.append(workloads.Tensor(c, 0, i, dtype))
            pop = workloads.Population("tail n=%d k=%d dt=%d" % (n, k, dtype), [ref], tensors, k, 0.005, 0.005,
                                       torch.ones(k, 1), torch.ones(1))
            check(evo, pop)


def test_edge_populations(evo):
    g = torch.Generator().manual_seed(11)
    n = 5 * 4096 + 77
    r = torch.randn(n, generator=g)
    # identical candidate; reference full of exact zeros (ReLU-like); tiny differences whose
    # squares underflow in binary32; huge values whose squares overflow binary32
    relu = torch.relu(r)
    tiny_r = r * 1e-25
    tiny_c = tiny_r * (1 + 1e-3)
    huge_r = r * 1e30
    huge_c = huge_r * 1.5
    pop = _pop([r, relu, tiny_r, huge_r],
               [(r.clone(), 0), (relu + 1e-3 * torch.rand(n, generator=g), 1), (relu.clone(), 1),
                (tiny_c, 2), (huge_c, 3), (r + 1e-3, 0)], 1e-2, 1e-2)
    got = check(evo, pop)
    assert got["sse"][0] == 0 and got["pass"][0] == 1
    assert got["sse"][3] > 0          # not flushed away


def test_results_are_reproducible_and_independent_of_other_tensors(evo):
    pop = workloads.config5("cpu", n_cand=40, log2_min=8.0, log2_max=16.0, trials=4)
    a, _ = run_gpu(evo, pop)
    b, _ = run_gpu(evo, pop)
    assert a.tobytes() == b.tobytes()
    # a tensor validated alone gives the same counts and maxima as inside the population
    t = pop.tensors[7]
    res, _ = evo.evo_validate([t.cand.cuda()], [pop.refs[t.ref_index].cuda()], pop.atol, pop.rtol)
    assert_results_equal(evo.results_to_numpy(res), a[7:8])


def test_prepared_population_gives_the_same_results(evo):
    pop = workloads.config5("cpu", n_cand=30, log2_min=8.0, log2_max=15.0, trials=4)
    dev_refs = [r.cuda() for r in pop.refs]
    cands = [t.cand.cuda() for t in pop.tensors]
    refs = [dev_refs[t.ref_index] for t in pop.tensors]
    groups = [t.group for t in pop.tensors]
    res, gp = evo.evo_validate(cands, refs, pop.atol, pop.rtol, groups=groups, n_group=pop.n_group)
    prep = evo.Prepared(cands, refs, groups, pop.n_group)
    for _ in range(2):
        res2, gp2 = evo.evo_validate(prep, None, pop.atol, pop.rtol)
        assert torch.equal(res, res2) and torch.equal(gp, gp2)
    prep_ng = evo.Prepared(cands, refs)
    res3, gp3 = evo.evo_validate(prep_ng, None, pop.atol, pop.rtol)
    assert torch.equal(res, res3) and gp3 is None


def test_plan_inspect_through_the_binding(evo):
    ref = torch.zeros(1 << 22, device="cuda")
    cands = [torch.zeros(1 << 22, device="cuda") for _ in range(16)]
    info = evo.plan_inspect(cands, [ref] * 16, 296)
    # 1024 tiles per tensor for 296 CTAs are fewer than six items each: the 16 members go into two sets of 8
    assert info["n_sets"] == 2 and info["n_ctas"] == 296 and info["total_tiles"] == 2048 and info["tile_elems"] == 4096
    assert info["weights"].sum() == 2048 * 9 and info["weights"].max() <= 8 * 9


def test_empty_call_and_empty_groups(evo):
    res, gp = evo.evo_validate([], [], 0.1, 0.1, groups=[], n_group=3)
    torch.cuda.synchronize()
    assert res.shape[0] == 0 and gp.cpu().tolist() == [1, 1, 1]
    z = torch.zeros(0, device="cuda")
    res, gp = evo.evo_validate([z, z], [z, z], 0.1, 0.1, groups=[2, 2], n_group=4)
    got = evo.results_to_numpy(res)
    assert got["pass"].tolist() == [1, 1] and got["n_mismatch"].sum() == 0 and gp.cpu().tolist() == [1, 1, 1, 1]


def test_argument_errors(evo):
    L, ctx = evo.load_library(), evo.default_context(0)
    c = torch.zeros(64, device="cuda")
    r = torch.zeros(64, device="cuda")
    out = torch.zeros(40, dtype=torch.uint8, device="cuda")
    for atol, rtol in [(-1.0, 0.0), (0.0, float("nan")), (float("inf"), 0.0)]:
        with pytest.raises(evo.EvoError) as e:
            evo.evo_validate([c], [r], atol, rtol)
        assert e.value.status == -1
    with pytest.raises(evo.EvoError) as e:
        evo.evo_validate([c], [r], 0.1, 0.1, groups=[5], n_group=2)
    assert e.value.status == -1
    # a tensor that is not aligned to its element size (torch cannot build such a view: raw call)
    import ctypes as C
    ptrs = np.array([c.data_ptr() + 2], dtype=np.uint64)
    desc = np.zeros(1, dtype=evo.binding._DESC_DTYPE)
    desc[0] = (8, r.data_ptr(), evo.EVO_F32, 0)
    st = L.evo_validate(ctx._h, C.c_void_p(ptrs.ctypes.data), None, C.c_void_p(desc.ctypes.data), 1, evo.EVO_F32,
                        0.1, 0.1, C.c_void_p(out.data_ptr()), None, 0, None)
    assert st == -2 and b"aligned" in L.evo_last_error(ctx._h)
    desc[0] = (8, r.data_ptr(), 9, 0)
    ptrs[0] = c.data_ptr()
    assert L.evo_validate(ctx._h, C.c_void_p(ptrs.ctypes.data), None, C.c_void_p(desc.ctypes.data), 1, evo.EVO_F32,
                          0.1, 0.1, C.c_void_p(out.data_ptr()), None, 0, None) == -3
    assert L.evo_validate(ctx._h, C.c_void_p(ptrs.ctypes.data), None, C.c_void_p(desc.ctypes.data), 1, evo.EVO_F32,
                          0.1, 0.1, None, None, 0, None) == -1
    # the context stays usable after errors
    res, _ = evo.evo_validate([c], [r], 0.1, 0.1)
    assert evo.results_to_numpy(res)["pass"][0] == 1
