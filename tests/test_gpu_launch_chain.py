"""The launch chain of evo_validate on the GPU: plans travel as kernel arguments or by copy, a repeated call reuses
the plan in device memory, every kernel may start while its predecessor still runs.  None of this may change a
result: every variant is compared with the oracle under the usual bars, and with each other byte for byte."""
import numpy as np
import pytest
import torch

import workloads
from parity import assert_results_equal, oracle_population

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def evo():
    import paper_2510_03760_b200 as evo
    return evo


def _dev(pop):
    refs = [r.cuda() for r in pop.refs]
    return [t.cand.cuda() for t in pop.tensors], [refs[t.ref_index] for t in pop.tensors], [t.group for t in pop.tensors]


def test_a_repeated_call_reuses_the_plan_but_reads_the_tensors_again(evo):
    """Same pointers, sizes and groups: the second call skips planning and upload.  The data behind the pointers has
    changed in between and the results must follow it."""
    ctx = evo.Context(0)
    pop = workloads.config2("cpu", n=(1 << 15) + 77, k=5, trials=4)
    cands, refs, groups = _dev(pop)
    prep = evo.Prepared(cands, refs, groups, pop.n_group)
    before = ctx.launches
    res1, gp1 = evo.evo_validate(prep, None, pop.atol, pop.rtol, ctx=ctx)
    first = ctx.launches - before
    want1, verdict1 = oracle_population(pop)
    assert_results_equal(evo.results_to_numpy(res1), want1, "first call")
    cands[2].add_(1.0)                                        # in place: the pointer stays, every element is now wrong
    pop.tensors[2].cand = pop.tensors[2].cand + 1.0
    before = ctx.launches
    res2, gp2 = evo.evo_validate(prep, None, pop.atol, pop.rtol, ctx=ctx)
    second = ctx.launches - before
    want2, verdict2 = oracle_population(pop)
    got2 = evo.results_to_numpy(res2)
    assert_results_equal(got2, want2, "second call")
    assert got2["pass"][2] == 0 and np.array_equal(gp2.cpu().numpy().view(np.uint32), verdict2)
    assert second == first - 1, "the repeated call should have launched everything but the plan's store"
    # other tolerances with the same plan
    res3, _ = evo.evo_validate(prep, None, 2.0, 0.0, ctx=ctx)
    pop.atol, pop.rtol = 2.0, 0.0
    assert_results_equal(evo.results_to_numpy(res3), oracle_population(pop)[0], "other tolerances")


def test_any_change_of_the_arguments_makes_a_new_plan(evo):
    ctx = evo.Context(0)
    pops = [workloads.config5("cpu", n_cand=20, log2_min=4.0, log2_max=15.0, trials=4),
            workloads.config2("cpu", n=5000, k=3, trials=4),
            workloads.config5("cpu", n_cand=21, log2_min=4.0, log2_max=15.0, trials=4)]
    devs = [_dev(p) for p in pops]
    wants = [oracle_population(p) for p in pops]
    for rnd in range(3):
        for p, (cands, refs, groups), (want, verdict) in zip(pops, devs, wants):
            res, gp = evo.evo_validate(cands, refs, p.atol, p.rtol, groups=groups, n_group=p.n_group, ctx=ctx)
            assert_results_equal(evo.results_to_numpy(res), want, "%s round %d" % (p.name, rnd))
            assert np.array_equal(gp.cpu().numpy().view(np.uint32), verdict)
    # the integer check shares the context's plan area: a float call after it must not trust the old plan
    p, (cands, refs, groups), (want, verdict) = pops[0], devs[0], wants[0]
    evo.evo_validate(cands, refs, p.atol, p.rtol, groups=groups, n_group=p.n_group, ctx=ctx)
    ints = torch.arange(10000, dtype=torch.int32, device="cuda")
    evo.evo_validate_exact([ints], [ints], ctx=ctx)
    res, gp = evo.evo_validate(cands, refs, p.atol, p.rtol, groups=groups, n_group=p.n_group, ctx=ctx)
    assert_results_equal(evo.results_to_numpy(res), want, "after an integer check")
    # without groups, then with: the verdict lists are part of the plan
    res, gp = evo.evo_validate(cands, refs, p.atol, p.rtol, ctx=ctx)
    assert gp is None
    res, gp = evo.evo_validate(cands, refs, p.atol, p.rtol, groups=groups, n_group=p.n_group, ctx=ctx)
    assert np.array_equal(gp.cpu().numpy().view(np.uint32), verdict)


def test_alternating_populations_back_to_back_without_a_host_wait(evo):
    """Two populations take turns on one context and one stream, fifty calls deep, nothing waits in between: the plan
    area, the partial records and the seeds are rewritten while earlier kernels may still be in flight.  With
    overlapped launches on and off, small plans (kernel arguments) and a large one (copy from pinned memory)."""
    small = workloads.config2("cpu", n=(1 << 16) + 5, k=4, trials=4)
    large = workloads.config5("cpu", n_cand=420, log2_min=3.0, log2_max=13.0, trials=4)        # a plan beyond 32 KiB
    mid = workloads.config3("cpu", n=1 << 15, k_per_dtype=20)
    pops = [small, large, mid]
    devs = [_dev(p) for p in pops]
    wants = [oracle_population(p) for p in pops]
    for overlapped in (True, False):
        ctx = evo.Context(0)
        ctx.set_overlapped_launch(overlapped)
        outs = []
        for i in range(48):
            j = i % 3
            p, (cands, refs, groups) = pops[j], devs[j]
            outs.append((j, *evo.evo_validate(cands, refs, p.atol, p.rtol, groups=groups, n_group=p.n_group, ctx=ctx)))
        ctx.synchronize()
        first = {}
        for j, res, gp in outs:
            got = evo.results_to_numpy(res)
            if j not in first:
                assert_results_equal(got, wants[j][0], "%s overlapped=%s" % (pops[j].name, overlapped))
                assert np.array_equal(gp.cpu().numpy().view(np.uint32), wants[j][1])
                first[j] = got.tobytes()
            assert got.tobytes() == first[j], "a later call of %s differs from its first" % pops[j].name


def test_whole_step_back_to_back_matches_the_oracle(evo):
    """gen -> validate -> fitness, many steps deep on one stream: the kernels of consecutive calls overlap their
    launches, and the last step's verdicts and speedups are still the oracle's."""
    import oracle
    ctx = evo.Context(0)
    pop = workloads.config2("cpu", n=20000, k=6, trials=9)
    cands, refs, groups = _dev(pop)
    prep = evo.Prepared(cands, refs, groups, pop.n_group)
    times, base = pop.times.cuda(), pop.base_times.cuda()
    buf = torch.empty(20000, dtype=torch.float32, device="cuda")
    for i in range(30):
        evo.evo_gen_inputs(i, 0, evo.EVO_F32, 20000, buf, ctx=ctx)
        res, gp = evo.evo_validate(prep, None, pop.atol, pop.rtol, ctx=ctx)
        fit = evo.evo_fitness(times, base, gp, ctx=ctx)
    ctx.synchronize()
    want, verdict = oracle_population(pop)
    assert_results_equal(evo.results_to_numpy(res), want)
    assert evo.fits_to_numpy(fit).tobytes() == oracle.fitness(pop.times.numpy(), pop.base_times.numpy(), verdict).tobytes()
    z = buf.cpu().numpy()
    wz = oracle.gen_inputs(29, 0, oracle.F32, 20000)
    from parity import ordered
    assert np.abs(ordered(z) - ordered(wz)).max() <= 4


def test_per_cta_clocks_cover_every_cta_and_lie_inside_the_call(evo):
    """evo_debug_cta_timing: one (begin, end) pair of the GPU's nanosecond clock per persistent CTA of the main kernel;
    begin <= end, all within a few milliseconds of each other, as many pairs as the plan has CTAs; off again afterwards."""
    ctx = evo.Context(0)
    pop = workloads.config5("cpu", n_cand=200, log2_min=8.0, log2_max=17.0, trials=4)
    cands, refs, groups = _dev(pop)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    ctx.cta_timing(True)
    res, gp = evo.evo_validate(cands, refs, pop.atol, pop.rtol, groups=groups, n_group=pop.n_group, ctx=ctx)
    t = ctx.read_cta_times()
    info = evo.plan_inspect(cands, refs, 2 * sms)
    assert len(t) == info["n_ctas"] and len(t) > 0
    assert (t[:, 1] >= t[:, 0]).all() and int(t[:, 1].max() - t[:, 0].min()) < 50_000_000
    assert_results_equal(evo.results_to_numpy(res), oracle_population(pop)[0], "with per-CTA clocks")
    ctx.cta_timing(False)
    evo.evo_validate(cands, refs, pop.atol, pop.rtol, groups=groups, n_group=pop.n_group, ctx=ctx)
    assert len(ctx.read_cta_times()) == 0


def test_a_repeated_call_can_be_captured_in_a_cuda_graph_and_replayed(evo):
    """After one ordinary call on the stream, the same call only launches kernels (its plan is in device memory), so
    check and fitness can be captured once and replayed; each replay reads the tensors as they are then."""
    import oracle
    ctx = evo.Context(0)
    pop = workloads.config2("cpu", n=30000, k=5, trials=7)
    cands, refs, groups = _dev(pop)
    prep = evo.Prepared(cands, refs, groups, pop.n_group)
    times, base = pop.times.cuda(), pop.base_times.cuda()
    res = torch.empty((len(cands), 40), dtype=torch.uint8, device="cuda")
    gp = torch.empty(pop.n_group, dtype=torch.int32, device="cuda")
    fit = torch.empty((pop.n_group, 16), dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        evo.evo_validate(prep, None, pop.atol, pop.rtol, results=res, group_pass=gp, ctx=ctx)
        evo.evo_fitness(times, base, gp, out=fit, ctx=ctx)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    before = ctx.launches
    with torch.cuda.graph(graph, stream=side):
        evo.evo_validate(prep, None, pop.atol, pop.rtol, results=res, group_pass=gp, ctx=ctx)
        evo.evo_fitness(times, base, gp, out=fit, ctx=ctx)
    assert ctx.launches - before == 3                       # first pass, second pass with the verdicts, fitness: no plan store
    for rnd in range(3):
        if rnd:
            cands[rnd].mul_(1.5)                             # in place, between replays
            pop.tensors[rnd].cand = pop.tensors[rnd].cand * 1.5
        res.fill_(0xAB)
        graph.replay()
        torch.cuda.synchronize()
        want, verdict = oracle_population(pop)
        assert_results_equal(evo.results_to_numpy(res), want, "replay %d" % rnd)
        assert np.array_equal(gp.cpu().numpy().view(np.uint32), verdict)
        assert evo.fits_to_numpy(fit).tobytes() == oracle.fitness(pop.times.numpy(), pop.base_times.numpy(), verdict).tobytes()
