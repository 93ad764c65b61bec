#!/usr/bin/env python
"""Benchmark of the candidate-evaluation step on B200.

One "step" is one pass of the whole evaluation path over one population of synthetic
candidate outputs: evo_gen_inputs (one test-input tensor), evo_validate (every candidate
tensor against its reference) and evo_fitness (median-of-trials speedup).  The metric is the
rate at which candidate outputs are validated: algorithmic bytes (every candidate tensor once,
every distinct reference once) per second, for inputs already resident in HBM (`value`) and
through the host-buffer entry points with the copies inside the timed region (`e2e`).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload config4|config3|config5|config2|config1]
    python bench.py --impl reference ...     # the CPU oracle on a bounded sample (baseline arm)

With N > 1 every rank evaluates its own replica of the population (one rank per GPU): candidates
are independent, there is no exchange between GPUs.  Started without a launcher, `--gpus N`
re-executes itself under torch.distributed.run with N local ranks.

The default run (config 4) also reports, under "per_config", the other synthetic populations
(configs 1, 2, 3 and 5): time of the main kernel, of the evo_validate call and of the whole step.
"""
import argparse
import json
import os
import statistics
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads  # noqa: E402

METRIC = "validated_bytes_per_second"
UNIT = "GB/s"
DATASHEET_HBM_GBS = 7700.0      # nominal HBM3e bandwidth of a 180 GB B200 (HGX figure; the DGX figure is 8000)
WORKLOAD_NOTES = {
    "config1": "1 fp32 candidate of 64 x 64 elements against its reference (fits in L2; latency)",
    "config4": "16 fp32 candidates x 2^28 elements (1 GiB each) sharing one 1 GiB reference",
    "config3": "64 fp16 + 64 bf16 candidates x 2^20 elements, one reference per dtype",
    "config5": "1024 candidates, 1-3 tensors each, 2^10..2^24 elements, fp32/fp16/bf16, own references",
    "config2": "8 fp32 candidates x 262144 elements sharing one reference (fits in L2)",
    "clean16": "8 bf16 candidates x 2^26 elements sharing one reference, noise far below the tolerance",
}


def build_population(name, device, log2_elems=None):
    if log2_elems is not None:
        return workloads.config4(device, n=1 << log2_elems)
    return getattr(workloads, name)(device)


def gen_elems(pop):
    """Size of the test-input tensor generated per step: one tensor as large as the largest output."""
    return max(t.cand.numel() for t in pop.tensors)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# DRAM traffic of validate_pass1 as counted by ncu (dram__bytes_read.sum + dram__bytes_write.sum) on a reduced
# config 4 (2^24 elements per tensor), per algorithmic byte (the capture is summarised under profiles/).
# It stands only for the kernel sources it was captured on: their hash is checked, and a mismatch reports null.
NCU_TRAFFIC = {"dram_bytes_per_algorithmic_byte": 1.0056, "sources_sha1": "f74fa22f289f3a07581d7d30302b1e0cbb9ac71d"}


def kernel_sources_sha1():
    import hashlib
    h = hashlib.sha1()
    for name in ("validate.cu", "plan.h", "plan.cu"):
        with open(os.path.join(ROOT, "paper_2510_03760_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def ncu_traffic(alg_bytes):
    if NCU_TRAFFIC["dram_bytes_per_algorithmic_byte"] is None or NCU_TRAFFIC["sources_sha1"] != kernel_sources_sha1():
        return None
    return NCU_TRAFFIC["dram_bytes_per_algorithmic_byte"] * alg_bytes


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while a region runs."""

    def __init__(self, index, period_s=0.02):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------- oracle arm
FULL_SHAPE = {"config4": dict(n=1 << 28, k=16), "config3": dict(n=1 << 20, k=128), "config2": dict(n=1 << 18, k=8),
              "config1": dict(n=1 << 12, k=1), "clean16": dict(n=1 << 26, k=8)}
FULL_TRIALS = {"config1": 5}


class OracleSample:
    """A bounded sample of a workload for the CPU oracle, and the factors that scale its
    timings (linear in elements) to one full step of that workload."""

    def __init__(self, workload, log2_elems, log2_gen, seed=None):
        if workload in FULL_SHAPE:
            n_full, k_full = FULL_SHAPE[workload]["n"], FULL_SHAPE[workload]["k"]
            n_s = min(n_full, 1 << log2_elems)
            if workload == "config4":
                pop = workloads.config4("cpu", n=n_s, k=4, **({} if seed is None else {"seed": seed}))
            elif workload == "config3":
                pop = workloads.config3("cpu", n=n_s, k_per_dtype=2)
            elif workload == "config1":
                pop = workloads.config1("cpu")
            elif workload == "clean16":
                pop = workloads.clean16("cpu", n=n_s, k=4)
            else:
                pop = workloads.config2("cpu", n=n_s, k=4)
            self.scale_val = (n_full * k_full) / float(n_s * len(pop.tensors))
            self.rows, self.n_gen_full = k_full, n_full
            what = "%d candidates x 2^%d elements of %s" % (len(pop.tensors), n_s.bit_length() - 1, workload)
        else:
            pop = workloads.config5("cpu", n_cand=48, log2_min=10.0, log2_max=float(min(22, log2_elems)))
            self.scale_val = 2048 * 1.73e6 / float(sum(t.cand.numel() for t in pop.tensors))
            self.rows, self.n_gen_full = 1024, 1 << 24
            what = "48 candidates of config5 with sizes up to 2^%d" % min(22, log2_elems)
        self.pop = pop
        self.refs = [workloads.to_host_bits(r) for r in pop.refs]
        self.cands = [workloads.to_host_bits(t.cand) for t in pop.tensors]
        self.n_gen = min(self.n_gen_full, 1 << log2_gen)
        import numpy as np
        self.times = np.repeat(pop.times.numpy()[:1], self.rows, axis=0)
        self.base = pop.base_times.numpy()
        self.what = "validate %s, generate 2^%d normals, fitness of %d rows" % (what, self.n_gen.bit_length() - 1, self.rows)
        self.description = ("oracle, 1 thread: %s; timings scaled linearly in elements to one full step" % self.what)

    def run(self):
        """One timed pass over the sample; returns (estimated seconds of a full step, seconds spent)."""
        import oracle
        t0 = time.perf_counter()
        for t, c in zip(self.pop.tensors, self.cands):
            oracle.validate(c, self.refs[t.ref_index], t.dtype, self.pop.atol, self.pop.rtol)
        t1 = time.perf_counter()
        oracle.gen_inputs(1, 0, oracle.F32, self.n_gen)
        t2 = time.perf_counter()
        oracle.fitness(self.times, self.base)
        t3 = time.perf_counter()
        est = (t1 - t0) * self.scale_val + (t2 - t1) * (self.n_gen_full / float(self.n_gen)) + (t3 - t2)
        return est, t3 - t0


# The sample both oracle legs time (the reference arm once per step, the cpu_baseline leg a few times over):
# log2 of the elements per sampled tensor and of the generated normals.
ORACLE_SAMPLE_LOG2 = (24, 22)


def full_algorithmic_bytes(workload):
    known = {"config4": 17 * (1 << 30), "config3": 130 * (1 << 21), "config2": 9 * (1 << 20), "config1": 2 * (1 << 14),
             "clean16": 9 * (1 << 27)}
    return known.get(workload, int(2048 * 1.73e6 * 3 * 2))


def config_keys(workload, n_gen, n_tensors, n_group, trials, alg_bytes, world):
    """The `config` object of a line: the same keys, built the same way, in both arms."""
    return {"workload": workload, "what": WORKLOAD_NOTES[workload],
            "step": "evo_gen_inputs(%d fp32 normals) + evo_validate(%d tensors) + evo_fitness(%d x %d trials)"
                    % (n_gen, n_tensors, n_group, trials),
            "algorithmic_bytes_per_step": alg_bytes,
            "l2": "inputs larger than L2" if alg_bytes > (1 << 28) else "inputs fit in L2", "replicas": world}


def _oracle_process(workload, seed, passes, barrier, queue):
    """One worker of the many-process baseline: its own sample (other tensors than every other worker's),
    built before the common start, then `passes` timed passes."""
    sample = OracleSample(workload, ORACLE_SAMPLE_LOG2[0], ORACLE_SAMPLE_LOG2[1], seed=seed)
    sample.run()
    barrier.wait()
    t0 = time.perf_counter()
    ests = [sample.run()[0] for _ in range(passes)]
    queue.put((sum(ests) / len(ests), time.perf_counter() - t0, sample.what))


def oracle_many_processes(workload, alg_bytes, passes):
    """The oracle as P independent single-threaded processes over disjoint candidates, P = the cores this process may
    use.  Processes are spawned (never forked: the parent holds a CUDA context).  Returns the cpu_baseline-style dict."""
    import multiprocessing as mp
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    ctx = mp.get_context("spawn")
    barrier, queue = ctx.Barrier(cores + 1), ctx.Queue()
    procs = [ctx.Process(target=_oracle_process, args=(workload, 4000 + 17 * (i + 1), passes, barrier, queue), daemon=True)
             for i in range(cores)]
    for p in procs:
        p.start()
    try:
        barrier.wait(timeout=600)
        t0 = time.perf_counter()
        got = [queue.get(timeout=600) for _ in procs]
        wall = time.perf_counter() - t0
    finally:
        for p in procs:
            p.join(timeout=30)
            if p.is_alive():
                p.kill()
    rate = sum(alg_bytes / g[0] for g in got) / 1e9
    return {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle, one single-threaded process per core, disjoint candidates",
            "sample": "each process: %d passes over its own sample (%s); the rates of the processes added up" % (passes, got[0][2]),
            "seconds": wall}


def run_reference(args):
    """Baseline arm: the CPU oracle, as it stands, on the host cores; rank 0 only.  Every step is one pass over a
    bounded sample of the workload; `value` scales the sample's timings to a full step."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    passes = args.steps + args.warmup
    shrink = 0 if passes <= 30 else 2 if passes <= 120 else 4 if passes <= 500 else 6      # about 1 s .. 20 ms per pass
    sample = OracleSample(args.workload, ORACLE_SAMPLE_LOG2[0] - shrink, ORACLE_SAMPLE_LOG2[1] - shrink)
    alg_bytes = full_algorithmic_bytes(args.workload)
    for _ in range(args.warmup):
        sample.run()
    ests, spent = [], 0.0
    for _ in range(args.steps):
        est, s = sample.run()
        ests.append(est)
        spent += s
    est = sum(ests) / len(ests)
    value = alg_bytes / est / 1e9
    shape = FULL_SHAPE.get(args.workload)
    if shape:
        config = config_keys(args.workload, shape["n"], shape["k"], shape["k"], FULL_TRIALS.get(args.workload, 100), alg_bytes, 1)
    else:
        config = config_keys(args.workload, 1 << 24, 2048, 1024, 100, alg_bytes, 1)
        config["step"] = config["step"].replace("2048 tensors", "about 2048 tensors")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": spent / max(1, args.steps) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample.description},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0, "full_step_ms_estimate": est * 1e3,
        "note": "each step is one pass over the bounded sample named in cpu_baseline.sample; ms_per_step is the measured "
                "time of that pass, value = algorithmic bytes of a full step / full_step_ms_estimate",
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------- GPU arm
def _clone_population(pop):
    refs = [r.clone() for r in pop.refs]
    tensors = [workloads.Tensor(t.cand.clone(), t.ref_index, t.group, t.dtype) for t in pop.tensors]
    return workloads.Population(pop.name, refs, tensors, pop.n_group, pop.atol, pop.rtol, pop.times, pop.base_times, pop.facts)


def measure_config(evo, ctx, name, device, peak, reps):
    """One of the smaller synthetic populations: device time of the main kernel alone, of the whole evo_validate call
    (calls issued back to back) and of the whole step, all with CUDA events on the launching stream.
    Populations that fit in L2 are labelled so; config 3 (272 MB, about twice L2) is run on three disjoint copies in
    rotation so that no call finds its tensors in L2."""
    pop = getattr(workloads, name)(device)
    alg_bytes = pop.algorithmic_bytes()
    copies = [pop] + ([_clone_population(pop), _clone_population(pop)] if name == "config3" else [])
    preps, n_tensors = [], len(pop.tensors)
    for p in copies:
        preps.append(evo.Prepared([t.cand for t in p.tensors], [p.refs[t.ref_index] for t in p.tensors],
                                  [t.group for t in p.tensors], p.n_group))
    n_gen = gen_elems(pop)
    gen_buf = torch.empty(n_gen, dtype=torch.float32, device=device)
    results = torch.empty((n_tensors, 40), dtype=torch.uint8, device=device)
    gpass = torch.empty(pop.n_group, dtype=torch.int32, device=device)
    fits = torch.empty((pop.n_group, 16), dtype=torch.uint8, device=device)

    def validate(i):
        evo.evo_validate(preps[i % len(preps)], None, pop.atol, pop.rtol, results=results, group_pass=gpass, ctx=ctx)

    def step(i):
        evo.evo_gen_inputs(3000 + i, 0, evo.EVO_F32, n_gen, gen_buf, ctx=ctx)
        validate(i)
        evo.evo_fitness(pop.times, pop.base_times, gpass, out=fits, ctx=ctx)

    def timed(fn):
        for i in range(3):
            fn(i)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(reps):
            fn(i)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    call_ms = timed(validate)
    step_ms = timed(step)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for a, b in evs:
        a.record()
        b.record()
    torch.cuda.synchronize()
    for i, (a, b) in enumerate(evs):
        ctx.set_timing_events(a, b)
        validate(i)
    torch.cuda.synchronize()
    kernel_ms = statistics.median(a.elapsed_time(b) for a, b in evs)
    fits_l2 = alg_bytes < 100 * (1 << 20)
    out = {
        "what": WORKLOAD_NOTES[name], "tensors": n_tensors, "candidates": pop.n_group, "algorithmic_bytes": alg_bytes,
        "reps": reps, "kernel_ms": kernel_ms, "call_ms": call_ms, "step_ms": step_ms,
        "kernel_gbs": alg_bytes / (kernel_ms * 1e-3) / 1e9, "call_gbs": alg_bytes / (call_ms * 1e-3) / 1e9,
        "step_gbs": alg_bytes / (step_ms * 1e-3) / 1e9,
        "kernel_frac_of_peak": alg_bytes / (kernel_ms * 1e-3) / 1e9 / peak, "step_frac_of_peak": alg_bytes / (step_ms * 1e-3) / 1e9 / peak,
        "candidates_per_s": pop.n_group / (step_ms * 1e-3),
        "memory": ("L2: the population fits in the 126 MB L2, the figures are not HBM rates" if fits_l2 else
                   "L2 defeated: three disjoint copies of the population in rotation" if len(copies) > 1 else
                   "inputs larger than L2"),
        "kernel": "validate_pass1 (CUDA events around the launch, median)",
        "call": "evo_validate, calls back to back (CUDA events around the loop)",
    }
    if fits_l2:
        # Launch-bound populations: the repeated call only launches kernels (the plan is reused), so check + fitness
        # can be captured once and replayed as a CUDA graph.
        side = torch.cuda.Stream(device)
        with torch.cuda.stream(side):
            for i in range(3):
                validate(0)
                evo.evo_fitness(pop.times, pop.base_times, gpass, out=fits, ctx=ctx)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            validate(0)
            evo.evo_fitness(pop.times, pop.base_times, gpass, out=fits, ctx=ctx)
        graph.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            graph.replay()
        b.record()
        torch.cuda.synchronize()
        out["graph_replay_ms"] = a.elapsed_time(b) / reps
        out["graph"] = "evo_validate + evo_fitness captured once in a CUDA graph, replays back to back"
        del graph
    if name == "config5":
        # load balance as measured: every CTA's own begin and end clock in one extra, untimed call
        ctx.cta_timing(True)
        validate(0)
        t = ctx.read_cta_times()
        ctx.cta_timing(False)
        if len(t):
            busy = (t[:, 1] - t[:, 0]).astype("float64")
            out["load_balance"] = {"ctas": int(len(t)), "max_over_mean_cta_time": float(busy.max() / busy.mean()),
                                   "min_over_mean_cta_time": float(busy.min() / busy.mean()),
                                   "mean_cta_ms": float(busy.mean() * 1e-6),
                                   "kernel_span_ms": float((t[:, 1].max() - t[:, 0].min()) * 1e-6),
                                   "how": "%globaltimer at the start and the end of every persistent CTA of validate_pass1"}
    del preps, copies, pop
    torch.cuda.empty_cache()
    return out


def measure_generated(evo, ctx, device, peak, log2_n=28, reps=10):
    """evo_validate_generated (reference regenerated in the kernel) against the two-step route evo_gen_inputs(raw words)
    + evo_validate_exact, for one candidate and for sixteen candidates of 2^log2_n words each."""
    n = 1 << log2_n
    ref = torch.empty(n, dtype=torch.int32, device=device)
    out = {"elements_per_tensor": n, "dtype": "u32 words compared as int32", "reps": reps}

    def timed(fn):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    evo.evo_gen_inputs(7, 0, evo.EVO_U32, n, ref, ctx=ctx)
    for k in (1, 16):
        cands = [ref.clone() for _ in range(k)]
        cands[-1][n // 3] += 1                                  # one wrong element in the last candidate
        fused_ms = timed(lambda: evo.evo_validate_generated(7, cands, offsets=0, dtype=evo.EVO_I32, ctx=ctx))

        def two_step():
            evo.evo_gen_inputs(7, 0, evo.EVO_U32, n, ref, ctx=ctx)
            evo.evo_validate_exact(cands, [ref] * k, ctx=ctx)
        two_ms = timed(two_step)
        got = evo.exact_to_numpy(evo.evo_validate_generated(7, cands, offsets=0, dtype=evo.EVO_I32, ctx=ctx)[0])
        assert got["n_mismatch"].sum() == 1 and got["n_mismatch"][-1] == 1, "fused check is wrong"
        cand_bytes = 4 * n * k
        out["k%d" % k] = {"fused_ms": fused_ms, "generate_then_check_ms": two_ms, "speedup": two_ms / fused_ms,
                          "fused_candidate_gbs": cand_bytes / (fused_ms * 1e-3) / 1e9,
                          "fused_frac_of_peak": cand_bytes / (fused_ms * 1e-3) / 1e9 / peak}
        del cands
    del ref
    torch.cuda.empty_cache()
    return out


def run_ours(args):
    import paper_2510_03760_b200 as evo

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    distributed = world > 1
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if distributed:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)

    def barrier():
        if distributed:
            dist.barrier()
        torch.cuda.synchronize()

    ctx = evo.Context(local_rank)
    pop = build_population(args.workload, device, args.log2_elems)
    cands = [t.cand for t in pop.tensors]
    refs = [pop.refs[t.ref_index] for t in pop.tensors]
    groups = [t.group for t in pop.tensors]
    n_group = pop.n_group
    alg_bytes = pop.algorithmic_bytes()
    n_gen = gen_elems(pop)
    gen_buf = torch.empty(n_gen, dtype=torch.float32, device=device)
    results = torch.empty((len(cands), 40), dtype=torch.uint8, device=device)
    gpass = torch.empty(n_group, dtype=torch.int32, device=device)
    fits = torch.empty((n_group, 16), dtype=torch.uint8, device=device)

    # the pointer and descriptor arrays of the population are marshalled once: the tensors do not move between steps
    prepared = evo.Prepared(cands, refs, groups, n_group)

    # The test inputs of the next case do not depend on this case's check: they are generated on a second stream
    # (a context of its own), launched after the check so that the check's persistent CTAs are resident first and the
    # generator fills the room they leave.  The timed region ends only when both streams have drained.
    main_stream = torch.cuda.current_stream(device)
    side_stream = torch.cuda.Stream(device) if args.overlap_gen else main_stream
    gen_ctx = evo.Context(local_rank) if args.overlap_gen else ctx

    def step(i, ev=None):
        if not args.overlap_gen:
            evo.evo_gen_inputs(1000 + i, 0, evo.EVO_F32, n_gen, gen_buf, ctx=ctx)
        if ev is not None:
            ctx.set_timing_events(ev[0], ev[1])
        evo.evo_validate(prepared, None, pop.atol, pop.rtol, results=results, group_pass=gpass, ctx=ctx)
        if args.overlap_gen:
            evo.evo_gen_inputs(1000 + i, 0, evo.EVO_F32, n_gen, gen_buf, stream=side_stream, ctx=gen_ctx)
        evo.evo_fitness(pop.times, pop.base_times, gpass, out=fits, ctx=ctx)

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()

    # per-step event pairs around the main validation kernel (recorded once so the handles exist)
    kern_events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, b in kern_events:
        a.record()
        b.record()
    torch.cuda.synchronize()

    sampler = ClockSampler(torch.cuda._get_nvml_device_index(local_rank) if hasattr(torch.cuda, "_get_nvml_device_index") else local_rank)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches_before, gen_launches_before = ctx.launches, gen_ctx.launches
    with sampler:
        barrier()
        start.record()
        for i in range(args.steps):
            step(i, kern_events[i])
        main_stream.wait_stream(side_stream)
        stop.record()
        barrier()
    launches = ctx.launches - launches_before + (gen_ctx.launches - gen_launches_before if gen_ctx is not ctx else 0)
    total_ms = start.elapsed_time(stop)
    kern_ms = [a.elapsed_time(b) for a, b in kern_events]

    # The main kernel by itself: a few more steps, outside the timed region, with nothing beside it on the device
    # (in the timed region the generator runs concurrently and takes its share of issue slots and of HBM writes).
    kern_alone_ms = None
    if args.overlap_gen:
        alone = kern_events[: min(20, len(kern_events))]
        torch.cuda.synchronize()
        for a, b in alone:
            ctx.set_timing_events(a, b)
            evo.evo_validate(prepared, None, pop.atol, pop.rtol, results=results, group_pass=gpass, ctx=ctx)
        torch.cuda.synchronize()
        kern_alone_ms = [a.elapsed_time(b) for a, b in alone]
    if distributed:
        t = torch.tensor([total_ms], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    ms_per_step = total_ms / args.steps
    value = world * alg_bytes / (ms_per_step * 1e-3) / 1e9
    cand_per_s = world * n_group / (ms_per_step * 1e-3)

    # correctness spot check of the timed configuration: verdicts known by construction
    res = evo.results_to_numpy(results)
    if "wrong" in pop.facts:
        assert res["pass"].sum() == len(cands) - 1 and res["pass"][pop.facts["wrong"]] == 0, "verdicts are wrong"

    # ---- end to end through the host-buffer entry points (pinned host tensors) ----
    e2e = None
    if not args.no_e2e:
        import psutil
        need = alg_bytes + (2 << 30)
        # every rank of the node pins its own copy at the same time: budget the host memory for all of them
        if psutil.virtual_memory().available > 2 * need * world and torch.cuda.mem_get_info()[0] > need:
            h_refs = [r.cpu().pin_memory() for r in pop.refs]
            h_cands = [t.cand.cpu().pin_memory() for t in pop.tensors]
            aliasing = False
        else:  # not enough host memory for a second copy of the population: reuse two host tensors
            h_refs = [r.cpu().pin_memory() for r in pop.refs[:1]]
            one = pop.tensors[0].cand.cpu().pin_memory()
            h_cands = [one for _ in pop.tensors]
            aliasing = True
        h_refl = [h_refs[t.ref_index if not aliasing else 0] for t in pop.tensors]
        h_times, h_base = pop.times.cpu().numpy(), pop.base_times.cpu().numpy()
        e2e_steps = max(1, min(args.steps, args.e2e_steps))

        def e2e_step(i):
            evo.evo_gen_inputs(2000 + i, 0, evo.EVO_F32, n_gen, gen_buf, ctx=ctx)
            r, gp = evo.evo_validate_host(h_cands, h_refl, pop.atol, pop.rtol, groups=groups, n_group=n_group,
                                          device=local_rank, ctx=ctx)
            f = evo.evo_fitness_host(h_times, h_base, gp, device=local_rank, ctx=ctx)
            return r, gp, f

        e2e_step(0)
        barrier()
        t0 = time.perf_counter()
        for i in range(e2e_steps):
            r, gp, f = e2e_step(i)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        if distributed:
            t = torch.tensor([dt], device=device, dtype=torch.float64)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            dt = float(t.item())
        h2d = alg_bytes + h_times.nbytes + h_base.nbytes + gp.nbytes
        d2h = r.nbytes + gp.nbytes + f.nbytes
        e2e = {"value": world * alg_bytes / (dt / e2e_steps) / 1e9, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "steps": e2e_steps, "ms_per_step": dt / e2e_steps * 1e3,
               "host_memory": "pinned", "timer": "host wall clock around synchronous calls, max over ranks",
               "host_tensors_aliased": aliasing}
        del h_cands, h_refs, h_refl

    if rank != 0:
        if distributed:
            dist.destroy_process_group()
        return

    # how evenly the fixed cut spreads the tiles over the persistent CTAs (host-side view of the schedule)
    pi = evo.plan_inspect(cands, refs, 2 * torch.cuda.get_device_properties(device).multi_processor_count)
    w = pi["weights"]
    plan_info = {"n_sets": pi["n_sets"], "n_ctas": pi["n_ctas"], "total_tiles": pi["total_tiles"],
                 "max_over_mean_tiles_per_cta": float(w.max() / w.mean()) if len(w) else None}
    peak, peak_kind = measured_peak()
    kern_avg_ms = sum(kern_ms) / len(kern_ms)
    achieved = alg_bytes / (kern_avg_ms * 1e-3) / 1e9
    traffic = ncu_traffic(alg_bytes) if args.workload == "config4" else None
    roofline = {"kernel": "validate_pass1", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": UNIT,
                "frac": achieved / peak, "peak_kind": "of " + peak_kind, "traffic": traffic,
                "algorithmic_bytes_per_launch": alg_bytes, "kernel_ms_avg": kern_avg_ms,
                "kernel_ms_min": min(kern_ms), "kernel_ms_max": max(kern_ms)}

    if kern_alone_ms:
        alone_avg = sum(kern_alone_ms) / len(kern_alone_ms)
        roofline["kernel_ms_alone"] = alone_avg
        roofline["achieved_alone"] = alg_bytes / (alone_avg * 1e-3) / 1e9
        roofline["frac_alone"] = roofline["achieved_alone"] / peak
        roofline["concurrency"] = ("achieved/frac: the kernel as it runs in the timed region, with evo_gen_inputs concurrent on a "
                                   "second stream (1 GiB of HBM writes and its arithmetic beside it); *_alone: %d more launches after "
                                   "the timed region with nothing else on the device" % len(kern_alone_ms))
    roofline["datasheet_peak"] = DATASHEET_HBM_GBS
    roofline["frac_of_datasheet"] = achieved / DATASHEET_HBM_GBS
    roofline["note"] = ("frac is against the measured copy bandwidth of this pool's B200s (a read+write copy; a read-only stream "
                        "can exceed it a little); frac_of_datasheet is against the nominal %d GB/s" % DATASHEET_HBM_GBS)

    # The generator is bound by plain arithmetic: 56 lane-slots per normal (ncu, smsp__inst_executed x 32 / normals)
    # against the issue peak of the part, SMs x 4 schedulers x 32 lanes x the SM clock.
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    g0.record()
    for i in range(5):
        evo.evo_gen_inputs(4000 + i, 0, evo.EVO_F32, n_gen, gen_buf, ctx=ctx)
    g1.record()
    torch.cuda.synchronize()
    gen_ms = g0.elapsed_time(g1) / 5
    props = torch.cuda.get_device_properties(device)
    sm_mhz_max = sampler.max_mhz or 1965
    issue_peak = props.multi_processor_count * 4 * 32 * sm_mhz_max * 1e6 / 1e12
    gen_info = {"kernel": "gen_kernel<f32>", "bound": "alu", "normals": n_gen, "kernel_ms": gen_ms,
                "lane_slots_per_normal": 56, "achieved": 56 * n_gen / (gen_ms * 1e-3) / 1e12, "peak": issue_peak,
                "unit": "T lane-slots/s", "frac": 56 * n_gen / (gen_ms * 1e-3) / 1e12 / issue_peak,
                "peak_kind": "SMs x 4 schedulers x 32 lanes x max SM clock"}

    # the other synthetic populations, with the main one out of the way
    config = config_keys(args.workload, n_gen, len(cands), n_group, int(pop.times.shape[1]), alg_bytes, world)
    streams = "evo_gen_inputs on a second stream, concurrent with evo_validate" if args.overlap_gen else "one stream"
    candidate_bytes = pop.candidate_bytes()
    per_config = None
    if args.per_config and world == 1:
        del prepared, cands, refs, pop, gen_buf
        torch.cuda.empty_cache()
        per_config = {}
        for name, reps in (("config1", 200), ("config2", 200), ("config3", 100), ("config5", 20), ("clean16", 20)):
            if name != args.workload:
                per_config[name] = measure_config(evo, ctx, name, device, peak, reps)
        per_config["fused_generate_compare"] = measure_generated(evo, ctx, device, peak)

    cpu = cpu_many = None
    if not args.no_cpu_baseline and world == 1:           # the baseline legs belong to the one-GPU run
        # about 10 s of single-thread work: the sample of the reference arm, several passes
        sample = OracleSample(args.workload, ORACLE_SAMPLE_LOG2[0], ORACLE_SAMPLE_LOG2[1])
        sample.run()
        ests, spent, passes = [], 0.0, 0
        while spent < 10.0 and passes < 64:
            est, s_ = sample.run()
            ests.append(est)
            spent += s_
            passes += 1
        est = sum(ests) / len(ests)
        cpu = {"value": alg_bytes / est / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": sample.description + "; %d passes" % passes, "seconds": spent,
               "host_cores_available": len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else os.cpu_count()}
        try:
            cpu_many = oracle_many_processes(args.workload, alg_bytes, max(2, passes // 2))
        except Exception as exc:        # a baseline leg must not take the benchmark line with it
            cpu_many = {"value": None, "error": repr(exc)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "n_gpus_requested": args.gpus, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": config, "streams": streams,
        "candidates_per_s": cand_per_s, "frac_of_hbm_peak": value / world / peak,
        "frac_of_datasheet_hbm": value / world / DATASHEET_HBM_GBS,
        "candidate_bytes_gbs": world * candidate_bytes / (ms_per_step * 1e-3) / 1e9, "plan": plan_info,
        "clocks": sampler.summary(), "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline, "roofline_generator": gen_info, "cpu_baseline": cpu, "cpu_baseline_all_cores": cpu_many, "per_config": per_config,
    }
    print(json.dumps(line))
    if distributed:
        dist.destroy_process_group()


def torchrun_command(n_gpus, argv):
    """The command line `--gpus N` re-executes itself as when no launcher started it: N local ranks, one per GPU."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n_gpus),
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", choices=sorted(WORKLOAD_NOTES), default="config4")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-overlap-gen", dest="overlap_gen", action="store_false",
                    help="generate the test inputs on the main stream, before the check, instead of on a second stream")
    ap.add_argument("--no-per-config", dest="per_config", action="store_false",
                    help="skip the figures of the other synthetic populations (configs 1, 2, 3, 5)")
    ap.add_argument("--log2-elems", type=int, default=None,
                    help="config4 only: shrink every tensor to 2^X elements (a small case for profiler captures; "
                         "not the benchmark configuration)")
    args = ap.parse_args()
    if args.log2_elems is not None:
        if args.workload != "config4" or not 12 <= args.log2_elems <= 28:
            ap.error("--log2-elems needs --workload config4 and 12 <= X <= 28")
        args.no_cpu_baseline = True
        WORKLOAD_NOTES["config4"] = "REDUCED: 16 fp32 candidates x 2^%d elements sharing one reference" % args.log2_elems
    if args.workload != "config4" or args.log2_elems is not None:
        args.per_config = False
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        cmd = torchrun_command(args.gpus, sys.argv[1:])
        os.execv(cmd[0], cmd)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != args.gpus:
        ap.error("--gpus %d, but the launcher started %d rank(s)" % (args.gpus, world))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
