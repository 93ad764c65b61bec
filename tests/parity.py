"""Helpers shared by the GPU parity tests: run a population through the oracle (CPU) and
compare evo_result records field by field under the stated bars."""
import math

import numpy as np

import oracle
import workloads

SSE_RTOL = 1e-5           # sum of squared error: relative agreement (summation order differs)


def oracle_population(pop):
    """evo_result of every tensor of `pop`, and the verdict per candidate id, by the oracle."""
    refs = [workloads.to_host_bits(r) for r in pop.refs]
    res = np.zeros(len(pop.tensors), dtype=oracle.RESULT_DTYPE)
    for i, t in enumerate(pop.tensors):
        res[i] = oracle.validate(workloads.to_host_bits(t.cand), refs[t.ref_index], t.dtype, pop.atol, pop.rtol)
    verdict = oracle.group_pass(res, [t.group for t in pop.tensors], pop.n_group)
    return res, verdict


def assert_results_equal(got, want, what=""):
    """Counts, flags, verdicts and the two maxima bit-exact; SSE within SSE_RTOL."""
    got = np.asarray(got)
    want = np.asarray(want)
    assert got.shape == want.shape, what
    for k in ("n_mismatch", "n_nonfinite", "flags", "pass"):
        bad = np.nonzero(got[k] != want[k])[0]
        assert bad.size == 0, "%s %s differs at %s: got %s want %s" % (what, k, bad[:5], got[k][bad[:5]], want[k][bad[:5]])
    for k in ("max_abs", "max_rel"):
        g, w = got[k].view(np.uint32), want[k].view(np.uint32)
        bad = np.nonzero(g != w)[0]
        assert bad.size == 0, "%s %s differs at %s: got %s want %s" % (what, k, bad[:5], got[k][bad[:5]], want[k][bad[:5]])
    for i, (g, w) in enumerate(zip(got["sse"], want["sse"])):
        if w == 0.0 or math.isinf(w) or math.isnan(w):
            assert (g == w) or (math.isnan(g) and math.isnan(w)), "%s sse[%d]: got %r want %r" % (what, i, g, w)
        else:
            assert abs(g - w) <= SSE_RTOL * abs(w), "%s sse[%d]: got %r want %r" % (what, i, g, w)


def ordered(x32):
    """Map float32 bit patterns to integers whose difference is the distance in ulps (+0 == -0)."""
    b = np.asarray(x32, dtype=np.float32).view(np.int32).astype(np.int64)
    return np.where(b < 0, -(b & 0x7FFFFFFF), b)


def ordered16(bits):
    b = np.asarray(bits, dtype=np.uint16).astype(np.int64)
    return np.where(b & 0x8000, -(b & 0x7FFF), b)
