"""ctypes front end of the CPU oracle (oracle/evo_oracle.cpp).

Test infrastructure only.  Every function takes and returns numpy arrays on the
host; nothing here touches CUDA or imports the product package.
"""
import ctypes as C

import numpy as np

from . import build as _build

U32, F32, F16, BF16 = 0, 1, 2, 3
_ELEM_BYTES = {U32: 4, F32: 4, F16: 2, BF16: 2}

RESULT_DTYPE = np.dtype(
    [("n_mismatch", "<u8"), ("n_nonfinite", "<u8"), ("sse", "<f8"), ("max_abs", "<f4"),
     ("max_rel", "<f4"), ("flags", "<u4"), ("pass", "<u4")], align=True)
FIT_DTYPE = np.dtype(
    [("median_ms", "<f4"), ("speedup", "<f4"), ("valid", "<u4"), ("status", "<u4")], align=True)
SUMMARY_DTYPE = np.dtype(
    [("median_speedup", "<f4"), ("validity", "<f4"), ("n_valid", "<u4"), ("n_cand", "<u4"), ("speedup_count", "<u4"),
     ("hist", "<u4", (5,)), ("n_kernel", "<u4"), ("n_run", "<u4")], align=True)
assert RESULT_DTYPE.itemsize == 40 and FIT_DTYPE.itemsize == 16 and SUMMARY_DTYPE.itemsize == 48
STAT_MEDIAN, STAT_MEAN, STAT_MIN, STAT_TRIMMED_MEAN = 0, 1, 2, 3
I32, I64, U8 = 5, 6, 7
_EXACT_NP = {I32: np.int32, I64: np.int64, U8: np.uint8}
EXACT_DTYPE = np.dtype([("n_mismatch", "<u8"), ("max_abs_diff", "<u8"), ("pass", "<u4"), ("pad", "<u4")], align=True)
assert EXACT_DTYPE.itemsize == 24
RESULT64_DTYPE = np.dtype(
    [("n_mismatch", "<u8"), ("n_nonfinite", "<u8"), ("sse", "<f8"), ("max_abs", "<f8"), ("max_rel", "<f8"),
     ("flags", "<u4"), ("pass", "<u4")], align=True)
assert RESULT64_DTYPE.itemsize == 48
OFFENDER_DTYPE = np.dtype([("index", "<u8"), ("cand", "<f4"), ("ref", "<f4")], align=True)
assert OFFENDER_DTYPE.itemsize == 16

_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.oracle_philox4x32_10.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.oracle_philox4x32_10.restype = None
        L.oracle_box_muller.argtypes = [C.c_uint32, C.c_uint32, C.c_void_p]
        L.oracle_box_muller.restype = None
        L.oracle_gen_u32.argtypes = [C.c_uint64, C.c_uint64, C.c_uint64, C.c_void_p]
        L.oracle_gen_u32.restype = None
        L.oracle_gen_normal_f64.argtypes = [C.c_uint64, C.c_uint64, C.c_uint64, C.c_void_p]
        L.oracle_gen_normal_f64.restype = None
        L.oracle_gen_inputs.argtypes = [C.c_uint64, C.c_uint64, C.c_int, C.c_uint64, C.c_void_p]
        L.oracle_gen_inputs.restype = C.c_int
        L.oracle_narrow.argtypes = [C.c_int, C.c_void_p, C.c_uint64, C.c_void_p]
        L.oracle_narrow.restype = None
        L.oracle_widen.argtypes = [C.c_int, C.c_void_p, C.c_uint64, C.c_void_p]
        L.oracle_widen.restype = None
        L.oracle_element_mismatch.argtypes = [C.c_float, C.c_float, C.c_float, C.c_float]
        L.oracle_element_mismatch.restype = C.c_int
        L.oracle_validate.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_int, C.c_float, C.c_float, C.c_void_p]
        L.oracle_validate.restype = C.c_int
        L.oracle_group_pass.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint64]
        L.oracle_group_pass.restype = None
        L.oracle_fitness.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p]
        L.oracle_fitness.restype = C.c_int
        L.oracle_fitness_ex.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32, C.c_void_p, C.c_uint32, C.c_void_p, C.c_int,
                                        C.c_uint32, C.c_uint32, C.c_void_p]
        L.oracle_fitness_ex.restype = C.c_int
        L.oracle_summary.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64, C.c_uint32, C.c_uint32, C.c_void_p,
                                     C.c_void_p, C.c_void_p]
        L.oracle_summary.restype = C.c_int
        L.oracle_select_elite.argtypes = [C.c_void_p, C.c_uint64, C.c_uint32, C.c_void_p, C.c_void_p]
        L.oracle_select_elite.restype = C.c_int
        L.oracle_mismatch_sample.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_int, C.c_float, C.c_float, C.c_uint64,
                                             C.c_void_p, C.c_void_p]
        L.oracle_mismatch_sample.restype = C.c_int
        L.oracle_validate_exact.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_int, C.c_void_p]
        L.oracle_validate_exact.restype = C.c_int
        L.oracle_group_pass_exact.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_void_p, C.c_uint64]
        L.oracle_group_pass_exact.restype = None
        L.oracle_validate_f64.argtypes = [C.c_void_p, C.c_void_p, C.c_uint64, C.c_double, C.c_double, C.c_void_p]
        L.oracle_validate_f64.restype = C.c_int
        _lib = L
    return _lib


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p)


def philox4x32_10(counter, key):
    """One Philox4x32-10 block: counter (4 x u32), key (2 x u32) -> 4 x u32."""
    c = np.ascontiguousarray(counter, dtype=np.uint32)
    k = np.ascontiguousarray(key, dtype=np.uint32)
    assert c.shape == (4,) and k.shape == (2,)
    out = np.empty(4, dtype=np.uint32)
    lib().oracle_philox4x32_10(_ptr(c), _ptr(k), _ptr(out))
    return out


def box_muller(xa, xb):
    """Two stream words -> (z_even, z_odd) in double, before rounding."""
    out = np.empty(2, dtype=np.float64)
    lib().oracle_box_muller(int(xa) & 0xFFFFFFFF, int(xb) & 0xFFFFFFFF, _ptr(out))
    return float(out[0]), float(out[1])


def gen_u32(seed, offset, n):
    out = np.empty(int(n), dtype=np.uint32)
    lib().oracle_gen_u32(int(seed), int(offset), int(n), _ptr(out))
    return out


def gen_normal_f64(seed, offset, n):
    """Standard normals of the stream before any rounding to a storage type."""
    out = np.empty(int(n), dtype=np.float64)
    lib().oracle_gen_normal_f64(int(seed), int(offset), int(n), _ptr(out))
    return out


def gen_inputs(seed, offset, dtype, n):
    """Raw words (U32 -> uint32), fp32 normals (F32 -> float32) or the bit
    patterns of fp16/bf16 normals (F16/BF16 -> uint16)."""
    np_dt = {U32: np.uint32, F32: np.float32, F16: np.uint16, BF16: np.uint16}[dtype]
    out = np.empty(int(n), dtype=np_dt)
    rc = lib().oracle_gen_inputs(int(seed), int(offset), int(dtype), int(n), _ptr(out))
    if rc != 0:
        raise ValueError("oracle_gen_inputs: status %d" % rc)
    return out


def narrow(dtype, x):
    """fp32 -> fp16/bf16 bit patterns, round-to-nearest-even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().oracle_narrow(int(dtype), _ptr(x), x.size, _ptr(out))
    return out


def widen(dtype, bits):
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float32)
    lib().oracle_widen(int(dtype), _ptr(bits), bits.size, _ptr(out))
    return out


def element_mismatch(c, r, atol, rtol):
    return int(lib().oracle_element_mismatch(float(np.float32(c)), float(np.float32(r)),
                                             float(np.float32(atol)), float(np.float32(rtol))))


def validate(cand, ref, dtype, atol, rtol):
    """One candidate tensor against its reference.  `cand`/`ref` are float32
    arrays (F32) or uint16 bit patterns (F16/BF16).  Returns a RESULT_DTYPE scalar."""
    np_dt = np.float32 if dtype == F32 else np.uint16
    cand = np.ascontiguousarray(cand)
    ref = np.ascontiguousarray(ref)
    if cand.dtype != np_dt or ref.dtype != np_dt:
        raise TypeError("validate: arrays must be %s for dtype %d" % (np_dt, dtype))
    if cand.size != ref.size:
        raise ValueError("validate: size mismatch")
    out = np.zeros(1, dtype=RESULT_DTYPE)
    rc = lib().oracle_validate(_ptr(cand), _ptr(ref), cand.size, int(dtype),
                               float(np.float32(atol)), float(np.float32(rtol)), _ptr(out))
    if rc != 0:
        raise ValueError("oracle_validate: status %d" % rc)
    return out[0]


def group_pass(results, group, n_group):
    results = np.ascontiguousarray(results, dtype=RESULT_DTYPE)
    group = np.ascontiguousarray(group, dtype=np.uint32)
    out = np.empty(int(n_group), dtype=np.uint32)
    lib().oracle_group_pass(_ptr(results), _ptr(group), results.size, _ptr(out), int(n_group))
    return out


def fitness(times, base_times, passed=None):
    """times [n_cand, trials] fp32, base_times [base_trials] fp32, passed optional
    [n_cand] u32.  Returns a FIT_DTYPE array of n_cand entries."""
    times = np.ascontiguousarray(times, dtype=np.float32)
    base = np.ascontiguousarray(base_times, dtype=np.float32)
    assert times.ndim == 2 and base.ndim == 1
    n_cand, trials = times.shape
    p = None
    if passed is not None:
        p = np.ascontiguousarray(passed, dtype=np.uint32)
        assert p.shape == (n_cand,)
    out = np.zeros(n_cand, dtype=FIT_DTYPE)
    rc = lib().oracle_fitness(_ptr(times), n_cand, trials, _ptr(base), base.size,
                              _ptr(p) if p is not None else None, _ptr(out))
    if rc != 0:
        raise ValueError("oracle_fitness: status %d" % rc)
    return out


def fitness_ex(times, base_times, passed=None, stat=STAT_MEDIAN, warmup=0, trim=0):
    """fitness() with the run-time statistic chosen (median, mean, min, trimmed mean), the first
    `warmup` runs left out and, for the trimmed mean, `trim` runs dropped at each end."""
    times = np.ascontiguousarray(times, dtype=np.float32)
    base = np.ascontiguousarray(base_times, dtype=np.float32)
    assert times.ndim == 2 and base.ndim == 1
    n_cand, trials = times.shape
    p = None
    if passed is not None:
        p = np.ascontiguousarray(passed, dtype=np.uint32)
        assert p.shape == (n_cand,)
    out = np.zeros(n_cand, dtype=FIT_DTYPE)
    rc = lib().oracle_fitness_ex(_ptr(times), n_cand, trials, _ptr(base), base.size, _ptr(p) if p is not None else None,
                                 int(stat), int(warmup), int(trim), _ptr(out))
    if rc != 0:
        raise ValueError("oracle_fitness_ex: status %d" % rc)
    return out


def summary(fits, kernel_of, n_kernel, run_of=None, n_run=1):
    """Reporting metrics of a population.  Returns (SUMMARY_DTYPE scalar, best [n_run, n_kernel],
    run_median [n_run])."""
    fits = np.ascontiguousarray(fits, dtype=FIT_DTYPE)
    k = np.ascontiguousarray(kernel_of, dtype=np.uint32)
    r = np.ascontiguousarray(run_of, dtype=np.uint32) if run_of is not None else None
    out = np.zeros(1, dtype=SUMMARY_DTYPE)
    best = np.zeros((int(n_run), int(n_kernel)), dtype=np.float32)
    med = np.zeros(int(n_run), dtype=np.float32)
    rc = lib().oracle_summary(_ptr(fits), _ptr(k), _ptr(r) if r is not None else None, fits.size, int(n_kernel), int(n_run),
                              _ptr(out), _ptr(best), _ptr(med))
    if rc != 0:
        raise ValueError("oracle_summary: status %d" % rc)
    return out[0], best, med


def select_elite(fits, k):
    """Indices of the k valid candidates with the largest speedup, best first (ties by index);
    returns (idx [k] uint32, padded with 0xffffffff, and the number of real entries)."""
    fits = np.ascontiguousarray(fits, dtype=FIT_DTYPE)
    idx = np.zeros(int(k), dtype=np.uint32)
    count = np.zeros(1, dtype=np.uint32)
    lib().oracle_select_elite(_ptr(fits), fits.size, int(k), _ptr(idx), _ptr(count))
    return idx, int(count[0])


def mismatch_sample(cand, ref, dtype, atol, rtol, max_out):
    """The first `max_out` elements (index order) that violate the closeness rule, as
    OFFENDER_DTYPE records, and the total number of violations."""
    np_dt = np.float32 if dtype == F32 else np.uint16
    cand = np.ascontiguousarray(cand)
    ref = np.ascontiguousarray(ref)
    if cand.dtype != np_dt or ref.dtype != np_dt or cand.size != ref.size:
        raise TypeError("mismatch_sample: arrays must be %s and of equal size" % np_dt)
    out = np.zeros(int(max_out), dtype=OFFENDER_DTYPE)
    found = np.zeros(1, dtype=np.uint64)
    rc = lib().oracle_mismatch_sample(_ptr(cand), _ptr(ref), cand.size, int(dtype), float(np.float32(atol)),
                                      float(np.float32(rtol)), int(max_out), _ptr(out), _ptr(found))
    if rc != 0:
        raise ValueError("oracle_mismatch_sample: status %d" % rc)
    return out[: min(int(max_out), int(found[0]))], int(found[0])


def validate_exact(cand, ref, dtype):
    """Integer / boolean tensors: equality, element by element.  Returns an EXACT_DTYPE scalar."""
    np_dt = _EXACT_NP[dtype]
    cand = np.ascontiguousarray(cand)
    ref = np.ascontiguousarray(ref)
    if cand.dtype == np.bool_:
        cand, ref = cand.view(np.uint8), ref.view(np.uint8)
    if cand.dtype != np_dt or ref.dtype != np_dt or cand.size != ref.size:
        raise TypeError("validate_exact: arrays must be %s and of equal size" % np_dt)
    out = np.zeros(1, dtype=EXACT_DTYPE)
    rc = lib().oracle_validate_exact(_ptr(cand), _ptr(ref), cand.size, int(dtype), _ptr(out))
    if rc != 0:
        raise ValueError("oracle_validate_exact: status %d" % rc)
    return out[0]


def group_pass_exact(results, group, n_group):
    results = np.ascontiguousarray(results, dtype=EXACT_DTYPE)
    group = np.ascontiguousarray(group, dtype=np.uint32)
    out = np.empty(int(n_group), dtype=np.uint32)
    lib().oracle_group_pass_exact(_ptr(results), _ptr(group), results.size, _ptr(out), int(n_group))
    return out


def validate_f64(cand, ref, atol, rtol):
    """binary64 tensors: the rule and statistics in binary64.  Returns a RESULT64_DTYPE scalar."""
    cand = np.ascontiguousarray(cand)
    ref = np.ascontiguousarray(ref)
    if cand.dtype != np.float64 or ref.dtype != np.float64 or cand.size != ref.size:
        raise TypeError("validate_f64: arrays must be float64 and of equal size")
    out = np.zeros(1, dtype=RESULT64_DTYPE)
    rc = lib().oracle_validate_f64(_ptr(cand), _ptr(ref), cand.size, float(atol), float(rtol), _ptr(out))
    if rc != 0:
        raise ValueError("oracle_validate_f64: status %d" % rc)
    return out[0]
