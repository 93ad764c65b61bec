"""ctypes binding of libevo (include/evo.h).  Argument marshalling only: every step of the
evaluation runs in the library's kernels.  torch supplies device memory and streams."""
import ctypes as C
import os

import numpy as np
import torch

EVO_U32, EVO_F32, EVO_F16, EVO_BF16 = 0, 1, 2, 3
EVO_F64, EVO_I32, EVO_I64, EVO_U8 = 4, 5, 6, 7
EVO_FLAG_INCOMPLETE = 0x40000000
_TORCH_TO_CODE = {torch.float32: EVO_F32, torch.float16: EVO_F16, torch.bfloat16: EVO_BF16,
                  torch.float64: EVO_F64, torch.int32: EVO_I32, torch.int64: EVO_I64, torch.uint8: EVO_U8, torch.bool: EVO_U8}

RESULT_DTYPE = np.dtype(
    [("n_mismatch", "<u8"), ("n_nonfinite", "<u8"), ("sse", "<f8"), ("max_abs", "<f4"),
     ("max_rel", "<f4"), ("flags", "<u4"), ("pass", "<u4")], align=True)
FIT_DTYPE = np.dtype(
    [("median_ms", "<f4"), ("speedup", "<f4"), ("valid", "<u4"), ("status", "<u4")], align=True)
_DESC_DTYPE = np.dtype([("n", "<u8"), ("ref", "<u8"), ("dtype", "<i4"), ("group", "<u4")], align=True)
SUMMARY_DTYPE = np.dtype(
    [("median_speedup", "<f4"), ("validity", "<f4"), ("n_valid", "<u4"), ("n_cand", "<u4"), ("speedup_count", "<u4"),
     ("hist", "<u4", (5,)), ("n_kernel", "<u4"), ("n_run", "<u4")], align=True)
EVO_STAT_MEDIAN, EVO_STAT_MEAN, EVO_STAT_MIN, EVO_STAT_TRIMMED_MEAN = 0, 1, 2, 3
assert RESULT_DTYPE.itemsize == 40 and FIT_DTYPE.itemsize == 16 and _DESC_DTYPE.itemsize == 24
EXACT_DTYPE = np.dtype([("n_mismatch", "<u8"), ("max_abs_diff", "<u8"), ("pass", "<u4"), ("pad", "<u4")], align=True)
assert EXACT_DTYPE.itemsize == 24
RESULT64_DTYPE = np.dtype(
    [("n_mismatch", "<u8"), ("n_nonfinite", "<u8"), ("sse", "<f8"), ("max_abs", "<f8"), ("max_rel", "<f8"),
     ("flags", "<u4"), ("pass", "<u4")], align=True)
assert RESULT64_DTYPE.itemsize == 48
OFFENDER_DTYPE = np.dtype([("index", "<u8"), ("cand", "<f4"), ("ref", "<f4")], align=True)
assert SUMMARY_DTYPE.itemsize == 48 and OFFENDER_DTYPE.itemsize == 16

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libevo.so")
_lib = None


class EvoError(RuntimeError):
    def __init__(self, status, message):
        super().__init__("libevo status %d: %s" % (status, message))
        self.status = status


def load_library():
    """Load libevo.so.  Fails loudly if it has not been built: there is no other code path."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError("%s is missing: build it with `python -m paper_2510_03760_b200.build`" % _LIB_PATH)
    L = C.CDLL(_LIB_PATH)
    vp, u64, u32, i32, f32 = C.c_void_p, C.c_uint64, C.c_uint32, C.c_int, C.c_float
    L.evo_create.argtypes = [C.POINTER(vp), i32]
    L.evo_create.restype = i32
    L.evo_destroy.argtypes = [vp]
    L.evo_destroy.restype = i32
    L.evo_strerror.argtypes = [i32]
    L.evo_strerror.restype = C.c_char_p
    L.evo_last_error.argtypes = [vp]
    L.evo_last_error.restype = C.c_char_p
    L.evo_launch_count.argtypes = [vp]
    L.evo_launch_count.restype = u64
    L.evo_set_timing_events.argtypes = [vp, vp, vp]
    L.evo_set_timing_events.restype = i32
    L.evo_check.argtypes = [vp, vp]
    L.evo_check.restype = i32
    L.evo_selftest_wait.argtypes = [vp, u32, vp]
    L.evo_selftest_wait.restype = i32
    L.evo_set_overlapped_launch.argtypes = [vp, i32]
    L.evo_set_overlapped_launch.restype = i32
    L.evo_debug_cta_timing.argtypes = [vp, i32]
    L.evo_debug_cta_timing.restype = i32
    L.evo_debug_read_cta_times.argtypes = [vp, vp, u32, vp]
    L.evo_debug_read_cta_times.restype = i32
    L.evo_gen_inputs.argtypes = [vp, u64, u64, i32, u64, vp, vp]
    L.evo_gen_inputs.restype = i32
    for name in ("evo_validate", "evo_validate_host"):
        fn = getattr(L, name)
        fn.argtypes = [vp, vp, vp, vp, u64, i32, f32, f32, vp, vp, u64, vp]
        fn.restype = i32
    L.evo_validate_static.argtypes = [vp, vp, vp, u64, i32, f32, f32, vp, vp, u64, vp]
    L.evo_validate_static.restype = i32
    L.evo_validate_static_error.argtypes = []
    L.evo_validate_static_error.restype = C.c_char_p
    for name in ("evo_fitness", "evo_fitness_host"):
        fn = getattr(L, name)
        fn.argtypes = [vp, vp, u64, u32, vp, u32, vp, vp, vp]
        fn.restype = i32
    L.evo_fitness_ex.argtypes = [vp, vp, u64, u32, vp, u32, vp, i32, u32, u32, vp, vp]
    L.evo_fitness_ex.restype = i32
    L.evo_summary.argtypes = [vp, vp, vp, vp, u64, u32, u32, vp, vp, vp, vp]
    L.evo_summary.restype = i32
    L.evo_select_elite.argtypes = [vp, vp, u64, u32, vp, vp, vp]
    L.evo_select_elite.restype = i32
    L.evo_mismatch_sample.argtypes = [vp, vp, vp, u64, i32, f32, f32, u64, vp, vp, vp]
    L.evo_mismatch_sample.restype = i32
    L.evo_validate_exact.argtypes = [vp, vp, vp, vp, u64, i32, vp, vp, u64, vp]
    L.evo_validate_exact.restype = i32
    L.evo_validate_generated.argtypes = [vp, u64, u64, vp, vp, vp, u64, i32, vp, vp, vp, u64, vp]
    L.evo_validate_generated.restype = i32
    L.evo_validate_f64.argtypes = [vp, vp, vp, vp, u64, C.c_double, C.c_double, vp, vp, u64, vp]
    L.evo_validate_f64.restype = i32
    L.evo_plan_inspect.argtypes = [vp, vp, vp, u64, i32, u32, vp, vp, vp, vp]
    L.evo_plan_inspect.restype = i32
    _lib = L
    return L


class Context:
    """Owns an evo_ctx (device workspace).  One per stream in use."""

    def __init__(self, device=0):
        L = load_library()
        h = C.c_void_p()
        st = L.evo_create(C.byref(h), int(device))
        if st != 0:
            raise EvoError(st, L.evo_strerror(st).decode())
        self._h = h
        self.device = int(device)

    def check(self, status):
        if status != 0:
            L = load_library()
            raise EvoError(status, "%s (%s)" % (L.evo_strerror(status).decode(), L.evo_last_error(self._h).decode()))

    @property
    def launches(self):
        return int(load_library().evo_launch_count(self._h))

    def set_timing_events(self, start, stop):
        """Have the next evo_validate on this context record torch CUDA events (created with
        enable_timing=True and already recorded once, so that their handles exist) around its
        main kernel."""
        st = load_library().evo_set_timing_events(
            self._h, C.c_void_p(start.cuda_event) if start is not None else None,
            C.c_void_p(stop.cuda_event) if stop is not None else None)
        self.check(st)

    def set_overlapped_launch(self, enable):
        """evo_set_overlapped_launch: programmatic dependent launch of this context's kernels on/off."""
        self.check(load_library().evo_set_overlapped_launch(self._h, 1 if enable else 0))

    def cta_timing(self, enable):
        """evo_debug_cta_timing: have evo_validate's main kernel record each CTA's begin and end clock."""
        self.check(load_library().evo_debug_cta_timing(self._h, 1 if enable else 0))

    def read_cta_times(self, capacity=4096):
        """evo_debug_read_cta_times: numpy uint64 array [n_ctas, 2] (begin, end) in ns of the last timed call."""
        buf = np.zeros((int(capacity), 2), dtype=np.uint64)
        n = C.c_uint32(0)
        self.check(load_library().evo_debug_read_cta_times(self._h, C.c_void_p(buf.ctypes.data), int(capacity), C.byref(n)))
        return buf[: min(int(n.value), int(capacity))]

    def synchronize(self, stream=None):
        """evo_check: wait for `stream` and raise EvoError(-6) if a device-side wait ran out."""
        self.check(load_library().evo_check(self._h, _stream_ptr(stream, torch.device("cuda", self.device))))

    def selftest_wait(self, limit_us=1000, stream=None):
        """evo_selftest_wait: enqueue a kernel whose bounded wait must run out (no fault)."""
        self.check(load_library().evo_selftest_wait(self._h, int(limit_us), _stream_ptr(stream, torch.device("cuda", self.device))))

    def close(self):
        if self._h is not None and _lib is not None:
            _lib.evo_destroy(self._h)
        self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


_default_ctx = {}


def default_context(device=None):
    device = torch.cuda.current_device() if device is None else int(device)
    ctx = _default_ctx.get(device)
    if ctx is None:
        ctx = _default_ctx[device] = Context(device)
    return ctx


def dtype_code(t):
    try:
        return _TORCH_TO_CODE[t]
    except KeyError:
        raise TypeError("unsupported tensor dtype %s" % t)


def _stream_ptr(stream, device):
    if stream is None:
        stream = torch.cuda.current_stream(device)
    return C.c_void_p(stream.cuda_stream)


def _dev_ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


def evo_gen_inputs(seed, offset, dtype, n, out, stream=None, ctx=None):
    """Fill the first n elements of the CUDA tensor `out` (uint32/int32 storage for EVO_U32,
    float32/float16/bfloat16 otherwise) with the stream of `seed` from position `offset`."""
    if not out.is_cuda or not out.is_contiguous() or out.numel() < n:
        raise ValueError("out must be a contiguous CUDA tensor with at least n elements")
    want = {EVO_U32: 4, EVO_F32: 4, EVO_F16: 2, EVO_BF16: 2}.get(dtype)
    if want is not None and out.element_size() != want:
        raise ValueError("out has the wrong element size for dtype %d" % dtype)
    ctx = ctx or default_context(out.device.index)
    st = load_library().evo_gen_inputs(ctx._h, int(seed), int(offset), int(dtype), int(n), _dev_ptr(out),
                                       _stream_ptr(stream, out.device))
    ctx.check(st)
    return out


def _marshal(cands, refs, groups, is_host):
    n = len(cands)
    if isinstance(refs, torch.Tensor):
        refs = [refs] * n
    if len(refs) != n:
        raise ValueError("need one reference per candidate tensor, or a single shared one")
    ptrs = np.empty(n, dtype=np.uint64)
    descs = np.zeros(n, dtype=_DESC_DTYPE)
    for i, (c, r) in enumerate(zip(cands, refs)):
        if c.is_cuda == is_host or r.is_cuda == is_host:
            raise ValueError("tensor %d lives on the wrong side for this call" % i)
        if c.dtype != r.dtype or c.numel() != r.numel():
            raise ValueError("tensor %d: candidate and reference differ in dtype or size" % i)
        if not (c.is_contiguous() and r.is_contiguous()):
            raise ValueError("tensor %d must be contiguous" % i)
        ptrs[i] = c.data_ptr()
        descs[i] = (c.numel(), r.data_ptr(), dtype_code(c.dtype), 0 if groups is None else int(groups[i]))
    return ptrs, descs


class Prepared:
    """The marshalled form of a population of CUDA tensors (pointer and descriptor arrays), built once
    and reusable for any number of evo_validate calls on the same tensors: marshalling a few thousand
    tensors in Python costs milliseconds, as much as checking them.  Keeps the tensors alive."""

    def __init__(self, cands, refs, groups=None, n_group=0):
        self.n = len(cands)
        self.device = cands[0].device if self.n else torch.device("cuda", torch.cuda.current_device())
        self.ptrs, self.descs = _marshal(cands, refs, groups, is_host=False)
        self.has_groups = groups is not None
        self.n_group = int(n_group) if self.has_groups else 0
        self._keep = (list(cands), refs if isinstance(refs, torch.Tensor) else list(refs))


def evo_validate(cands, refs, atol, rtol, groups=None, n_group=0, results=None, group_pass=None, stream=None, ctx=None):
    """Check CUDA tensors `cands[i]` against `refs[i]` (or one shared tensor).  Returns
    (results, group_pass): a uint8 CUDA tensor of len(cands) x 40 bytes (evo_result records,
    see results_to_numpy) and, if `groups` is given, an int32 tensor of n_group verdicts.
    `cands` may be a Prepared population (then refs, groups and n_group are taken from it)."""
    if isinstance(cands, Prepared):
        prep = cands
        n, device, ptrs, descs = prep.n, prep.device, prep.ptrs, prep.descs
        groups, n_group = (True if prep.has_groups else None), prep.n_group
    else:
        n = len(cands)
        device = cands[0].device if n else torch.device("cuda", torch.cuda.current_device())
        ptrs, descs = _marshal(cands, refs, groups, is_host=False)
    ctx = ctx or default_context(device.index)
    if results is None:
        results = torch.empty((n, RESULT_DTYPE.itemsize), dtype=torch.uint8, device=device)
    if groups is not None and group_pass is None:
        group_pass = torch.empty(int(n_group), dtype=torch.int32, device=device)
    st = load_library().evo_validate(
        ctx._h, C.c_void_p(ptrs.ctypes.data), None, C.c_void_p(descs.ctypes.data), n, EVO_F32,
        float(atol), float(rtol), _dev_ptr(results), _dev_ptr(group_pass) if groups is not None else None,
        int(n_group) if groups is not None else 0, _stream_ptr(stream, device))
    ctx.check(st)
    return results, group_pass


_PLAN_SUMMARY = np.dtype([("n_sets", "<u4"), ("n_ctas", "<u4"), ("n_parts", "<u4"), ("tile_elems", "<u4"),
                          ("total_tiles", "<u8")], align=True)
_PLAN_RANGE = np.dtype([("tile_begin", "<u8"), ("tile_end", "<u8"), ("set_begin", "<u4"), ("set_end", "<u4")], align=True)


def plan_inspect(cands, refs, max_ctas):
    """The schedule evo_validate would use for these CUDA tensors on a device running `max_ctas` persistent CTAs
    (evo_plan_inspect; host only).  Returns a dict: n_sets, n_ctas, total_tiles, tile_elems, and `weights`, the
    tiles each CTA moves (tiles of its run times members + 1), as a numpy array."""
    ptrs, descs = _marshal(cands, refs, None, is_host=False)
    n = len(cands)
    summ = np.zeros(1, _PLAN_SUMMARY)
    ranges = np.zeros(int(max_ctas), _PLAN_RANGE)
    set_of = np.zeros(max(n, 1), np.uint32)
    set_k = np.zeros(max(n, 1), np.uint32)
    st = load_library().evo_plan_inspect(C.c_void_p(ptrs.ctypes.data), None, C.c_void_p(descs.ctypes.data), n, EVO_F32,
                                         int(max_ctas), C.c_void_p(summ.ctypes.data), C.c_void_p(ranges.ctypes.data),
                                         C.c_void_p(set_of.ctypes.data), C.c_void_p(set_k.ctypes.data))
    if st != 0:
        raise EvoError(st, load_library().evo_strerror(st).decode())
    s = summ[0]
    te = int(s["tile_elems"])
    set_tiles = np.zeros(int(s["n_sets"]), np.int64)
    for i in range(n):
        set_tiles[set_of[i]] = (int(descs["n"][i]) + te - 1) // te
    weights = np.zeros(int(s["n_ctas"]), np.int64)
    for b, r in enumerate(ranges[: int(s["n_ctas"])]):
        for q in range(int(r["set_begin"]), int(r["set_end"]) + 1):
            t0 = int(r["tile_begin"]) if q == r["set_begin"] else 0
            t1 = int(r["tile_end"]) if q == r["set_end"] else int(set_tiles[q])
            weights[b] += max(0, t1 - t0) * (int(set_k[q]) + 1)
    return {"n_sets": int(s["n_sets"]), "n_ctas": int(s["n_ctas"]), "total_tiles": int(s["total_tiles"]),
            "tile_elems": te, "weights": weights}


def evo_validate_exact(cands, refs, groups=None, n_group=0, stream=None, ctx=None):
    """Integer / boolean CUDA tensors (int32, int64, uint8, bool) checked by equality.  Returns
    (results: uint8 CUDA tensor of len(cands) x 24 bytes, see exact_to_numpy; group_pass or None)."""
    n = len(cands)
    device = cands[0].device if n else torch.device("cuda", torch.cuda.current_device())
    ctx = ctx or default_context(device.index)
    ptrs, descs = _marshal(cands, refs, groups, is_host=False)
    results = torch.empty((n, EXACT_DTYPE.itemsize), dtype=torch.uint8, device=device)
    group_pass = torch.empty(int(n_group), dtype=torch.int32, device=device) if groups is not None else None
    st = load_library().evo_validate_exact(
        ctx._h, C.c_void_p(ptrs.ctypes.data), None, C.c_void_p(descs.ctypes.data), n, EVO_I32, _dev_ptr(results),
        _dev_ptr(group_pass) if groups is not None else None, int(n_group) if groups is not None else 0,
        _stream_ptr(stream, device))
    ctx.check(st)
    return results, group_pass


def evo_validate_generated(seed, cands, offsets=0, dtype=EVO_U32, groups=None, n_group=0, stream=None, ctx=None):
    """int32 / uint32-storage CUDA tensors checked for equality against windows of the random stream of `seed`,
    regenerated in the kernel: tensor i against stream elements [offsets[i], offsets[i] + numel) (`offsets` may be one
    number for all).  dtype EVO_U32 or EVO_I32 says how the words compare.  Returns (results as evo_validate_exact,
    group_pass or None)."""
    n = len(cands)
    device = cands[0].device if n else torch.device("cuda", torch.cuda.current_device())
    ctx = ctx or default_context(device.index)
    for i, c in enumerate(cands):
        if not c.is_cuda or not c.is_contiguous() or c.element_size() != 4:
            raise ValueError("tensor %d must be a contiguous CUDA tensor of 32-bit elements" % i)
    ptrs = np.array([c.data_ptr() for c in cands], dtype=np.uint64)
    counts = np.array([c.numel() for c in cands], dtype=np.uint64)
    one = isinstance(offsets, int)
    offs = None if one else np.ascontiguousarray(offsets, dtype=np.uint64)
    if offs is not None and offs.size != n:
        raise ValueError("need one stream offset per tensor, or a single number")
    grp = np.ascontiguousarray(groups, dtype=np.uint32) if groups is not None else None
    results = torch.empty((n, EXACT_DTYPE.itemsize), dtype=torch.uint8, device=device)
    group_pass = torch.empty(int(n_group), dtype=torch.int32, device=device) if groups is not None else None
    st = load_library().evo_validate_generated(
        ctx._h, int(seed), int(offsets) if one else 0, C.c_void_p(offs.ctypes.data) if offs is not None else None,
        C.c_void_p(ptrs.ctypes.data), C.c_void_p(counts.ctypes.data), n, int(dtype),
        C.c_void_p(grp.ctypes.data) if grp is not None else None, _dev_ptr(results),
        _dev_ptr(group_pass) if groups is not None else None, int(n_group) if groups is not None else 0,
        _stream_ptr(stream, device))
    ctx.check(st)
    return results, group_pass


def evo_validate_f64(cands, refs, atol, rtol, groups=None, n_group=0, stream=None, ctx=None):
    """float64 CUDA tensors judged by the rule in binary64.  Returns (results: uint8 CUDA tensor of
    len(cands) x 48 bytes, see results64_to_numpy; group_pass or None)."""
    n = len(cands)
    device = cands[0].device if n else torch.device("cuda", torch.cuda.current_device())
    ctx = ctx or default_context(device.index)
    ptrs, descs = _marshal(cands, refs, groups, is_host=False)
    results = torch.empty((n, RESULT64_DTYPE.itemsize), dtype=torch.uint8, device=device)
    group_pass = torch.empty(int(n_group), dtype=torch.int32, device=device) if groups is not None else None
    st = load_library().evo_validate_f64(
        ctx._h, C.c_void_p(ptrs.ctypes.data), None, C.c_void_p(descs.ctypes.data), n, float(atol), float(rtol),
        _dev_ptr(results), _dev_ptr(group_pass) if groups is not None else None,
        int(n_group) if groups is not None else 0, _stream_ptr(stream, device))
    ctx.check(st)
    return results, group_pass


def results64_to_numpy(results):
    return results.cpu().numpy().view(RESULT64_DTYPE).reshape(-1)


def exact_to_numpy(results):
    return results.cpu().numpy().view(EXACT_DTYPE).reshape(-1)


def evo_validate_static(cands, refs, atol, rtol, results, groups=None, n_group=0, group_pass=None, stream=None):
    """evo_validate for callers that must not allocate device memory (a process whose allocator
    owns the device, a no-allocation serving loop): no context, fixed 1 MiB scratch inside the
    library, current device.  The caller passes the output tensors: `results` (uint8 CUDA,
    len(cands) x 40 bytes) and, with `groups`, `group_pass` (int32 CUDA, n_group).  Populations
    that need more scratch than the fixed array raise EvoError (status -5)."""
    n = len(cands)
    device = results.device
    ptrs, descs = _marshal(cands, refs, groups, is_host=False)
    L = load_library()
    st = L.evo_validate_static(
        C.c_void_p(ptrs.ctypes.data), None, C.c_void_p(descs.ctypes.data), n, EVO_F32, float(atol), float(rtol),
        _dev_ptr(results), _dev_ptr(group_pass) if groups is not None else None,
        int(n_group) if groups is not None else 0, _stream_ptr(stream, device))
    if st != 0:
        raise EvoError(st, "%s (%s)" % (L.evo_strerror(st).decode(), L.evo_validate_static_error().decode()))
    return results, group_pass


def evo_validate_host(cands, refs, atol, rtol, groups=None, n_group=0, device=None, stream=None, ctx=None):
    """The same check for host tensors (pinned or not): copies, checks and copies the results
    back inside the library; returns numpy arrays (RESULT_DTYPE records, uint32 verdicts)."""
    n = len(cands)
    device = torch.device("cuda", torch.cuda.current_device() if device is None else int(device))
    ctx = ctx or default_context(device.index)
    ptrs, descs = _marshal(cands, refs, groups, is_host=True)
    results = np.zeros(n, dtype=RESULT_DTYPE)
    gp = np.zeros(int(n_group), dtype=np.uint32) if groups is not None else None
    st = load_library().evo_validate_host(
        ctx._h, C.c_void_p(ptrs.ctypes.data), None, C.c_void_p(descs.ctypes.data), n, EVO_F32,
        float(atol), float(rtol), C.c_void_p(results.ctypes.data),
        C.c_void_p(gp.ctypes.data) if gp is not None else None, int(n_group) if gp is not None else 0,
        _stream_ptr(stream, device))
    ctx.check(st)
    return results, gp


def evo_fitness(times, base_times, passed=None, out=None, stream=None, ctx=None, stat=EVO_STAT_MEDIAN, warmup=0, trim=0):
    """times [n_cand, trials] float32 CUDA, base_times [base_trials] float32 CUDA, passed
    optional int32/uint32 [n_cand].  Returns a uint8 CUDA tensor of n_cand x 16 bytes (evo_fit).
    `stat`, `warmup`, `trim` choose the run-time statistic (evo_fitness_ex)."""
    if times.dtype != torch.float32 or base_times.dtype != torch.float32 or times.dim() != 2:
        raise ValueError("times must be a 2-D float32 tensor and base_times float32")
    if not (times.is_contiguous() and base_times.is_contiguous()):
        raise ValueError("times and base_times must be contiguous")
    n_cand, trials = times.shape
    ctx = ctx or default_context(times.device.index)
    if out is None:
        out = torch.empty((n_cand, FIT_DTYPE.itemsize), dtype=torch.uint8, device=times.device)
    L = load_library()
    if stat == EVO_STAT_MEDIAN and warmup == 0:
        st = L.evo_fitness(ctx._h, _dev_ptr(times), n_cand, trials, _dev_ptr(base_times), base_times.numel(),
                           _dev_ptr(passed), _dev_ptr(out), _stream_ptr(stream, times.device))
    else:
        st = L.evo_fitness_ex(ctx._h, _dev_ptr(times), n_cand, trials, _dev_ptr(base_times), base_times.numel(),
                              _dev_ptr(passed), int(stat), int(warmup), int(trim), _dev_ptr(out),
                              _stream_ptr(stream, times.device))
    ctx.check(st)
    return out


def evo_summary(fits, kernel_of, n_kernel, run_of=None, n_run=1, stream=None, ctx=None):
    """Reporting metrics of a population: `fits` is the uint8 CUDA tensor evo_fitness returned,
    `kernel_of` (and optionally `run_of`) int32 CUDA tensors with one id per candidate.  Returns
    (summary: uint8 CUDA tensor of 48 bytes, see summary_to_numpy; best: float32 [n_run, n_kernel];
    run_median: float32 [n_run])."""
    n_cand = fits.shape[0]
    dev = fits.device
    ctx = ctx or default_context(dev.index)
    for t in (kernel_of, run_of):
        if t is not None and (t.dtype not in (torch.int32, torch.uint32) or t.numel() != n_cand or not t.is_contiguous()):
            raise ValueError("kernel_of / run_of must be contiguous 32-bit integer tensors with one entry per candidate")
    out = torch.empty(SUMMARY_DTYPE.itemsize, dtype=torch.uint8, device=dev)
    best = torch.empty((int(n_run), int(n_kernel)), dtype=torch.float32, device=dev)
    med = torch.empty(int(n_run), dtype=torch.float32, device=dev)
    st = load_library().evo_summary(ctx._h, _dev_ptr(fits), _dev_ptr(kernel_of), _dev_ptr(run_of), n_cand, int(n_kernel),
                                    int(n_run), _dev_ptr(out), _dev_ptr(best), _dev_ptr(med), _stream_ptr(stream, dev))
    ctx.check(st)
    return out, best, med


def evo_select_elite(fits, k, stream=None, ctx=None):
    """Indices (int32 CUDA tensor of k entries, -1 where there is none) of the k valid candidates
    with the largest speedup, best first, and their number (int32 CUDA tensor of one entry)."""
    dev = fits.device
    ctx = ctx or default_context(dev.index)
    idx = torch.empty(int(k), dtype=torch.int32, device=dev)
    count = torch.empty(1, dtype=torch.int32, device=dev)
    st = load_library().evo_select_elite(ctx._h, _dev_ptr(fits), fits.shape[0], int(k), _dev_ptr(idx), _dev_ptr(count),
                                         _stream_ptr(stream, dev))
    ctx.check(st)
    return idx, count


def evo_mismatch_sample(cand, ref, atol, rtol, max_out, stream=None, ctx=None):
    """The first `max_out` elements of CUDA tensor `cand` that violate the closeness rule against
    `ref` (index order).  Returns (numpy OFFENDER_DTYPE records, total number of violations);
    synchronises to read them back."""
    if not (cand.is_cuda and ref.is_cuda and cand.is_contiguous() and ref.is_contiguous()):
        raise ValueError("cand and ref must be contiguous CUDA tensors")
    if cand.dtype != ref.dtype or cand.numel() != ref.numel():
        raise ValueError("candidate and reference differ in dtype or size")
    dev = cand.device
    ctx = ctx or default_context(dev.index)
    out = torch.zeros((int(max_out), OFFENDER_DTYPE.itemsize), dtype=torch.uint8, device=dev)
    found = torch.zeros(1, dtype=torch.int64, device=dev)
    st = load_library().evo_mismatch_sample(ctx._h, _dev_ptr(cand), _dev_ptr(ref), cand.numel(), dtype_code(cand.dtype),
                                            float(atol), float(rtol), int(max_out), _dev_ptr(out) if max_out else None,
                                            _dev_ptr(found), _stream_ptr(stream, dev))
    ctx.check(st)
    n_found = int(found.cpu().item())
    recs = out.cpu().numpy().view(OFFENDER_DTYPE).reshape(-1)[: min(int(max_out), n_found)]
    return recs, n_found


def summary_to_numpy(summary):
    return summary.cpu().numpy().view(SUMMARY_DTYPE)[0]


def evo_fitness_host(times, base_times, passed=None, device=None, stream=None, ctx=None):
    """evo_fitness for host arrays (numpy float32); returns a numpy array of FIT_DTYPE records."""
    times = np.ascontiguousarray(times, dtype=np.float32)
    base = np.ascontiguousarray(base_times, dtype=np.float32)
    n_cand, trials = times.shape
    device = torch.device("cuda", torch.cuda.current_device() if device is None else int(device))
    ctx = ctx or default_context(device.index)
    p = np.ascontiguousarray(passed, dtype=np.uint32) if passed is not None else None
    out = np.zeros(n_cand, dtype=FIT_DTYPE)
    st = load_library().evo_fitness_host(
        ctx._h, C.c_void_p(times.ctypes.data), n_cand, trials, C.c_void_p(base.ctypes.data), base.size,
        C.c_void_p(p.ctypes.data) if p is not None else None, C.c_void_p(out.ctypes.data), _stream_ptr(stream, device))
    ctx.check(st)
    return out


def results_to_numpy(results):
    """Device evo_result records -> numpy structured array (synchronises)."""
    return results.cpu().numpy().view(RESULT_DTYPE).reshape(-1)


def fits_to_numpy(fits):
    return fits.cpu().numpy().view(FIT_DTYPE).reshape(-1)
