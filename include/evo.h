/*
 * evo.h - C ABI of the candidate-evaluation library (CUDA, sm_100a).
 *
 * The EvoEngineer paper states kernel optimisation as a constrained problem
 * (Section 3.1, Eq. 1): minimise a performance objective f(p) subject to a
 * correctness constraint g(p) = 0, and reports validity rate and median speedup
 * as metrics (Section 5.1 "Evaluation Metric").  Its evaluator (Section 4.3
 * "Modular Architecture Design") runs functional testing on random test inputs
 * against the reference implementation and then times the kernel over repeated
 * runs.  This library is the data-parallel part of that evaluator:
 *
 *   evo_gen_inputs   seeded random test inputs            (Section 4.3; Appendix A.8.1 "Evaluation Method")
 *   evo_validate     the functional-correctness part of g (Section 3.1 Eq. 1; Section 4.3 functional testing)
 *   evo_fitness      f: median run time -> speedup         (Section 4.3 timing; Appendix A.7.1; Section 5.1)
 *
 * The paper fixes neither the random generator, nor the comparison formula, nor
 * the treatment of NaN/Inf; those are fixed here and stated with each call.
 *
 * Conventions
 *   - Every function returns an int status: EVO_OK (0) or a negative EVO_ERR_*.
 *     Nothing throws, aborts or traps.  evo_last_error() gives a message for the
 *     last failing call on a context.
 *   - "device" pointers are CUDA device addresses on the context's device; "host"
 *     pointers are ordinary process memory.  The caller owns every buffer it
 *     passes; the library keeps no pointer to them after the call's stream work
 *     has run.
 *   - Calls taking a `stream` (a cudaStream_t passed as void*, NULL = the default
 *     stream) only enqueue work; results are in device memory once the stream
 *     reaches that point.  The *_host variants synchronise the stream before they
 *     return.
 *   - The kernels of a context's calls are launched so that each may begin its
 *     set-up while the kernel before it in the stream is still running
 *     (programmatic dependent launch); each waits for that kernel to complete
 *     before it reads or writes any global memory, so stream order is kept for
 *     every buffer.  evo_set_overlapped_launch(ctx, 0) turns this off.
 *   - A context owns a scratch workspace that grows on demand (cudaMalloc inside
 *     the call that needs it, never during stream capture by design of the
 *     caller) and is released by evo_destroy.  Use one context per stream; calls
 *     on one context must not overlap on the device.
 *   - There is no CPU fallback: without a CUDA device every call but
 *     evo_strerror fails with EVO_ERR_CUDA.
 */
#ifndef EVO_H_
#define EVO_H_

#include <stdint.h>

#if defined(__GNUC__)
#define EVO_API __attribute__((visibility("default")))
#else
#define EVO_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

enum {
    EVO_OK = 0,
    EVO_ERR_ARG = -1,        /* null pointer, bad count, tolerance negative or not finite, ... */
    EVO_ERR_ALIGN = -2,      /* pointer not aligned to its element size */
    EVO_ERR_DTYPE = -3,      /* dtype code not accepted by this call */
    EVO_ERR_CUDA = -4,       /* a CUDA runtime call failed; evo_last_error has its text */
    EVO_ERR_WORKSPACE = -5,  /* scratch memory could not be obtained or a fixed limit was exceeded */
    EVO_ERR_TIMEOUT = -6     /* a bounded device-side wait gave up (reported through the context status word) */
};

/* Element types. EVO_U32 is accepted by evo_gen_inputs and evo_validate_generated only; EVO_I32, EVO_I64 and EVO_U8 (also
 * the storage of bool) by evo_validate_exact only; EVO_F64 by evo_validate_f64 only. */
enum { EVO_U32 = 0, EVO_F32 = 1, EVO_F16 = 2, EVO_BF16 = 3, EVO_F64 = 4, EVO_I32 = 5, EVO_I64 = 6, EVO_U8 = 7 };

/* Bits of evo_result.flags. */
enum {
    EVO_FLAG_CAND_NAN = 1, EVO_FLAG_CAND_PINF = 2, EVO_FLAG_CAND_NINF = 4,
    EVO_FLAG_REF_NAN = 8, EVO_FLAG_REF_INF = 16,
    EVO_FLAG_INCOMPLETE = 0x40000000   /* the check did not finish (see evo_check); pass is 0, the statistics are 0 */
};

typedef struct evo_ctx evo_ctx;

/* Create / destroy a context bound to CUDA device `device`.  evo_create allocates
 * a small workspace; evo_destroy synchronises the device work of the context's
 * last calls and frees everything the context owns. */
EVO_API int evo_create(evo_ctx** ctx, int device);
EVO_API int evo_destroy(evo_ctx* ctx);

/* Static text for a status code; never NULL. */
EVO_API const char* evo_strerror(int status);
/* Message of the last failing call on `ctx` (owned by the context, valid until
 * the next call on it); "" if none. */
EVO_API const char* evo_last_error(const evo_ctx* ctx);

/*
 * evo_gen_inputs - fill `out` with n elements of the random stream of `seed`,
 * starting at stream position `offset` (counted in elements, any value).
 * Paper: test inputs are random (Section 4.3, five test cases; Appendix A.8.1,
 * five random inputs).  Generator (fixed here): Philox4x32-10 (Salmon et al.,
 * SC'11).  Stream element g is word (g mod 4) of the block with counter
 * (lo32(g/4), hi32(g/4), 0, 0) under key (lo32(seed), hi32(seed)), so
 * gen(seed, a, n)[i] == gen(seed, 0, a + n)[a + i] for every a.
 *   dtype EVO_U32 : the raw words.
 *   dtype EVO_F32 : standard normals by Box-Muller on word pairs (x0,x1),(x2,x3) of a block:
 *                   u1 = ((xa >> 8) + 1) / 2^24,  u2 = (xb >> 8) / 2^24,
 *                   z_even = sqrt(-2 ln u1) cos(2 pi u2),  z_odd = sqrt(-2 ln u1) sin(2 pi u2),
 *                   computed in binary32 (within 4 ulp of the exactly rounded value).
 *   dtype EVO_F16 / EVO_BF16 : the binary32 value rounded to nearest even.
 * out: device, n elements of the type, aligned to the element size, written
 * completely.  n == 0 is a no-op.  Errors: EVO_ERR_ARG (null ctx/out),
 * EVO_ERR_DTYPE, EVO_ERR_ALIGN, EVO_ERR_CUDA.
 */
EVO_API int evo_gen_inputs(evo_ctx* ctx, uint64_t seed, uint64_t offset, int dtype, uint64_t n,
                   void* out /* device */, void* stream);

/* One candidate output tensor to check. */
typedef struct {
    uint64_t n;        /* elements; 0 is legal (passes, all statistics zero) */
    const void* ref;   /* device; NULL = use the call's ref_ptr */
    int32_t dtype;     /* EVO_F32/F16/BF16; -1 = use the call's dtype.  Candidate and reference share it. */
    uint32_t group;    /* candidate id in [0, n_group): tensors / test cases of one candidate share a verdict */
} evo_desc;

typedef struct {
    uint64_t n_mismatch;   /* elements violating the closeness rule */
    uint64_t n_nonfinite;  /* elements where candidate or reference is NaN or +-Inf */
    double sse;            /* sum of d^2 over elements with both values finite (partial sums of up to 512 elements are
                              formed in binary32, the rest in binary64: within 1e-5 relative of the exact sum) */
    float max_abs;         /* max d over those elements (0 if none; +Inf if a finite difference overflows) */
    float max_rel;         /* max d / |r| over those elements with r != 0 (0 if none) */
    uint32_t flags;        /* EVO_FLAG_* */
    uint32_t pass;         /* 1 iff n_mismatch == 0 */
} evo_result;              /* 40 bytes */

/*
 * evo_validate - the functional-correctness constraint over a population.
 * Paper: Section 3.1 Eq. 1 (g(p) = 0, "output must match the reference
 * implementation across test cases"); Section 4.3 (functional testing against
 * the reference outputs).  Rule (fixed here), per element, candidate c and
 * reference r widened exactly to binary32, each operation rounded once, no fused
 * multiply-add, subnormals kept:
 *     d = |c - r|,  tol = atol + rtol * |r|,
 *     close = (c == r) or (d is finite and d <= tol);   mismatch = not close.
 * So NaN never matches, equal infinities match (but are flagged), +0 matches -0.
 * Elements with a NaN/Inf on either side are counted in n_nonfinite, flagged,
 * judged by the rule, and left out of max_abs, max_rel and sse.
 *
 * cand_ptrs : host array of n_desc device pointers, one candidate tensor each.
 * ref_ptr   : device reference shared by all descriptors whose .ref is NULL (may be NULL if none is).
 * descs     : host array of n_desc descriptors.  Descriptors with the same (reference, n, dtype)
 *             are found and their reference is read from memory once for all of them.
 * dtype     : default element type for descriptors with .dtype == -1.
 * atol,rtol : finite and >= 0.
 * results   : device, n_desc entries, written completely; entry i belongs to descriptor i.
 * group_pass: device, n_group words, optional (NULL with n_group 0): word g = AND of .pass over the
 *             descriptors with .group == g (1 for a group without descriptors).
 * Tensors need only element alignment; 16-byte aligned tensors take the fast path.
 * The host arrays are consumed before the call returns.  n_desc == 0 is legal.
 * A call whose pointer and descriptor arrays, reference, dtype, groups and stream equal those of
 * the call before it on the same context (an evaluation loop that reuses its buffers for every
 * test case) reuses that call's schedule, which is still in device memory, and only launches the
 * kernels; the tensors are read again, the tolerances may differ.  Such a repeated call makes no
 * copy, no allocation and no host wait, so after one ordinary call on the stream it can be
 * captured in a CUDA graph (together with evo_fitness) and replayed.  Schedules of up to 32 KiB
 * (a few hundred tensors) reach the device as kernel arguments, larger ones by a copy from a
 * pinned block of the context.
 * Errors: EVO_ERR_ARG, EVO_ERR_DTYPE, EVO_ERR_ALIGN, EVO_ERR_WORKSPACE, EVO_ERR_CUDA.
 */
EVO_API int evo_validate(evo_ctx* ctx, const void* const* cand_ptrs /* host array of device ptrs */,
                 const void* ref_ptr /* device */, const evo_desc* descs /* host */, uint64_t n_desc,
                 int dtype, float atol, float rtol, evo_result* results /* device */,
                 uint32_t* group_pass /* device, optional */, uint64_t n_group, void* stream);

/*
 * evo_validate_host - the same check for tensors that live in host memory: every
 * pointer (cand_ptrs[i], ref_ptr, descs[i].ref, results, group_pass) is a HOST
 * address.  The tensors are copied to a staging area owned by the context
 * (distinct references once), checked there by the same kernels, and the results
 * are copied back; the stream is synchronised before returning.  Pinned host
 * memory makes the copies faster but is not required.
 */
EVO_API int evo_validate_host(evo_ctx* ctx, const void* const* cand_ptrs /* host array of host ptrs */,
                      const void* ref_ptr /* host */, const evo_desc* descs /* host */, uint64_t n_desc,
                      int dtype, float atol, float rtol, evo_result* results /* host */,
                      uint32_t* group_pass /* host, optional */, uint64_t n_group, void* stream);

typedef struct {
    float median_ms;   /* median of the candidate's run times (0 if status == 1) */
    float speedup;     /* baseline median / candidate median; 0 if not valid */
    uint32_t valid;    /* 1 iff status == 0 and the candidate passed (pass NULL = all passed) */
    uint32_t status;   /* 0 ok; 1 a candidate time is NaN, Inf or <= 0; 2 a baseline time is */
} evo_fit;             /* 16 bytes */

/*
 * evo_fitness - the performance objective f(p): speedup over the baseline kernel
 * from the medians of the run times.
 * Paper: Section 4.3 (run times collected over 100 runs); Appendix A.7.1 (the
 * median of multiple runs is taken; Section 4.3 says "average": the two passages
 * disagree, the median is what this call computes); Section 5.1 "Evaluation
 * Metric" (speedup over the baseline).  Median = middle order statistic, or
 * 0.5 * (a + b) of the two middle ones; speedup = base_median / median; all in
 * binary32, one rounding per operation.  The floor of 1.0 that the paper applies
 * when reporting across kernels is not applied here.
 * times      : device, n_cand rows of `trials` floats (milliseconds), row-major.
 * base_times : device, base_trials floats.
 * pass       : device, n_cand words (e.g. group_pass of evo_validate), optional.
 * out        : device, n_cand entries.
 * 1 <= trials, base_trials <= 4096.  Errors: EVO_ERR_ARG, EVO_ERR_CUDA.
 */
EVO_API int evo_fitness(evo_ctx* ctx, const float* times /* device */, uint64_t n_cand, uint32_t trials,
                const float* base_times /* device */, uint32_t base_trials,
                const uint32_t* pass /* device, optional */, evo_fit* out /* device */, void* stream);

/*
 * evo_fitness_ex - evo_fitness with the run-time statistic chosen.
 * Paper: Section 4.3 says the run times are averaged, Appendix A.7.1 that their median is
 * taken; this call offers both, the minimum and a trimmed mean, and can leave out the first
 * `warmup` runs of every row (and of the baseline).  The statistic is reported in
 * evo_fit.median_ms; speedup = baseline statistic / candidate statistic, of the same kind.
 *   EVO_STAT_MEDIAN        as evo_fitness
 *   EVO_STAT_MEAN          binary64 sum of the kept runs in run order / their count, rounded once to binary32
 *   EVO_STAT_MIN           the smallest kept run
 *   EVO_STAT_TRIMMED_MEAN  kept runs in ascending order, `trim` dropped at each end, binary64 sum of the rest in
 *                          that order / their count, rounded once to binary32
 * warmup < trials and < base_trials; 2 * trim < kept runs (trimmed mean only; ignored otherwise).
 * Errors: as evo_fitness.
 */
enum { EVO_STAT_MEDIAN = 0, EVO_STAT_MEAN = 1, EVO_STAT_MIN = 2, EVO_STAT_TRIMMED_MEAN = 3 };
EVO_API int evo_fitness_ex(evo_ctx* ctx, const float* times /* device */, uint64_t n_cand, uint32_t trials,
                           const float* base_times /* device */, uint32_t base_trials, const uint32_t* pass /* device, optional */,
                           int stat, uint32_t warmup, uint32_t trim, evo_fit* out /* device */, void* stream);

/* evo_fitness for host arrays (all four pointers are HOST addresses); synchronises the stream. */
EVO_API int evo_fitness_host(evo_ctx* ctx, const float* times, uint64_t n_cand, uint32_t trials,
                     const float* base_times, uint32_t base_trials,
                     const uint32_t* pass, evo_fit* out, void* stream);

/*
 * evo_summary - the reporting metrics of a population from its evo_fit records.
 * Paper: Section 5.1 "Evaluation Metric" (the median speedup across kernels, 1.0 for a kernel
 * where no candidate beats the baseline, averaged over the independent runs; Pass@1 = the
 * share of trials that yield a valid kernel); Appendix A.5 (kernels counted by speedup range).
 *   best[r][k]      largest speedup among the valid candidates of kernel k in run r (0 if none)
 *   run_median[r]   median over the kernels of max(best[r][k], 1.0) (middle value, or
 *                   0.5 * (a + b) of the two middle ones, binary32)
 *   median_speedup  mean of the run medians (binary64 sum in run order, rounded once)
 *   validity        n_valid / n_cand (binary64 quotient of the counts, rounded once)
 *   speedup_count   kernels whose best over all runs exceeds 1.0
 *   hist[0..4]      kernels by their best over all runs: < 1, [1, 2), [2, 5), [5, 10), >= 10
 *                   (the paper prints the ranges without saying where the boundaries belong)
 * fits       : device, n_cand records (as written by evo_fitness).
 * kernel_of  : device, n_cand kernel ids in [0, n_kernel).
 * run_of     : device, n_cand run ids in [0, n_run); NULL = all in run 0.
 * out        : device, one record.
 * best       : device, n_run * n_kernel floats, written (it doubles as the call's workspace).
 * run_median : device, n_run floats, optional.
 * 1 <= n_kernel <= 8192, 1 <= n_run <= 1024.  An id out of range makes the next evo_check
 * return EVO_ERR_ARG (the record is skipped).  Errors: EVO_ERR_ARG, EVO_ERR_ALIGN, EVO_ERR_CUDA.
 */
typedef struct {
    float median_speedup, validity;
    uint32_t n_valid, n_cand, speedup_count;
    uint32_t hist[5];
    uint32_t n_kernel, n_run;
} evo_summary_rec;         /* 48 bytes */
EVO_API int evo_summary(evo_ctx* ctx, const evo_fit* fits /* device */, const uint32_t* kernel_of /* device */,
                        const uint32_t* run_of /* device, optional */, uint64_t n_cand, uint32_t n_kernel, uint32_t n_run,
                        evo_summary_rec* out /* device */, float* best /* device */, float* run_median /* device, optional */,
                        void* stream);

/*
 * evo_validate_exact - the correctness constraint for integer and boolean outputs (index
 * results such as an argmax, masks, counts).
 * Paper: Section 3.1 Eq. 1 and Section 4.3 (the output must match the reference); for these
 * types "match" is read as equality, element by element.  Arguments as evo_validate, without
 * tolerances; descriptor and call dtypes are EVO_I32, EVO_I64 or EVO_U8.  Per tensor it
 * reports the number of unequal elements and the largest |c - r| (exact, as an unsigned
 * 64-bit integer: the difference of two int64 values always fits); pass = (n_mismatch == 0).
 * Tensors that share (reference, n, dtype) are found and their reference is read once.
 * Errors: EVO_ERR_ARG, EVO_ERR_DTYPE, EVO_ERR_ALIGN, EVO_ERR_WORKSPACE, EVO_ERR_CUDA.
 */
typedef struct { uint64_t n_mismatch; uint64_t max_abs_diff; uint32_t pass; uint32_t pad; } evo_result_exact;   /* 24 bytes */
EVO_API int evo_validate_exact(evo_ctx* ctx, const void* const* cand_ptrs /* host array of device ptrs */,
                               const void* ref_ptr /* device */, const evo_desc* descs /* host */, uint64_t n_desc, int dtype,
                               evo_result_exact* results /* device */, uint32_t* group_pass /* device, optional */,
                               uint64_t n_group, void* stream);

/*
 * evo_validate_generated - the equality check of evo_validate_exact against a reference that is
 * not stored anywhere: a window of the random stream of evo_gen_inputs, regenerated inside the
 * checking kernel.
 * Paper: Section 4.3 (functional testing on random test cases; the stream of a test case is
 * reproducible from its seed) and Section 3.1 Eq. 1.  Use: a buffer that must still hold, or must
 * have been reproduced as, the raw words that evo_gen_inputs(seed, start, EVO_U32, n) writes - the
 * inputs of a test case after the candidate ran (a kernel must not overwrite its inputs), or the
 * output of a copying / reordering-free candidate - is checked without keeping a second copy and
 * without reading one: per element the kernel spends ten Philox rounds per four words instead of
 * four bytes of memory traffic.
 * Tensor i holds counts[i] 32-bit elements and is compared with stream elements
 * [start_i, start_i + counts[i]) of `seed`, start_i = offsets[i] (offsets NULL: `offset` for all);
 * any start is accepted, multiples of 4 cost one Philox block per four elements, others two.
 * dtype EVO_U32 compares the words as unsigned, EVO_I32 as two's-complement integers (only
 * max_abs_diff differs).  Tensors with the same window are found and checked together.
 * cand_ptrs : host array of n_desc device pointers (4-byte aligned; 16-byte aligned ones take the vector path).
 * counts, offsets, groups : host arrays of n_desc entries (groups may be NULL without group_pass).
 * results, group_pass, n_group : as evo_validate_exact.
 * Errors: EVO_ERR_ARG, EVO_ERR_DTYPE, EVO_ERR_ALIGN, EVO_ERR_WORKSPACE, EVO_ERR_CUDA.
 */
EVO_API int evo_validate_generated(evo_ctx* ctx, uint64_t seed, uint64_t offset, const uint64_t* offsets /* host, optional */,
                                   const void* const* cand_ptrs /* host array of device ptrs */, const uint64_t* counts /* host */,
                                   uint64_t n_desc, int dtype, const uint32_t* groups /* host, optional */,
                                   evo_result_exact* results /* device */, uint32_t* group_pass /* device, optional */,
                                   uint64_t n_group, void* stream);

/*
 * evo_validate_f64 - the correctness constraint for binary64 outputs.
 * Paper: Section 3.1 Eq. 1 and Section 4.3, as evo_validate.  The same rule and statistics
 * with every operation an individually rounded binary64 operation (no fused multiply-add on
 * the rule's chain): d = |c - r|, tol = atol + rtol * |r|, close = (c == r) or (d finite and
 * d <= tol); NaN/Inf elements are counted, flagged, judged by the rule and left out of
 * max_abs, max_rel and sse (every square d*d is a binary64 product, so a square below the
 * binary64 range is lost and one in its subnormal range keeps only the bits that fit; the sum of
 * the squares is within 1e-12 relative of their exact sum).
 * Arguments as evo_validate; descriptor dtypes are EVO_F64 (or -1);
 * tensors are aligned to 8 bytes (16-byte aligned ones take the vector path).
 * Errors: EVO_ERR_ARG, EVO_ERR_DTYPE, EVO_ERR_ALIGN, EVO_ERR_WORKSPACE, EVO_ERR_CUDA.
 */
typedef struct {
    uint64_t n_mismatch, n_nonfinite;
    double sse, max_abs, max_rel;
    uint32_t flags, pass;
} evo_result64;            /* 48 bytes */
EVO_API int evo_validate_f64(evo_ctx* ctx, const void* const* cand_ptrs /* host array of device ptrs */,
                             const void* ref_ptr /* device */, const evo_desc* descs /* host */, uint64_t n_desc,
                             double atol, double rtol, evo_result64* results /* device */,
                             uint32_t* group_pass /* device, optional */, uint64_t n_group, void* stream);

/*
 * evo_mismatch_sample - where a failing candidate is wrong.
 * Paper: Section 4.3 (the third step of the system collects feedback for the next round of
 * generation).  Judges one candidate tensor against its reference by the rule of evo_validate
 * and writes the first max_out violating elements in index order: their index and the two
 * values widened to binary32 (a NaN is reported as some NaN: its payload is not kept);
 * *n_found receives the total number of violations (so min(max_out, *n_found) entries of
 * `out` are written; the rest is left untouched).
 * cand, ref : device, n elements of `dtype` (EVO_F32/F16/BF16), aligned to the element size.
 * out       : device, max_out entries (may be NULL with max_out 0: count only).
 * n_found   : device, one 64-bit word.
 * The context's workspace grows by 8 bytes per 2048 elements.  Errors: EVO_ERR_ARG,
 * EVO_ERR_DTYPE, EVO_ERR_ALIGN, EVO_ERR_WORKSPACE, EVO_ERR_CUDA.
 */
typedef struct { uint64_t index; float cand, ref; } evo_offender;   /* 16 bytes */
EVO_API int evo_mismatch_sample(evo_ctx* ctx, const void* cand /* device */, const void* ref /* device */, uint64_t n,
                                int dtype, float atol, float rtol, uint64_t max_out, evo_offender* out /* device */,
                                uint64_t* n_found /* device */, void* stream);

/*
 * evo_select_elite - which candidates to keep.
 * Paper: Section 4.2 "Population Management" (the single-solution strategy keeps the current
 * best solution, elite preservation a small set of high-performing ones).  Writes the indices
 * of the k valid candidates with the largest speedup, best first, candidates with equal
 * speedup in order of their index; if fewer than k are valid, the remaining entries are
 * 0xffffffff.  k = 1 is the single-solution strategy.
 * fits  : device, n_cand records (as written by evo_fitness); n_cand <= 65536.
 * idx   : device, k words, written.   count : device, one word: min(k, valid candidates).
 * Errors: EVO_ERR_ARG, EVO_ERR_ALIGN, EVO_ERR_CUDA.
 */
EVO_API int evo_select_elite(evo_ctx* ctx, const evo_fit* fits /* device */, uint64_t n_cand, uint32_t k,
                             uint32_t* idx /* device */, uint32_t* count /* device */, void* stream);

/*
 * evo_validate_static - evo_validate for callers that cannot allocate device memory.
 * (The paper has no counterpart: this entry point exists for the sake of such callers.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a memory pool or a
 * framework allocator that owns the whole device, under a "no allocation after start-up"
 * rule of a serving process, or while another part of the program has a CUDA graph capture
 * open on the thread (an allocation would break the capture).  evo_validate grows its
 * context's workspace with cudaMalloc when a population needs more room, and creating a
 * context allocates too; this variant needs no context and never allocates: its scratch
 * (the schedule and the per-CTA partial results) is a fixed array of 1 MiB that is part of the
 * library image, so every GPU that loads the library carries that 1 MiB until the process ends.
 *
 * Arguments, results, rule and errors are those of evo_validate (all tensor, result and verdict
 * pointers are device addresses; the caller still provides inputs and outputs), on the CURRENT
 * device.  Differences:
 *   - Limit: schedule plus partial results must fit the 1 MiB.  That is roughly 4000 tensors in
 *     one call (fewer when very many share a reference); the exact need depends on the
 *     population and is checked per call.  Beyond it the call does nothing and returns
 *     EVO_ERR_WORKSPACE; evo_validate_static_error() then says how many bytes were needed.
 *     Split the population over several calls, or use evo_validate.
 *   - The first call on each device looks up the scratch's device address (no allocation, but a
 *     runtime query): make that first call before starting any stream capture.
 *   - All calls on one device share the one scratch array.  It keeps whatever the previous call
 *     left.  The only word that must start at zero, the status word that a kernel raises when one
 *     of its bounded waits runs out, is cleared on the stream at the head of every call; everything
 *     else a call reads it has written itself.  So a call reports its own waits only: results
 *     carry EVO_FLAG_INCOMPLETE (pass = 0) exactly when a wait of THAT call ran out, and the next
 *     call starts clean - no restart and no extra call is needed to recover.
 *     But two calls whose kernels overlap on the GPU (different streams, or different threads)
 *     would overwrite each other's schedule: keep calls on one device ordered, e.g. on one stream.
 *   - The schedule reaches the device as the arguments of small kernels (one launch per 16 KiB of
 *     schedule, a few KiB for typical populations): the call hands the runtime no pointer into
 *     host memory that it frees afterwards, and the host does not wait for the stream.
 *   - It calls no cudaMalloc, cudaFree, cudaMallocHost nor any other allocating CUDA routine.
 * evo_validate_static_error: message of the calling thread's last failing evo_validate_static
 * call ("" if it succeeded); static storage, never NULL.
 */
EVO_API int evo_validate_static(const void* const* cand_ptrs /* host array of device ptrs */, const void* ref_ptr /* device */,
                                const evo_desc* descs /* host */, uint64_t n_desc, int dtype, float atol, float rtol,
                                evo_result* results /* device */, uint32_t* group_pass /* device, optional */,
                                uint64_t n_group, void* stream);
EVO_API const char* evo_validate_static_error(void);

/*
 * evo_plan_inspect - host-only view of the schedule evo_validate would use on a device that
 * runs `max_ctas` persistent CTAs: how descriptors were merged into sets that share one
 * reference read, and which contiguous run of (set, tile) items each CTA walks.  Touches no
 * device and dereferences no tensor; meant for inspection and for testing the scheduler.
 * (The persistent grid over ragged descriptors is this library's design; the paper has no
 * counterpart.)
 * summary    : host, written.
 * ranges     : host, optional, max_ctas entries; entry b is CTA b's run
 *              [(set_begin, tile_begin), (set_end, tile_end)), tile_end exclusive inside
 *              set_end.  Only summary->n_ctas entries are written (runs are never empty).
 * set_of_desc: host, optional, n_desc entries: the set each descriptor joined.
 * set_k      : host, optional, n_desc entries (only the first n_sets are written): members per set.
 * Errors: as evo_validate's argument checks.
 */
typedef struct { uint32_t n_sets, n_ctas, n_parts, tile_elems; uint64_t total_tiles; } evo_plan_summary;
typedef struct { uint64_t tile_begin, tile_end; uint32_t set_begin, set_end; } evo_plan_range;
EVO_API int evo_plan_inspect(const void* const* cand_ptrs, const void* ref_ptr, const evo_desc* descs, uint64_t n_desc,
                             int dtype, uint32_t max_ctas, evo_plan_summary* summary, evo_plan_range* ranges,
                             uint32_t* set_of_desc, uint32_t* set_k);

/*
 * evo_set_timing_events - ask the next evo_validate / evo_validate_host call on `ctx` to record
 * two CUDA events (cudaEvent_t passed as void*, created by the caller with timing enabled) on
 * its stream: `start` right before and `stop` right after the launch of the main checking
 * kernel (the first pass over the tensors).  The request is consumed by that call; pass NULLs
 * to cancel, and a call that fails consumes it too.  The small kernels before it (the store of
 * the schedule, the warm start of the max d/|r| filter on short runs) lie outside the pair.
 * For measuring the kernel alone inside a longer stream of work.  (The paper has no
 * counterpart.)
 */
EVO_API int evo_set_timing_events(evo_ctx* ctx, void* start, void* stop);

/*
 * evo_check - wait for the work enqueued on `stream` and report whether the device side of
 * the context's calls ran to completion.  The kernels never wait without a limit (a copy
 * into shared memory that does not land within 2 s makes the CTA stop, raise a status word
 * and return); when that happened, evo_validate's results carry EVO_FLAG_INCOMPLETE with
 * pass = 0, and this call returns EVO_ERR_TIMEOUT once and clears the word.  The *_host
 * variants do this check themselves.  It also reports, as EVO_ERR_ARG, an id out of range
 * that evo_summary met on the device.  (The paper has no counterpart.)
 * Errors: EVO_ERR_ARG, EVO_ERR_CUDA, EVO_ERR_TIMEOUT.
 */
EVO_API int evo_check(evo_ctx* ctx, void* stream);

/*
 * evo_selftest_wait - exercise the bounded device-side wait without any fault: enqueues a
 * one-warp kernel that waits, through the routine the checking kernel uses, on a barrier that
 * nothing completes, with a limit of `limit_us` microseconds (1..1000000).  The kernel gives
 * up at the limit, raises the context's status word and returns normally; the next evo_check
 * then reports EVO_ERR_TIMEOUT once and the context stays usable.  (The paper has no
 * counterpart.)  Errors: EVO_ERR_ARG, EVO_ERR_CUDA.
 */
EVO_API int evo_selftest_wait(evo_ctx* ctx, uint32_t limit_us, void* stream);

/* Number of kernels this context has launched so far (for accounting in benchmarks). */
EVO_API uint64_t evo_launch_count(const evo_ctx* ctx);

/*
 * evo_set_overlapped_launch - turn programmatic dependent launch of the context's kernels on
 * (default) or off.  Off, every kernel starts only after the work before it in the stream has
 * finished, as with an ordinary launch.  (The paper has no counterpart.)
 */
EVO_API int evo_set_overlapped_launch(evo_ctx* ctx, int enable);

/*
 * evo_debug_cta_timing / evo_debug_read_cta_times - how evenly a population spreads over the
 * persistent CTAs of evo_validate's main kernel, measured rather than planned.  While enabled,
 * every CTA of that kernel writes the GPU's nanosecond clock (%globaltimer) when it starts
 * working and when it is done, into a buffer of the context (allocated by the next
 * evo_validate call).  evo_debug_read_cta_times waits for the device and copies the pairs
 * (begin, end) of the last such call to `begin_end_ns` (host, 2 * capacity words; CTA b at
 * 2b, 2b + 1); *n_ctas receives how many CTAs that call ran.  Meant for benchmarks; leave it
 * off otherwise.  (The paper has no counterpart.)  Errors: EVO_ERR_ARG, EVO_ERR_CUDA.
 */
EVO_API int evo_debug_cta_timing(evo_ctx* ctx, int enable);
EVO_API int evo_debug_read_cta_times(evo_ctx* ctx, uint64_t* begin_end_ns /* host */, uint32_t capacity, uint32_t* n_ctas /* host */);

#ifdef __cplusplus
}
#endif
#endif /* EVO_H_ */
