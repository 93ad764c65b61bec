// evo_validate: the functional-correctness constraint over a population of candidate
// outputs (paper Section 3.1 Eq. 1, g(p) = 0; Section 4.3, functional testing against the
// reference outputs), with the error statistics reported alongside the verdict.
//
// Shape of the computation: a pure streaming read.  Every candidate element and every
// distinct reference element has to come from HBM once; per element there are five to
// eight binary32 operations.  The design therefore spends its effort on (1) never reading a
// reference tile more than once per set of candidates that share it, (2) keeping many
// bytes in flight per SM independently of the arithmetic, and (3) keeping reductions and
// everything that depends on the reference alone off the per-candidate path.
//
//   plan (host)   tensors with the same (reference, n, dtype) form a set of up to kMaxK
//                 members; the flat list of (set, tile) items, weighted by the tiles they
//                 move, is cut into one contiguous range per CTA (a fixed cut: no work
//                 queue, no atomics, results reproducible run to run).  A small plan reaches
//                 the device as kernel arguments (plan_store), a large one by one copy; a call
//                 with the arguments of the call before reuses the plan that is already there.
//   pass 1        persistent CTAs walk their range.  A producer warp streams the tiles
//                 (reference, then each member) into a ring of shared-memory stages with
//                 bulk asynchronous copies that complete on mbarriers; eight consumer warps
//                 take a reference tile into registers once (values, smallest tolerance), then
//                 compare each member's tile against it.  Per (tile, member) a warp folds
//                 its lanes with redux/shuffles into a warp-private accumulator in shared
//                 memory.  When a CTA leaves a set it writes one partial record per member.
//   pass 2        one warp per tensor folds the partial records of the CTAs that touched
//                 it, in a fixed order, and writes the evo_result.
//   verdict       one thread per candidate id ANDs the verdicts of its tensors (inside
//                 pass 2 when one CTA holds every tensor).
//
// Every kernel is launched so that it may begin under the tail of its predecessor
// (programmatic dependent launch) and waits for it before touching global memory.
//
// Every wait on an mbarrier is bounded: after kWaitLimitNs the CTA stops working, lets its
// outstanding copies land, raises the status word and returns; pass 2 then marks every
// result as incomplete instead of reporting numbers.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <string>
#include <unordered_map>
#include <vector>

#include "evo_internal.h"
#include "plan.h"
#include "rule.cuh"

namespace {

using namespace evo;

constexpr int kCtasPerSm = 2;
constexpr int kCtasPerSm16 = 3;                     // for populations of 16-bit tensors only
constexpr int kStages = 6;                          // ring depth per CTA
constexpr int kStageBytes = kTileElems * 4;         // 16 KiB: one fp32 tile (a 16-bit tile uses half)
constexpr size_t kRingBytes = static_cast<size_t>(kStages) * kStageBytes;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s per wait, then give up
constexpr uint64_t kSeedBelowTilesPerCta = 32;               // runs shorter than this get the seed pass

// ---- shared-memory barriers and bulk copies (PTX) -------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait, cold part: polls until the phase completes, another warp of the CTA has given
// up, or the limit has passed (then raises the CTA's abort flag itself).
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                            unsigned long long limit_ns) {
    const unsigned long long t0 = global_ns();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_ns() - t0 > limit_ns) { *abort_flag = 1; return false; }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          unsigned long long limit_ns = kWaitLimitNs) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, limit_ns);
}
__device__ __forceinline__ unsigned long long policy_evict_first() {
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// One contiguous block global -> this CTA's shared memory; completion is counted in bytes on
// `bar`.  Source, destination and size are multiples of 16 bytes.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, unsigned long long pol) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, %0;" ::"n"(kThreads) : "memory"); }

// Programmatic dependent launch.  Every kernel of a call is launched so that it may start while
// its predecessor in the stream is still running: it does its set-up, then waits here until the
// predecessor has completed and its writes are visible, and only then touches global memory.
// Every kernel waits (even one that needs nothing from its predecessor), so completion stays
// transitive along the stream.  Launched without the attribute, both are no-ops.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependents_may_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
__device__ __forceinline__ float rcp_approx(float x) {
    float y;
    asm("rcp.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// Position in the ring: both the producer and the consumers count the same sequence of tiles.
struct Ring {
    uint32_t full0, empty0;     // shared-memory addresses of full[0], empty[0]
    uint32_t data0;             // ... and of stage 0
    uint32_t stage_bytes;       // 16 KiB, or 8 KiB in the kernel for populations of 16-bit tensors only
    uint32_t stage = 0, phase = 0;
    bool dead = false;          // this warp has given up (warp-uniform)
    volatile int* abort_flag;
    __device__ __forceinline__ uint32_t full() const { return full0 + 8u * stage; }
    __device__ __forceinline__ uint32_t empty() const { return empty0 + 8u * stage; }
    __device__ __forceinline__ uint32_t data() const { return data0 + stage_bytes * stage; }
    __device__ __forceinline__ void advance() { if (++stage == kStages) { stage = 0; phase ^= 1u; } }
};

// ---- the rule, exact form ----------------------------------------------------------------
// Per-lane state for one (tile, member) on the exact path.
struct Lane {
    uint32_t cnt = 0;        // mismatches
    float ma = 0.f;          // max d
    float mr = 0.f;          // max d/|r|
    double dsse = 0.0;       // sum d^2, binary64
    uint32_t nf = 0;         // non-finite elements
    uint32_t flags = 0;
};

// The rule with every special case, and the true quotient: d = |c - r|, tol = atol + rtol*|r|
// (one rounding per operation, no fused multiply-add), close = (c == r) or (d finite and
// d <= tol); NaN/Inf elements are counted and flagged and stay out of the statistics.
__device__ __forceinline__ void exact_elem(float c, float r, float atol, float rtol, Lane& s) {
    const float d = fabsf(__fsub_rn(c, r));
    const float ar = fabsf(r);
    s.cnt += rule_mismatch(c, r, atol, rtol) ? 1u : 0u;
    const uint32_t cb = __float_as_uint(c), rb = __float_as_uint(r);
    const uint32_t cm = cb & 0x7fffffffu, rm = rb & 0x7fffffffu;
    uint32_t f = 0;
    if (cm > 0x7f800000u) f |= EVO_FLAG_CAND_NAN;
    if (cb == 0x7f800000u) f |= EVO_FLAG_CAND_PINF;
    if (cb == 0xff800000u) f |= EVO_FLAG_CAND_NINF;
    if (rm > 0x7f800000u) f |= EVO_FLAG_REF_NAN;
    if (rm == 0x7f800000u) f |= EVO_FLAG_REF_INF;
    if (f) {
        s.nf += 1;
        s.flags |= f;
    } else {
        s.ma = fmaxf(s.ma, d);                                      // d may be +Inf (overflow), never NaN
        if (ar != 0.f) s.mr = fmaxf(s.mr, __fdiv_rn(d, ar));
        s.dsse += static_cast<double>(d) * static_cast<double>(d);
    }
}

// Fold the 32 lanes (all fields) and add the result to the warp's accumulator for this member.
__device__ __forceinline__ void warp_commit_exact(const Lane& s, Acc* acc, int lane) {
    const unsigned full = 0xffffffffu;
    const uint32_t cnt = __reduce_add_sync(full, s.cnt);
    const uint32_t ma = __reduce_max_sync(full, __float_as_uint(s.ma));
    const uint32_t mr = __reduce_max_sync(full, __float_as_uint(s.mr));
    const uint32_t nf = __reduce_add_sync(full, s.nf);
    const uint32_t fl = __reduce_or_sync(full, s.flags);
    double x = s.dsse;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(full, x, o);
    if (lane == 0) {
        acc->mism += cnt;
        acc->nonfin += nf;
        acc->sse += x;
        acc->max_abs = max(acc->max_abs, ma);
        acc->max_rel = max(acc->max_rel, mr);
        acc->flags |= fl;
    }
    __syncwarp();
}

// The exact rule over this thread's 16 elements of a full tile, read again from global
// memory (they were just streamed: L2 hits at best).  Reached only when the fast path
// cannot vouch for its numbers: a NaN/Inf, an overflowing difference, or differences so
// small that their squares underflow in binary32.
template <int DT>
__device__ __noinline__ void exact_redo(const uint4* __restrict__ cp, const uint4* __restrict__ rp,
                                        float atol, float rtol, Lane* out) {
    using E = Elem<DT>;
    Lane st;
#pragma unroll 1
    for (int v = 0; v < E::kVecs; ++v) {
        const uint4 c = cp[v * kThreads], r = rp[v * kThreads];
#pragma unroll
        for (int e = 0; e < E::kPerVec; ++e) exact_elem(E::at(c, e), E::at(r, e), atol, rtol, st);
    }
    *out = st;
}

// ---- consumers ---------------------------------------------------------------------------
// Wait until the producer's copy into the current stage has landed.  The answer is the same
// for all lanes of the warp; after a failed wait the warp does no further work.
__device__ __forceinline__ bool ring_acquire(Ring& g) {
    const bool ok = mbar_wait(g.full(), g.phase, g.abort_flag);
    if (!__all_sync(0xffffffffu, ok)) { g.dead = true; return false; }
    return true;
}
// The warp has copied its share of the stage into registers: hand the stage back.
__device__ __forceinline__ void ring_release(Ring& g, int lane) {
    __syncwarp();
    if (lane == 0) mbar_arrive(g.empty());
    g.advance();
}

// One tile (kTileElems elements of one tensor) out of the ring into registers: thread t takes
// vectors v * kThreads + t of the stage, which is handed back as soon as the warp has its share.
// False if a wait ran out.
template <int DT>
__device__ __forceinline__ bool take_tile(Ring& g, uint4 (&v)[Elem<DT>::kVecs], int lane) {
    constexpr uint32_t kVecStride = kThreads * 16;
    if (!ring_acquire(g)) return false;
    const uint32_t a = g.data() + threadIdx.x * 16;
#pragma unroll
    for (int q = 0; q < Elem<DT>::kVecs; ++q) v[q] = lds128(a + q * kVecStride);
    ring_release(g, lane);
    return true;
}

// IEEE division, kept out of line: the walks below name it at 16 unrolled positions and run it
// at one or two of them, so its body would only bloat the hot loop's instruction footprint.
__device__ __noinline__ float div_rn(float a, float b) { return __fdiv_rn(a, b); }

constexpr float kInf = __builtin_huge_valf();

// One full, 16-byte aligned tile: reference into registers once, then every member.
//
// Fast path per element, valid when c and r are finite and d does not overflow: d = |c - r|,
// its maximum and its square; mismatches are counted only for a thread whose largest d exceeds the
// smallest tolerance of its 16 elements.  With atol, rtol >= 0 and finite data c == r implies
// d = 0 <= tol, so the equality clause needs no test here.
// The quotient d/|r| is not formed.  With m the running maximum of the quotient (a binary32 value),
// fl(d/|r|) > m implies d/|r| > m (rounding is monotone and m is representable), hence
// d > m*|r| >= RZ(m*|r|): the test d > RZ(m*|r|) never misses a new maximum, and an element that only
// ties the maximum does not pass it.  A thread whose filter fired walks its 16 elements again in
// registers and divides only where r != 0 and the filter still fires against its own, rising maximum.
template <int DT>
__device__ __forceinline__ void fast_tile(const void* ref, int K, uint64_t t, float atol, float rtol, Acc (*s_acc)[kWarps],
                                          uint32_t* s_mr, const void* const* s_cand, Ring& g, int warp, int lane) {
    using E = Elem<DT>;
    if (g.dead) return;
    float r[kEpt];
    {
        uint4 rv[E::kVecs];
        if (!take_tile<DT>(g, rv, lane)) return;
#pragma unroll
        for (int v = 0; v < E::kVecs; ++v)
#pragma unroll
            for (int e = 0; e < E::kPerVec; ++e) r[v * E::kPerVec + e] = E::at(rv[v], e);
    }
    // The smallest tolerance among this thread's 16 reference elements: tol = atol + rtol*|r| does not decrease
    // with |r| (each rounding is monotone), so it is the tolerance of the smallest |r|.  A member whose largest
    // difference over these elements stays within it has no mismatch here, and none is counted element by element.
    // (Finer groups - a tolerance per 16-byte vector - and a walk shared out over the warp were measured: no gain on
    // data with values on the boundary, a loss on candidates that are wrong everywhere.)
    float armin = kInf;
#pragma unroll
    for (int e = 0; e < kEpt; ++e) armin = fminf(armin, fabsf(r[e]));
    const float tolmin = __fadd_rn(atol, __fmul_rn(rtol, armin));
    const uint64_t vec0 = t * (kTileElems / E::kPerVec) + threadIdx.x;   // this thread's first vector of the tile
#pragma unroll 1
    for (int k = 0; k < K; ++k) {
        uint4 cv[E::kVecs];
        if (!take_tile<DT>(g, cv, lane)) return;
        Acc* acc = &s_acc[k][warp];
        // Running maximum of d/|r| of this member, shared by the CTA's warps.  A stale (smaller)
        // value only makes the filter fire more often.
        const float m = __uint_as_float(*reinterpret_cast<volatile uint32_t*>(&s_mr[k]));
        uint32_t cnt = 0;
        float ma = 0.f, sse = 0.f;
        bool trig = false;
#pragma unroll
        for (int v = 0; v < E::kVecs; ++v)
#pragma unroll
            for (int e = 0; e < E::kPerVec; e += 2) {
                const int i = v * E::kPerVec + e;
                const float d0 = fabsf(__fsub_rn(E::at(cv[v], e), r[i]));
                const float d1 = fabsf(__fsub_rn(E::at(cv[v], e + 1), r[i + 1]));
                ma = max3(ma, d0, d1);
                sse = fmaf(d0, d0, sse);
                sse = fmaf(d1, d1, sse);
                trig |= d0 > __fmul_rz(m, fabsf(r[i]));
                trig |= d1 > __fmul_rz(m, fabsf(r[i + 1]));
            }
        // The fast numbers do not stand if something was NaN/Inf or overflowed (the sum of
        // squares is then NaN/Inf) or if every d is so small that d^2 underflows in binary32.
        const bool redo = !(sse < kInf) || (ma < 9.094947017729282e-13f /* 2^-40 */ && ma > 0.f);
        if (ma > tolmin && !redo) {
            // some difference may exceed its tolerance: count, element by element
#pragma unroll
            for (int v = 0; v < E::kVecs; ++v)
#pragma unroll
                for (int e = 0; e < E::kPerVec; ++e) {
                    const int i = v * E::kPerVec + e;
                    const float d = fabsf(__fsub_rn(E::at(cv[v], e), r[i]));
                    const float tol = __fadd_rn(atol, __fmul_rn(rtol, fabsf(r[i])));
                    cnt += (d > tol) ? 1u : 0u;
                }
        }
        float mt = m;
        float lo = m;
        bool scan = trig && !redo;
        const unsigned full = 0xffffffffu;
        if (m == 0.f && __any_sync(full, scan)) {
            // No maximum yet (m is the same for the whole warp): every lane with some d > 0 would
            // scan, each dividing at its own elements.  Instead all lanes first form approximate
            // quotients (reciprocal approximation, relative error below 2^-21), the warp takes
            // their maximum A, and only lanes that come within 2^-17 of A scan, starting from a
            // threshold 2^-18 below A: the element with the exact maximum passes it.
            float qa = 0.f;
            if (!redo) {
#pragma unroll
                for (int v = 0; v < E::kVecs; ++v)
#pragma unroll
                    for (int e = 0; e < E::kPerVec; ++e) {
                        const int i = v * E::kPerVec + e;
                        const float ar = fabsf(r[i]);
                        const float d = fabsf(__fsub_rn(E::at(cv[v], e), r[i]));
                        qa = fmaxf(qa, d * rcp_approx(ar == 0.f ? kInf : ar));      // r == 0 contributes 0
                    }
            }
            const float A = __uint_as_float(__reduce_max_sync(full, __float_as_uint(qa)));
            // Outside the range where the error bound of the approximation holds, scan from 0.
            if (A > 7.888609052210118e-31f /* 2^-100 */ && A < kInf) {
                lo = __fmul_rz(A, 0.999996185302734375f /* 1 - 2^-18 */);
                scan = scan && qa >= __fmul_rz(A, 0.99999237060546875f /* 1 - 2^-17 */);
            }
        }
        if (scan) {
#pragma unroll
            for (int v = 0; v < E::kVecs; ++v)
#pragma unroll
                for (int e = 0; e < E::kPerVec; ++e) {
                    const int i = v * E::kPerVec + e;
                    const float d = fabsf(__fsub_rn(E::at(cv[v], e), r[i]));
                    const float ar = fabsf(r[i]);
                    if (ar != 0.f && d > __fmul_rz(lo, ar)) {
                        const float q = div_rn(d, ar);
                        if (q > mt) { mt = q; lo = q; }
                    }
                }
        }
        if (__any_sync(full, redo)) {
            Lane st;
            if (redo) {
                exact_redo<DT>(static_cast<const uint4*>(s_cand[k]) + vec0, static_cast<const uint4*>(ref) + vec0,
                               atol, rtol, &st);
            } else {
                st.cnt = cnt; st.ma = ma; st.mr = mt; st.dsse = static_cast<double>(sse);
            }
            const uint32_t mr_w = __reduce_max_sync(full, __float_as_uint(st.mr));
            if (lane == 0 && mr_w > __float_as_uint(m)) atomicMax(&s_mr[k], mr_w);
            warp_commit_exact(st, acc, lane);
        } else {
            const uint32_t cnt_w = __reduce_add_sync(full, cnt);
            const uint32_t ma_w = __reduce_max_sync(full, __float_as_uint(ma));
            const uint32_t mr_w = __reduce_max_sync(full, __float_as_uint(mt));
            float x = sse;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(full, x, o);
            if (lane == 0) {
                acc->mism += cnt_w;
                acc->sse += static_cast<double>(x);
                acc->max_abs = max(acc->max_abs, ma_w);
                if (mr_w > __float_as_uint(m)) atomicMax(&s_mr[k], mr_w);
            }
        }
    }
}

// Tensors that are not 16-byte aligned: scalar loads straight from global memory, exact
// rule.  These tiles do not pass through the ring.
template <int DT>
__device__ __noinline__ void slow_tile(const SetRec& S, uint64_t t, float atol, float rtol,
                                       Acc (*s_acc)[kWarps], const void* const* s_cand, int warp, int lane) {
    using E = Elem<DT>;
    using T = typename E::T;
    const uint64_t e0 = t * kTileElems;
    const uint64_t e1 = min(S.n, e0 + kTileElems);
    const T* rp = static_cast<const T*>(S.ref);
    for (uint32_t k = 0; k < S.k; ++k) {
        const T* cp = static_cast<const T*>(s_cand[k]);
        Lane st;
        for (uint64_t e = e0 + threadIdx.x; e < e1; e += kThreads) exact_elem(E::widen(cp[e]), E::widen(rp[e]), atol, rtol, st);
        warp_commit_exact(st, &s_acc[k][warp], lane);
    }
}

// The whole vectors of a ragged last tile (`valid_vecs` of them); vectors that do not exist read as zero.
template <int DT>
__device__ __forceinline__ bool take_tail(Ring& g, uint4 (&v)[Elem<DT>::kVecs], uint32_t valid_vecs, int lane) {
    constexpr uint32_t kVecStride = kThreads * 16;
    if (!ring_acquire(g)) return false;
    const uint32_t a = g.data() + threadIdx.x * 16;
#pragma unroll
    for (int q = 0; q < Elem<DT>::kVecs; ++q)
        v[q] = q * kThreads + threadIdx.x < valid_vecs ? lds128(a + q * kVecStride) : make_uint4(0u, 0u, 0u, 0u);
    ring_release(g, lane);
    return true;
}

// The ragged last tile of an aligned tensor.  Its whole 16-byte vectors (`valid_vecs` of
// them) come through the ring like a full tile; a thread takes the same vectors as in
// fast_tile but only those that exist, and applies the exact rule to each element.  Once per
// tensor, so kept out of line and simple.
// The ring position travels by value (in and out, packed), so that the caller's copy can
// stay in registers.
template <int DT>
__device__ __noinline__ uint32_t tail_tile(uint32_t n_members, uint32_t valid_vecs, float atol, float rtol,
                                           Acc (*s_acc)[kWarps], Ring g, int warp, int lane) {
    using E = Elem<DT>;
    uint4 rv[E::kVecs];
    if (take_tail<DT>(g, rv, valid_vecs, lane)) {
        for (uint32_t k = 0; k < n_members; ++k) {
            uint4 cv[E::kVecs];
            if (!take_tail<DT>(g, cv, valid_vecs, lane)) break;
            Lane st;
#pragma unroll
            for (int v = 0; v < E::kVecs; ++v) {
                if (v * kThreads + threadIdx.x < valid_vecs) {
#pragma unroll
                    for (int e = 0; e < E::kPerVec; ++e) exact_elem(E::at(cv[v], e), E::at(rv[v], e), atol, rtol, st);
                }
            }
            warp_commit_exact(st, &s_acc[k][warp], lane);
        }
    }
    return g.stage | (g.phase << 8) | (g.dead ? 1u << 16 : 0u);       // ring_pack
}

// The last few elements of an aligned tensor that do not fill a 16-byte vector (at most 3
// fp32 or 7 fp16/bf16 values): thread (8k + j) takes element j of member k, so one round of
// scalar loads serves all members; groups of 8 lanes fold with shuffles and the group's first
// lane adds to the accumulator its own warp owns.
template <int DT>
__device__ __noinline__ void leftover_pass(const SetRec& S, uint64_t e_first, uint32_t left, float atol, float rtol,
                                           Acc (*s_acc)[kWarps], const void* const* s_cand, int warp, int lane) {
    using E = Elem<DT>;
    using T = typename E::T;
    const uint32_t k = threadIdx.x >> 3, j = threadIdx.x & 7;
    Lane st;
    if (k < S.k && j < left) {
        const T c = static_cast<const T*>(s_cand[k])[e_first + j];
        const T r = static_cast<const T*>(S.ref)[e_first + j];
        exact_elem(E::widen(c), E::widen(r), atol, rtol, st);
    }
    const unsigned full = 0xffffffffu;
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) {
        st.cnt += __shfl_xor_sync(full, st.cnt, o);
        st.nf += __shfl_xor_sync(full, st.nf, o);
        st.flags |= __shfl_xor_sync(full, st.flags, o);
        st.ma = fmaxf(st.ma, __shfl_xor_sync(full, st.ma, o));
        st.mr = fmaxf(st.mr, __shfl_xor_sync(full, st.mr, o));
        st.dsse += __shfl_xor_sync(full, st.dsse, o);
    }
    if (j == 0 && k < S.k) {
        Acc* acc = &s_acc[k][warp];                 // warp == k / 4: touched by this warp only
        acc->mism += st.cnt;
        acc->nonfin += st.nf;
        acc->sse += st.dsse;
        acc->max_abs = max(acc->max_abs, __float_as_uint(st.ma));
        acc->max_rel = max(acc->max_rel, __float_as_uint(st.mr));
        acc->flags |= st.flags;
    }
    __syncwarp();
}

// What of set s belongs to this CTA's range, and how its tiles travel.  Producer and
// consumers derive the sequence of ring stages from this, so they must agree on it.
struct Span {
    uint64_t t0, t1;         // this CTA's tiles of the set
    uint64_t full_tiles;     // tiles [0, full_tiles) are complete and go through the ring (0 if not 16-byte aligned)
    uint32_t tail_vecs;      // whole 16-byte vectors of the ragged last tile, copied through the ring as well
    uint32_t left;           // elements after those (less than one vector): leftover pass
};
__device__ __forceinline__ Span set_span(const CtaRange& rg, uint32_t s, const SetRec& S) {
    Span sp;
    const uint64_t tiles = (S.n + kTileElems - 1) / kTileElems;
    sp.t0 = (s == rg.s_begin) ? rg.t_begin : 0;
    sp.t1 = (s == rg.s_end) ? rg.t_end : tiles;
    const uint32_t rem = static_cast<uint32_t>(S.n % kTileElems);
    const uint32_t per_vec = S.dtype == EVO_F32 ? 4u : 8u;
    sp.full_tiles = S.vec_ok ? S.n / kTileElems : 0;
    sp.tail_vecs = S.vec_ok ? rem / per_vec : 0;
    sp.left = S.vec_ok ? rem % per_vec : 0;
    return sp;
}

// All full tiles [t_begin, t_end) of a set: the hot loop, a function of its own so that its
// registers are allocated without regard to the rarely used paths around it.  The ring
// position travels by value, in and packed out.
__device__ __forceinline__ uint32_t ring_pack(const Ring& g) { return g.stage | (g.phase << 8) | (g.dead ? 1u << 16 : 0u); }
__device__ __forceinline__ void ring_unpack(Ring& g, uint32_t pos) {
    g.stage = pos & 0xffu; g.phase = (pos >> 8) & 1u; g.dead = (pos >> 16) != 0;
}
template <int DT>
__device__ __noinline__ uint32_t fast_run(const void* ref, int K, uint64_t t_begin, uint64_t t_end, float atol, float rtol,
                                          Acc (*s_acc)[kWarps], uint32_t* s_mr, const void* const* s_cand, Ring g,
                                          int warp, int lane) {
#pragma unroll 1
    for (uint64_t t = t_begin; t < t_end; ++t) fast_tile<DT>(ref, K, t, atol, rtol, s_acc, s_mr, s_cand, g, warp, lane);
    return ring_pack(g);
}

template <int DT>
__device__ __forceinline__ void run_set(const SetRec& S, const Span& sp, float atol, float rtol, Acc (*s_acc)[kWarps],
                                        uint32_t* s_mr, const void* const* s_cand, Ring& g, int warp, int lane) {
    using E = Elem<DT>;
    if (!S.vec_ok) {
        for (uint64_t t = sp.t0; t < sp.t1; ++t) slow_tile<DT>(S, t, atol, rtol, s_acc, s_cand, warp, lane);
        return;
    }
    const uint64_t t_full = sp.t1 < sp.full_tiles ? sp.t1 : sp.full_tiles;
    if (sp.t0 < t_full)
        ring_unpack(g, fast_run<DT>(S.ref, static_cast<int>(S.k), sp.t0, t_full, atol, rtol, s_acc, s_mr, s_cand, g, warp, lane));
    if (sp.t1 > sp.full_tiles) {        // the ragged last tile is in this CTA's range
        if (sp.tail_vecs && !g.dead) ring_unpack(g, tail_tile<DT>(S.k, sp.tail_vecs, atol, rtol, s_acc, g, warp, lane));
        if (sp.left && !g.dead)
            leftover_pass<DT>(S, sp.full_tiles * kTileElems + static_cast<uint64_t>(sp.tail_vecs) * E::kPerVec, sp.left,
                              atol, rtol, s_acc, s_cand, warp, lane);
    }
}

// ---- producer ----------------------------------------------------------------------------
// One warp walks the CTA's range ahead of the consumers and fills the ring: per tile the
// reference, then each member.  Lane k keeps member k's base address; lane 0 waits for the
// stage to be free, arms its barrier with the byte count and issues the copy.
// Returns how many copies were issued.
__device__ __forceinline__ uint32_t producer_loop(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members,
                                                  const CtaRange& rg, Ring& g, int lane) {
    const unsigned full = 0xffffffffu;
    const unsigned long long pol = policy_evict_first();
    uint32_t issued = 0;
    for (uint32_t s = rg.s_begin; s <= rg.s_end && !g.dead; ++s) {
        const SetRec S = sets[s];
        const Span sp = set_span(rg, s, S);
        const uint64_t ring_end = sp.full_tiles + (sp.tail_vecs ? 1 : 0);     // tiles [0, ring_end) use the ring
        const uint64_t t0 = sp.t0, t1 = sp.t1 < ring_end ? sp.t1 : ring_end;
        if (t0 >= t1) continue;
        const uint32_t full_bytes = kTileElems * (S.dtype == EVO_F32 ? 4u : 2u);
        const unsigned long long mine = (static_cast<uint32_t>(lane) < S.k)
            ? reinterpret_cast<unsigned long long>(members[S.member_off + lane].cand) : 0ull;
        const unsigned long long ref = reinterpret_cast<unsigned long long>(S.ref);
        for (uint64_t t = t0; t < t1 && !g.dead; ++t) {
            const unsigned long long off = t * full_bytes;
            const uint32_t tile_bytes = t < sp.full_tiles ? full_bytes : sp.tail_vecs * 16u;
            for (uint32_t j = 0; j <= S.k; ++j) {
                const unsigned long long base = __shfl_sync(full, mine, j == 0 ? 0 : static_cast<int>(j - 1));
                const unsigned long long src = (j == 0 ? ref : base) + off;
                int ok = 1;
                if (lane == 0) {
                    ok = mbar_wait(g.empty(), g.phase ^ 1u, g.abort_flag) ? 1 : 0;
                    if (ok) {
                        mbar_arrive_expect_tx(g.full(), tile_bytes);
                        bulk_load(g.data(), reinterpret_cast<const void*>(src), tile_bytes, g.full(), pol);
                    }
                }
                ok = __shfl_sync(full, ok, 0);
                if (!ok) { g.dead = true; break; }
                g.advance();
                ++issued;
            }
        }
    }
    return issued;
}

// The body of the first pass.  kOnly16: the population holds fp16/bf16 tensors only; the fp32 path (more
// registers, 16 KiB stages) is then left out, which lets a third CTA share the SM (see validate_pass1_16bit).
template <bool kOnly16>
__device__ __forceinline__ void pass1_body(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members,
               const CtaRange* __restrict__ ranges, Acc* __restrict__ partials, float atol, float rtol,
               uint32_t* __restrict__ status, const uint32_t* __restrict__ seeds /* optional: see seed_kernel */,
               unsigned long long* __restrict__ cta_times /* optional: %globaltimer at start and end of every CTA */) {
    extern __shared__ __align__(128) unsigned char s_ring[];
    __shared__ Acc s_acc[kMaxK][kWarps];
    __shared__ const void* s_cand[kMaxK];
    __shared__ uint32_t s_mr[kMaxK];         // per member: running maximum of d/|r| found on the fast path (bit pattern)
    __shared__ __align__(8) unsigned long long s_full[kStages], s_empty[kStages];
    __shared__ int s_abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(smem_u32(&s_full[i]), 1);          // the producer's arrive + the copy's bytes
            mbar_init(smem_u32(&s_empty[i]), kWarps);    // one arrive per consumer warp
        }
        s_abort = 0;
        mbar_fence_init();
    }
    __syncthreads();
    // Up to here nothing depended on earlier work in the stream; the plan, the seeds and the tensors do.
    if (!kOnly16) grid_dependents_may_launch();
    grid_dependency_wait();
    if (cta_times && threadIdx.x == 0) cta_times[2 * blockIdx.x] = global_ns();
    const CtaRange rg = ranges[blockIdx.x];
    Ring g;
    g.full0 = smem_u32(&s_full[0]);
    g.empty0 = smem_u32(&s_empty[0]);
    g.data0 = smem_u32(s_ring);
    g.stage_bytes = kOnly16 ? kStageBytes / 2 : kStageBytes;
    g.abort_flag = &s_abort;
    uint32_t issued = 0;

    if (warp == kWarps) {
        issued = producer_loop(sets, members, rg, g, lane);
    } else {
        for (uint32_t s = rg.s_begin; s <= rg.s_end; ++s) {
            const SetRec S = sets[s];
            const Span sp = set_span(rg, s, S);
            if (sp.t0 >= sp.t1) continue;
            for (uint32_t i = threadIdx.x; i < S.k * kWarps; i += kThreads) {
                Acc z;
                z.mism = 0; z.nonfin = 0; z.sse = 0.0; z.max_abs = 0; z.max_rel = 0; z.flags = 0; z.pad = 0;
                s_acc[i / kWarps][i % kWarps] = z;
            }
            if (threadIdx.x < S.k) {
                s_cand[threadIdx.x] = members[S.member_off + threadIdx.x].cand;
                s_mr[threadIdx.x] = seeds ? seeds[S.member_off + threadIdx.x] : 0u;
            }
            consumer_bar();
            if (!kOnly16 && S.dtype == EVO_F32) run_set<EVO_F32>(S, sp, atol, rtol, s_acc, s_mr, s_cand, g, warp, lane);
            else if (S.dtype == EVO_F16) run_set<EVO_F16>(S, sp, atol, rtol, s_acc, s_mr, s_cand, g, warp, lane);
            else run_set<EVO_BF16>(S, sp, atol, rtol, s_acc, s_mr, s_cand, g, warp, lane);
            consumer_bar();
            if (threadIdx.x < S.k) {
                Acc a = s_acc[threadIdx.x][0];
#pragma unroll
                for (int w = 1; w < kWarps; ++w) {
                    const Acc b = s_acc[threadIdx.x][w];
                    a.mism += b.mism; a.nonfin += b.nonfin; a.sse += b.sse;
                    a.max_abs = max(a.max_abs, b.max_abs); a.max_rel = max(a.max_rel, b.max_rel); a.flags |= b.flags;
                }
                a.max_rel = max(a.max_rel, s_mr[threadIdx.x]);
                partials[rg.part_base + (S.member_off - rg.first_member) + threadIdx.x] = a;
            }
            consumer_bar();
        }
    }
    // With three CTAs per SM the register file is full: kernels that start early would only take the places of
    // this kernel's own CTAs and wait there (measured: 20 us lost per call on 128 x 2 MiB); they may start once
    // this CTA's work is done.
    if (kOnly16) grid_dependents_may_launch();
    __syncthreads();
    if (s_abort) {
        // A wait ran out.  Before the CTA gives its shared memory back, let the copies that
        // are still outstanding land (bounded again), then report.
        if (warp == kWarps && lane == 0) {
            const uint32_t pending = issued < kStages ? issued : kStages;
            for (uint32_t q = 0; q < pending; ++q) {
                const uint32_t i = issued - 1 - q;
                const uint32_t bar = g.full0 + 8u * (i % kStages);
                const uint32_t parity = (i / kStages) & 1u;
                const unsigned long long t0 = global_ns();
                while (!mbar_try_wait(bar, parity) && global_ns() - t0 < kWaitLimitNs) {}
            }
        }
        if (threadIdx.x == 0) atomicOr(status, 1u);
    }
    if (cta_times && threadIdx.x == 0) cta_times[2 * blockIdx.x + 1] = global_ns();
}

__global__ void __launch_bounds__(kBlock, kCtasPerSm)
validate_pass1(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members,
               const CtaRange* __restrict__ ranges, Acc* __restrict__ partials, float atol, float rtol,
               uint32_t* __restrict__ status, const uint32_t* __restrict__ seeds, unsigned long long* __restrict__ cta_times) {
    pass1_body<false>(sets, members, ranges, partials, atol, rtol, status, seeds, cta_times);
}

// The same pass for populations without fp32 tensors.  16-bit tiles are 8 KiB, so the ring is half as large, and
// the 16-bit path needs fewer registers: three CTAs (27 warps) share an SM instead of two, which is what a pass
// bound by instruction issue rather than by memory (two bytes per element for the same arithmetic) can use.
__global__ void __launch_bounds__(kBlock, kCtasPerSm16)
validate_pass1_16bit(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members,
                     const CtaRange* __restrict__ ranges, Acc* __restrict__ partials, float atol, float rtol,
                     uint32_t* __restrict__ status, const uint32_t* __restrict__ seeds, unsigned long long* __restrict__ cta_times) {
    pass1_body<true>(sets, members, ranges, partials, atol, rtol, status, seeds, cta_times);
}

// Warm start for the filter of max d/|r|.  A CTA that begins a run knows no maximum for its
// members yet, so on its first tile every lane's filter fires and the exact handling runs for
// the whole tile; with short runs (a few tiles per CTA and member) that is a large share of the
// work.  This small kernel, run before the first pass when runs are short, takes the exact
// maximum quotient over the first tile of every member (one CTA per member, a division per
// element) and the first pass starts every run from it.  The seed is a true quotient of that
// member, so folding it into the result changes nothing: the maximum is the maximum.
__global__ void __launch_bounds__(kThreads)
seed_kernel(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members, uint32_t* __restrict__ seeds) {
    __shared__ uint32_t s_max[kWarps];
    grid_dependents_may_launch();
    grid_dependency_wait();
    const MemberRec M = members[blockIdx.x];
    const SetRec S = sets[M.set];
    const uint32_t n = static_cast<uint32_t>(S.n < static_cast<uint64_t>(kTileElems) ? S.n : static_cast<uint64_t>(kTileElems));
    // all 16 element pairs of the thread are loaded before any is used: one round of memory latency, not sixteen
    float c[kEpt], r[kEpt];
#pragma unroll
    for (int j = 0; j < kEpt; ++j) {
        const uint32_t e = threadIdx.x + j * kThreads;
        c[j] = 0.f; r[j] = 0.f;
        if (e < n) {
            if (S.dtype == EVO_F32) { c[j] = static_cast<const float*>(M.cand)[e]; r[j] = static_cast<const float*>(S.ref)[e]; }
            else if (S.dtype == EVO_F16) { c[j] = __half2float(static_cast<const __half*>(M.cand)[e]); r[j] = __half2float(static_cast<const __half*>(S.ref)[e]); }
            else { c[j] = __bfloat162float(static_cast<const __nv_bfloat16*>(M.cand)[e]); r[j] = __bfloat162float(static_cast<const __nv_bfloat16*>(S.ref)[e]); }
        }
    }
    float best = 0.f;
#pragma unroll
    for (int j = 0; j < kEpt; ++j) {
        const float d = fabsf(__fsub_rn(c[j], r[j])), ar = fabsf(r[j]);
        const bool usable = d > 0.f && ar > 0.f && d < kInf && ar < kInf && fabsf(c[j]) < kInf;   // as the statistics: finite pairs, r != 0
        if (usable) best = fmaxf(best, __fdiv_rn(d, ar));
    }
    const uint32_t w = __reduce_max_sync(0xffffffffu, __float_as_uint(best));
    if ((threadIdx.x & 31) == 0) s_max[threadIdx.x >> 5] = w;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t m = 0;
        for (int i = 0; i < kWarps; ++i) m = max(m, s_max[i]);
        seeds[blockIdx.x] = m;
    }
}

// One warp per tensor: fold the partial records of the CTAs [cta_first, cta_last] in a
// fixed order (lane-strided, then a xor tree).  If the first pass gave up on a wait, the
// records are incomplete: every result then says so instead of carrying numbers.
// `fused` (a single CTA holds every tensor: small populations) also takes the candidate
// verdicts afterwards, which saves a launch where launches are all the time there is.
struct VerdictArgs { const uint32_t* offsets; const uint32_t* desc_of; uint32_t n_group; uint32_t* group_pass; };

__device__ __forceinline__ void fold_partials(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members,
                                              const CtaRange* __restrict__ ranges, const Acc* __restrict__ partials,
                                              uint32_t m, int lane, evo_result* __restrict__ results,
                                              const uint32_t* __restrict__ status);

__global__ void __launch_bounds__(1024)
validate_pass2(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members,
               const CtaRange* __restrict__ ranges, const Acc* __restrict__ partials,
               uint32_t n_members, evo_result* __restrict__ results, const uint32_t* __restrict__ status,
               bool fused, VerdictArgs va) {
    grid_dependents_may_launch();
    grid_dependency_wait();
    const uint32_t m = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (m < n_members) fold_partials(sets, members, ranges, partials, m, threadIdx.x & 31, results, status);
    if (!fused) return;
    __syncthreads();              // the CTA's own writes to results[] are visible to it from here on
    for (uint32_t g = threadIdx.x; g < va.n_group; g += blockDim.x) {
        uint32_t ok = 1;
        for (uint32_t i = va.offsets[g]; i < va.offsets[g + 1]; ++i) ok &= results[va.desc_of[i]].pass;
        va.group_pass[g] = ok;
    }
}

__device__ __forceinline__ void fold_partials(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members,
                                              const CtaRange* __restrict__ ranges, const Acc* __restrict__ partials,
                                              uint32_t m, int lane, evo_result* __restrict__ results,
                                              const uint32_t* __restrict__ status) {
    const MemberRec M = members[m];
    if (*status != 0) {
        if (lane == 0) {
            evo_result r;
            r.n_mismatch = 0; r.n_nonfinite = 0; r.sse = 0.0; r.max_abs = 0.f; r.max_rel = 0.f;
            r.flags = EVO_FLAG_INCOMPLETE; r.pass = 0;
            results[M.desc] = r;
        }
        return;
    }
    const SetRec S = sets[M.set];
    unsigned long long mism = 0, nonfin = 0;
    double sse = 0.0;
    uint32_t ma = 0, mr = 0, fl = 0;
    if (S.cta_first <= S.cta_last) {
        for (uint32_t b = S.cta_first + lane; b <= S.cta_last; b += 32) {
            const CtaRange R = ranges[b];
            const Acc p = partials[R.part_base + (m - R.first_member)];
            mism += p.mism; nonfin += p.nonfin; sse += p.sse;
            ma = max(ma, p.max_abs); mr = max(mr, p.max_rel); fl |= p.flags;
        }
    }
    const unsigned full = 0xffffffffu;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        mism += __shfl_xor_sync(full, mism, o);
        nonfin += __shfl_xor_sync(full, nonfin, o);
        sse += __shfl_xor_sync(full, sse, o);
    }
    ma = __reduce_max_sync(full, ma);
    mr = __reduce_max_sync(full, mr);
    fl = __reduce_or_sync(full, fl);
    if (lane == 0) {
        evo_result r;
        r.n_mismatch = mism; r.n_nonfinite = nonfin; r.sse = sse;
        r.max_abs = __uint_as_float(ma); r.max_rel = __uint_as_float(mr);
        r.flags = fl; r.pass = mism == 0 ? 1u : 0u;
        results[M.desc] = r;
    }
}

// Candidate verdicts: AND over the tensors of each candidate id.
__global__ void group_verdict(const uint32_t* __restrict__ offsets, const uint32_t* __restrict__ desc_of,
                              const evo_result* __restrict__ results, uint32_t n_group, uint32_t* __restrict__ group_pass) {
    grid_dependents_may_launch();
    grid_dependency_wait();
    const uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= n_group) return;
    uint32_t ok = 1;
    for (uint32_t i = offsets[g]; i < offsets[g + 1]; ++i) ok &= results[desc_of[i]].pass;
    group_pass[g] = ok;
}

// Small plans travel as kernel arguments: this kernel writes one chunk of a packed plan to its
// place in device memory.  No staging buffer on the host, no copy engine, nothing the host has
// to wait for before it may build the next plan; the launch itself carries the bytes.
constexpr uint32_t kPlanChunkBytes = 16 * 1024;
struct PlanChunk { uint4 w[kPlanChunkBytes / 16]; };
__global__ void __launch_bounds__(256)
plan_store(const __grid_constant__ PlanChunk chunk, uint4* __restrict__ dst, uint32_t n_vec, uint32_t* __restrict__ clear_word) {
    grid_dependents_may_launch();
    grid_dependency_wait();
    for (uint32_t i = threadIdx.x; i < n_vec; i += blockDim.x) dst[i] = chunk.w[i];
    if (clear_word && threadIdx.x == 0) *clear_word = 0u;
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing will ever complete,
// through the same wait routine as the first pass, with a short limit; it must come back,
// raise the status word and leave the context usable.
__global__ void wait_selftest_kernel(unsigned long long limit_ns, uint32_t* __restrict__ status) {
    __shared__ __align__(8) unsigned long long s_bar;
    __shared__ int s_abort;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&s_bar), 1);
        s_abort = 0;
        mbar_fence_init();
    }
    __syncthreads();
    const bool ok = mbar_wait(smem_u32(&s_bar), 0, &s_abort, limit_ns);
    const bool all_ok = __all_sync(0xffffffffu, ok);
    __syncthreads();
    if (threadIdx.x == 0 && (!all_ok || s_abort)) atomicOr(status, 2u);
}

// ---- host side ------------------------------------------------------------------------

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Where the parts of a packed plan sit, as byte offsets from the start of the plan area.
struct PlanLayout { size_t o_sets, o_members, o_ranges, o_goff, o_gdesc, bytes; };

PlanLayout layout_of(const Plan& plan, size_t first) {
    PlanLayout L;
    L.o_sets = first;
    L.o_members = align_up(L.o_sets + plan.sets.size() * sizeof(SetRec), 256);
    L.o_ranges = align_up(L.o_members + plan.members.size() * sizeof(MemberRec), 256);
    L.o_goff = align_up(L.o_ranges + plan.ranges.size() * sizeof(CtaRange), 256);
    L.o_gdesc = align_up(L.o_goff + plan.group_off.size() * 4, 256);
    L.bytes = align_up(L.o_gdesc + plan.group_desc.size() * 4, 256);
    return L;
}

// Packs the plan into `dst`, whose first byte stands for offset `first` of the layout.
void pack_plan(const Plan& plan, const PlanLayout& L, size_t first, unsigned char* dst) {
    auto put = [&](size_t o, const void* src, size_t bytes) { if (bytes) std::memcpy(dst + (o - first), src, bytes); };
    put(L.o_sets, plan.sets.data(), plan.sets.size() * sizeof(SetRec));
    put(L.o_members, plan.members.data(), plan.members.size() * sizeof(MemberRec));
    put(L.o_ranges, plan.ranges.data(), plan.ranges.size() * sizeof(CtaRange));
    put(L.o_goff, plan.group_off.data(), plan.group_off.size() * 4);
    put(L.o_gdesc, plan.group_desc.data(), plan.group_desc.size() * 4);
}

// `bytes` of a packed plan from host memory to `dst` on the device as the arguments of one
// plan_store launch per chunk (16-byte granules; dst is 16-byte aligned).  The first chunk may
// also clear a word (the status word of a caller that has no other moment to do so).
cudaError_t store_plan(const unsigned char* src, size_t bytes, unsigned char* dst, uint32_t* clear_word, bool pdl,
                       cudaStream_t stream, uint64_t* launches) {
    PlanChunk chunk;
    size_t done = 0;
    do {
        const size_t piece = std::min<size_t>(bytes - done, kPlanChunkBytes);
        if (piece) std::memcpy(chunk.w, src + done, piece);
        const uint32_t n_vec = static_cast<uint32_t>((piece + 15) / 16);
        const cudaError_t e = evo::launch(plan_store, dim3(1), dim3(256), 0, stream, pdl, chunk,
                                          reinterpret_cast<uint4*>(dst + done), n_vec, done == 0 ? clear_word : nullptr);
        if (e != cudaSuccess) return e;
        if (launches) *launches += 1;
        done += piece;
    } while (done < bytes);
    return cudaSuccess;
}

// Everything a call launches once its plan is in device memory: seed pass (optional), first
// pass, second pass, verdicts.  Shared by the context-based and the allocation-free entry points.
struct ChainArgs {
    const unsigned char* d_plan;      // device address of layout offset 0
    PlanLayout L;
    Acc* d_parts;
    uint32_t* d_status;
    uint32_t* d_seeds;                // nullptr: no seed pass
    unsigned long long* d_cta_times;  // nullptr: no per-CTA clock readings
    float atol, rtol;
    evo_result* results;
    uint32_t* group_pass;
    uint64_t n_group;
    bool pdl;
    bool only16;                      // no fp32 tensor in the population: the three-CTAs-per-SM kernel
    cudaEvent_t ev_start, ev_stop;    // optional: around the first pass
};

cudaError_t launch_chain(uint32_t n_members, uint32_t n_ctas, const ChainArgs& a, cudaStream_t stream, uint64_t* launches) {
    const SetRec* d_sets = reinterpret_cast<const SetRec*>(a.d_plan + a.L.o_sets);
    const MemberRec* d_members = reinterpret_cast<const MemberRec*>(a.d_plan + a.L.o_members);
    const CtaRange* d_ranges = reinterpret_cast<const CtaRange*>(a.d_plan + a.L.o_ranges);
    const uint32_t* d_goff = reinterpret_cast<const uint32_t*>(a.d_plan + a.L.o_goff);
    const uint32_t* d_gdesc = reinterpret_cast<const uint32_t*>(a.d_plan + a.L.o_gdesc);
    cudaError_t e;
    auto count = [&]() { if (launches) *launches += 1; };
    if (a.d_seeds && n_members > 0) {
        e = evo::launch(seed_kernel, dim3(n_members), dim3(kThreads), 0, stream, a.pdl, d_sets, d_members, a.d_seeds);
        if (e != cudaSuccess) return e;
        count();
    }
    if (a.ev_start && (e = cudaEventRecord(a.ev_start, stream)) != cudaSuccess) return e;
    if (n_ctas > 0) {
        e = evo::launch(a.only16 ? validate_pass1_16bit : validate_pass1, dim3(n_ctas), dim3(kBlock),
                        a.only16 ? kRingBytes / 2 : kRingBytes, stream, a.pdl, d_sets, d_members, d_ranges,
                        a.d_parts, a.atol, a.rtol, a.d_status, static_cast<const uint32_t*>(a.d_seeds && n_members ? a.d_seeds : nullptr),
                        a.d_cta_times);
        if (e != cudaSuccess) return e;
        count();
    }
    if (a.ev_stop && (e = cudaEventRecord(a.ev_stop, stream)) != cudaSuccess) return e;
    // Up to 32 tensors: one CTA, one warp per tensor, takes the second pass and then the verdicts.
    const bool fused = a.group_pass != nullptr && n_members <= 32;
    VerdictArgs va{d_goff, d_gdesc, static_cast<uint32_t>(a.n_group), a.group_pass};
    if (n_members > 0 || fused) {
        const uint32_t block = fused ? std::max<uint32_t>(32u, 32u * n_members) : static_cast<uint32_t>(kThreads);
        const uint32_t grid = fused ? 1u : (n_members + kWarps - 1) / kWarps;
        e = evo::launch(validate_pass2, dim3(grid), dim3(block), 0, stream, a.pdl, d_sets, d_members, d_ranges,
                        static_cast<const Acc*>(a.d_parts), n_members, a.results, static_cast<const uint32_t*>(a.d_status), fused, va);
        if (e != cudaSuccess) return e;
        count();
    }
    if (a.group_pass && !fused) {
        e = evo::launch(group_verdict, dim3(static_cast<unsigned>((a.n_group + 255) / 256)), dim3(256), 0, stream, a.pdl, d_goff,
                        d_gdesc, static_cast<const evo_result*>(a.results), static_cast<uint32_t>(a.n_group), a.group_pass);
        if (e != cudaSuccess) return e;
        count();
    }
    return cudaSuccess;
}

constexpr size_t kPlanAsArgumentsLimit = 2 * kPlanChunkBytes;      // larger plans go up with a copy from pinned memory

// Byte image of everything the plan depends on.
void plan_key_of(const void* const* cand_ptrs, const void* ref_ptr, const evo_desc* descs, uint64_t n_desc, int dtype,
                 bool want_groups, uint64_t n_group, uint32_t max_ctas, cudaStream_t stream, std::vector<unsigned char>* key) {
    // (the stream is part of it: the upload is ordered on the stream of the call that made it)
    struct Head { const void* ref; const void* stream; uint64_t n_desc, n_group; int32_t dtype; uint32_t max_ctas; uint32_t groups; uint32_t pad; } head;
    std::memset(&head, 0, sizeof head);
    head.ref = ref_ptr; head.stream = stream; head.n_desc = n_desc; head.n_group = n_group; head.dtype = dtype; head.max_ctas = max_ctas;
    head.groups = want_groups ? 1u : 0u;
    key->resize(sizeof head + n_desc * (sizeof(void*) + sizeof(evo_desc)));
    unsigned char* p = key->data();
    std::memcpy(p, &head, sizeof head);
    if (n_desc) {
        std::memcpy(p + sizeof head, cand_ptrs, n_desc * sizeof(void*));
        std::memcpy(p + sizeof head + n_desc * sizeof(void*), descs, n_desc * sizeof(evo_desc));
    }
}

int validate_device(evo_ctx* ctx, const void* const* cand_ptrs, const void* ref_ptr, const evo_desc* descs,
                    uint64_t n_desc, int dtype, float atol, float rtol, evo_result* results,
                    uint32_t* group_pass, uint64_t n_group, cudaStream_t stream, const char* who) {
    // the one-shot timing request belongs to this call, whether it succeeds or not
    const cudaEvent_t ev_start = ctx->time_start, ev_stop = ctx->time_stop;
    ctx->time_start = ctx->time_stop = nullptr;
    if (n_desc > 0 && !results) return evo::fail(ctx, EVO_ERR_ARG, "%s: results must not be NULL", who);
    if (!(atol >= 0.f) || !(rtol >= 0.f) || std::isinf(atol) || std::isinf(rtol))
        return evo::fail(ctx, EVO_ERR_ARG, "%s: atol and rtol must be finite and >= 0", who);
    if (n_desc > 0 && (!cand_ptrs || !descs)) return evo::fail(ctx, EVO_ERR_ARG, "%s: cand_ptrs and descs must not be NULL", who);
    bool only16 = n_desc > 0;
    for (uint64_t i = 0; i < n_desc && only16; ++i) {
        const int dt = descs[i].dtype == -1 ? dtype : descs[i].dtype;
        only16 = dt == EVO_F16 || dt == EVO_BF16;
    }
    const uint32_t max_ctas = static_cast<uint32_t>(ctx->sm_count) * (only16 ? kCtasPerSm16 : kCtasPerSm);

    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");

    // The same tensors as in the call before (an evaluation loop that reuses its buffers): the plan that is
    // already in device memory stands, only the kernels are launched again.
    std::vector<unsigned char>& key = ctx->plan_scratch_key;
    plan_key_of(cand_ptrs, ref_ptr, descs, n_desc, dtype, group_pass != nullptr, n_group, max_ctas, stream, &key);
    const bool hit = ctx->plan_key_valid && key.size() == ctx->plan_key.size() &&
                     std::memcmp(key.data(), ctx->plan_key.data(), key.size()) == 0;
    PlanLayout L;
    uint32_t n_members, n_ctas;
    bool seed;
    if (hit) {
        L = PlanLayout{ctx->plan_layout[0], ctx->plan_layout[1], ctx->plan_layout[2], ctx->plan_layout[3], ctx->plan_layout[4],
                       ctx->plan_layout[5]};
        n_members = ctx->plan_n_members; n_ctas = ctx->plan_n_ctas; seed = ctx->plan_seed;
    } else {
        Plan plan;
        std::string err;
        int st = build_plan(cand_ptrs, ref_ptr, descs, n_desc, dtype, atol, rtol, group_pass != nullptr, n_group, max_ctas,
                            &plan, &err);
        if (st != EVO_OK) return evo::fail(ctx, st, "%s: %s", who, err.c_str());
        ctx->plan_key_valid = false;
        L = layout_of(plan, 0);
        n_members = static_cast<uint32_t>(plan.members.size());
        n_ctas = static_cast<uint32_t>(plan.ranges.size());
        st = evo::reserve_device(ctx, &ctx->d_plan, &ctx->d_plan_bytes, L.bytes + 256);
        if (st != EVO_OK) return st;
        st = evo::reserve_device(ctx, &ctx->d_partials, &ctx->d_partials_bytes, std::max<size_t>(plan.n_parts, 1) * sizeof(Acc));
        if (st != EVO_OK) return st;
        // Short runs (few tiles per CTA and member): seed the filter of max d/|r| first, see seed_kernel.
        // (Not for populations with fewer tiles than CTAs: those are bound by launch latency, which a further
        // kernel only adds to.)
        seed = plan.total_tiles >= max_ctas && plan.total_tiles / max_ctas < kSeedBelowTilesPerCta && n_desc > 0;
        if (seed) {
            st = evo::reserve_device(ctx, &ctx->d_seeds, &ctx->d_seeds_bytes, n_desc * sizeof(uint32_t));
            if (st != EVO_OK) return st;
        }
        // ---- the plan goes up: as kernel arguments when it is small, else with a copy from pinned memory ----
        if (L.bytes <= kPlanAsArgumentsLimit) {
            std::vector<unsigned char> h(L.bytes);
            pack_plan(plan, L, 0, h.data());
            cudaError_t e = store_plan(h.data(), L.bytes, static_cast<unsigned char*>(ctx->d_plan), nullptr, ctx->pdl, stream, &ctx->launches);
            if (e != cudaSuccess) return evo::fail_cuda(ctx, e, "plan_store launch");
        } else {
            st = evo::reserve_pinned(ctx, &ctx->h_plan, &ctx->h_plan_bytes, L.bytes);
            if (st != EVO_OK) return st;
            if (ctx->plan_in_flight) {
                // the pinned staging block is about to be overwritten: the previous upload must have been read
                EVO_CUDA_TRY(ctx, cudaEventSynchronize(ctx->plan_consumed));
                ctx->plan_in_flight = false;
            }
            pack_plan(plan, L, 0, static_cast<unsigned char*>(ctx->h_plan));
            EVO_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_plan, ctx->h_plan, L.bytes, cudaMemcpyHostToDevice, stream));
            EVO_CUDA_TRY(ctx, cudaEventRecord(ctx->plan_consumed, stream));
            ctx->plan_in_flight = true;
        }
        ctx->plan_key.swap(key);
        ctx->plan_layout[0] = L.o_sets; ctx->plan_layout[1] = L.o_members; ctx->plan_layout[2] = L.o_ranges;
        ctx->plan_layout[3] = L.o_goff; ctx->plan_layout[4] = L.o_gdesc; ctx->plan_layout[5] = L.bytes;
        ctx->plan_n_members = n_members; ctx->plan_n_ctas = n_ctas; ctx->plan_seed = seed;
        ctx->plan_key_valid = true;
    }
    if (ctx->cta_timing) {
        const int st = evo::reserve_device(ctx, &ctx->d_cta_times, &ctx->d_cta_times_bytes, std::max<size_t>(max_ctas, 1) * 16);
        if (st != EVO_OK) return st;
        ctx->cta_times_n = n_ctas;
    }

    if (n_ctas > 0 && !ctx->pass1_ready) {
        EVO_CUDA_TRY(ctx, cudaFuncSetAttribute(validate_pass1, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               static_cast<int>(kRingBytes)));
        EVO_CUDA_TRY(ctx, cudaFuncSetAttribute(validate_pass1_16bit, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               static_cast<int>(kRingBytes / 2)));
        ctx->pass1_ready = true;
    }
    ChainArgs a{};
    a.d_plan = static_cast<const unsigned char*>(ctx->d_plan);
    a.L = L;
    a.d_parts = static_cast<Acc*>(ctx->d_partials);
    a.d_status = evo::status_word(ctx);
    a.d_seeds = seed ? static_cast<uint32_t*>(ctx->d_seeds) : nullptr;
    a.d_cta_times = ctx->cta_timing ? static_cast<unsigned long long*>(ctx->d_cta_times) : nullptr;
    a.atol = atol; a.rtol = rtol;
    a.results = results; a.group_pass = group_pass; a.n_group = n_group;
    a.pdl = ctx->pdl;
    a.only16 = only16;
    a.ev_start = ev_start; a.ev_stop = ev_stop;
    const cudaError_t e = launch_chain(n_members, n_ctas, a, stream, &ctx->launches);
    if (e != cudaSuccess) return evo::fail_cuda(ctx, e, "kernel launch");
    return EVO_OK;
}

}  // namespace

extern "C" int evo_validate(evo_ctx* ctx, const void* const* cand_ptrs, const void* ref_ptr, const evo_desc* descs,
                            uint64_t n_desc, int dtype, float atol, float rtol, evo_result* results,
                            uint32_t* group_pass, uint64_t n_group, void* stream) {
    if (!ctx) return EVO_ERR_ARG;
    return validate_device(ctx, cand_ptrs, ref_ptr, descs, n_desc, dtype, atol, rtol, results, group_pass, n_group,
                           static_cast<cudaStream_t>(stream), "evo_validate");
}

extern "C" int evo_validate_host(evo_ctx* ctx, const void* const* cand_ptrs, const void* ref_ptr, const evo_desc* descs,
                                 uint64_t n_desc, int dtype, float atol, float rtol, evo_result* results,
                                 uint32_t* group_pass, uint64_t n_group, void* stream_) {
    if (!ctx) return EVO_ERR_ARG;
    const char* who = "evo_validate_host";
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (n_desc > 0 && (!cand_ptrs || !descs || !results))
        return evo::fail(ctx, EVO_ERR_ARG, "%s: cand_ptrs, descs and results must not be NULL", who);
    if ((group_pass == nullptr) != (n_group == 0))
        return evo::fail(ctx, EVO_ERR_ARG, "%s: group_pass and n_group must be given together", who);
    // Lay the tensors out in the staging area: every candidate, each distinct reference once,
    // then the results and the verdict words.
    struct Copy { const void* src; size_t dst_off; size_t bytes; };
    std::vector<Copy> copies;
    std::vector<size_t> cand_off(n_desc), ref_off(n_desc);
    std::unordered_map<const void*, std::pair<size_t, size_t>> ref_slot;      // host ref -> (offset, bytes staged)
    size_t total = 0;
    for (uint64_t i = 0; i < n_desc; ++i) {
        const evo_desc& d = descs[i];
        const int dt = d.dtype == -1 ? dtype : d.dtype;
        if (dt != EVO_F32 && dt != EVO_F16 && dt != EVO_BF16)
            return evo::fail(ctx, EVO_ERR_DTYPE, "%s: descriptor %llu has dtype %d", who, (unsigned long long)i, dt);
        if (d.n > (1ull << 60)) return evo::fail(ctx, EVO_ERR_ARG, "%s: descriptor %llu too large", who, (unsigned long long)i);
        const size_t bytes = d.n * evo::elem_bytes(dt);
        const void* ref = d.ref ? d.ref : ref_ptr;
        if (d.n > 0 && (!ref || !cand_ptrs[i]))
            return evo::fail(ctx, EVO_ERR_ARG, "%s: descriptor %llu has a NULL tensor", who, (unsigned long long)i);
        cand_off[i] = total;
        if (bytes) copies.push_back({cand_ptrs[i], total, bytes});
        total = align_up(total + bytes, 256);
        auto it = ref_slot.find(ref);
        if (it == ref_slot.end() || it->second.second < bytes) {
            // first use of this reference, or a longer prefix of it than staged so far
            ref_slot[ref] = {total, bytes};
            ref_off[i] = total;
            if (bytes) copies.push_back({ref, total, bytes});
            total = align_up(total + bytes, 256);
        } else {
            ref_off[i] = it->second.first;
        }
    }
    const size_t o_results = total;
    total = align_up(total + n_desc * sizeof(evo_result), 256);
    const size_t o_gpass = total;
    total = align_up(total + n_group * sizeof(uint32_t), 256);

    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");
    int st = evo::reserve_device(ctx, &ctx->d_stage, &ctx->d_stage_bytes, std::max<size_t>(total, 256));
    if (st != EVO_OK) return st;
    char* base = static_cast<char*>(ctx->d_stage);
    for (const Copy& c : copies)
        EVO_CUDA_TRY(ctx, cudaMemcpyAsync(base + c.dst_off, c.src, c.bytes, cudaMemcpyHostToDevice, stream));
    std::vector<const void*> d_cands(n_desc);
    std::vector<evo_desc> d_descs(descs, descs + n_desc);
    for (uint64_t i = 0; i < n_desc; ++i) {
        d_cands[i] = base + cand_off[i];
        d_descs[i].ref = base + ref_off[i];
    }
    evo_result* d_results = reinterpret_cast<evo_result*>(base + o_results);
    uint32_t* d_gpass = group_pass ? reinterpret_cast<uint32_t*>(base + o_gpass) : nullptr;
    st = validate_device(ctx, d_cands.data(), nullptr, d_descs.data(), n_desc, dtype, atol, rtol, d_results, d_gpass,
                         n_group, stream, who);
    if (st != EVO_OK) return st;
    if (n_desc) EVO_CUDA_TRY(ctx, cudaMemcpyAsync(results, d_results, n_desc * sizeof(evo_result), cudaMemcpyDeviceToHost, stream));
    if (group_pass) EVO_CUDA_TRY(ctx, cudaMemcpyAsync(group_pass, d_gpass, n_group * sizeof(uint32_t), cudaMemcpyDeviceToHost, stream));
    return evo::sync_and_check(ctx, stream, who);
}

extern "C" int evo_selftest_wait(evo_ctx* ctx, uint32_t limit_us, void* stream) {
    if (!ctx) return EVO_ERR_ARG;
    if (limit_us == 0 || limit_us > 1000000u) return evo::fail(ctx, EVO_ERR_ARG, "evo_selftest_wait: limit must be 1..1000000 us");
    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");
    wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(1000ull * limit_us, evo::status_word(ctx));
    ctx->launches += 1;
    EVO_CUDA_TRY(ctx, cudaGetLastError());
    return EVO_OK;
}

// ---- evo_validate_static: the same check without any allocation --------------------------
//
// Scratch of the variant below.  It is part of the library image: every GPU that loads the
// library holds these bytes until the process exits.  In host code `g_static_scratch` is only
// a stand-in for the symbol; the address a kernel can use comes from cudaGetSymbolAddress.
constexpr size_t kStaticScratchBytes = 1u << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {

constexpr int kMaxDevices = 64;
struct StaticDevice { unsigned char* scratch; int sm_count; bool ready; };
constexpr size_t kStaticStatusBytes = 256;      // the scratch starts with the status word (zero when the library loads)
StaticDevice g_static_dev[kMaxDevices];
std::mutex g_static_mutex;
thread_local char g_static_error[256] = "";

int static_fail(int status, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_static_error, sizeof g_static_error, fmt, ap);
    va_end(ap);
    return status;
}

}  // namespace

extern "C" const char* evo_validate_static_error(void) { return g_static_error; }

extern "C" int evo_validate_static(const void* const* cand_ptrs, const void* ref_ptr, const evo_desc* descs, uint64_t n_desc,
                                   int dtype, float atol, float rtol, evo_result* results, uint32_t* group_pass,
                                   uint64_t n_group, void* stream_) {
    g_static_error[0] = '\0';
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (n_desc > 0 && !results) return static_fail(EVO_ERR_ARG, "evo_validate_static: results must not be NULL");
    int device = -1;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess) return static_fail(EVO_ERR_CUDA, "evo_validate_static: cudaGetDevice: %s", cudaGetErrorString(e));
    if (device < 0 || device >= kMaxDevices) return static_fail(EVO_ERR_ARG, "evo_validate_static: device %d out of range", device);

    // Set-up, once per device, with that device current: the device address of the scratch.
    StaticDevice dev;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_dev[device].ready) {
            unsigned char* ptr = nullptr;
            e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch);
            if (e != cudaSuccess || !ptr)
                return static_fail(EVO_ERR_CUDA, "evo_validate_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
            int sms = 0;
            e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
            if (e != cudaSuccess) return static_fail(EVO_ERR_CUDA, "evo_validate_static: %s", cudaGetErrorString(e));
            e = cudaFuncSetAttribute(validate_pass1, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kRingBytes));
            if (e != cudaSuccess) return static_fail(EVO_ERR_CUDA, "evo_validate_static: %s", cudaGetErrorString(e));
            g_static_dev[device].scratch = ptr;
            g_static_dev[device].sm_count = sms;
            g_static_dev[device].ready = true;
        }
        dev = g_static_dev[device];
    }

    Plan plan;
    std::string err;
    const uint32_t max_ctas = static_cast<uint32_t>(dev.sm_count) * kCtasPerSm;
    const int st = build_plan(cand_ptrs, ref_ptr, descs, n_desc, dtype, atol, rtol, group_pass != nullptr, n_group, max_ctas,
                              &plan, &err);
    if (st != EVO_OK) return static_fail(st, "evo_validate_static: %s", err.c_str());

    // Layout inside the scratch: the status word, the plan, then the partial records.
    const PlanLayout L = layout_of(plan, kStaticStatusBytes);
    const size_t o_parts = L.bytes;
    const size_t need = o_parts + static_cast<size_t>(plan.n_parts) * sizeof(Acc);
    if (need > kStaticScratchBytes)
        return static_fail(EVO_ERR_WORKSPACE,
                           "evo_validate_static: this population needs %zu bytes of scratch, the fixed scratch holds %zu "
                           "(%llu tensors in %zu sets); use evo_validate or split the call",
                           need, kStaticScratchBytes, (unsigned long long)n_desc, plan.sets.size());

    // The plan travels as the arguments of small store kernels (one per 16 KiB), so the call never
    // hands the runtime a pointer into this function's own memory and never makes the host wait
    // for the stream.  The first store also clears the status word: each call reports its own
    // waits only, and one that ran out long ago does not mark later results incomplete.
    // Nothing else in the scratch has to start at zero: the first pass writes every partial record
    // that the second pass reads.
    std::vector<unsigned char> h(L.bytes - kStaticStatusBytes);
    pack_plan(plan, L, kStaticStatusBytes, h.data());
    uint32_t* d_status = reinterpret_cast<uint32_t*>(dev.scratch);
    e = store_plan(h.data(), h.size(), dev.scratch + kStaticStatusBytes, d_status, false, stream, nullptr);
    if (e != cudaSuccess) return static_fail(EVO_ERR_CUDA, "evo_validate_static: plan store: %s", cudaGetErrorString(e));
    ChainArgs a{};
    a.d_plan = dev.scratch;
    a.L = L;
    a.d_parts = reinterpret_cast<Acc*>(dev.scratch + o_parts);
    a.d_status = d_status;
    a.atol = atol; a.rtol = rtol;
    a.results = results; a.group_pass = group_pass; a.n_group = n_group;
    a.pdl = false;
    e = launch_chain(static_cast<uint32_t>(plan.members.size()), static_cast<uint32_t>(plan.ranges.size()), a, stream, nullptr);
    if (e != cudaSuccess) return static_fail(EVO_ERR_CUDA, "evo_validate_static: launch: %s", cudaGetErrorString(e));
    return EVO_OK;
}
