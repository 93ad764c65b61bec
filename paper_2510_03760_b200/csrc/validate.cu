// evo_validate: the functional-correctness constraint over a population of candidate
// outputs (paper Section 3.1 Eq. 1, g(p) = 0; Section 4.3, functional testing against the
// reference outputs), with the error statistics reported alongside the verdict.
//
// Shape of the computation: a pure streaming read.  Every candidate element and every
// distinct reference element has to come from HBM once; per element there are about ten
// binary32 operations.  The design therefore spends its effort on (1) never reading a
// reference tile more than once per set of candidates that share it, (2) keeping many
// 16-byte loads in flight per SM, and (3) keeping reductions off the per-element path.
//
//   plan (host)   tensors with the same (reference, n, dtype) form a set of up to kMaxK
//                 members; the flat list of (set, tile) items, weighted by the bytes they
//                 move, is cut into one contiguous range per CTA (a fixed cut: no work
//                 queue, no atomics, results reproducible run to run).
//   pass 1        persistent CTAs walk their range.  Per tile the reference is loaded
//                 once into registers (128-bit loads) and compared against each member's
//                 tile; per (tile, member) the warp folds its lanes with redux/shuffles
//                 into a warp-private accumulator in shared memory.  When a CTA leaves a
//                 set it writes one partial record per member to global memory.
//   pass 2        one warp per tensor folds the partial records of the CTAs that touched
//                 it, in a fixed order, and writes the evo_result.
//   verdict       one thread per candidate id ANDs the verdicts of its tensors.
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

namespace {

using namespace evo;

constexpr int kCtasPerSm = 3;

// ---- loads ---------------------------------------------------------------------------
// Streaming 128-bit load: the data is used exactly once by this SM.
__device__ __forceinline__ uint4 load_stream(const uint4* p) { return __ldcs(p); }

template <int DT> struct Elem;
template <> struct Elem<EVO_F32> {
    static constexpr int kPerVec = 4;
    using T = float;
    static __device__ __forceinline__ float at(const uint4& v, int i) {
        return __uint_as_float(i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w);
    }
    static __device__ __forceinline__ float widen(T x) { return x; }
};
template <> struct Elem<EVO_F16> {
    static constexpr int kPerVec = 8;
    using T = __half;
    static __device__ __forceinline__ float at(const uint4& v, int i) {
        const uint32_t w = (i >> 1) == 0 ? v.x : (i >> 1) == 1 ? v.y : (i >> 1) == 2 ? v.z : v.w;
        const __half2 h = *reinterpret_cast<const __half2*>(&w);
        return (i & 1) ? __high2float(h) : __low2float(h);
    }
    static __device__ __forceinline__ float widen(T x) { return __half2float(x); }
};
template <> struct Elem<EVO_BF16> {
    static constexpr int kPerVec = 8;
    using T = __nv_bfloat16;
    static __device__ __forceinline__ float at(const uint4& v, int i) {
        const uint32_t w = (i >> 1) == 0 ? v.x : (i >> 1) == 1 ? v.y : (i >> 1) == 2 ? v.z : v.w;
        return __uint_as_float((i & 1) ? (w & 0xffff0000u) : (w << 16));
    }
    static __device__ __forceinline__ float widen(T x) { return __bfloat162float(x); }
};

// ---- per-lane state for one (tile, member) ----------------------------------------------
struct Lane {
    uint32_t cnt = 0;        // mismatches
    float ma = 0.f;          // max d
    float mr = 0.f;          // max d/|r| found by this lane (exact path only)
    float sse = 0.f;         // sum d^2, binary32 (fast path)
    double dsse = 0.0;       // sum d^2, binary64 (exact path)
    uint32_t nf = 0;         // non-finite elements
    uint32_t flags = 0;
    bool trig = false;       // some quotient may exceed the running maximum
    bool exact = false;      // values above come from the exact path
};

// Fast path, valid when c and r are finite and d does not overflow.  Operations and
// rounding follow the rule literally: d = |c - r|, tol = atol + rtol*|r|, no fused
// multiply-add on that chain.  With atol, rtol >= 0 and finite data, c == r implies
// d = 0 <= tol, so the equality clause needs no separate test here.
// The quotient d/|r| is not formed: `mlo` is a value slightly below the running maximum m
// of the quotient, and d > RZ(mlo*|r|) holds whenever fl(d/|r|) > m could (rounding the
// product toward zero keeps the test one-sided), so a miss never loses a maximum.
__device__ __forceinline__ void fast_elem(float c, float r, float atol, float rtol, float mlo, Lane& s) {
    const float d = fabsf(__fsub_rn(c, r));
    const float ar = fabsf(r);
    const float tol = __fadd_rn(atol, __fmul_rn(rtol, ar));
    s.cnt += (d > tol) ? 1u : 0u;
    s.ma = fmaxf(s.ma, d);
    s.sse = fmaf(d, d, s.sse);
    s.trig |= (d > __fmul_rz(mlo, ar));
}

// Exact path: the rule with every special case, and the true quotient.
__device__ __forceinline__ void exact_elem(float c, float r, float atol, float rtol, Lane& s) {
    const float d = fabsf(__fsub_rn(c, r));
    const float ar = fabsf(r);
    const float tol = __fadd_rn(atol, __fmul_rn(rtol, ar));
    const bool d_finite = d < __int_as_float(0x7f800000);          // false for NaN and Inf
    const bool close = (c == r) || (d_finite && d <= tol);
    s.cnt += close ? 0u : 1u;
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

// Fold the 32 lanes and add the result to the warp's accumulator for this member.
__device__ __forceinline__ void warp_commit(const Lane& s, Acc* acc, int lane) {
    const unsigned full = 0xffffffffu;
    const uint32_t cnt = __reduce_add_sync(full, s.cnt);
    const uint32_t ma = __reduce_max_sync(full, __float_as_uint(s.ma));
    const bool any_exact = __any_sync(full, s.exact);
    double sse;
    uint32_t mr = 0, nf = 0, fl = 0;
    if (any_exact) {
        double x = s.exact ? s.dsse : static_cast<double>(s.sse);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(full, x, o);
        sse = x;
        mr = __reduce_max_sync(full, __float_as_uint(s.mr));
        nf = __reduce_add_sync(full, s.nf);
        fl = __reduce_or_sync(full, s.flags);
    } else {
        float x = s.sse;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(full, x, o);
        sse = static_cast<double>(x);
    }
    if (lane == 0) {
        acc->mism += cnt;
        acc->sse += sse;
        acc->max_abs = max(acc->max_abs, ma);
        if (any_exact) {
            acc->nonfin += nf;
            acc->max_rel = max(acc->max_rel, mr);
            acc->flags |= fl;
        }
    }
    __syncwarp();
}

// The exact path over this thread's share of a full tile.  Reached rarely (first tile of a
// set, a new maximum of the quotient, NaN/Inf, overflow or all-tiny differences), so it
// re-reads its 16-byte vectors (they were just loaded: L2 hits) instead of holding the hot
// loop's registers hostage.
template <int DT>
__device__ __noinline__ void exact_redo(const uint4* __restrict__ cp, const uint4* __restrict__ rp,
                                        float atol, float rtol, Lane& st) {
    using E = Elem<DT>;
    st = Lane();
    st.exact = true;
#pragma unroll 1
    for (int v = 0; v < kVpt; ++v) {
        const uint4 c = cp[v * kThreads], r = rp[v * kThreads];
#pragma unroll
        for (int e = 0; e < E::kPerVec; ++e) exact_elem(E::at(c, e), E::at(r, e), atol, rtol, st);
    }
}

// One full, 16-byte aligned tile: reference into registers once, then every member.
template <int DT>
__device__ __forceinline__ void fast_tile(const SetRec& S, uint64_t t, float atol, float rtol,
                                          Acc (*s_acc)[kWarps], const void* const* s_cand, int warp, int lane) {
    using E = Elem<DT>;
    const uint64_t base = t * kTileVecs + threadIdx.x;
    const uint4* rp = static_cast<const uint4*>(S.ref) + base;
    uint4 r[kVpt];
#pragma unroll
    for (int v = 0; v < kVpt; ++v) r[v] = load_stream(rp + v * kThreads);
    const int K = static_cast<int>(S.k);
#pragma unroll 1
    for (int k = 0; k < K; ++k) {
        const uint4* cp = static_cast<const uint4*>(s_cand[k]) + base;
        uint4 c[kVpt];
#pragma unroll
        for (int v = 0; v < kVpt; ++v) c[v] = load_stream(cp + v * kThreads);
        Acc* acc = &s_acc[k][warp];
        const float m = __uint_as_float(acc->max_rel);
        const float mlo = __fmul_rz(m, 0.99999904632568359375f);      // 1 - 2^-20
        Lane st;
#pragma unroll
        for (int v = 0; v < kVpt; ++v)
#pragma unroll
            for (int e = 0; e < E::kPerVec; ++e) fast_elem(E::at(c[v], e), E::at(r[v], e), atol, rtol, mlo, st);
        // Leave the fast path if (a) something was NaN/Inf or overflowed (the sum of squares
        // is then NaN/Inf), (b) a quotient may beat the running maximum, or (c) every d is so
        // small that d^2 underflows in binary32.
        const bool redo = !(st.sse < __int_as_float(0x7f800000)) || st.trig ||
                          (st.ma < 9.094947017729282e-13f /* 2^-40 */ && st.ma > 0.f);
        if (redo) exact_redo<DT>(cp, rp, atol, rtol, st);
        warp_commit(st, acc, lane);
    }
}

// Ragged last tile, or tensors that are not 16-byte aligned: scalar loads, exact path.
template <int DT>
__device__ __noinline__ void slow_tile(const SetRec& S, uint64_t t, float atol, float rtol,
                                       Acc (*s_acc)[kWarps], const void* const* s_cand, int warp, int lane) {
    using E = Elem<DT>;
    using T = typename E::T;
    const uint64_t e0 = t * tile_elems(DT);
    const uint64_t e1 = min(S.n, e0 + tile_elems(DT));
    const T* rp = static_cast<const T*>(S.ref);
    for (uint32_t k = 0; k < S.k; ++k) {
        const T* cp = static_cast<const T*>(s_cand[k]);
        Lane st;
        st.exact = true;
        for (uint64_t e = e0 + threadIdx.x; e < e1; e += kThreads) exact_elem(E::widen(cp[e]), E::widen(rp[e]), atol, rtol, st);
        warp_commit(st, &s_acc[k][warp], lane);
    }
}

template <int DT>
__device__ __forceinline__ void run_set(const SetRec& S, uint64_t t0, uint64_t t1, float atol, float rtol,
                                        Acc (*s_acc)[kWarps], const void* const* s_cand, int warp, int lane) {
    const uint64_t full_tiles = S.vec_ok ? S.n / tile_elems(DT) : 0;
    for (uint64_t t = t0; t < t1; ++t) {
        if (t < full_tiles) fast_tile<DT>(S, t, atol, rtol, s_acc, s_cand, warp, lane);
        else slow_tile<DT>(S, t, atol, rtol, s_acc, s_cand, warp, lane);
    }
}

__global__ void __launch_bounds__(kThreads, kCtasPerSm)
validate_pass1(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members,
               const CtaRange* __restrict__ ranges, Acc* __restrict__ partials, float atol, float rtol) {
    __shared__ Acc s_acc[kMaxK][kWarps];
    __shared__ const void* s_cand[kMaxK];
    const CtaRange rg = ranges[blockIdx.x];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (uint32_t s = rg.s_begin; s <= rg.s_end && rg.s_begin <= rg.s_end; ++s) {
        const SetRec S = sets[s];
        const uint64_t tiles = (S.n + tile_elems(S.dtype) - 1) / tile_elems(S.dtype);
        const uint64_t t0 = (s == rg.s_begin) ? rg.t_begin : 0;
        const uint64_t t1 = (s == rg.s_end) ? rg.t_end : tiles;
        if (t0 >= t1) continue;
        for (uint32_t i = threadIdx.x; i < S.k * kWarps; i += kThreads) {
            Acc z;
            z.mism = 0; z.nonfin = 0; z.sse = 0.0; z.max_abs = 0; z.max_rel = 0; z.flags = 0; z.pad = 0;
            s_acc[i / kWarps][i % kWarps] = z;
        }
        if (threadIdx.x < S.k) s_cand[threadIdx.x] = members[S.member_off + threadIdx.x].cand;
        __syncthreads();
        if (S.dtype == EVO_F32) run_set<EVO_F32>(S, t0, t1, atol, rtol, s_acc, s_cand, warp, lane);
        else if (S.dtype == EVO_F16) run_set<EVO_F16>(S, t0, t1, atol, rtol, s_acc, s_cand, warp, lane);
        else run_set<EVO_BF16>(S, t0, t1, atol, rtol, s_acc, s_cand, warp, lane);
        __syncthreads();
        if (threadIdx.x < S.k) {
            Acc a = s_acc[threadIdx.x][0];
#pragma unroll
            for (int w = 1; w < kWarps; ++w) {
                const Acc b = s_acc[threadIdx.x][w];
                a.mism += b.mism; a.nonfin += b.nonfin; a.sse += b.sse;
                a.max_abs = max(a.max_abs, b.max_abs); a.max_rel = max(a.max_rel, b.max_rel); a.flags |= b.flags;
            }
            partials[rg.part_base + (S.member_off - rg.first_member) + threadIdx.x] = a;
        }
        __syncthreads();
    }
}

// One warp per tensor: fold the partial records of the CTAs [cta_first, cta_last] in a
// fixed order (lane-strided, then a xor tree).
__global__ void __launch_bounds__(kThreads)
validate_pass2(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members,
               const CtaRange* __restrict__ ranges, const Acc* __restrict__ partials,
               uint32_t n_members, evo_result* __restrict__ results) {
    const uint32_t m = blockIdx.x * kWarps + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (m >= n_members) return;
    const MemberRec M = members[m];
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
    const uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= n_group) return;
    uint32_t ok = 1;
    for (uint32_t i = offsets[g]; i < offsets[g + 1]; ++i) ok &= results[desc_of[i]].pass;
    group_pass[g] = ok;
}

// ---- host side ------------------------------------------------------------------------

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int validate_device(evo_ctx* ctx, const void* const* cand_ptrs, const void* ref_ptr, const evo_desc* descs,
                    uint64_t n_desc, int dtype, float atol, float rtol, evo_result* results,
                    uint32_t* group_pass, uint64_t n_group, cudaStream_t stream, const char* who) {
    if (n_desc > 0 && !results) return evo::fail(ctx, EVO_ERR_ARG, "%s: results must not be NULL", who);
    Plan plan;
    std::string err;
    const uint32_t max_ctas = static_cast<uint32_t>(ctx->sm_count) * kCtasPerSm;
    int st = build_plan(cand_ptrs, ref_ptr, descs, n_desc, dtype, atol, rtol, group_pass != nullptr, n_group, max_ctas,
                        &plan, &err);
    if (st != EVO_OK) return evo::fail(ctx, st, "%s: %s", who, err.c_str());

    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");

    // ---- pack and upload the plan ----
    const size_t o_sets = 0;
    const size_t o_members = align_up(o_sets + plan.sets.size() * sizeof(SetRec), 256);
    const size_t o_ranges = align_up(o_members + plan.members.size() * sizeof(MemberRec), 256);
    const size_t o_goff = align_up(o_ranges + plan.ranges.size() * sizeof(CtaRange), 256);
    const size_t o_gdesc = align_up(o_goff + plan.group_off.size() * 4, 256);
    const size_t plan_bytes = align_up(o_gdesc + plan.group_desc.size() * 4, 256) + 256;
    st = evo::reserve_pinned(ctx, &ctx->h_plan, &ctx->h_plan_bytes, plan_bytes);
    if (st != EVO_OK) return st;
    st = evo::reserve_device(ctx, &ctx->d_plan, &ctx->d_plan_bytes, plan_bytes);
    if (st != EVO_OK) return st;
    st = evo::reserve_device(ctx, &ctx->d_partials, &ctx->d_partials_bytes, std::max<size_t>(plan.n_parts, 1) * sizeof(Acc));
    if (st != EVO_OK) return st;
    if (ctx->plan_in_flight) {
        // the pinned staging block is about to be overwritten: the previous upload must have been read
        EVO_CUDA_TRY(ctx, cudaEventSynchronize(ctx->plan_consumed));
        ctx->plan_in_flight = false;
    }
    char* h = static_cast<char*>(ctx->h_plan);
    auto put = [&](size_t o, const void* src, size_t bytes) { if (bytes) std::memcpy(h + o, src, bytes); };
    put(o_sets, plan.sets.data(), plan.sets.size() * sizeof(SetRec));
    put(o_members, plan.members.data(), plan.members.size() * sizeof(MemberRec));
    put(o_ranges, plan.ranges.data(), plan.ranges.size() * sizeof(CtaRange));
    put(o_goff, plan.group_off.data(), plan.group_off.size() * 4);
    put(o_gdesc, plan.group_desc.data(), plan.group_desc.size() * 4);
    EVO_CUDA_TRY(ctx, cudaMemcpyAsync(ctx->d_plan, h, plan_bytes, cudaMemcpyHostToDevice, stream));
    EVO_CUDA_TRY(ctx, cudaEventRecord(ctx->plan_consumed, stream));
    ctx->plan_in_flight = true;

    const char* d = static_cast<const char*>(ctx->d_plan);
    const SetRec* d_sets = reinterpret_cast<const SetRec*>(d + o_sets);
    const MemberRec* d_members = reinterpret_cast<const MemberRec*>(d + o_members);
    const CtaRange* d_ranges = reinterpret_cast<const CtaRange*>(d + o_ranges);
    Acc* d_parts = static_cast<Acc*>(ctx->d_partials);

    const uint32_t n_ctas = static_cast<uint32_t>(plan.ranges.size());
    const cudaEvent_t ev_start = ctx->time_start, ev_stop = ctx->time_stop;
    ctx->time_start = ctx->time_stop = nullptr;
    if (ev_start) EVO_CUDA_TRY(ctx, cudaEventRecord(ev_start, stream));
    if (n_ctas > 0) {
        validate_pass1<<<n_ctas, kThreads, 0, stream>>>(d_sets, d_members, d_ranges, d_parts, atol, rtol);
        ctx->launches += 1;
        EVO_CUDA_TRY(ctx, cudaGetLastError());
    }
    if (ev_stop) EVO_CUDA_TRY(ctx, cudaEventRecord(ev_stop, stream));
    const uint32_t n_members = static_cast<uint32_t>(n_desc);
    if (n_members > 0) {
        validate_pass2<<<(n_members + kWarps - 1) / kWarps, kThreads, 0, stream>>>(d_sets, d_members, d_ranges, d_parts,
                                                                                    n_members, results);
        ctx->launches += 1;
        EVO_CUDA_TRY(ctx, cudaGetLastError());
    }
    if (group_pass) {
        group_verdict<<<static_cast<unsigned>((n_group + 255) / 256), 256, 0, stream>>>(
            reinterpret_cast<const uint32_t*>(d + o_goff), reinterpret_cast<const uint32_t*>(d + o_gdesc), results,
            static_cast<uint32_t>(n_group), group_pass);
        ctx->launches += 1;
        EVO_CUDA_TRY(ctx, cudaGetLastError());
    }
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
    EVO_CUDA_TRY(ctx, cudaStreamSynchronize(stream));
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

    // Layout inside the scratch: the plan, then the partial records.
    const size_t o_sets = 0;
    const size_t o_members = align_up(o_sets + plan.sets.size() * sizeof(SetRec), 256);
    const size_t o_ranges = align_up(o_members + plan.members.size() * sizeof(MemberRec), 256);
    const size_t o_goff = align_up(o_ranges + plan.ranges.size() * sizeof(CtaRange), 256);
    const size_t o_gdesc = align_up(o_goff + plan.group_off.size() * 4, 256);
    const size_t plan_bytes = align_up(o_gdesc + plan.group_desc.size() * 4, 256);
    const size_t o_parts = plan_bytes;
    const size_t need = o_parts + static_cast<size_t>(plan.n_parts) * sizeof(Acc);
    if (need > kStaticScratchBytes)
        return static_fail(EVO_ERR_WORKSPACE,
                           "evo_validate_static: this population needs %zu bytes of scratch, the fixed scratch holds %zu "
                           "(%llu tensors in %zu sets); use evo_validate or split the call",
                           need, kStaticScratchBytes, (unsigned long long)n_desc, plan.sets.size());

    // The plan goes up from ordinary host memory: the copy call returns once the runtime has
    // taken the bytes, so the local buffer may go out of scope.
    std::vector<unsigned char> h(plan_bytes ? plan_bytes : 1);
    auto put = [&](size_t o, const void* src, size_t bytes) { if (bytes) std::memcpy(h.data() + o, src, bytes); };
    put(o_sets, plan.sets.data(), plan.sets.size() * sizeof(SetRec));
    put(o_members, plan.members.data(), plan.members.size() * sizeof(MemberRec));
    put(o_ranges, plan.ranges.data(), plan.ranges.size() * sizeof(CtaRange));
    put(o_goff, plan.group_off.data(), plan.group_off.size() * 4);
    put(o_gdesc, plan.group_desc.data(), plan.group_desc.size() * 4);
    if (plan_bytes) {
        e = cudaMemcpyAsync(dev.scratch, h.data(), plan_bytes, cudaMemcpyHostToDevice, stream);
        if (e != cudaSuccess) return static_fail(EVO_ERR_CUDA, "evo_validate_static: plan upload: %s", cudaGetErrorString(e));
    }
    const unsigned char* d = dev.scratch;
    const SetRec* d_sets = reinterpret_cast<const SetRec*>(d + o_sets);
    const MemberRec* d_members = reinterpret_cast<const MemberRec*>(d + o_members);
    const CtaRange* d_ranges = reinterpret_cast<const CtaRange*>(d + o_ranges);
    Acc* d_parts = reinterpret_cast<Acc*>(dev.scratch + o_parts);
    // Nothing in the scratch has to start at zero: pass 1 writes every partial record that
    // pass 2 reads, so what an earlier call left behind is never looked at.
    const uint32_t n_ctas = static_cast<uint32_t>(plan.ranges.size());
    if (n_ctas > 0) validate_pass1<<<n_ctas, kThreads, 0, stream>>>(d_sets, d_members, d_ranges, d_parts, atol, rtol);
    const uint32_t n_members = static_cast<uint32_t>(n_desc);
    if (n_members > 0)
        validate_pass2<<<(n_members + kWarps - 1) / kWarps, kThreads, 0, stream>>>(d_sets, d_members, d_ranges, d_parts,
                                                                                    n_members, results);
    if (group_pass)
        group_verdict<<<static_cast<unsigned>((n_group + 255) / 256), 256, 0, stream>>>(
            reinterpret_cast<const uint32_t*>(d + o_goff), reinterpret_cast<const uint32_t*>(d + o_gdesc), results,
            static_cast<uint32_t>(n_group), group_pass);
    e = cudaGetLastError();
    if (e != cudaSuccess) return static_fail(EVO_ERR_CUDA, "evo_validate_static: launch: %s", cudaGetErrorString(e));
    return EVO_OK;
}
