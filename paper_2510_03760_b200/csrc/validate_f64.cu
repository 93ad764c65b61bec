// evo_validate_f64: the correctness constraint for binary64 outputs (paper Section 3.1 Eq. 1,
// Section 4.3: the output must match the reference).  The rule and the statistics of
// evo_validate, with every operation an individually rounded binary64 operation.
//
// Same plan as evo_validate (sets of tensors sharing a reference, (set, tile) items cut into
// one contiguous run per persistent CTA; a reference tile is read once per set).  Eight bytes
// per element and about ten binary64 operations: plain 128-bit streaming loads into registers
// keep up, so there is no shared-memory ring and nothing to wait on.  max d/|r| uses the same
// one-sided filter as the binary32 kernel (d > RZ(mlo*|r|) with mlo just below the running
// maximum), a thread whose filter fired walks its 16 elements again and divides only where it
// still fires.  A thread whose sum of squares comes out NaN/Inf (a NaN/Inf input or an
// overflowing difference) applies the rule in its exact form, flags included, to its elements.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <string>

#include "evo_internal.h"
#include "plan.h"

namespace {

using namespace evo;

constexpr int kCtasPerSm64 = 2;
constexpr int kVecs64 = kEpt / 2;                           // 16-byte vectors (two doubles) per thread per tile
constexpr int kTileVecs64 = kTileElems / 2;
constexpr double kShrink64 = 0.99999999999909050530;        // 1 - 2^-40

struct Acc64 {                 // partial result of one tensor (48 bytes)
    unsigned long long mism, nonfin;
    double sse;
    unsigned long long max_abs, max_rel;      // bit patterns of non-negative doubles: unsigned order == numeric order
    uint32_t flags, pad;
};

struct Lane64 {
    uint32_t cnt = 0, nf = 0, flags = 0;
    double ma = 0.0, mr = 0.0, sse = 0.0;
};

__device__ __forceinline__ double dinf() { return __longlong_as_double(0x7ff0000000000000ll); }
__device__ __forceinline__ double lo_of(const uint4& v) { return __hiloint2double(static_cast<int>(v.y), static_cast<int>(v.x)); }
__device__ __forceinline__ double hi_of(const uint4& v) { return __hiloint2double(static_cast<int>(v.w), static_cast<int>(v.z)); }

// The rule with every special case (see evo.h), and the true quotient.
__device__ __forceinline__ void exact_elem64(double c, double r, double atol, double rtol, Lane64& s) {
    const double d = fabs(__dsub_rn(c, r));
    const double ar = fabs(r);
    const double tol = __dadd_rn(atol, __dmul_rn(rtol, ar));
    const bool close = (c == r) || (d < dinf() && d <= tol);
    s.cnt += close ? 0u : 1u;
    uint32_t f = 0;
    if (c != c) f |= EVO_FLAG_CAND_NAN;
    if (c == dinf()) f |= EVO_FLAG_CAND_PINF;
    if (c == -dinf()) f |= EVO_FLAG_CAND_NINF;
    if (r != r) f |= EVO_FLAG_REF_NAN;
    if (ar == dinf()) f |= EVO_FLAG_REF_INF;
    if (f) {
        s.nf += 1;
        s.flags |= f;
    } else {
        s.ma = fmax(s.ma, d);
        if (ar != 0.0) s.mr = fmax(s.mr, __ddiv_rn(d, ar));
        s.sse = __fma_rn(d, d, s.sse);
    }
}

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long y = __shfl_xor_sync(0xffffffffu, x, o);
        x = y > x ? y : x;
    }
    return x;
}

__device__ __forceinline__ void commit64(const Lane64& s, Acc64* acc, unsigned long long* mr_shared, int lane) {
    const unsigned full = 0xffffffffu;
    const uint32_t cnt = __reduce_add_sync(full, s.cnt);
    const uint32_t nf = __reduce_add_sync(full, s.nf);
    const uint32_t fl = __reduce_or_sync(full, s.flags);
    const unsigned long long ma = warp_max_u64(static_cast<unsigned long long>(__double_as_longlong(s.ma)));
    const unsigned long long mr = warp_max_u64(static_cast<unsigned long long>(__double_as_longlong(s.mr)));
    double x = s.sse;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(full, x, o);
    if (lane == 0) {
        acc->mism += cnt;
        acc->nonfin += nf;
        acc->sse += x;
        acc->max_abs = ma > acc->max_abs ? ma : acc->max_abs;
        acc->flags |= fl;
        if (mr > *mr_shared) atomicMax(mr_shared, mr);
    }
    __syncwarp();
}

__device__ __forceinline__ void run_set64(const SetRec& S, uint64_t t0, uint64_t t1, double atol, double rtol,
                                          Acc64 (*s_acc)[kWarps], unsigned long long* s_mr, const void* const* s_cand,
                                          int warp, int lane) {
    const uint64_t full_tiles = S.vec_ok ? S.n / kTileElems : 0;
    for (uint64_t t = t0; t < t1; ++t) {
        if (t < full_tiles) {
            const uint64_t base = t * kTileVecs64 + threadIdx.x;
            const uint4* rp = static_cast<const uint4*>(S.ref) + base;
            double r[kEpt];
#pragma unroll
            for (int v = 0; v < kVecs64; ++v) {
                const uint4 x = __ldcs(rp + v * kThreads);
                r[2 * v] = lo_of(x);
                r[2 * v + 1] = hi_of(x);
            }
#pragma unroll 1
            for (uint32_t k = 0; k < S.k; ++k) {
                const uint4* cp = static_cast<const uint4*>(s_cand[k]) + base;
                double c[kEpt];
#pragma unroll
                for (int v = 0; v < kVecs64; ++v) {
                    const uint4 x = __ldcs(cp + v * kThreads);
                    c[2 * v] = lo_of(x);
                    c[2 * v + 1] = hi_of(x);
                }
                const double m = __longlong_as_double(static_cast<long long>(*reinterpret_cast<volatile unsigned long long*>(&s_mr[k])));
                const double mlo = __dmul_rz(m, kShrink64);
                Lane64 st;
                bool trig = false;
#pragma unroll
                for (int i = 0; i < kEpt; ++i) {
                    const double d = fabs(__dsub_rn(c[i], r[i]));
                    const double ar = fabs(r[i]);
                    const double tol = __dadd_rn(atol, __dmul_rn(rtol, ar));
                    st.cnt += d > tol ? 1u : 0u;
                    st.ma = fmax(st.ma, d);
                    st.sse = __fma_rn(d, d, st.sse);
                    trig |= d > __dmul_rz(mlo, ar);
                }
                st.mr = m;
                if (!(st.sse < dinf())) {
                    // something was NaN/Inf or a difference overflowed: the exact form, for this thread's elements
                    st = Lane64();
#pragma unroll
                    for (int i = 0; i < kEpt; ++i) exact_elem64(c[i], r[i], atol, rtol, st);
                } else if (trig) {
                    double lo = mlo;
#pragma unroll
                    for (int i = 0; i < kEpt; ++i) {
                        const double d = fabs(__dsub_rn(c[i], r[i]));
                        const double ar = fabs(r[i]);
                        if (ar != 0.0 && d > __dmul_rz(lo, ar)) {
                            const double q = __ddiv_rn(d, ar);
                            if (q > st.mr) { st.mr = q; lo = __dmul_rz(q, kShrink64); }
                        }
                    }
                }
                commit64(st, &s_acc[k][warp], &s_mr[k], lane);
            }
        } else {
            // ragged last tile, or tensors that are not 16-byte aligned: element loads, exact form
            const uint64_t e0 = t * kTileElems;
            const uint64_t e1 = min(S.n, e0 + kTileElems);
            const double* rp = static_cast<const double*>(S.ref);
            for (uint32_t k = 0; k < S.k; ++k) {
                const double* cp = static_cast<const double*>(s_cand[k]);
                Lane64 st;
                for (uint64_t e = e0 + threadIdx.x; e < e1; e += kThreads) exact_elem64(cp[e], rp[e], atol, rtol, st);
                commit64(st, &s_acc[k][warp], &s_mr[k], lane);
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads, kCtasPerSm64)
f64_pass1(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members, const CtaRange* __restrict__ ranges,
          Acc64* __restrict__ partials, double atol, double rtol) {
    __shared__ Acc64 s_acc[kMaxK][kWarps];
    __shared__ unsigned long long s_mr[kMaxK];
    __shared__ const void* s_cand[kMaxK];
    const CtaRange rg = ranges[blockIdx.x];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (uint32_t s = rg.s_begin; s <= rg.s_end; ++s) {
        const SetRec S = sets[s];
        const uint64_t tiles = (S.n + kTileElems - 1) / kTileElems;
        const uint64_t t0 = (s == rg.s_begin) ? rg.t_begin : 0;
        const uint64_t t1 = (s == rg.s_end) ? rg.t_end : tiles;
        if (t0 >= t1) continue;
        for (uint32_t i = threadIdx.x; i < S.k * kWarps; i += kThreads) {
            Acc64 z;
            z.mism = 0; z.nonfin = 0; z.sse = 0.0; z.max_abs = 0; z.max_rel = 0; z.flags = 0; z.pad = 0;
            s_acc[i / kWarps][i % kWarps] = z;
        }
        if (threadIdx.x < S.k) {
            s_cand[threadIdx.x] = members[S.member_off + threadIdx.x].cand;
            s_mr[threadIdx.x] = 0;
        }
        __syncthreads();
        run_set64(S, t0, t1, atol, rtol, s_acc, s_mr, s_cand, warp, lane);
        __syncthreads();
        if (threadIdx.x < S.k) {
            Acc64 a = s_acc[threadIdx.x][0];
#pragma unroll
            for (int w = 1; w < kWarps; ++w) {
                const Acc64 b = s_acc[threadIdx.x][w];
                a.mism += b.mism; a.nonfin += b.nonfin; a.sse += b.sse;
                a.max_abs = b.max_abs > a.max_abs ? b.max_abs : a.max_abs;
                a.flags |= b.flags;
            }
            a.max_rel = s_mr[threadIdx.x];
            partials[rg.part_base + (S.member_off - rg.first_member) + threadIdx.x] = a;
        }
        __syncthreads();
    }
}

// One warp per tensor: fold the partial records of the CTAs [cta_first, cta_last] in a fixed order.
__global__ void __launch_bounds__(kThreads)
f64_pass2(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members, const CtaRange* __restrict__ ranges,
          const Acc64* __restrict__ partials, uint32_t n_members, evo_result64* __restrict__ results) {
    const uint32_t m = blockIdx.x * kWarps + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (m >= n_members) return;
    const MemberRec M = members[m];
    const SetRec S = sets[M.set];
    unsigned long long mism = 0, nonfin = 0, ma = 0, mr = 0;
    double sse = 0.0;
    uint32_t fl = 0;
    if (S.cta_first <= S.cta_last) {
        for (uint32_t b = S.cta_first + lane; b <= S.cta_last; b += 32) {
            const CtaRange R = ranges[b];
            const Acc64 p = partials[R.part_base + (m - R.first_member)];
            mism += p.mism; nonfin += p.nonfin; sse += p.sse;
            ma = p.max_abs > ma ? p.max_abs : ma;
            mr = p.max_rel > mr ? p.max_rel : mr;
            fl |= p.flags;
        }
    }
    const unsigned full = 0xffffffffu;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        mism += __shfl_xor_sync(full, mism, o);
        nonfin += __shfl_xor_sync(full, nonfin, o);
        sse += __shfl_xor_sync(full, sse, o);
    }
    ma = warp_max_u64(ma);
    mr = warp_max_u64(mr);
    fl = __reduce_or_sync(full, fl);
    if (lane == 0) {
        evo_result64 r;
        r.n_mismatch = mism; r.n_nonfinite = nonfin; r.sse = sse;
        r.max_abs = __longlong_as_double(static_cast<long long>(ma));
        r.max_rel = __longlong_as_double(static_cast<long long>(mr));
        r.flags = fl; r.pass = mism == 0 ? 1u : 0u;
        results[M.desc] = r;
    }
}

__global__ void f64_verdict(const uint32_t* __restrict__ offsets, const uint32_t* __restrict__ desc_of,
                            const evo_result64* __restrict__ results, uint32_t n_group, uint32_t* __restrict__ group_pass) {
    const uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= n_group) return;
    uint32_t ok = 1;
    for (uint32_t i = offsets[g]; i < offsets[g + 1]; ++i) ok &= results[desc_of[i]].pass;
    group_pass[g] = ok;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace

extern "C" int evo_validate_f64(evo_ctx* ctx, const void* const* cand_ptrs, const void* ref_ptr, const evo_desc* descs,
                                uint64_t n_desc, double atol, double rtol, evo_result64* results, uint32_t* group_pass,
                                uint64_t n_group, void* stream_) {
    if (!ctx) return EVO_ERR_ARG;
    const char* who = "evo_validate_f64";
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (n_desc > 0 && !results) return evo::fail(ctx, EVO_ERR_ARG, "%s: results must not be NULL", who);
    if (!(atol >= 0.0) || !(rtol >= 0.0) || std::isinf(atol) || std::isinf(rtol))
        return evo::fail(ctx, EVO_ERR_ARG, "%s: atol and rtol must be finite and >= 0", who);
    Plan plan;
    std::string err;
    const uint32_t max_ctas = static_cast<uint32_t>(ctx->sm_count) * kCtasPerSm64;
    int st = build_plan(cand_ptrs, ref_ptr, descs, n_desc, EVO_F64, 0.f, 0.f, group_pass != nullptr, n_group, max_ctas, &plan,
                        &err, 1u << EVO_F64);
    if (st != EVO_OK) return evo::fail(ctx, st, "%s: %s", who, err.c_str());
    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");

    const size_t o_sets = 0;
    const size_t o_members = align_up(o_sets + plan.sets.size() * sizeof(SetRec), 256);
    const size_t o_ranges = align_up(o_members + plan.members.size() * sizeof(MemberRec), 256);
    const size_t o_goff = align_up(o_ranges + plan.ranges.size() * sizeof(CtaRange), 256);
    const size_t o_gdesc = align_up(o_goff + plan.group_off.size() * 4, 256);
    const size_t plan_bytes = align_up(o_gdesc + plan.group_desc.size() * 4, 256) + 256;
    ctx->plan_key_valid = false;          // the plan area is about to hold this call's plan
    st = evo::reserve_pinned(ctx, &ctx->h_plan, &ctx->h_plan_bytes, plan_bytes);
    if (st != EVO_OK) return st;
    st = evo::reserve_device(ctx, &ctx->d_plan, &ctx->d_plan_bytes, plan_bytes);
    if (st != EVO_OK) return st;
    st = evo::reserve_device(ctx, &ctx->d_partials, &ctx->d_partials_bytes, std::max<size_t>(plan.n_parts, 1) * sizeof(Acc64));
    if (st != EVO_OK) return st;
    if (ctx->plan_in_flight) {
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
    Acc64* d_parts = static_cast<Acc64*>(ctx->d_partials);
    const uint32_t n_ctas = static_cast<uint32_t>(plan.ranges.size());
    if (n_ctas > 0) {
        f64_pass1<<<n_ctas, kThreads, 0, stream>>>(d_sets, d_members, d_ranges, d_parts, atol, rtol);
        ctx->launches += 1;
        EVO_CUDA_TRY(ctx, cudaGetLastError());
    }
    const uint32_t n_members = static_cast<uint32_t>(n_desc);
    if (n_members > 0) {
        f64_pass2<<<(n_members + kWarps - 1) / kWarps, kThreads, 0, stream>>>(d_sets, d_members, d_ranges, d_parts, n_members, results);
        ctx->launches += 1;
        EVO_CUDA_TRY(ctx, cudaGetLastError());
    }
    if (group_pass) {
        f64_verdict<<<static_cast<unsigned>((n_group + 255) / 256), 256, 0, stream>>>(
            reinterpret_cast<const uint32_t*>(d + o_goff), reinterpret_cast<const uint32_t*>(d + o_gdesc), results,
            static_cast<uint32_t>(n_group), group_pass);
        ctx->launches += 1;
        EVO_CUDA_TRY(ctx, cudaGetLastError());
    }
    return EVO_OK;
}
