// evo_validate_exact: the correctness constraint for integer and boolean outputs (paper
// Section 3.1 Eq. 1, Section 4.3: the output must match the reference; read as equality for
// index results, masks and counts).  Per tensor: the number of unequal elements and the
// largest |c - r|, exact.
//
// Same plan as evo_validate (sets of tensors sharing a reference, (set, tile) items cut into
// one contiguous run per persistent CTA) and the same property that matters: a reference tile
// is read once per set.  The arithmetic is two or three integer operations per element, so
// plain 128-bit streaming loads into registers keep up; there is no shared-memory ring and
// nothing to wait on.  Per (tile, member) a warp folds its lanes into a warp-private
// accumulator in shared memory; a CTA leaving a set writes one partial record per member; a
// second pass folds the records per tensor in a fixed order.
#include <algorithm>
#include <cstring>
#include <string>

#include <unordered_map>
#include <vector>

#include "evo_internal.h"
#include "philox.cuh"
#include "plan.h"

namespace {

using namespace evo;

constexpr int kCtasPerSmExact = 4;

__device__ __forceinline__ uint4 load_stream(const uint4* p) { return __ldcs(p); }

// Per element type: elements per 16-byte vector, and (count, largest difference) of one vector pair.
template <int DT> struct IntElem;
template <> struct IntElem<EVO_I32> {
    using T = int32_t;
    static constexpr int kPerVec = 4;
    static __device__ __forceinline__ unsigned long long diff(T c, T r) {
        const long long a = c, b = r;
        return static_cast<unsigned long long>(a > b ? a - b : b - a);
    }
    static __device__ __forceinline__ void vec(const uint4& c, const uint4& r, uint32_t& cnt, unsigned long long& md) {
        const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, rw[4] = {r.x, r.y, r.z, r.w};
        uint32_t m = 0;                                     // |c - r| of two int32 values fits 32 unsigned bits
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int32_t a = static_cast<int32_t>(cw[i]), b = static_cast<int32_t>(rw[i]);
            const uint32_t d = a > b ? cw[i] - rw[i] : rw[i] - cw[i];
            cnt += d != 0 ? 1u : 0u;
            m = max(m, d);
        }
        md = m > md ? m : md;
    }
};
template <> struct IntElem<EVO_I64> {
    using T = long long;
    static constexpr int kPerVec = 2;
    // the true difference of two int64 values may not fit int64: subtract as unsigned (exact, below 2^64)
    static __device__ __forceinline__ unsigned long long diff(T c, T r) {
        return c > r ? static_cast<unsigned long long>(c) - static_cast<unsigned long long>(r)
                     : static_cast<unsigned long long>(r) - static_cast<unsigned long long>(c);
    }
    static __device__ __forceinline__ void vec(const uint4& c, const uint4& r, uint32_t& cnt, unsigned long long& md) {
        const long long c0 = static_cast<long long>((static_cast<unsigned long long>(c.y) << 32) | c.x);
        const long long c1 = static_cast<long long>((static_cast<unsigned long long>(c.w) << 32) | c.z);
        const long long r0 = static_cast<long long>((static_cast<unsigned long long>(r.y) << 32) | r.x);
        const long long r1 = static_cast<long long>((static_cast<unsigned long long>(r.w) << 32) | r.z);
        const unsigned long long d0 = diff(c0, r0), d1 = diff(c1, r1);
        cnt += (d0 != 0 ? 1u : 0u) + (d1 != 0 ? 1u : 0u);
        md = d0 > md ? d0 : md;
        md = d1 > md ? d1 : md;
    }
};
template <> struct IntElem<EVO_U8> {
    using T = uint8_t;
    static constexpr int kPerVec = 16;
    static __device__ __forceinline__ unsigned long long diff(T c, T r) {
        const int a = c, b = r;
        return static_cast<unsigned long long>(a > b ? a - b : b - a);
    }
    static __device__ __forceinline__ void vec(const uint4& c, const uint4& r, uint32_t& cnt, unsigned long long& md) {
        const uint32_t cw[4] = {c.x, c.y, c.z, c.w}, rw[4] = {r.x, r.y, r.z, r.w};
        uint32_t m4 = 0;                                    // per-byte running maximum of |c - r|
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (cw[i] == rw[i]) continue;
            cnt += __popc(__vcmpne4(cw[i], rw[i])) >> 3;    // 0xff per unequal byte
            m4 = __vmaxu4(m4, __vabsdiffu4(cw[i], rw[i]));
        }
        const uint32_t m = max(max(m4 & 0xffu, (m4 >> 8) & 0xffu), max((m4 >> 16) & 0xffu, m4 >> 24));
        md = m > md ? m : md;
    }
};

struct AccExact { unsigned long long mism, maxdiff; };

__device__ __forceinline__ void commit(uint32_t cnt, unsigned long long md, AccExact* acc, int lane) {
    const unsigned full = 0xffffffffu;
    cnt = __reduce_add_sync(full, cnt);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long other = __shfl_xor_sync(full, md, o);
        md = other > md ? other : md;
    }
    if (lane == 0) {
        acc->mism += cnt;
        acc->maxdiff = md > acc->maxdiff ? md : acc->maxdiff;
    }
    __syncwarp();
}

template <int DT>
__device__ __forceinline__ void run_set_exact(const SetRec& S, uint64_t t0, uint64_t t1, AccExact (*s_acc)[kWarps],
                                              const void* const* s_cand, int warp, int lane) {
    using E = IntElem<DT>;
    using T = typename E::T;
    constexpr int kVecs = kEpt / E::kPerVec > 0 ? kEpt / E::kPerVec : 1;     // 16-byte vectors per thread per tile
    constexpr int kTileVecs = kTileElems / E::kPerVec;
    const uint64_t full_tiles = S.vec_ok ? S.n / kTileElems : 0;
    for (uint64_t t = t0; t < t1; ++t) {
        if (t < full_tiles) {
            // a whole, 16-byte aligned tile: the reference into registers once, then every member
            const uint64_t base = t * kTileVecs + threadIdx.x;
            const bool mine = E::kPerVec <= kEpt || threadIdx.x < kTileVecs;           // uint8: 256 vectors per tile
            const uint4* rp = static_cast<const uint4*>(S.ref) + base;
            uint4 r[kVecs];
            if (mine) {
#pragma unroll
                for (int v = 0; v < kVecs; ++v) r[v] = load_stream(rp + v * kThreads);
            }
#pragma unroll 1
            for (uint32_t k = 0; k < S.k; ++k) {
                uint32_t cnt = 0;
                unsigned long long md = 0;
                if (mine) {
                    const uint4* cp = static_cast<const uint4*>(s_cand[k]) + base;
                    uint4 c[kVecs];
#pragma unroll
                    for (int v = 0; v < kVecs; ++v) c[v] = load_stream(cp + v * kThreads);
#pragma unroll
                    for (int v = 0; v < kVecs; ++v) E::vec(c[v], r[v], cnt, md);
                }
                commit(cnt, md, &s_acc[k][warp], lane);
            }
        } else {
            // ragged last tile, or tensors that are not 16-byte aligned: element loads
            const uint64_t e0 = t * kTileElems;
            const uint64_t e1 = min(S.n, e0 + kTileElems);
            const T* rp = static_cast<const T*>(S.ref);
            for (uint32_t k = 0; k < S.k; ++k) {
                const T* cp = static_cast<const T*>(s_cand[k]);
                uint32_t cnt = 0;
                unsigned long long md = 0;
                for (uint64_t e = e0 + threadIdx.x; e < e1; e += kThreads) {
                    const unsigned long long d = E::diff(cp[e], rp[e]);
                    cnt += d != 0 ? 1u : 0u;
                    md = d > md ? d : md;
                }
                commit(cnt, md, &s_acc[k][warp], lane);
            }
        }
    }
}

// A thread should keep about 128 bytes of every tensor in flight; a tile gives it 16 (uint8) or 64 (int32).
// kGroup consecutive whole tiles are contiguous in memory, so they are taken together as one group with
// kGroup times the vectors per thread; what does not fill a group goes through the generic routine tile by tile.
// Functions of their own, so that their registers do not weigh on the other loops.
template <int DT, int kGroup>
__device__ __noinline__ void run_set_grouped(const SetRec& S, uint64_t t0, uint64_t t1, AccExact (*s_acc)[kWarps],
                                             const void* const* s_cand, int warp, int lane) {
    using E = IntElem<DT>;
    constexpr int kTileVecs = kTileElems / E::kPerVec;
    constexpr int kVecs = kGroup * kTileVecs / kThreads;                // vectors per thread per group
    const uint64_t full_tiles = S.vec_ok ? S.n / kTileElems : 0;
    uint64_t t = t0;
    for (; t + kGroup <= t1 && t + kGroup <= full_tiles; t += kGroup) {
        const uint64_t base = t * kTileVecs + threadIdx.x;
        const uint4* rp = static_cast<const uint4*>(S.ref) + base;
        uint4 r[kVecs];
#pragma unroll
        for (int v = 0; v < kVecs; ++v) r[v] = load_stream(rp + v * kThreads);
#pragma unroll 1
        for (uint32_t k = 0; k < S.k; ++k) {
            const uint4* cp = static_cast<const uint4*>(s_cand[k]) + base;
            uint4 c[kVecs];
#pragma unroll
            for (int v = 0; v < kVecs; ++v) c[v] = load_stream(cp + v * kThreads);
            uint32_t cnt = 0;
            unsigned long long md = 0;
#pragma unroll
            for (int v = 0; v < kVecs; ++v) E::vec(c[v], r[v], cnt, md);
            commit(cnt, md, &s_acc[k][warp], lane);
        }
    }
    if (t < t1) run_set_exact<DT>(S, t, t1, s_acc, s_cand, warp, lane);
}

__global__ void __launch_bounds__(kThreads, kCtasPerSmExact)
exact_pass1(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members, const CtaRange* __restrict__ ranges,
            AccExact* __restrict__ partials) {
    __shared__ AccExact s_acc[kMaxK][kWarps];
    __shared__ const void* s_cand[kMaxK];
    const CtaRange rg = ranges[blockIdx.x];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (uint32_t s = rg.s_begin; s <= rg.s_end; ++s) {
        const SetRec S = sets[s];
        const uint64_t tiles = (S.n + kTileElems - 1) / kTileElems;
        const uint64_t t0 = (s == rg.s_begin) ? rg.t_begin : 0;
        const uint64_t t1 = (s == rg.s_end) ? rg.t_end : tiles;
        if (t0 >= t1) continue;
        for (uint32_t i = threadIdx.x; i < S.k * kWarps; i += kThreads) s_acc[i / kWarps][i % kWarps] = AccExact{0ull, 0ull};
        if (threadIdx.x < S.k) s_cand[threadIdx.x] = members[S.member_off + threadIdx.x].cand;
        __syncthreads();
        if (S.dtype == EVO_I32) run_set_grouped<EVO_I32, 2>(S, t0, t1, s_acc, s_cand, warp, lane);
        else if (S.dtype == EVO_I64) run_set_exact<EVO_I64>(S, t0, t1, s_acc, s_cand, warp, lane);
        else run_set_grouped<EVO_U8, 4>(S, t0, t1, s_acc, s_cand, warp, lane);
        __syncthreads();
        if (threadIdx.x < S.k) {
            AccExact a = s_acc[threadIdx.x][0];
#pragma unroll
            for (int w = 1; w < kWarps; ++w) {
                const AccExact b = s_acc[threadIdx.x][w];
                a.mism += b.mism;
                a.maxdiff = b.maxdiff > a.maxdiff ? b.maxdiff : a.maxdiff;
            }
            partials[rg.part_base + (S.member_off - rg.first_member) + threadIdx.x] = a;
        }
        __syncthreads();
    }
}

// ---- the reference regenerated in the kernel (evo_validate_generated) ----------------------
// The reference of a set is a window of a Philox stream: SetRec::ref holds the stream position of
// its first element instead of an address.  A thread produces the four words of a 16-byte vector
// with one Philox block (two when the window does not start on a block boundary), so the reference
// costs arithmetic and no memory traffic; the candidates stream through registers as above.
template <bool SIGNED>
__device__ __forceinline__ void word_pair(uint32_t c, uint32_t r, uint32_t& cnt, uint32_t& md) {
    const bool gt = SIGNED ? static_cast<int32_t>(c) > static_cast<int32_t>(r) : c > r;
    const uint32_t d = gt ? c - r : r - c;            // |c - r| of two 32-bit values fits 32 unsigned bits
    cnt += d != 0 ? 1u : 0u;
    md = max(md, d);
}

// Words [pos, pos + 4) of the stream, pos any value.
__device__ __forceinline__ uint4 stream_vector(uint64_t pos, const RoundKeys& rk) {
    const uint4 a = philox4x32_10(pos >> 2, rk);
    const uint32_t lead = static_cast<uint32_t>(pos) & 3u;
    if (lead == 0) return a;
    const uint4 b = philox4x32_10((pos >> 2) + 1, rk);
    const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint4 v;
    v.x = lead == 1 ? w[1] : lead == 2 ? w[2] : w[3];
    v.y = lead == 1 ? w[2] : lead == 2 ? w[3] : w[4];
    v.z = lead == 1 ? w[3] : lead == 2 ? w[4] : w[5];
    v.w = lead == 1 ? w[4] : lead == 2 ? w[5] : w[6];
    return v;
}

__device__ __forceinline__ uint32_t stream_word(uint64_t pos, const RoundKeys& rk) {
    const uint4 a = philox4x32_10(pos >> 2, rk);
    const uint32_t lane = static_cast<uint32_t>(pos) & 3u;
    return lane == 0 ? a.x : lane == 1 ? a.y : lane == 2 ? a.z : a.w;
}

template <bool SIGNED>
__device__ __forceinline__ void run_set_generated(const RoundKeys& rk, const SetRec& S, uint64_t t0, uint64_t t1,
                                                  AccExact (*s_acc)[kWarps], const void* const* s_cand, int warp, int lane) {
    constexpr int kVecs = kEpt / 4;                       // 16-byte vectors per thread per tile
    constexpr int kTileVecs = kTileElems / 4;
    const uint64_t first = reinterpret_cast<uint64_t>(S.ref);       // stream position of element 0
    const uint64_t full_tiles = S.vec_ok ? S.n / kTileElems : 0;
    for (uint64_t t = t0; t < t1; ++t) {
        if (t < full_tiles) {
            const uint64_t base = t * kTileVecs + threadIdx.x;
            // the first member's loads are on their way while the reference is generated
            uint4 c[kVecs];
            {
                const uint4* cp = static_cast<const uint4*>(s_cand[0]) + base;
#pragma unroll
                for (int v = 0; v < kVecs; ++v) c[v] = load_stream(cp + v * kThreads);
            }
            uint4 r[kVecs];
#pragma unroll
            for (int v = 0; v < kVecs; ++v) r[v] = stream_vector(first + 4 * (base + static_cast<uint64_t>(v) * kThreads), rk);
#pragma unroll 1
            for (uint32_t k = 0; k < S.k; ++k) {
                if (k > 0) {
                    const uint4* cp = static_cast<const uint4*>(s_cand[k]) + base;
#pragma unroll
                    for (int v = 0; v < kVecs; ++v) c[v] = load_stream(cp + v * kThreads);
                }
                uint32_t cnt = 0, md = 0;
#pragma unroll
                for (int v = 0; v < kVecs; ++v) {
                    // equal vectors (the rule, not the exception) cost four xors and a branch
                    if (((c[v].x ^ r[v].x) | (c[v].y ^ r[v].y) | (c[v].z ^ r[v].z) | (c[v].w ^ r[v].w)) == 0u) continue;
                    word_pair<SIGNED>(c[v].x, r[v].x, cnt, md); word_pair<SIGNED>(c[v].y, r[v].y, cnt, md);
                    word_pair<SIGNED>(c[v].z, r[v].z, cnt, md); word_pair<SIGNED>(c[v].w, r[v].w, cnt, md);
                }
                commit(cnt, md, &s_acc[k][warp], lane);
            }
        } else {
            // ragged last tile, or candidates that are not 16-byte aligned: element by element
            const uint64_t e0 = t * kTileElems;
            const uint64_t e1 = min(S.n, e0 + kTileElems);
            for (uint64_t e = e0 + threadIdx.x; e < e0 + kTileElems; e += kThreads) {      // uniform trip count: commit is collective
                const bool in = e < e1;
                const uint32_t r = in ? stream_word(first + e, rk) : 0u;
                for (uint32_t k = 0; k < S.k; ++k) {
                    uint32_t cnt = 0, md = 0;
                    if (in) word_pair<SIGNED>(static_cast<const uint32_t*>(s_cand[k])[e], r, cnt, md);
                    commit(cnt, md, &s_acc[k][warp], lane);
                }
            }
        }
    }
}

__global__ void __launch_bounds__(kThreads, kCtasPerSmExact)
generated_pass1(const __grid_constant__ RoundKeys rk, const SetRec* __restrict__ sets, const MemberRec* __restrict__ members,
                const CtaRange* __restrict__ ranges, AccExact* __restrict__ partials) {
    __shared__ AccExact s_acc[kMaxK][kWarps];
    __shared__ const void* s_cand[kMaxK];
    const CtaRange rg = ranges[blockIdx.x];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (uint32_t s = rg.s_begin; s <= rg.s_end; ++s) {
        const SetRec S = sets[s];
        const uint64_t tiles = (S.n + kTileElems - 1) / kTileElems;
        const uint64_t t0 = (s == rg.s_begin) ? rg.t_begin : 0;
        const uint64_t t1 = (s == rg.s_end) ? rg.t_end : tiles;
        if (t0 >= t1) continue;
        for (uint32_t i = threadIdx.x; i < S.k * kWarps; i += kThreads) s_acc[i / kWarps][i % kWarps] = AccExact{0ull, 0ull};
        if (threadIdx.x < S.k) s_cand[threadIdx.x] = members[S.member_off + threadIdx.x].cand;
        __syncthreads();
        if (S.dtype == EVO_I32) run_set_generated<true>(rk, S, t0, t1, s_acc, s_cand, warp, lane);
        else run_set_generated<false>(rk, S, t0, t1, s_acc, s_cand, warp, lane);
        __syncthreads();
        if (threadIdx.x < S.k) {
            AccExact a = s_acc[threadIdx.x][0];
#pragma unroll
            for (int w = 1; w < kWarps; ++w) {
                const AccExact b = s_acc[threadIdx.x][w];
                a.mism += b.mism;
                a.maxdiff = b.maxdiff > a.maxdiff ? b.maxdiff : a.maxdiff;
            }
            partials[rg.part_base + (S.member_off - rg.first_member) + threadIdx.x] = a;
        }
        __syncthreads();
    }
}

// One warp per tensor: fold the partial records of the CTAs [cta_first, cta_last] of its set.
__global__ void __launch_bounds__(kThreads)
exact_pass2(const SetRec* __restrict__ sets, const MemberRec* __restrict__ members, const CtaRange* __restrict__ ranges,
            const AccExact* __restrict__ partials, uint32_t n_members, evo_result_exact* __restrict__ results) {
    const uint32_t m = blockIdx.x * kWarps + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (m >= n_members) return;
    const MemberRec M = members[m];
    const SetRec S = sets[M.set];
    unsigned long long mism = 0, md = 0;
    if (S.cta_first <= S.cta_last) {
        for (uint32_t b = S.cta_first + lane; b <= S.cta_last; b += 32) {
            const CtaRange R = ranges[b];
            const AccExact p = partials[R.part_base + (m - R.first_member)];
            mism += p.mism;
            md = p.maxdiff > md ? p.maxdiff : md;
        }
    }
    const unsigned full = 0xffffffffu;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        mism += __shfl_xor_sync(full, mism, o);
        const unsigned long long other = __shfl_xor_sync(full, md, o);
        md = other > md ? other : md;
    }
    if (lane == 0) {
        evo_result_exact r;
        r.n_mismatch = mism; r.max_abs_diff = md; r.pass = mism == 0 ? 1u : 0u; r.pad = 0;
        results[M.desc] = r;
    }
}

__global__ void exact_verdict(const uint32_t* __restrict__ offsets, const uint32_t* __restrict__ desc_of,
                              const evo_result_exact* __restrict__ results, uint32_t n_group, uint32_t* __restrict__ group_pass) {
    const uint32_t g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= n_group) return;
    uint32_t ok = 1;
    for (uint32_t i = offsets[g]; i < offsets[g + 1]; ++i) ok &= results[desc_of[i]].pass;
    group_pass[g] = ok;
}

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Device addresses of an uploaded plan.
struct DevicePlan {
    const SetRec* sets; const MemberRec* members; const CtaRange* ranges; const uint32_t* goff; const uint32_t* gdesc;
    AccExact* parts;
};

// Packs the plan into the context's pinned block, copies it to the device on `stream` and sizes the
// partial records (one pinned block, one copy, as evo_validate does for large plans).
int upload_plan(evo_ctx* ctx, const Plan& plan, cudaStream_t stream, DevicePlan* out) {
    const size_t o_sets = 0;
    const size_t o_members = align_up(o_sets + plan.sets.size() * sizeof(SetRec), 256);
    const size_t o_ranges = align_up(o_members + plan.members.size() * sizeof(MemberRec), 256);
    const size_t o_goff = align_up(o_ranges + plan.ranges.size() * sizeof(CtaRange), 256);
    const size_t o_gdesc = align_up(o_goff + plan.group_off.size() * 4, 256);
    const size_t plan_bytes = align_up(o_gdesc + plan.group_desc.size() * 4, 256) + 256;
    ctx->plan_key_valid = false;          // the plan area is about to hold this call's plan
    int st = evo::reserve_pinned(ctx, &ctx->h_plan, &ctx->h_plan_bytes, plan_bytes);
    if (st != EVO_OK) return st;
    st = evo::reserve_device(ctx, &ctx->d_plan, &ctx->d_plan_bytes, plan_bytes);
    if (st != EVO_OK) return st;
    st = evo::reserve_device(ctx, &ctx->d_partials, &ctx->d_partials_bytes, std::max<size_t>(plan.n_parts, 1) * sizeof(Acc));
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
    out->sets = reinterpret_cast<const SetRec*>(d + o_sets);
    out->members = reinterpret_cast<const MemberRec*>(d + o_members);
    out->ranges = reinterpret_cast<const CtaRange*>(d + o_ranges);
    out->goff = reinterpret_cast<const uint32_t*>(d + o_goff);
    out->gdesc = reinterpret_cast<const uint32_t*>(d + o_gdesc);
    out->parts = static_cast<AccExact*>(ctx->d_partials);          // 16-byte records in a block sized for 40-byte ones
    return EVO_OK;
}

// Second pass and verdicts, the same after either first pass.
int finish_exact(evo_ctx* ctx, const DevicePlan& d, uint64_t n_desc, evo_result_exact* results, uint32_t* group_pass,
                 uint64_t n_group, cudaStream_t stream) {
    const uint32_t n_members = static_cast<uint32_t>(n_desc);
    if (n_members > 0) {
        exact_pass2<<<(n_members + kWarps - 1) / kWarps, kThreads, 0, stream>>>(d.sets, d.members, d.ranges, d.parts, n_members,
                                                                                 results);
        ctx->launches += 1;
        EVO_CUDA_TRY(ctx, cudaGetLastError());
    }
    if (group_pass) {
        exact_verdict<<<static_cast<unsigned>((n_group + 255) / 256), 256, 0, stream>>>(d.goff, d.gdesc, results,
                                                                                        static_cast<uint32_t>(n_group), group_pass);
        ctx->launches += 1;
        EVO_CUDA_TRY(ctx, cudaGetLastError());
    }
    return EVO_OK;
}

}  // namespace

extern "C" int evo_validate_exact(evo_ctx* ctx, const void* const* cand_ptrs, const void* ref_ptr, const evo_desc* descs,
                                  uint64_t n_desc, int dtype, evo_result_exact* results, uint32_t* group_pass,
                                  uint64_t n_group, void* stream_) {
    if (!ctx) return EVO_ERR_ARG;
    const char* who = "evo_validate_exact";
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (n_desc > 0 && !results) return evo::fail(ctx, EVO_ERR_ARG, "%s: results must not be NULL", who);
    Plan plan;
    std::string err;
    const uint32_t max_ctas = static_cast<uint32_t>(ctx->sm_count) * kCtasPerSmExact;
    int st = build_plan(cand_ptrs, ref_ptr, descs, n_desc, dtype, 0.f, 0.f, group_pass != nullptr, n_group, max_ctas, &plan,
                        &err, kIntTypes);
    if (st != EVO_OK) return evo::fail(ctx, st, "%s: %s", who, err.c_str());
    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");
    DevicePlan d;
    st = upload_plan(ctx, plan, stream, &d);
    if (st != EVO_OK) return st;
    const uint32_t n_ctas = static_cast<uint32_t>(plan.ranges.size());
    if (n_ctas > 0) {
        exact_pass1<<<n_ctas, kThreads, 0, stream>>>(d.sets, d.members, d.ranges, d.parts);
        ctx->launches += 1;
        EVO_CUDA_TRY(ctx, cudaGetLastError());
    }
    return finish_exact(ctx, d, n_desc, results, group_pass, n_group, stream);
}

extern "C" int evo_validate_generated(evo_ctx* ctx, uint64_t seed, uint64_t offset, const uint64_t* offsets,
                                      const void* const* cand_ptrs, const uint64_t* counts, uint64_t n_desc, int dtype,
                                      const uint32_t* groups, evo_result_exact* results, uint32_t* group_pass,
                                      uint64_t n_group, void* stream_) {
    if (!ctx) return EVO_ERR_ARG;
    const char* who = "evo_validate_generated";
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (dtype != EVO_I32 && dtype != EVO_U32) return evo::fail(ctx, EVO_ERR_DTYPE, "%s: dtype %d (EVO_I32 or EVO_U32)", who, dtype);
    if (n_desc > 0 && (!results || !counts || !cand_ptrs))
        return evo::fail(ctx, EVO_ERR_ARG, "%s: cand_ptrs, counts and results must not be NULL", who);
    if (group_pass && n_desc > 0 && !groups) return evo::fail(ctx, EVO_ERR_ARG, "%s: group_pass without groups", who);
    // Descriptors for the planner: tensors with the same window of the stream form a set, exactly as tensors
    // with the same reference do.  The planner keys sets by the reference's address, so every distinct window
    // start gets a stand-in address (16-byte aligned, never dereferenced), replaced by the stream position below.
    std::vector<evo_desc> descs(n_desc);
    std::unordered_map<uint64_t, uintptr_t> token_of;
    std::vector<uint64_t> start_of_token;
    for (uint64_t i = 0; i < n_desc; ++i) {
        const uint64_t start = offsets ? offsets[i] : offset;
        if (counts[i] > (1ull << 60)) return evo::fail(ctx, EVO_ERR_ARG, "%s: tensor %llu is too large", who, (unsigned long long)i);
        auto it = token_of.find(start);
        if (it == token_of.end()) {
            start_of_token.push_back(start);
            it = token_of.emplace(start, static_cast<uintptr_t>(16 * start_of_token.size())).first;
        }
        descs[i].n = counts[i];
        descs[i].ref = reinterpret_cast<const void*>(it->second);
        descs[i].dtype = dtype;
        descs[i].group = groups ? groups[i] : 0u;
    }
    Plan plan;
    std::string err;
    const uint32_t max_ctas = static_cast<uint32_t>(ctx->sm_count) * kCtasPerSmExact;
    int st = build_plan(cand_ptrs, nullptr, descs.data(), n_desc, dtype, 0.f, 0.f, group_pass != nullptr, n_group, max_ctas,
                        &plan, &err, kWordTypes);
    if (st != EVO_OK) return evo::fail(ctx, st, "%s: %s", who, err.c_str());
    for (SetRec& S : plan.sets) {
        const uintptr_t token = reinterpret_cast<uintptr_t>(S.ref);
        S.ref = reinterpret_cast<const void*>(static_cast<uintptr_t>(token ? start_of_token[token / 16 - 1] : 0));
    }
    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");
    DevicePlan d;
    st = upload_plan(ctx, plan, stream, &d);
    if (st != EVO_OK) return st;
    const uint32_t n_ctas = static_cast<uint32_t>(plan.ranges.size());
    if (n_ctas > 0) {
        generated_pass1<<<n_ctas, kThreads, 0, stream>>>(round_keys(seed), d.sets, d.members, d.ranges, d.parts);
        ctx->launches += 1;
        EVO_CUDA_TRY(ctx, cudaGetLastError());
    }
    return finish_exact(ctx, d, n_desc, results, group_pass, n_group, stream);
}
