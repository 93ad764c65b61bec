// evo_mismatch_sample: feedback on a failing candidate (paper Section 4.3: the third step of
// the system is feedback collection for the next round of generation) - where its output is
// wrong.  The first max_out elements, in index order, that violate the closeness rule, with
// their values, and the total number of violations.
//
// A diagnostic for candidates that already failed evo_validate, so simplicity wins over the
// last bit of bandwidth: the tensor is read twice with coalesced element loads.
//   count  per chunk of 2048 elements the number of violations
//   scan   one CTA: exclusive prefix over the chunks (64-bit), total -> n_found
//   write  chunks whose prefix is below max_out judge their elements again and write each
//          offender at prefix + its rank inside the chunk (ballots and a scan over the warps),
//          which is its rank in index order: the output is unique, no atomics involved.
#include <algorithm>
#include <cmath>

#include "evo_internal.h"
#include "rule.cuh"

namespace {

using namespace evo;

constexpr int kFbThreads = 256;
constexpr int kFbRows = 8;
constexpr uint32_t kChunk = kFbThreads * kFbRows;       // 2048 elements; element (row, tid) = chunk*2048 + row*256 + tid

template <int DT>
__global__ void __launch_bounds__(kFbThreads)
offender_count(const void* __restrict__ cand_, const void* __restrict__ ref_, uint64_t n, float atol, float rtol,
               uint64_t n_chunks, unsigned long long* __restrict__ counts) {
    using T = typename Elem<DT>::T;
    const T* cand = static_cast<const T*>(cand_);
    const T* ref = static_cast<const T*>(ref_);
    __shared__ uint32_t s_warp[kFbThreads / 32];
    for (uint64_t ch = blockIdx.x; ch < n_chunks; ch += gridDim.x) {
        uint32_t mine = 0;
#pragma unroll
        for (int row = 0; row < kFbRows; ++row) {
            const uint64_t e = ch * kChunk + row * kFbThreads + threadIdx.x;
            if (e < n) mine += rule_mismatch(Elem<DT>::widen(cand[e]), Elem<DT>::widen(ref[e]), atol, rtol) ? 1u : 0u;
        }
        mine = __reduce_add_sync(0xffffffffu, mine);
        if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = mine;
        __syncthreads();
        if (threadIdx.x == 0) {
            uint32_t t = 0;
            for (int w = 0; w < kFbThreads / 32; ++w) t += s_warp[w];
            counts[ch] = t;
        }
        __syncthreads();
    }
}

// In place: counts[] -> exclusive prefix; *n_found = total.  One CTA walks the array in
// slices of blockDim.x with a carried running total.
__global__ void __launch_bounds__(1024)
offender_scan(unsigned long long* __restrict__ counts, uint64_t n_chunks, unsigned long long* __restrict__ n_found) {
    __shared__ unsigned long long s_warp[32];
    __shared__ unsigned long long s_carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) s_carry = 0;
    __syncthreads();
    for (uint64_t base = 0; base < n_chunks; base += blockDim.x) {
        const uint64_t i = base + threadIdx.x;
        const unsigned long long x = i < n_chunks ? counts[i] : 0ull;
        unsigned long long incl = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long y = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += y;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            unsigned long long w = s_warp[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned long long y = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o) w += y;
            }
            s_warp[lane] = w;                     // inclusive over the warps
        }
        __syncthreads();
        const unsigned long long before = s_carry + (warp ? s_warp[warp - 1] : 0ull) + (incl - x);
        if (i < n_chunks) counts[i] = before;
        __syncthreads();
        if (threadIdx.x == blockDim.x - 1) s_carry = before + x;
        __syncthreads();
    }
    if (threadIdx.x == 0) *n_found = s_carry;
}

template <int DT>
__global__ void __launch_bounds__(kFbThreads)
offender_write(const void* __restrict__ cand_, const void* __restrict__ ref_, uint64_t n, float atol, float rtol,
               uint64_t n_chunks, const unsigned long long* __restrict__ prefix, const unsigned long long* __restrict__ n_found,
               uint64_t max_out, evo_offender* __restrict__ out) {
    using T = typename Elem<DT>::T;
    const T* cand = static_cast<const T*>(cand_);
    const T* ref = static_cast<const T*>(ref_);
    __shared__ uint32_t s_warp[kFbThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned long long total = *n_found;
    for (uint64_t ch = blockIdx.x; ch < n_chunks; ch += gridDim.x) {
        const unsigned long long first = prefix[ch];
        const unsigned long long next = ch + 1 < n_chunks ? prefix[ch + 1] : total;
        if (first >= max_out || next == first) continue;          // the same for the whole CTA
        unsigned long long pos = first;
#pragma unroll 1
        for (int row = 0; row < kFbRows; ++row) {
            const uint64_t e = ch * kChunk + row * kFbThreads + threadIdx.x;
            float c = 0.f, r = 0.f;
            bool bad = false;
            if (e < n) {
                c = Elem<DT>::widen(cand[e]);
                r = Elem<DT>::widen(ref[e]);
                bad = rule_mismatch(c, r, atol, rtol);
            }
            const uint32_t ballot = __ballot_sync(0xffffffffu, bad);
            if (lane == 0) s_warp[warp] = __popc(ballot);
            __syncthreads();
            uint32_t before = 0, row_total = 0;
#pragma unroll
            for (int w = 0; w < kFbThreads / 32; ++w) {
                const uint32_t cw = s_warp[w];
                before += w < warp ? cw : 0u;
                row_total += cw;
            }
            if (bad) {
                const unsigned long long at = pos + before + __popc(ballot & ((1u << lane) - 1u));
                if (at < max_out) { evo_offender o; o.index = e; o.cand = c; o.ref = r; out[at] = o; }
            }
            pos += row_total;
            __syncthreads();
        }
    }
}

template <int DT>
int run(evo_ctx* ctx, const void* cand, const void* ref, uint64_t n, float atol, float rtol, uint64_t max_out,
        evo_offender* out, unsigned long long* n_found, unsigned long long* counts, uint64_t n_chunks, cudaStream_t stream) {
    const unsigned grid = static_cast<unsigned>(std::min<uint64_t>(n_chunks, static_cast<uint64_t>(ctx->sm_count) * 16));
    offender_count<DT><<<grid, kFbThreads, 0, stream>>>(cand, ref, n, atol, rtol, n_chunks, counts);
    EVO_CUDA_TRY(ctx, cudaGetLastError());
    offender_scan<<<1, 1024, 0, stream>>>(counts, n_chunks, n_found);
    EVO_CUDA_TRY(ctx, cudaGetLastError());
    ctx->launches += 2;
    if (max_out > 0) {
        offender_write<DT><<<grid, kFbThreads, 0, stream>>>(cand, ref, n, atol, rtol, n_chunks, counts, n_found, max_out, out);
        EVO_CUDA_TRY(ctx, cudaGetLastError());
        ctx->launches += 1;
    }
    return EVO_OK;
}

}  // namespace

extern "C" int evo_mismatch_sample(evo_ctx* ctx, const void* cand, const void* ref, uint64_t n, int dtype, float atol,
                                   float rtol, uint64_t max_out, evo_offender* out, uint64_t* n_found, void* stream_) {
    if (!ctx) return EVO_ERR_ARG;
    const char* who = "evo_mismatch_sample";
    if (dtype != EVO_F32 && dtype != EVO_F16 && dtype != EVO_BF16) return evo::fail(ctx, EVO_ERR_DTYPE, "%s: dtype %d", who, dtype);
    if (!(atol >= 0.f) || !(rtol >= 0.f) || std::isinf(atol) || std::isinf(rtol))
        return evo::fail(ctx, EVO_ERR_ARG, "%s: atol and rtol must be finite and >= 0", who);
    if (!n_found || (max_out > 0 && !out) || (n > 0 && (!cand || !ref)))
        return evo::fail(ctx, EVO_ERR_ARG, "%s: cand, ref, out and n_found must not be NULL", who);
    if (n > (1ull << 60)) return evo::fail(ctx, EVO_ERR_ARG, "%s: n too large", who);
    const size_t eb = evo::elem_bytes(dtype);
    if (reinterpret_cast<uintptr_t>(cand) % eb || reinterpret_cast<uintptr_t>(ref) % eb || reinterpret_cast<uintptr_t>(out) % 8 ||
        reinterpret_cast<uintptr_t>(n_found) % 8)
        return evo::fail(ctx, EVO_ERR_ALIGN, "%s: tensors must be aligned to their element size, out and n_found to 8 bytes", who);
    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (n == 0) {
        EVO_CUDA_TRY(ctx, cudaMemsetAsync(n_found, 0, sizeof(uint64_t), stream));
        return EVO_OK;
    }
    const uint64_t n_chunks = (n + kChunk - 1) / kChunk;
    int st = evo::reserve_device(ctx, &ctx->d_feedback, &ctx->d_feedback_bytes, n_chunks * sizeof(unsigned long long));
    if (st != EVO_OK) return st;
    unsigned long long* counts = static_cast<unsigned long long*>(ctx->d_feedback);
    unsigned long long* found = reinterpret_cast<unsigned long long*>(n_found);
    switch (dtype) {
        case EVO_F32: return run<EVO_F32>(ctx, cand, ref, n, atol, rtol, max_out, out, found, counts, n_chunks, stream);
        case EVO_F16: return run<EVO_F16>(ctx, cand, ref, n, atol, rtol, max_out, out, found, counts, n_chunks, stream);
        default:      return run<EVO_BF16>(ctx, cand, ref, n, atol, rtol, max_out, out, found, counts, n_chunks, stream);
    }
}
