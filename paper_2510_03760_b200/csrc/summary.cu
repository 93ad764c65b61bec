// evo_summary: the paper's reporting metrics (Section 5.1 "Evaluation Metric": median speedup
// across kernels with 1.0 where no candidate beats the baseline, averaged over the independent
// runs; Pass@1 = share of trials that are valid; Appendix A.5: kernels counted by speedup
// range) from the device-resident per-candidate records that evo_fitness wrote.
//
// A few thousand records and about a hundred kernels: latency only.  Three small launches:
//   1. per (run, kernel) the best valid speedup, by a maximum on the bit patterns (non-negative
//      binary32 values order like unsigned integers; a maximum does not depend on the order of
//      arrival, so the atomics do not cost reproducibility), and the count of valid candidates;
//   2. one CTA: per run the median over kernels of max(best, 1) by rank counting, the mean of
//      those medians in binary64 in run order, the counts per speedup range.
#include <algorithm>

#include "evo_internal.h"

namespace {

constexpr uint32_t kMaxKernels = 8192;      // one run's values must fit the final CTA's shared memory
constexpr uint32_t kMaxRuns = 1024;
constexpr int kFinalThreads = 1024;

__global__ void summary_best(const evo_fit* __restrict__ fits, const uint32_t* __restrict__ kernel_of,
                             const uint32_t* __restrict__ run_of, uint64_t n_cand, uint32_t n_kernel, uint32_t n_run,
                             uint32_t* __restrict__ best_bits, uint32_t* __restrict__ n_valid, uint32_t* __restrict__ status) {
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    uint32_t mine = 0;
    for (uint64_t i = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x; i < n_cand; i += stride) {
        const uint32_t k = kernel_of[i], r = run_of ? run_of[i] : 0u;
        if (k >= n_kernel || r >= n_run) { atomicOr(status, 4u); continue; }
        const evo_fit f = fits[i];
        if (!f.valid) continue;
        ++mine;
        atomicMax(&best_bits[static_cast<size_t>(r) * n_kernel + k], __float_as_uint(f.speedup));
    }
    mine = __reduce_add_sync(0xffffffffu, mine);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(n_valid, mine);
}

__global__ void __launch_bounds__(kFinalThreads)
summary_final(const float* __restrict__ best, uint64_t n_cand, uint32_t n_kernel, uint32_t n_run,
              const uint32_t* __restrict__ n_valid, evo_summary_rec* __restrict__ out, float* __restrict__ run_median) {
    extern __shared__ float s_v[];                 // n_kernel floored values of the current run
    __shared__ float s_mid[2];
    __shared__ uint32_t s_hist[5], s_count;
    __shared__ double s_sum;
    const uint32_t tid = threadIdx.x;
    if (tid < 5) s_hist[tid] = 0;
    if (tid == 0) { s_count = 0; s_sum = 0.0; }
    const uint32_t lo = (n_kernel - 1) / 2, hi = n_kernel / 2;
    for (uint32_t r = 0; r < n_run; ++r) {
        __syncthreads();
        for (uint32_t k = tid; k < n_kernel; k += kFinalThreads) {
            const float x = best[static_cast<size_t>(r) * n_kernel + k];
            s_v[k] = x > 1.0f ? x : 1.0f;
        }
        __syncthreads();
        for (uint32_t i = tid; i < n_kernel; i += kFinalThreads) {
            const float x = s_v[i];
            uint32_t rank = 0;
            for (uint32_t j = 0; j < n_kernel; ++j) {
                const float y = s_v[j];
                rank += (y < x || (y == x && j < i)) ? 1u : 0u;
            }
            if (rank == lo) s_mid[0] = x;
            if (rank == hi) s_mid[1] = x;
        }
        __syncthreads();
        if (tid == 0) {
            const float med = (lo == hi) ? s_mid[0] : __fmul_rn(0.5f, __fadd_rn(s_mid[0], s_mid[1]));
            if (run_median) run_median[r] = med;
            s_sum += static_cast<double>(med);     // run order: one thread, fixed sequence
        }
    }
    // kernels by their best over all runs
    for (uint32_t k = tid; k < n_kernel; k += kFinalThreads) {
        float top = 0.f;
        for (uint32_t r = 0; r < n_run; ++r) top = fmaxf(top, best[static_cast<size_t>(r) * n_kernel + k]);
        if (top > 1.0f) atomicAdd(&s_count, 1u);
        const int bin = top < 1.0f ? 0 : top < 2.0f ? 1 : top < 5.0f ? 2 : top < 10.0f ? 3 : 4;
        atomicAdd(&s_hist[bin], 1u);
    }
    __syncthreads();
    if (tid == 0) {
        evo_summary_rec s;
        s.median_speedup = static_cast<float>(s_sum / static_cast<double>(n_run));
        s.n_valid = *n_valid;
        s.n_cand = static_cast<uint32_t>(n_cand);
        s.validity = n_cand ? static_cast<float>(static_cast<double>(s.n_valid) / static_cast<double>(n_cand)) : 0.f;
        s.speedup_count = s_count;
        for (int b = 0; b < 5; ++b) s.hist[b] = s_hist[b];
        s.n_kernel = n_kernel;
        s.n_run = n_run;
        *out = s;
    }
}

}  // namespace

extern "C" int evo_summary(evo_ctx* ctx, const evo_fit* fits, const uint32_t* kernel_of, const uint32_t* run_of,
                           uint64_t n_cand, uint32_t n_kernel, uint32_t n_run, evo_summary_rec* out, float* best,
                           float* run_median, void* stream_) {
    if (!ctx) return EVO_ERR_ARG;
    const char* who = "evo_summary";
    if (n_kernel == 0 || n_kernel > kMaxKernels || n_run == 0 || n_run > kMaxRuns)
        return evo::fail(ctx, EVO_ERR_ARG, "%s: n_kernel must be in [1, %u] and n_run in [1, %u]", who, kMaxKernels, kMaxRuns);
    if (!out || !best || (n_cand > 0 && (!fits || !kernel_of)))
        return evo::fail(ctx, EVO_ERR_ARG, "%s: fits, kernel_of, out and best must not be NULL", who);
    if (n_cand >= (1ull << 32)) return evo::fail(ctx, EVO_ERR_ARG, "%s: too many candidates", who);
    if (reinterpret_cast<uintptr_t>(fits) % 4 || reinterpret_cast<uintptr_t>(out) % 4 || reinterpret_cast<uintptr_t>(best) % 4)
        return evo::fail(ctx, EVO_ERR_ALIGN, "%s: arrays must be 4-byte aligned", who);
    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    uint32_t* d_valid = reinterpret_cast<uint32_t*>(static_cast<char*>(ctx->d_small) + 64);
    EVO_CUDA_TRY(ctx, cudaMemsetAsync(best, 0, static_cast<size_t>(n_run) * n_kernel * sizeof(float), stream));
    EVO_CUDA_TRY(ctx, cudaMemsetAsync(d_valid, 0, sizeof(uint32_t), stream));
    if (n_cand > 0) {
        const unsigned grid = static_cast<unsigned>(std::min<uint64_t>((n_cand + 255) / 256, static_cast<uint64_t>(ctx->sm_count) * 8));
        summary_best<<<grid, 256, 0, stream>>>(fits, kernel_of, run_of, n_cand, n_kernel, n_run,
                                               reinterpret_cast<uint32_t*>(best), d_valid, evo::status_word(ctx));
        ctx->launches += 1;
        EVO_CUDA_TRY(ctx, cudaGetLastError());
    }
    summary_final<<<1, kFinalThreads, n_kernel * sizeof(float), stream>>>(best, n_cand, n_kernel, n_run, d_valid, out, run_median);
    ctx->launches += 1;
    EVO_CUDA_TRY(ctx, cudaGetLastError());
    return EVO_OK;
}

// ---- evo_select_elite -----------------------------------------------------------------------
// Population management (Section 4.2: the single-solution strategy keeps the best candidate,
// elite preservation a small set of high-performing ones): the k valid candidates with the
// largest speedup, best first, equal speedups by index.  Rank counting again: a candidate's
// place is the number of valid candidates ahead of it, so there is no sort and the outcome
// is unique.  Quadratic in the population, which is a few thousand records.
namespace {

constexpr uint32_t kMaxEliteCands = 1u << 16;
constexpr int kEliteThreads = 256;

__global__ void __launch_bounds__(kEliteThreads)
elite_kernel(const evo_fit* __restrict__ fits, uint32_t n_cand, uint32_t k, uint32_t* __restrict__ idx,
             uint32_t* __restrict__ count) {
    __shared__ float s_speed[kEliteThreads];
    __shared__ uint32_t s_valid[kEliteThreads];
    const uint32_t i = blockIdx.x * kEliteThreads + threadIdx.x;
    float mine = 0.f;
    bool valid = false;
    if (i < n_cand) { const evo_fit f = fits[i]; mine = f.speedup; valid = f.valid != 0; }
    uint32_t ahead = 0;
    for (uint32_t base = 0; base < n_cand; base += kEliteThreads) {
        const uint32_t j = base + threadIdx.x;
        __syncthreads();
        if (j < n_cand) { const evo_fit f = fits[j]; s_speed[threadIdx.x] = f.speedup; s_valid[threadIdx.x] = f.valid; }
        else s_valid[threadIdx.x] = 0;
        __syncthreads();
        const uint32_t lim = min(static_cast<uint32_t>(kEliteThreads), n_cand - base);
        for (uint32_t q = 0; q < lim; ++q) {
            const float s = s_speed[q];
            ahead += (s_valid[q] && (s > mine || (s == mine && base + q < i))) ? 1u : 0u;
        }
    }
    if (valid && ahead < k) {
        idx[ahead] = i;
        atomicAdd(count, 1u);           // an integer count: the order of arrival does not matter
    }
}

}  // namespace

extern "C" int evo_select_elite(evo_ctx* ctx, const evo_fit* fits, uint64_t n_cand, uint32_t k, uint32_t* idx,
                                uint32_t* count, void* stream_) {
    if (!ctx) return EVO_ERR_ARG;
    const char* who = "evo_select_elite";
    if (n_cand > kMaxEliteCands) return evo::fail(ctx, EVO_ERR_ARG, "%s: at most %u candidates per call", who, kMaxEliteCands);
    if (!count || (k > 0 && !idx) || (n_cand > 0 && !fits)) return evo::fail(ctx, EVO_ERR_ARG, "%s: fits, idx and count must not be NULL", who);
    if (reinterpret_cast<uintptr_t>(fits) % 4 || reinterpret_cast<uintptr_t>(idx) % 4 || reinterpret_cast<uintptr_t>(count) % 4)
        return evo::fail(ctx, EVO_ERR_ALIGN, "%s: arrays must be 4-byte aligned", who);
    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    if (k > 0) EVO_CUDA_TRY(ctx, cudaMemsetAsync(idx, 0xff, static_cast<size_t>(k) * sizeof(uint32_t), stream));
    EVO_CUDA_TRY(ctx, cudaMemsetAsync(count, 0, sizeof(uint32_t), stream));
    if (n_cand > 0 && k > 0) {
        const unsigned grid = static_cast<unsigned>((n_cand + kEliteThreads - 1) / kEliteThreads);
        elite_kernel<<<grid, kEliteThreads, 0, stream>>>(fits, static_cast<uint32_t>(n_cand), k, idx, count);
        ctx->launches += 1;
        EVO_CUDA_TRY(ctx, cudaGetLastError());
    }
    return EVO_OK;
}
