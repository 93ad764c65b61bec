// evo_fitness: the performance objective f(p) of the paper's formulation (Section 3.1 Eq. 1):
// the speedup of a candidate over the baseline kernel (Section 5.1 "Evaluation Metric") from
// the medians of their run times (Section 4.3: times over repeated runs; Appendix A.7.1: the
// median of the runs is taken).
//
// A few hundred floats per candidate: this is latency, not bandwidth.  One warp owns one row
// of times in shared memory and selects the middle order statistic(s) by rank counting
// (rank of x_i = number of j with x_j < x_i, or x_j == x_i and j < i), which needs no sort and
// is independent of the order in which the trials arrive.
#include <algorithm>

#include "evo_internal.h"

namespace {

constexpr int kWarpsPerCta = 4;
constexpr uint32_t kMaxTrials = 4096;

struct RowMedian { float median; uint32_t ok; };

// Statistic of row[0..m) held in shared memory, computed by one warp.  ok = 0 when a time is
// NaN, Inf or not positive.  All lanes return the same value.
//   median        middle order statistic, or 0.5 * (a + b) of the two middle ones (binary32)
//   mean          binary64 sum in run order, one division, one rounding to binary32
//   min           the smallest run
//   trimmed mean  runs ranked, `trim` dropped at each end, binary64 sum in ascending order
// Order statistics come from rank counting (rank of x_i = number of j with x_j < x_i, or
// x_j == x_i and j < i): no sort, and the result does not depend on the order of the runs.
// The sums are taken by one lane in a fixed order, so they are reproducible bit for bit.
__device__ RowMedian warp_statistic(const float* row, uint32_t m, int stat, uint32_t trim, int lane,
                                    float* slot /* 2 floats */, float* sorted /* m floats, trimmed mean only */) {
    const unsigned full = 0xffffffffu;
    bool bad = false;
    for (uint32_t i = lane; i < m; i += 32) {
        const float x = row[i];
        bad |= !(x > 0.f && x < __int_as_float(0x7f800000));
    }
    if (__any_sync(full, bad)) return RowMedian{0.f, 0u};
    if (stat == EVO_STAT_MEAN) {
        if (lane == 0) {
            double sum = 0.0;
            for (uint32_t i = 0; i < m; ++i) sum += static_cast<double>(row[i]);
            slot[0] = static_cast<float>(sum / static_cast<double>(m));
        }
        __syncwarp();
        const float v = slot[0];
        __syncwarp();
        return RowMedian{v, 1u};
    }
    if (stat == EVO_STAT_MIN) {
        float lo = __int_as_float(0x7f800000);
        for (uint32_t i = lane; i < m; i += 32) lo = fminf(lo, row[i]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) lo = fminf(lo, __shfl_xor_sync(full, lo, o));
        return RowMedian{lo, 1u};
    }
    const uint32_t lo = (m - 1) / 2, hi = m / 2;     // equal when m is odd
    for (uint32_t i = lane; i < m; i += 32) {
        const float x = row[i];
        uint32_t rank = 0;
        for (uint32_t j = 0; j < m; ++j) {
            const float y = row[j];
            rank += (y < x || (y == x && j < i)) ? 1u : 0u;
        }
        if (stat == EVO_STAT_TRIMMED_MEAN) {
            sorted[rank] = x;
        } else {
            if (rank == lo) slot[0] = x;
            if (rank == hi) slot[1] = x;
        }
    }
    __syncwarp();
    if (stat == EVO_STAT_TRIMMED_MEAN) {
        if (lane == 0) {
            double sum = 0.0;
            for (uint32_t i = trim; i < m - trim; ++i) sum += static_cast<double>(sorted[i]);
            slot[0] = static_cast<float>(sum / static_cast<double>(m - 2 * trim));
        }
        __syncwarp();
        const float v = slot[0];
        __syncwarp();
        return RowMedian{v, 1u};
    }
    const float a = slot[0], b = slot[1];
    __syncwarp();
    const float med = (lo == hi) ? a : __fmul_rn(0.5f, __fadd_rn(a, b));
    return RowMedian{med, 1u};
}

// One launch: warps 0..3 of a CTA take one row of candidate times each, warp 4 takes the
// baseline row (every CTA computes the baseline's statistic again: a hundred floats, cheaper
// than a launch of its own and a dependency on it).
__global__ void __launch_bounds__((kWarpsPerCta + 1) * 32)
fitness_kernel(const float* __restrict__ times, uint64_t n_rows, uint32_t trials, const float* __restrict__ base_times,
               uint32_t base_trials, int stat, uint32_t warmup, uint32_t trim, const uint32_t* __restrict__ pass,
               evo_fit* __restrict__ out) {
    extern __shared__ float smem[];
    __shared__ RowMedian s_base;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");       // the verdicts in `pass` come from the kernel before
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool is_base = warp == kWarpsPerCta;
    const uint32_t m = (is_base ? base_trials : trials) - warmup;            // runs that count
    const uint32_t per_row = (stat == EVO_STAT_TRIMMED_MEAN ? 2 * (trials - warmup) : trials - warmup) + 2;
    float* row = smem + static_cast<size_t>(warp) * per_row;                 // the baseline's area comes last
    float* slot = row + m;
    float* sorted = slot + 2;
    const uint64_t r = static_cast<uint64_t>(blockIdx.x) * kWarpsPerCta + warp;
    RowMedian med{0.f, 0u};
    if (is_base || r < n_rows) {
        const float* src = (is_base ? base_times : times + r * trials) + warmup;
        for (uint32_t i = lane; i < m; i += 32) row[i] = src[i];
        __syncwarp();
        med = warp_statistic(row, m, stat, trim, lane, slot, sorted);
        if (is_base && lane == 0) s_base = med;
    }
    __syncthreads();
    if (is_base || r >= n_rows || lane != 0) return;
    const RowMedian b = s_base;
    evo_fit f;
    f.median_ms = med.ok ? med.median : 0.f;
    f.speedup = 0.f;
    f.valid = 0u;
    f.status = !med.ok ? 1u : (!b.ok ? 2u : 0u);
    if (f.status == 0u && (!pass || pass[r] != 0u)) {
        f.valid = 1u;
        f.speedup = __fdiv_rn(b.median, med.median);
    }
    out[r] = f;
}

size_t row_floats(uint32_t trials, int stat, uint32_t warmup) {
    const size_t m = trials - warmup;
    return (stat == EVO_STAT_TRIMMED_MEAN ? 2 * m : m) + 2;
}

int fitness_device(evo_ctx* ctx, const float* times, uint64_t n_cand, uint32_t trials, const float* base_times,
                   uint32_t base_trials, const uint32_t* pass, int stat, uint32_t warmup, uint32_t trim, evo_fit* out,
                   cudaStream_t stream) {
    if (n_cand == 0) return EVO_OK;
    const size_t smem = (kWarpsPerCta * row_floats(trials, stat, warmup) + row_floats(base_trials, stat, warmup)) * sizeof(float);
    if (smem > 48 * 1024)
        EVO_CUDA_TRY(ctx, cudaFuncSetAttribute(fitness_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                               static_cast<int>((kWarpsPerCta + 1) * row_floats(kMaxTrials, EVO_STAT_TRIMMED_MEAN, 0) * sizeof(float))));
    const unsigned grid = static_cast<unsigned>((n_cand + kWarpsPerCta - 1) / kWarpsPerCta);
    EVO_CUDA_TRY(ctx, evo::launch(fitness_kernel, dim3(grid), dim3((kWarpsPerCta + 1) * 32), smem, stream, ctx->pdl, times, n_cand,
                                  trials, base_times, base_trials, stat, warmup, trim, pass, out));
    ctx->launches += 1;
    return EVO_OK;
}

int check_args(evo_ctx* ctx, const char* who, const float* times, uint64_t n_cand, uint32_t trials,
               const float* base_times, uint32_t base_trials, int stat, uint32_t warmup, uint32_t trim, evo_fit* out) {
    if (stat < EVO_STAT_MEDIAN || stat > EVO_STAT_TRIMMED_MEAN) return evo::fail(ctx, EVO_ERR_ARG, "%s: stat %d", who, stat);
    if (warmup >= trials || warmup >= base_trials)
        return evo::fail(ctx, EVO_ERR_ARG, "%s: warmup must leave at least one run", who);
    if (stat == EVO_STAT_TRIMMED_MEAN && (2ull * trim >= trials - warmup || 2ull * trim >= base_trials - warmup))
        return evo::fail(ctx, EVO_ERR_ARG, "%s: trim must leave at least one run", who);
    if (trials == 0 || base_trials == 0 || trials > kMaxTrials || base_trials > kMaxTrials)
        return evo::fail(ctx, EVO_ERR_ARG, "%s: trials and base_trials must be in [1, %u]", who, kMaxTrials);
    if (!base_times || (n_cand > 0 && (!times || !out)))
        return evo::fail(ctx, EVO_ERR_ARG, "%s: times, base_times and out must not be NULL", who);
    if (n_cand > (1ull << 31) * kWarpsPerCta) return evo::fail(ctx, EVO_ERR_ARG, "%s: too many candidates", who);
    if (reinterpret_cast<uintptr_t>(times) % 4 || reinterpret_cast<uintptr_t>(base_times) % 4 || reinterpret_cast<uintptr_t>(out) % 4)
        return evo::fail(ctx, EVO_ERR_ALIGN, "%s: arrays must be 4-byte aligned", who);
    return EVO_OK;
}

}  // namespace

extern "C" int evo_fitness_ex(evo_ctx* ctx, const float* times, uint64_t n_cand, uint32_t trials, const float* base_times,
                              uint32_t base_trials, const uint32_t* pass, int stat, uint32_t warmup, uint32_t trim,
                              evo_fit* out, void* stream) {
    if (!ctx) return EVO_ERR_ARG;
    int st = check_args(ctx, "evo_fitness", times, n_cand, trials, base_times, base_trials, stat, warmup, trim, out);
    if (st != EVO_OK) return st;
    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");
    return fitness_device(ctx, times, n_cand, trials, base_times, base_trials, pass, stat, warmup, trim, out,
                          static_cast<cudaStream_t>(stream));
}

extern "C" int evo_fitness(evo_ctx* ctx, const float* times, uint64_t n_cand, uint32_t trials, const float* base_times,
                           uint32_t base_trials, const uint32_t* pass, evo_fit* out, void* stream) {
    return evo_fitness_ex(ctx, times, n_cand, trials, base_times, base_trials, pass, EVO_STAT_MEDIAN, 0, 0, out, stream);
}

extern "C" int evo_fitness_host(evo_ctx* ctx, const float* times, uint64_t n_cand, uint32_t trials, const float* base_times,
                                uint32_t base_trials, const uint32_t* pass, evo_fit* out, void* stream_) {
    if (!ctx) return EVO_ERR_ARG;
    int st = check_args(ctx, "evo_fitness_host", times, n_cand, trials, base_times, base_trials, EVO_STAT_MEDIAN, 0, 0, out);
    if (st != EVO_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");
    auto up = [](size_t x) { return (x + 255) / 256 * 256; };
    const size_t b_times = n_cand * trials * sizeof(float), b_base = base_trials * sizeof(float);
    const size_t o_base = up(b_times), o_pass = o_base + up(b_base), o_out = o_pass + up(n_cand * 4);
    const size_t total = o_out + up(n_cand * sizeof(evo_fit));
    st = evo::reserve_device(ctx, &ctx->d_stage, &ctx->d_stage_bytes, std::max<size_t>(total, 256));
    if (st != EVO_OK) return st;
    char* base = static_cast<char*>(ctx->d_stage);
    if (b_times) EVO_CUDA_TRY(ctx, cudaMemcpyAsync(base, times, b_times, cudaMemcpyHostToDevice, stream));
    EVO_CUDA_TRY(ctx, cudaMemcpyAsync(base + o_base, base_times, b_base, cudaMemcpyHostToDevice, stream));
    if (pass && n_cand) EVO_CUDA_TRY(ctx, cudaMemcpyAsync(base + o_pass, pass, n_cand * 4, cudaMemcpyHostToDevice, stream));
    st = fitness_device(ctx, reinterpret_cast<const float*>(base), n_cand, trials, reinterpret_cast<const float*>(base + o_base),
                        base_trials, pass ? reinterpret_cast<const uint32_t*>(base + o_pass) : nullptr, EVO_STAT_MEDIAN, 0, 0,
                        reinterpret_cast<evo_fit*>(base + o_out), stream);
    if (st != EVO_OK) return st;
    if (n_cand) EVO_CUDA_TRY(ctx, cudaMemcpyAsync(out, base + o_out, n_cand * sizeof(evo_fit), cudaMemcpyDeviceToHost, stream));
    EVO_CUDA_TRY(ctx, cudaStreamSynchronize(stream));
    return EVO_OK;
}
