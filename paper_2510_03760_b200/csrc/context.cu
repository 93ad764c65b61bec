// Context life cycle, error reporting and workspace management of libevo.
#include <cstdarg>
#include <cstdio>
#include <new>

#include "evo_internal.h"

namespace evo {

int fail(evo_ctx* ctx, int status, const char* fmt, ...) {
    if (ctx) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        ctx->last_error = buf;
    }
    return status;
}

int fail_cuda(evo_ctx* ctx, cudaError_t e, const char* what) {
    return fail(ctx, EVO_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

int reserve_device(evo_ctx* ctx, void** ptr, size_t* have, size_t bytes) {
    if (*have >= bytes) return EVO_OK;
    if (*ptr) {
        // Earlier launches on any stream may still read the old block.
        EVO_CUDA_TRY(ctx, cudaDeviceSynchronize());
        EVO_CUDA_TRY(ctx, cudaFree(*ptr));
        *ptr = nullptr;
        *have = 0;
    }
    size_t want = bytes + bytes / 4;
    cudaError_t e = cudaMalloc(ptr, want);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        want = bytes;
        e = cudaMalloc(ptr, want);
    }
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        *ptr = nullptr;
        return fail(ctx, EVO_ERR_WORKSPACE, "workspace of %zu bytes: %s", bytes, cudaGetErrorString(e));
    }
    *have = want;
    return EVO_OK;
}

int reserve_pinned(evo_ctx* ctx, void** ptr, size_t* have, size_t bytes) {
    if (*have >= bytes) return EVO_OK;
    if (*ptr) {
        EVO_CUDA_TRY(ctx, cudaDeviceSynchronize());
        EVO_CUDA_TRY(ctx, cudaFreeHost(*ptr));
        *ptr = nullptr;
        *have = 0;
    }
    const size_t want = bytes + bytes / 4;
    cudaError_t e = cudaMallocHost(ptr, want);
    if (e != cudaSuccess) {
        (void)cudaGetLastError();
        *ptr = nullptr;
        return fail(ctx, EVO_ERR_WORKSPACE, "pinned staging of %zu bytes: %s", bytes, cudaGetErrorString(e));
    }
    *have = want;
    return EVO_OK;
}

DeviceGuard::DeviceGuard(int device) {
    err = cudaGetDevice(&prev);
    if (err == cudaSuccess && prev != device) {
        err = cudaSetDevice(device);
        switched = (err == cudaSuccess);
    }
}

DeviceGuard::~DeviceGuard() {
    if (switched) (void)cudaSetDevice(prev);
}

int sync_and_check(evo_ctx* ctx, cudaStream_t stream, const char* who) {
    EVO_CUDA_TRY(ctx, cudaStreamSynchronize(stream));
    uint32_t word = 0;
    EVO_CUDA_TRY(ctx, cudaMemcpy(&word, status_word(ctx), sizeof word, cudaMemcpyDeviceToHost));
    if (word == 0) return EVO_OK;
    EVO_CUDA_TRY(ctx, cudaMemset(status_word(ctx), 0, sizeof word));
    if (word & 3u)
        return fail(ctx, EVO_ERR_TIMEOUT, "%s: a device-side wait ran out (status word 0x%x); results are marked incomplete", who, word);
    return fail(ctx, EVO_ERR_ARG, "%s: a kernel or run id was out of range (status word 0x%x); that record was skipped", who, word);
}

}  // namespace evo

extern "C" {

int evo_create(evo_ctx** out, int device) {
    if (!out) return EVO_ERR_ARG;
    *out = nullptr;
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess || device < 0 || device >= count) {
        (void)cudaGetLastError();
        return e != cudaSuccess ? EVO_ERR_CUDA : EVO_ERR_ARG;
    }
    evo_ctx* ctx = new (std::nothrow) evo_ctx();
    if (!ctx) return EVO_ERR_WORKSPACE;
    ctx->device = device;
    evo::DeviceGuard guard(device);
    int status = EVO_OK;
    if (guard.err != cudaSuccess) status = EVO_ERR_CUDA;
    if (status == EVO_OK && cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
        status = EVO_ERR_CUDA;
    if (status == EVO_OK && cudaMalloc(&ctx->d_small, 256) != cudaSuccess) status = EVO_ERR_CUDA;
    if (status == EVO_OK && cudaMemset(ctx->d_small, 0, 256) != cudaSuccess) status = EVO_ERR_CUDA;
    if (status == EVO_OK && cudaEventCreateWithFlags(&ctx->plan_consumed, cudaEventDisableTiming) != cudaSuccess)
        status = EVO_ERR_CUDA;
    if (status != EVO_OK) {
        (void)cudaGetLastError();
        if (ctx->d_small) (void)cudaFree(ctx->d_small);
        delete ctx;
        return status;
    }
    *out = ctx;
    return EVO_OK;
}

int evo_destroy(evo_ctx* ctx) {
    if (!ctx) return EVO_OK;
    evo::DeviceGuard guard(ctx->device);
    (void)cudaDeviceSynchronize();
    if (ctx->d_plan) (void)cudaFree(ctx->d_plan);
    if (ctx->h_plan) (void)cudaFreeHost(ctx->h_plan);
    if (ctx->d_partials) (void)cudaFree(ctx->d_partials);
    if (ctx->d_stage) (void)cudaFree(ctx->d_stage);
    if (ctx->d_feedback) (void)cudaFree(ctx->d_feedback);
    if (ctx->d_seeds) (void)cudaFree(ctx->d_seeds);
    if (ctx->d_cta_times) (void)cudaFree(ctx->d_cta_times);
    if (ctx->d_small) (void)cudaFree(ctx->d_small);
    if (ctx->plan_consumed) (void)cudaEventDestroy(ctx->plan_consumed);
    delete ctx;
    return EVO_OK;
}

const char* evo_strerror(int status) {
    switch (status) {
        case EVO_OK: return "ok";
        case EVO_ERR_ARG: return "invalid argument";
        case EVO_ERR_ALIGN: return "pointer not aligned to its element size";
        case EVO_ERR_DTYPE: return "unsupported element type";
        case EVO_ERR_CUDA: return "CUDA runtime error";
        case EVO_ERR_WORKSPACE: return "workspace unavailable or limit exceeded";
        case EVO_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

const char* evo_last_error(const evo_ctx* ctx) { return ctx ? ctx->last_error.c_str() : ""; }

int evo_set_timing_events(evo_ctx* ctx, void* start, void* stop) {
    if (!ctx || ((start == nullptr) != (stop == nullptr))) return EVO_ERR_ARG;
    ctx->time_start = static_cast<cudaEvent_t>(start);
    ctx->time_stop = static_cast<cudaEvent_t>(stop);
    return EVO_OK;
}

int evo_check(evo_ctx* ctx, void* stream) {
    if (!ctx) return EVO_ERR_ARG;
    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");
    return evo::sync_and_check(ctx, static_cast<cudaStream_t>(stream), "evo_check");
}

uint64_t evo_launch_count(const evo_ctx* ctx) { return ctx ? ctx->launches : 0; }

int evo_debug_cta_timing(evo_ctx* ctx, int enable) {
    if (!ctx) return EVO_ERR_ARG;
    ctx->cta_timing = enable != 0;
    if (!ctx->cta_timing) ctx->cta_times_n = 0;
    return EVO_OK;
}

int evo_debug_read_cta_times(evo_ctx* ctx, uint64_t* begin_end_ns, uint32_t capacity, uint32_t* n_ctas) {
    if (!ctx || !n_ctas || (capacity > 0 && !begin_end_ns)) return EVO_ERR_ARG;
    *n_ctas = ctx->cta_times_n;
    const uint32_t n = ctx->cta_times_n < capacity ? ctx->cta_times_n : capacity;
    if (n == 0) return EVO_OK;
    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");
    EVO_CUDA_TRY(ctx, cudaDeviceSynchronize());
    EVO_CUDA_TRY(ctx, cudaMemcpy(begin_end_ns, ctx->d_cta_times, static_cast<size_t>(n) * 16, cudaMemcpyDeviceToHost));
    return EVO_OK;
}

int evo_set_overlapped_launch(evo_ctx* ctx, int enable) {
    if (!ctx) return EVO_ERR_ARG;
    ctx->pdl = enable != 0;
    return EVO_OK;
}

}  // extern "C"
