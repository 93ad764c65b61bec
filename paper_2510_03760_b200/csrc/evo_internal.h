// Internal declarations shared by the translation units of libevo (host side).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "evo.h"

struct evo_ctx {
    int device = 0;
    int sm_count = 0;
    std::string last_error;
    uint64_t launches = 0;

    // Scratch owned by the context (see evo.h: grows on demand, freed by evo_destroy).
    void* d_plan = nullptr;      size_t d_plan_bytes = 0;       // validation plan (device copy)
    void* h_plan = nullptr;      size_t h_plan_bytes = 0;       // pinned staging of the plan
    void* d_partials = nullptr;  size_t d_partials_bytes = 0;   // per-(CTA, tensor) partial results
    void* d_stage = nullptr;     size_t d_stage_bytes = 0;      // tensors of the *_host calls
    void* d_seeds = nullptr;     size_t d_seeds_bytes = 0;      // per tensor: warm start of the max d/|r| filter
    void* d_feedback = nullptr;  size_t d_feedback_bytes = 0;   // per-chunk counts of evo_mismatch_sample
    void* d_small = nullptr;                                   // 256 bytes: summary scratch (64..), status word (128)
    bool pass1_ready = false;                                  // the first pass's shared-memory size has been set
    cudaEvent_t plan_consumed = nullptr;                       // the last plan upload has been read
    bool plan_in_flight = false;
    cudaEvent_t time_start = nullptr, time_stop = nullptr;     // one-shot request of evo_set_timing_events
    // What d_plan holds: the arguments of the evo_validate call whose plan was uploaded last (byte image), and what
    // launching it takes.  A call with the same arguments skips planning and upload.
    bool plan_key_valid = false;
    std::vector<unsigned char> plan_key, plan_scratch_key;
    size_t plan_layout[6] = {0, 0, 0, 0, 0, 0};
    uint32_t plan_n_members = 0, plan_n_ctas = 0;
    bool plan_seed = false;
    bool pdl = true;                                           // launch kernels so that they may overlap their predecessor's tail
    bool cta_timing = false;                                   // evo_debug_cta_timing: the first pass records per-CTA clocks
    void* d_cta_times = nullptr; size_t d_cta_times_bytes = 0; // two 64-bit %globaltimer readings per CTA
    uint32_t cta_times_n = 0;                                  // CTAs of the last timed first pass
};

namespace evo {

int fail(evo_ctx* ctx, int status, const char* fmt, ...);
int fail_cuda(evo_ctx* ctx, cudaError_t e, const char* what);

// Grows *ptr to at least `bytes` (device memory, contents not preserved).
int reserve_device(evo_ctx* ctx, void** ptr, size_t* have, size_t bytes);
int reserve_pinned(evo_ctx* ctx, void** ptr, size_t* have, size_t bytes);

// Sets the context's device for the scope and restores the previous one.
struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    cudaError_t err = cudaSuccess;
    explicit DeviceGuard(int device);
    ~DeviceGuard();
};

// Device word that a kernel raises when one of its bounded waits ran out.
inline uint32_t* status_word(evo_ctx* ctx) { return reinterpret_cast<uint32_t*>(static_cast<char*>(ctx->d_small) + 128); }
// Synchronises `stream`, then reads and clears the status word: EVO_OK or EVO_ERR_TIMEOUT.
int sync_and_check(evo_ctx* ctx, cudaStream_t stream, const char* who);

// Launches `kernel`; with `pdl` the launch carries the programmatic-stream-serialization
// attribute, so the kernel may begin (up to its griddepcontrol.wait) while the kernel before it
// in the stream is still running.  If a launch with the attribute is refused, it is repeated
// without.
template <typename... KArgs, typename... Args>
inline cudaError_t launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, bool pdl,
                          const Args&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
    if (e != cudaSuccess && pdl) {
        (void)cudaGetLastError();
        cfg.numAttrs = 0;
        e = cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
    }
    return e;
}

inline size_t elem_bytes(int dtype) { return dtype == EVO_F16 || dtype == EVO_BF16 ? 2 : 4; }

}  // namespace evo

#define EVO_CUDA_TRY(ctx, expr)                                            \
    do {                                                                   \
        cudaError_t evo_e_ = (expr);                                       \
        if (evo_e_ != cudaSuccess) return evo::fail_cuda((ctx), evo_e_, #expr); \
    } while (0)
