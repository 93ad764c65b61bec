// evo_gen_inputs: seeded random test inputs (paper Section 4.3, functional testing on
// random test cases; Appendix A.8.1).  Philox4x32-10 counter stream (Salmon et al., SC'11)
// and a Box-Muller normal fill in binary32.
//
// One thread produces one Philox block (4 stream elements) per loop trip: ten rounds of
// two 32x32->64 multiplies, then for the normal fill two log/sqrt/sincospi evaluations.
// The kernel is bound by the integer/float pipes, not by memory (4 bytes stored per
// ~50 instructions), so the only memory-side care is a full-width store per thread.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "evo_internal.h"
#include "philox.cuh"

namespace {

using namespace evo;

// (xa, xb) -> (rho cos, rho sin).  u1 and 2*u2 are exact in binary32; the angle is handed
// to sincospif as a multiple of pi so that no rounded 2*pi enters and the zeros at the
// axis crossings are exact.
__device__ __forceinline__ float2 box_muller(uint32_t xa, uint32_t xb) {
    const float u1 = static_cast<float>((xa >> 8) + 1u) * 5.9604644775390625e-08f;   // 2^-24
    const float two_u2 = static_cast<float>(xb >> 8) * 1.1920928955078125e-07f;      // 2^-23
    const float rho = sqrtf(-2.0f * logf(u1));
    float s, c;
    sincospif(two_u2, &s, &c);
    return make_float2(rho * c, rho * s);
}

template <int DT> struct Out;
template <> struct Out<EVO_U32>  { using T = uint32_t;      static __device__ T make(uint32_t w, float) { return w; } };
template <> struct Out<EVO_F32>  { using T = float;         static __device__ T make(uint32_t, float z) { return z; } };
template <> struct Out<EVO_F16>  { using T = __half;        static __device__ T make(uint32_t, float z) { return __float2half_rn(z); } };
template <> struct Out<EVO_BF16> { using T = __nv_bfloat16; static __device__ T make(uint32_t, float z) { return __float2bfloat16_rn(z); } };

template <int DT> struct alignas(4 * sizeof(typename Out<DT>::T)) Quad { typename Out<DT>::T v[4]; };

// Stream blocks first_block .. first_block + n_blocks - 1 cover stream elements
// [offset, offset + n); `lead` = offset mod 4 elements of the first block are skipped.
// VEC: lead == 0 and `out` is aligned for one store of four elements per block.
template <int DT, bool VEC>
__global__ void __launch_bounds__(256) gen_kernel(const __grid_constant__ RoundKeys rk, uint64_t first_block, uint64_t n_blocks,
                                                  uint32_t lead, uint64_t n, typename Out<DT>::T* __restrict__ out) {
    using T = typename Out<DT>::T;
    // may start while the kernel before it in the stream still runs; `out` is not written before that one is done
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const uint64_t stride = static_cast<uint64_t>(gridDim.x) * blockDim.x;
    for (uint64_t j = static_cast<uint64_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < n_blocks; j += stride) {
        const uint4 w = philox4x32_10(first_block + j, rk);
        Quad<DT> q;
        if (DT == EVO_U32) {
            q.v[0] = Out<DT>::make(w.x, 0.f); q.v[1] = Out<DT>::make(w.y, 0.f);
            q.v[2] = Out<DT>::make(w.z, 0.f); q.v[3] = Out<DT>::make(w.w, 0.f);
        } else {
            const float2 a = box_muller(w.x, w.y), b = box_muller(w.z, w.w);
            q.v[0] = Out<DT>::make(0u, a.x); q.v[1] = Out<DT>::make(0u, a.y);
            q.v[2] = Out<DT>::make(0u, b.x); q.v[3] = Out<DT>::make(0u, b.y);
        }
        if (VEC && 4 * j + 4 <= n) {
            *reinterpret_cast<Quad<DT>*>(out + 4 * j) = q;
        } else {
#pragma unroll
            for (int l = 0; l < 4; ++l) {
                const uint64_t g = 4 * j + l;          // position relative to the first block's start
                if (g >= lead && g - lead < n) out[g - lead] = q.v[l];
            }
        }
    }
}

template <int DT>
cudaError_t launch(evo_ctx* ctx, uint64_t seed, uint64_t offset, uint64_t n, void* out, cudaStream_t stream) {
    using T = typename Out<DT>::T;
    const uint32_t lead = static_cast<uint32_t>(offset & 3u);
    const uint64_t n_blocks = (lead + n + 3) / 4;
    const bool vec = lead == 0 && (reinterpret_cast<uintptr_t>(out) % (4 * sizeof(T))) == 0;
    const uint64_t want = (n_blocks + 255) / 256;
    const uint64_t cap = static_cast<uint64_t>(ctx->sm_count) * 8 * 4;   // a few waves of 8 resident CTAs per SM
    const unsigned grid = static_cast<unsigned>(want < cap ? want : cap);
    const RoundKeys rk = round_keys(seed);
    ctx->launches += 1;
    if (vec) return evo::launch(gen_kernel<DT, true>, dim3(grid), dim3(256), 0, stream, ctx->pdl, rk, offset >> 2, n_blocks, lead, n, static_cast<T*>(out));
    return evo::launch(gen_kernel<DT, false>, dim3(grid), dim3(256), 0, stream, ctx->pdl, rk, offset >> 2, n_blocks, lead, n, static_cast<T*>(out));
}

}  // namespace

extern "C" int evo_gen_inputs(evo_ctx* ctx, uint64_t seed, uint64_t offset, int dtype, uint64_t n, void* out, void* stream) {
    if (!ctx) return EVO_ERR_ARG;
    if (dtype != EVO_U32 && dtype != EVO_F32 && dtype != EVO_F16 && dtype != EVO_BF16)
        return evo::fail(ctx, EVO_ERR_DTYPE, "evo_gen_inputs: dtype %d", dtype);
    if (n == 0) return EVO_OK;
    if (!out) return evo::fail(ctx, EVO_ERR_ARG, "evo_gen_inputs: out is NULL");
    if (n > (UINT64_MAX >> 3)) return evo::fail(ctx, EVO_ERR_ARG, "evo_gen_inputs: n too large");
    if (reinterpret_cast<uintptr_t>(out) % evo::elem_bytes(dtype))
        return evo::fail(ctx, EVO_ERR_ALIGN, "evo_gen_inputs: out not aligned to %zu bytes", evo::elem_bytes(dtype));
    evo::DeviceGuard guard(ctx->device);
    if (guard.err != cudaSuccess) return evo::fail_cuda(ctx, guard.err, "cudaSetDevice");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    switch (dtype) {
        case EVO_U32: e = launch<EVO_U32>(ctx, seed, offset, n, out, s); break;
        case EVO_F32: e = launch<EVO_F32>(ctx, seed, offset, n, out, s); break;
        case EVO_F16: e = launch<EVO_F16>(ctx, seed, offset, n, out, s); break;
        default:      e = launch<EVO_BF16>(ctx, seed, offset, n, out, s); break;
    }
    if (e != cudaSuccess) return evo::fail_cuda(ctx, e, "gen_kernel launch");
    return EVO_OK;
}
