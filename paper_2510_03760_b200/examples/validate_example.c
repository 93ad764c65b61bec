/*
 * Using the library from plain C: generate a reference tensor on the device, derive three candidates from it on
 * the host, validate them in one call, turn run times into speedups and print the records.
 *
 *   gcc -std=c99 -I include -I /usr/local/cuda/include validate_example.c \
 *       -L paper_2510_03760_b200 -levo -L /usr/local/cuda/lib64 -lcudart -Wl,-rpath,... -o validate_example
 *
 * Prints one line per candidate: "cand <i> n_mismatch <..> max_abs <..> pass <0|1> speedup <..>", then "ok".
 */
#include <cuda_runtime_api.h>
#include <stdio.h>
#include <stdlib.h>

#include "evo.h"

#define CHECK_CUDA(x) do { cudaError_t e_ = (x); if (e_ != cudaSuccess) { fprintf(stderr, "%s: %s\n", #x, cudaGetErrorString(e_)); return 2; } } while (0)
#define CHECK_EVO(x) do { int s_ = (x); if (s_ != EVO_OK) { fprintf(stderr, "%s: %s (%s)\n", #x, evo_strerror(s_), evo_last_error(ctx)); return 3; } } while (0)

int main(void) {
    enum { N = 3 * 4096 + 77, K = 3, TRIALS = 5 };
    evo_ctx* ctx = NULL;
    if (evo_create(&ctx, 0) != EVO_OK) { fprintf(stderr, "evo_create failed\n"); return 1; }

    /* reference: standard normals of stream (seed 7, offset 0), generated on the device */
    float *d_ref = NULL, *d_cand[K];
    CHECK_CUDA(cudaMalloc((void**)&d_ref, N * sizeof(float)));
    CHECK_EVO(evo_gen_inputs(ctx, 7, 0, EVO_F32, N, d_ref, NULL));
    float* h = (float*)malloc(N * sizeof(float));
    CHECK_CUDA(cudaMemcpy(h, d_ref, N * sizeof(float), cudaMemcpyDeviceToHost));

    /* candidate 0: identical; candidate 1: 5 elements off by 1.0; candidate 2: everything off by 1e-3 (inside 1e-2) */
    for (int k = 0; k < K; ++k) {
        float* c = (float*)malloc(N * sizeof(float));
        for (int i = 0; i < N; ++i) c[i] = h[i] + (k == 2 ? 1e-3f : 0.0f);
        if (k == 1) for (int j = 0; j < 5; ++j) c[1000 * j + 3] += 1.0f;
        CHECK_CUDA(cudaMalloc((void**)&d_cand[k], N * sizeof(float)));
        CHECK_CUDA(cudaMemcpy(d_cand[k], c, N * sizeof(float), cudaMemcpyHostToDevice));
        free(c);
    }

    const void* cand_ptrs[K];
    evo_desc descs[K];
    for (int k = 0; k < K; ++k) {
        cand_ptrs[k] = d_cand[k];
        descs[k].n = N; descs[k].ref = NULL; descs[k].dtype = -1; descs[k].group = (uint32_t)k;
    }
    evo_result* d_res = NULL;
    uint32_t* d_pass = NULL;
    CHECK_CUDA(cudaMalloc((void**)&d_res, K * sizeof(evo_result)));
    CHECK_CUDA(cudaMalloc((void**)&d_pass, K * sizeof(uint32_t)));
    CHECK_EVO(evo_validate(ctx, cand_ptrs, d_ref, descs, K, EVO_F32, 1e-2f, 1e-2f, d_res, d_pass, K, NULL));

    /* run times: candidate k takes (k + 1) ms per trial, the baseline 6 ms */
    float times[K * TRIALS], base[TRIALS];
    for (int k = 0; k < K; ++k) for (int t = 0; t < TRIALS; ++t) times[k * TRIALS + t] = (float)(k + 1);
    for (int t = 0; t < TRIALS; ++t) base[t] = 6.0f;
    float *d_times = NULL, *d_base = NULL;
    evo_fit* d_fit = NULL;
    CHECK_CUDA(cudaMalloc((void**)&d_times, sizeof times));
    CHECK_CUDA(cudaMalloc((void**)&d_base, sizeof base));
    CHECK_CUDA(cudaMalloc((void**)&d_fit, K * sizeof(evo_fit)));
    CHECK_CUDA(cudaMemcpy(d_times, times, sizeof times, cudaMemcpyHostToDevice));
    CHECK_CUDA(cudaMemcpy(d_base, base, sizeof base, cudaMemcpyHostToDevice));
    CHECK_EVO(evo_fitness(ctx, d_times, K, TRIALS, d_base, TRIALS, d_pass, d_fit, NULL));
    CHECK_EVO(evo_check(ctx, NULL));

    evo_result res[K];
    evo_fit fit[K];
    CHECK_CUDA(cudaMemcpy(res, d_res, sizeof res, cudaMemcpyDeviceToHost));
    CHECK_CUDA(cudaMemcpy(fit, d_fit, sizeof fit, cudaMemcpyDeviceToHost));
    for (int k = 0; k < K; ++k)
        printf("cand %d n_mismatch %llu max_abs %.6g pass %u speedup %.6g\n", k, (unsigned long long)res[k].n_mismatch,
               (double)res[k].max_abs, res[k].pass, (double)fit[k].speedup);

    int ok = res[0].n_mismatch == 0 && res[0].pass == 1 && res[0].max_abs == 0.0f && fit[0].speedup == 6.0f &&
             res[1].n_mismatch == 5 && res[1].pass == 0 && fit[1].valid == 0 && fit[1].speedup == 0.0f &&
             res[2].n_mismatch == 0 && res[2].pass == 1 && fit[2].speedup == 2.0f;
    free(h);
    cudaFree(d_ref); cudaFree(d_res); cudaFree(d_pass); cudaFree(d_times); cudaFree(d_base); cudaFree(d_fit);
    for (int k = 0; k < K; ++k) cudaFree(d_cand[k]);
    evo_destroy(ctx);
    puts(ok ? "ok" : "UNEXPECTED");
    return ok ? 0 : 4;
}
