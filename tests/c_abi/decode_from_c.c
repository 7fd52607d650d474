/* A plain C caller of the library: no Python, no C++.  Builds a tiny problem in host memory,
 * runs a few decode steps and Exact Top-K through the C interface and checks what can be
 * checked by hand: with identical keys everywhere the Top-K support is the K lowest indices
 * (ties go to the lower index) and the output equals the common value row. */
#include <cuda_runtime_api.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "retopk.h"

#define CHECK(call)                                                              \
    do {                                                                         \
        int rc_ = (call);                                                        \
        if (rc_ != 0) { printf("FAIL %s -> %d (%s)\n", #call, rc_, retopk_strerror(rc_)); return 1; } \
    } while (0)
#define CUDA(call)                                                               \
    do {                                                                         \
        cudaError_t e_ = (call);                                                 \
        if (e_ != cudaSuccess) { printf("FAIL %s -> %s\n", #call, cudaGetErrorString(e_)); return 1; } \
    } while (0)

int main(void) {
    enum { B = 1, HQ = 4, HKV = 2, D = 64, M = 4, R_RECALL = 2, W = 8, K = 16, LMAX = 600, L0 = 500 };
    const uint16_t one = 0x3F80, half = 0x3F00;            /* bf16 1.0 and 0.5 */
    size_t nkv = (size_t)B * HKV * LMAX * D, nq = (size_t)B * HQ * D;
    uint16_t* hk = (uint16_t*)malloc(nkv * 2);
    uint16_t* hv = (uint16_t*)malloc(nkv * 2);
    uint16_t* hq = (uint16_t*)malloc(nq * 2);
    uint16_t* ho = (uint16_t*)malloc(nq * 2);
    int32_t* hidx = (int32_t*)malloc((size_t)B * HQ * K * 4);
    for (size_t i = 0; i < nkv; ++i) { hk[i] = one; hv[i] = half; }
    for (size_t i = 0; i < nq; ++i) hq[i] = one;

    void *dk, *dv, *dq, *dout, *didx;
    CUDA(cudaMalloc(&dk, nkv * 2)); CUDA(cudaMalloc(&dv, nkv * 2)); CUDA(cudaMalloc(&dq, nq * 2));
    CUDA(cudaMalloc(&dout, nq * 2)); CUDA(cudaMalloc(&didx, (size_t)B * HQ * K * 4));
    CUDA(cudaMemcpy(dk, hk, nkv * 2, cudaMemcpyHostToDevice));
    CUDA(cudaMemcpy(dv, hv, nkv * 2, cudaMemcpyHostToDevice));
    CUDA(cudaMemcpy(dq, hq, nq * 2, cudaMemcpyHostToDevice));

    retopk_ctx* ctx = NULL;
    CHECK(retopk_create_batched(&ctx, B, HQ, HKV, D, M, R_RECALL, W, K, 0.85f, 0, LMAX));
    for (int t = 0; t < 5; ++t) CHECK(retopk_decode_step(ctx, dq, dk, dv, L0 + t + 1, dout, NULL));
    CHECK(exact_topk_decode(ctx, dq, dk, dv, L0, dout, (int32_t*)didx, NULL));
    retopk_stats_t st;
    CHECK(retopk_stats(ctx, &st));
    CUDA(cudaMemcpy(ho, dout, nq * 2, cudaMemcpyDeviceToHost));
    CUDA(cudaMemcpy(hidx, didx, (size_t)B * HQ * K * 4, cudaMemcpyDeviceToHost));

    int bad = 0;
    /* step 0 falls back (empty cache); the identical queries of the later steps have similarity 1 */
    if (st.steps != 5 * HQ || st.fallback != HQ || st.reuse != 4 * HQ || st.status != 0) bad |= 1;
    for (int h = 0; h < HQ; ++h)
        for (int i = 0; i < K; ++i)
            if (hidx[h * K + i] != i) bad |= 2;
    for (size_t i = 0; i < nq; ++i)
        if (ho[i] != half) bad |= 4;
    /* argument checks answer with error codes */
    if (retopk_decode_step(ctx, dq, dk, dv, LMAX + 1, dout, NULL) != RETOPK_EINVAL) bad |= 8;
    if (retopk_decode_step(NULL, dq, dk, dv, 10, dout, NULL) != RETOPK_EINVAL) bad |= 16;
    CHECK(retopk_destroy(ctx));
    printf("steps %lld reuse %lld fallback %lld refresh %lld bad %d\n", (long long)st.steps, (long long)st.reuse,
           (long long)st.fallback, (long long)st.refresh, bad);
    puts(bad ? "FAIL" : "OK");
    return bad ? 1 : 0;
}
