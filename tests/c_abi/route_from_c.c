/* A plain C program that drives libdirector.so through its C ABI (no Python, no C++): gate a small batch and check
 * the winners against a scalar search.  Exit code 0 = pass.  Built and run by tests/test_gpu_c_abi.py. */
#include <cuda_runtime_api.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>

#include "director.h"

#define CHECK(call)                                                                  \
    do {                                                                             \
        int rc_ = (call);                                                            \
        if (rc_ != 0) { fprintf(stderr, "%s -> %d\n", #call, rc_); return 2; }      \
    } while (0)

int main(void) {
    enum { T = 300, E = 24, K = 3, R = 4, C = 6 };
    director_shape shape = {T, 256, 128, E, K, 0, R, C};
    director_ctx* ctx = NULL;
    CHECK(director_create(&shape, &ctx));

    uint8_t X[E][R] = {{0}};
    for (int e = 0; e < E; ++e) X[e][e % R] = 1;
    CHECK(director_set_placement(ctx, &X[0][0], NULL));

    float* h_logits = (float*)malloc(sizeof(float) * T * E);
    for (int t = 0; t < T; ++t)
        for (int e = 0; e < E; ++e)
            h_logits[t * E + e] = sinf(0.37f * (float)(t * 31 + e * 17)) * 3.0f;   /* distinct values, no ties */

    float *d_logits, *d_w;
    int32_t* d_idx;
    CHECK(cudaMalloc((void**)&d_logits, sizeof(float) * T * E));
    CHECK(cudaMalloc((void**)&d_idx, sizeof(int32_t) * T * K));
    CHECK(cudaMalloc((void**)&d_w, sizeof(float) * T * K));
    CHECK(cudaMemcpy(d_logits, h_logits, sizeof(float) * T * E, cudaMemcpyHostToDevice));
    CHECK(director_route(ctx, T, d_logits, d_idx, d_w, NULL));
    CHECK(cudaDeviceSynchronize());
    CHECK(director_last_status(ctx, NULL));

    int32_t* idx = (int32_t*)malloc(sizeof(int32_t) * T * K);
    float* w = (float*)malloc(sizeof(float) * T * K);
    CHECK(cudaMemcpy(idx, d_idx, sizeof(int32_t) * T * K, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(w, d_w, sizeof(float) * T * K, cudaMemcpyDeviceToHost));

    int bad = 0;
    for (int t = 0; t < T; ++t) {
        int taken[E] = {0};
        double sum = 0.0, wsum = 0.0, ex[K];
        for (int s = 0; s < K; ++s) {                     /* the s-th largest logit by plain search */
            int best = -1;
            for (int e = 0; e < E; ++e)
                if (!taken[e] && (best < 0 || h_logits[t * E + e] > h_logits[t * E + best])) best = e;
            taken[best] = 1;
            if (idx[t * K + s] != best) ++bad;
            ex[s] = exp((double)h_logits[t * E + best] - (double)h_logits[t * E + idx[t * K]]);
            sum += ex[s];
        }
        for (int s = 0; s < K; ++s) {
            if (fabs((double)w[t * K + s] - ex[s] / sum) > 1e-6) ++bad;
            wsum += w[t * K + s];
        }
        if (fabs(wsum - 1.0) > 1e-6) ++bad;
    }
    printf("route_from_c: %d tokens, %d mismatches, %s\n", T, bad, director_status_string(0));
    cudaFree(d_logits); cudaFree(d_idx); cudaFree(d_w);
    free(h_logits); free(idx); free(w);
    CHECK(director_destroy(ctx));
    return bad ? 1 : 0;
}
