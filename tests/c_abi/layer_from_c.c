/* A plain C program that drives every stage of libdirector.so through its C ABI (no Python, no C++) on a small
 * layer and checks, in C, the facts the method fixes:
 *   - the segment table ends at T*K and every assignment's row points back at its token,
 *   - the per-rank loads of Eq. 1 sum to T*K and the workload matrix sums to T*K,
 *   - dispatch followed by combine with identity experts (yp := xp) returns x bit for bit,
 *   - the stage calls in order and director_layer_forward give the same bits (y and all histograms),
 *   - the combining down projection (director_expert_ffn_combine) agrees with expert_ffn + combine to bf16 rounding.
 * Exit code 0 = pass.  Built and run by tests/test_gpu_c_abi.py. */
#include <cuda_runtime_api.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "director.h"

#define CHECK(call)                                                                  \
    do {                                                                             \
        int rc_ = (int)(call);                                                       \
        if (rc_ != 0) { fprintf(stderr, "%s -> %d\n", #call, rc_); return 2; }      \
    } while (0)

static uint32_t lcg(uint32_t* s) { *s = *s * 1664525u + 1013904223u; return *s >> 8; }

/* bf16 bit pattern of a small value in (-scale, scale): fp32 rounded to nearest even */
static uint16_t bf16_of(float v) {
    uint32_t u;
    memcpy(&u, &v, 4);
    u += 0x7FFFu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

static void* dev_copy(const void* h, size_t bytes) {
    void* d = NULL;
    if (cudaMalloc(&d, bytes) != cudaSuccess) return NULL;
    if (h != NULL && cudaMemcpy(d, h, bytes, cudaMemcpyHostToDevice) != cudaSuccess) return NULL;
    return d;
}

int main(void) {
    enum { T = 300, H = 256, F = 128, E = 24, K = 3, R = 4, C = 7, G = R * C, A = T * K };
    director_shape shape = {T, H, F, E, K, 0, R, C};
    director_ctx* ctx = NULL;
    CHECK(director_create(&shape, &ctx));

    uint8_t X[E][R];
    memset(X, 0, sizeof X);
    for (int e = 0; e < E; ++e) X[e][e % R] = 1;
    X[0][1] = X[0][2] = X[5][0] = 1;                       /* replicas: expert 0 on three ranks, expert 5 on two */
    CHECK(director_set_placement(ctx, &X[0][0], NULL));

    uint32_t seed = 12345u;
    float* h_logits = (float*)malloc(sizeof(float) * T * E);
    uint16_t* h_x = (uint16_t*)malloc(2 * T * H);
    uint16_t* h_wg = (uint16_t*)malloc(2 * (size_t)E * F * H);
    uint16_t* h_wu = (uint16_t*)malloc(2 * (size_t)E * F * H);
    uint16_t* h_wd = (uint16_t*)malloc(2 * (size_t)E * H * F);
    for (int i = 0; i < T * E; ++i) h_logits[i] = (float)(lcg(&seed) % 20001) * 1e-3f - 10.0f - 0.3f * (float)(i % E);
    for (int i = 0; i < T * H; ++i) h_x[i] = bf16_of(((float)(lcg(&seed) % 2001) - 1000.0f) * 1e-3f);
    for (size_t i = 0; i < (size_t)E * F * H; ++i) {
        h_wg[i] = bf16_of(((float)(lcg(&seed) % 2001) - 1000.0f) * 4e-5f);
        h_wu[i] = bf16_of(((float)(lcg(&seed) % 2001) - 1000.0f) * 4e-5f);
        h_wd[i] = bf16_of(((float)(lcg(&seed) % 2001) - 1000.0f) * 4e-5f);
    }

    float* d_logits = (float*)dev_copy(h_logits, sizeof(float) * T * E);
    void* d_x = dev_copy(h_x, 2 * T * H);
    void* d_wg = dev_copy(h_wg, 2 * (size_t)E * F * H);
    void* d_wu = dev_copy(h_wu, 2 * (size_t)E * F * H);
    void* d_wd = dev_copy(h_wd, 2 * (size_t)E * H * F);
    int32_t* d_idx = (int32_t*)dev_copy(NULL, 4 * A);
    float* d_w = (float*)dev_copy(NULL, 4 * A);
    void* d_xp = dev_copy(NULL, 2 * (size_t)A * H);
    void* d_yp = dev_copy(NULL, 2 * (size_t)A * H);
    int32_t* d_row_token = (int32_t*)dev_copy(NULL, 4 * A);
    int32_t* d_inv_row = (int32_t*)dev_copy(NULL, 4 * A);
    int32_t* d_dest = (int32_t*)dev_copy(NULL, 4 * A);
    int32_t* d_seg = (int32_t*)dev_copy(NULL, 4 * (G + 1));
    void* d_y = dev_copy(NULL, 2 * T * H);
    void* d_y2 = dev_copy(NULL, 2 * T * H);
    int64_t* d_cost = (int64_t*)dev_copy(NULL, 8 * (R * E + R + 2 * R * R));      /* W | lambda | D tokens | D bytes */
    int64_t* d_cost2 = (int64_t*)dev_copy(NULL, 8 * (R * E + R + 2 * R * R));
    if (!d_logits || !d_x || !d_wg || !d_wu || !d_wd || !d_idx || !d_w || !d_xp || !d_yp || !d_row_token || !d_inv_row ||
        !d_dest || !d_seg || !d_y || !d_y2 || !d_cost || !d_cost2) {
        fprintf(stderr, "device allocation failed\n");
        return 2;
    }

    /* ---- the five stages, one call each ---- */
    CHECK(director_route(ctx, T, d_logits, d_idx, d_w, NULL));
    CHECK(director_dispatch(ctx, T, d_x, d_idx, d_xp, d_row_token, d_inv_row, d_dest, d_seg, NULL));
    CHECK(director_expert_ffn(ctx, T, d_xp, d_seg, d_wg, d_wu, d_wd, d_yp, NULL, NULL, NULL, NULL, NULL, NULL));
    CHECK(director_combine(ctx, T, d_yp, d_inv_row, d_w, NULL, d_y, NULL));
    CHECK(director_placement_cost(ctx, T, d_idx, NULL, d_cost, d_cost + R * E, d_cost + R * E + R,
                                  (uint64_t*)(d_cost + R * E + R + R * R), NULL));
    CHECK(cudaDeviceSynchronize());
    CHECK(director_last_status(ctx, NULL));

    int32_t seg[G + 1], *row_token = (int32_t*)malloc(4 * A), *inv_row = (int32_t*)malloc(4 * A), *dest = (int32_t*)malloc(4 * A);
    int32_t* idx = (int32_t*)malloc(4 * A);
    int64_t cost[R * E + R + 2 * R * R], cost2[R * E + R + 2 * R * R];
    uint16_t* y = (uint16_t*)malloc(2 * T * H);
    uint16_t* y2 = (uint16_t*)malloc(2 * T * H);
    CHECK(cudaMemcpy(seg, d_seg, sizeof seg, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(row_token, d_row_token, 4 * A, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(inv_row, d_inv_row, 4 * A, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(dest, d_dest, 4 * A, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(idx, d_idx, 4 * A, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(cost, d_cost, sizeof cost, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(y, d_y, 2 * T * H, cudaMemcpyDeviceToHost));

    int bad = 0;
    /* segment table: starts at 0, never decreases, ends at T*K */
    if (seg[0] != 0 || seg[G] != A) ++bad;
    for (int g = 0; g < G; ++g) if (seg[g + 1] < seg[g]) ++bad;
    /* every assignment's row points back at its token, lies in a segment of its destination rank, and that rank hosts the expert */
    for (int t = 0; t < T; ++t)
        for (int s = 0; s < K; ++s) {
            const int row = inv_row[t * K + s], k = dest[t * K + s], e = idx[t * K + s];
            if (row < 0 || row >= A || row_token[row] != t) { ++bad; continue; }
            if (k < 0 || k >= R || !X[e][k]) ++bad;
            if (row < seg[k * C] || row >= seg[(k + 1) * C]) ++bad;
        }
    /* Eq. 1: the loads sum to T*K; so do W and D; bytes = tokens * 2H */
    int64_t sum_load = 0, sum_w = 0, sum_d = 0;
    for (int j = 0; j < R; ++j) sum_load += cost[R * E + j];
    for (int i = 0; i < R * E; ++i) sum_w += cost[i];
    for (int i = 0; i < R * R; ++i) {
        sum_d += cost[R * E + R + i];
        if (cost[R * E + R + R * R + i] != cost[R * E + R + i] * 2 * H) ++bad;
    }
    if (sum_load != A || sum_w != A || sum_d != A) ++bad;
    /* the loads equal the segment lengths per rank */
    for (int j = 0; j < R; ++j) if (cost[R * E + j] != seg[(j + 1) * C] - seg[j * C]) ++bad;
    int y_nonzero = 0;
    for (int i = 0; i < T * H; ++i) y_nonzero += (y[i] & 0x7FFFu) != 0;
    if (y_nonzero < T * H / 2) ++bad;                      /* the experts did compute something */

    /* ---- identity experts: combine(dispatch(x)) == x, bit for bit ---- */
    CHECK(director_combine(ctx, T, d_xp, d_inv_row, d_w, NULL, d_y2, NULL));
    CHECK(cudaMemcpy(y2, d_y2, 2 * T * H, cudaMemcpyDeviceToHost));
    const int identity_ok = memcmp(y2, h_x, 2 * T * H) == 0;
    if (!identity_ok) ++bad;

    /* ---- the one-call layer gives the same bits as the stage calls ---- */
    CHECK(cudaMemset(d_y2, 0, 2 * T * H));
    CHECK(director_layer_forward(ctx, T, d_logits, d_x, d_wg, d_wu, d_wd, NULL, NULL, NULL, d_y2, d_cost2, d_cost2 + R * E,
                                 d_cost2 + R * E + R, (uint64_t*)(d_cost2 + R * E + R + R * R), NULL));
    CHECK(cudaDeviceSynchronize());
    CHECK(director_last_status(ctx, NULL));
    CHECK(cudaMemcpy(y2, d_y2, 2 * T * H, cudaMemcpyDeviceToHost));
    CHECK(cudaMemcpy(cost2, d_cost2, sizeof cost2, cudaMemcpyDeviceToHost));
    const int layer_ok = memcmp(y2, y, 2 * T * H) == 0 && memcmp(cost2, cost, sizeof cost) == 0;
    if (!layer_ok) ++bad;

    /* ---- which FFN kernels a batch takes: the streaming ones up to 4 tokens ---- */
    if (director_batch_streams_weights(ctx, T) != 0 || director_batch_streams_weights(ctx, 2) != 1 ||
        director_batch_streams_weights(ctx, 0) >= 0 || director_batch_streams_weights(NULL, 1) >= 0)
        ++bad;

    /* ---- the combining down projection agrees with expert_ffn + combine to a bf16 unit or two ---- */
    float* d_yacc = (float*)dev_copy(NULL, sizeof(float) * T * H);
    float* d_rw = (float*)dev_copy(NULL, sizeof(float) * A);
    if (!d_yacc || !d_rw) return 3;
    CHECK(cudaMemset(d_y2, 0, 2 * T * H));
    CHECK(director_expert_ffn_combine(ctx, T, d_xp, d_seg, d_row_token, d_inv_row, d_w, d_wg, d_wu, d_wd, NULL, NULL, NULL,
                                      NULL, d_yacc, d_rw, d_y2, NULL));
    CHECK(cudaDeviceSynchronize());
    CHECK(director_last_status(ctx, NULL));
    CHECK(cudaMemcpy(y2, d_y2, 2 * T * H, cudaMemcpyDeviceToHost));
    int fused_far = 0;
    for (int i = 0; i < T * H; ++i) {
        uint32_t ua = (uint32_t)y[i] << 16, ub = (uint32_t)y2[i] << 16;
        float a, b;
        memcpy(&a, &ua, 4);
        memcpy(&b, &ub, 4);
        const float d = a > b ? a - b : b - a, m = (a < 0 ? -a : a) > (b < 0 ? -b : b) ? (a < 0 ? -a : a) : (b < 0 ? -b : b);
        if (d > m / 64.0f + 1e-3f) ++fused_far;
    }
    if (fused_far) ++bad;

    printf("layer_from_c: %d tokens, %d assignments, identity %s, one-call layer %s, fused combine %d far, %d mismatches\n",
           T, A, identity_ok ? "exact" : "DIFFERS", layer_ok ? "identical" : "DIFFERS", fused_far, bad);
    CHECK(director_destroy(ctx));
    return bad ? 1 : 0;
}
