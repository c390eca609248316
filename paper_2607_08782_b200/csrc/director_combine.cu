// (a4) Weighted un-permute / combine (Section II-A: a token's result is the sum of its experts' outputs weighted by
// the gate's scores; Section II-B: the second all-to-all brings those outputs back to the token's rank).
//
//   y[t,:] = bf16( sum_s w[t,s] * float(yp[inv_row[t,s],:]) (+ float(y_shared[t,:])) )
//
// One warp per (token, 1 KB column slice): each lane owns 2 x 8 consecutive bf16 columns, gathers
// them from the K rows with 16-byte loads (all K loads in flight), accumulates in fp32 in slot
// order and writes 16 bytes.  HBM-bound gather: 2HK + 8K (+2H) bytes read, 2H written per token.
#include "director_common.cuh"

#include <cuda_bf16.h>

namespace director {

namespace {

constexpr int kCombineWarps = 8;
constexpr int kVecPerLane = 2;                      // uint4 per lane per row
constexpr int kCombineSliceVec = 32 * kVecPerLane;  // uint4 per slice

__device__ __forceinline__ void fma_bf16x8(float (&acc)[8], const uint4& v, float w) {
    const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        acc[2 * i] = fmaf(w, __uint_as_float(u[i] << 16), acc[2 * i]);
        acc[2 * i + 1] = fmaf(w, __uint_as_float(u[i] & 0xFFFF0000u), acc[2 * i + 1]);
    }
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&p);
}

template <int K_T>   // K_T > 0: compile-time top-k (fully unrolled gathers); 0: runtime K
__global__ void __launch_bounds__(kCombineWarps * 32)
combine_kernel(const uint4* __restrict__ yp, const int32_t* __restrict__ inv_row, const float* __restrict__ topk_w,
               const uint4* __restrict__ y_shared, uint4* __restrict__ y, int T, int K_rt, int row_vec,
               int slices_per_row) {
    chain_prologue();
    const int K = K_T > 0 ? K_T : K_rt;
    const int lane = threadIdx.x & 31;
    const long long item = (long long)blockIdx.x * kCombineWarps + (threadIdx.x >> 5);
    if (item >= (long long)T * slices_per_row) return;
    const int t = (int)(item / slices_per_row);
    const int v0 = (int)(item % slices_per_row) * kCombineSliceVec + lane;

    int my_row = -1;
    float my_w = 0.0f;
    if (lane < K) {
        my_row = __ldg(inv_row + (size_t)t * K + lane);
        my_w = __ldg(topk_w + (size_t)t * K + lane);
    }
    float acc[kVecPerLane][8];
#pragma unroll
    for (int i = 0; i < kVecPerLane; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;

    if constexpr (K_T > 0) {
        uint4 v[K_T][kVecPerLane];
        int rows[K_T];
        float ws[K_T];
#pragma unroll
        for (int s = 0; s < K_T; ++s) {
            rows[s] = __shfl_sync(0xFFFFFFFFu, my_row, s);
            ws[s] = __shfl_sync(0xFFFFFFFFu, my_w, s);
#pragma unroll
            for (int i = 0; i < kVecPerLane; ++i) {
                v[s][i] = make_uint4(0u, 0u, 0u, 0u);
                if (rows[s] >= 0 && v0 + 32 * i < row_vec) v[s][i] = __ldcs(yp + (size_t)rows[s] * row_vec + v0 + 32 * i);
            }
        }
#pragma unroll
        for (int s = 0; s < K_T; ++s)
#pragma unroll
            for (int i = 0; i < kVecPerLane; ++i) fma_bf16x8(acc[i], v[s][i], ws[s]);
    } else {
        for (int s = 0; s < K; ++s) {
            const int row = __shfl_sync(0xFFFFFFFFu, my_row, s);
            const float w = __shfl_sync(0xFFFFFFFFu, my_w, s);
            if (row < 0) continue;
#pragma unroll
            for (int i = 0; i < kVecPerLane; ++i)
                if (v0 + 32 * i < row_vec) fma_bf16x8(acc[i], __ldcs(yp + (size_t)row * row_vec + v0 + 32 * i), w);
        }
    }
#pragma unroll
    for (int i = 0; i < kVecPerLane; ++i) {
        if (v0 + 32 * i >= row_vec) continue;
        if (y_shared) fma_bf16x8(acc[i], __ldcs(y_shared + (size_t)t * row_vec + v0 + 32 * i), 1.0f);
        uint4 o;
        o.x = pack_bf16x2(acc[i][0], acc[i][1]);
        o.y = pack_bf16x2(acc[i][2], acc[i][3]);
        o.z = pack_bf16x2(acc[i][4], acc[i][5]);
        o.w = pack_bf16x2(acc[i][6], acc[i][7]);
        y[(size_t)t * row_vec + v0 + 32 * i] = o;
    }
}

}  // namespace

int launch_combine(director_ctx* ctx, int T, const void* yp, const int32_t* inv_row, const float* topk_w,
                   const void* y_shared, void* y, cudaStream_t st) {
    StageScope stage(ctx, st, "stage_combine");
    const director_shape& s = ctx->shape;
    const int row_vec = s.H * 2 / 16;
    const int slices = (row_vec + kCombineSliceVec - 1) / kCombineSliceVec;
    const long long items = (long long)T * slices;
    const unsigned grid = (unsigned)((items + kCombineWarps - 1) / kCombineWarps);
    LaunchScope scope(ctx, st, "combine_kernel");
#define COMBINE_LAUNCH(KT)                                                                                      \
    launch_chained(combine_kernel<KT>, dim3(grid), dim3(kCombineWarps * 32), 0, st, static_cast<const uint4*>(yp),  \
                   inv_row, topk_w, static_cast<const uint4*>(y_shared), static_cast<uint4*>(y), T, (int)s.K, row_vec,  \
                   slices)
    switch (s.K) {
        case 1: COMBINE_LAUNCH(1); break;
        case 2: COMBINE_LAUNCH(2); break;
        case 4: COMBINE_LAUNCH(4); break;
        case 6: COMBINE_LAUNCH(6); break;
        case 8: COMBINE_LAUNCH(8); break;
        default: COMBINE_LAUNCH(0); break;
    }
#undef COMBINE_LAUNCH
    return cuda_status(cudaGetLastError());
}

}  // namespace director
