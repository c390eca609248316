// (a1) Top-k softmax gating: Section II-A "the gating network computes relevance scores and
// selects a small subset of experts ... weighted summation based on the scores".
//
// One warp per token.  Lane values live in registers; K rounds of a warp arg-max pick the
// experts in (logit descending, expert id ascending) order; the weights are the softmax over
// the K winning logits, which equals the full softmax renormalised over the winners.
// HBM-bound: reads 4*E bytes and writes 8*K bytes per token.
#include "director_common.cuh"

namespace director {

namespace {

constexpr int kRouteWarps = 8;

// Monotone map float -> uint32 (larger float => larger key).  -0.0 is folded onto +0.0 so that
// signed zeros tie.  Keys: 0 = "no candidate", 1 = NaN, real values are >= 0x007FFFFF.
__device__ __forceinline__ uint32_t ordered_key(float v, bool& nonfinite) {
    if (v != v) { nonfinite = true; return 1u; }
    if (fabsf(v) == INFINITY) nonfinite = true;
    uint32_t u = __float_as_uint(v + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_to_float(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// VPL = values per lane.  CONTIG: lane owns experts [lane*VPL, lane*VPL+VPL) and loads them with
// one vector load (E == 32*VPL); otherwise lane owns experts lane + 32*i (any E <= 32*VPL).
template <int VPL, bool CONTIG>
__global__ void __launch_bounds__(kRouteWarps * 32)
route_topk_kernel(const float* __restrict__ logits, int32_t* __restrict__ topk_idx, float* __restrict__ topk_w,
                  int T, int E, int K, int32_t* __restrict__ status) {
    const int lane = threadIdx.x & 31;
    const int t = blockIdx.x * kRouteWarps + (threadIdx.x >> 5);
    if (t >= T) return;
    const float* row = logits + (size_t)t * E;

    uint32_t key[VPL];
    bool nonfinite = false;
    if constexpr (CONTIG) {
        float v[VPL];
        if constexpr (VPL == 4) {
            const float4 q = __ldg(reinterpret_cast<const float4*>(row) + lane);
            v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
        } else if constexpr (VPL == 2) {
            const float2 q = __ldg(reinterpret_cast<const float2*>(row) + lane);
            v[0] = q.x; v[1] = q.y;
        } else if constexpr (VPL == 8) {
            const float4 q0 = __ldg(reinterpret_cast<const float4*>(row) + 2 * lane);
            const float4 q1 = __ldg(reinterpret_cast<const float4*>(row) + 2 * lane + 1);
            v[0] = q0.x; v[1] = q0.y; v[2] = q0.z; v[3] = q0.w;
            v[4] = q1.x; v[5] = q1.y; v[6] = q1.z; v[7] = q1.w;
        } else {
            v[0] = __ldg(row + lane);
        }
#pragma unroll
        for (int i = 0; i < VPL; ++i) key[i] = ordered_key(v[i], nonfinite);
    } else {
#pragma unroll
        for (int i = 0; i < VPL; ++i) {
            const int e = lane + 32 * i;
            key[i] = (e < E) ? ordered_key(__ldg(row + e), nonfinite) : 0u;
        }
    }
    if (__any_sync(0xFFFFFFFFu, nonfinite) && lane == 0) director_set_status(status, DIRECTOR_ERR_NONFINITE);

    float my_logit = 0.0f;      // lane s keeps the s-th winner
    int my_expert = 0;
    for (int s = 0; s < K; ++s) {
        uint32_t best = 0u;
        int best_i = 0;
#pragma unroll
        for (int i = 0; i < VPL; ++i)
            if (key[i] > best) { best = key[i]; best_i = i; }   // strict: lowest local index wins ties
        const uint32_t top = __reduce_max_sync(0xFFFFFFFFu, best);
        const uint32_t my_e = CONTIG ? (uint32_t)(lane * VPL + best_i) : (uint32_t)(lane + 32 * best_i);
        const uint32_t cand = (best == top && best != 0u) ? my_e : 0xFFFFFFFFu;
        const uint32_t win = __reduce_min_sync(0xFFFFFFFFu, cand);
        if (cand == win) {
#pragma unroll
            for (int i = 0; i < VPL; ++i)
                if (i == best_i) key[i] = 0u;                    // taken
        }
        if (lane == s) { my_logit = key_to_float(top); my_expert = (int)win; }
    }
    // softmax over the K winners, relative to the largest (lane 0 holds it)
    const float l0 = __shfl_sync(0xFFFFFFFFu, my_logit, 0);
    float p = (lane < K) ? expf(my_logit - l0) : 0.0f;
    float sum = p;
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);   // K <= 8 lanes
    if (lane < K) {
        topk_idx[(size_t)t * K + lane] = my_expert;
        topk_w[(size_t)t * K + lane] = p / sum;
    }
}

}  // namespace

int launch_route(director_ctx* ctx, int T, const float* logits, int32_t* topk_idx, float* topk_w, cudaStream_t st) {
    const int E = ctx->shape.E, K = ctx->shape.K;
    const dim3 grid((T + kRouteWarps - 1) / kRouteWarps), block(kRouteWarps * 32);
    LaunchScope scope(ctx, st, "route_topk_kernel");
#define ROUTE_LAUNCH(VPL, CONTIG) \
    route_topk_kernel<VPL, CONTIG><<<grid, block, 0, st>>>(logits, topk_idx, topk_w, T, E, K, ctx->d_status)
    if (E == 256) ROUTE_LAUNCH(8, true);
    else if (E == 128) ROUTE_LAUNCH(4, true);
    else if (E == 64) ROUTE_LAUNCH(2, true);
    else if (E == 32) ROUTE_LAUNCH(1, true);
    else if (E <= 32) ROUTE_LAUNCH(1, false);
    else if (E <= 64) ROUTE_LAUNCH(2, false);
    else if (E <= 128) ROUTE_LAUNCH(4, false);
    else ROUTE_LAUNCH(8, false);
#undef ROUTE_LAUNCH
    return cuda_status(cudaGetLastError());
}

}  // namespace director
