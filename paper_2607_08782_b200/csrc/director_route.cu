// (a1) Top-k softmax gating: Section II-A "the gating network computes relevance scores and
// selects a small subset of experts ... weighted summation based on the scores".
//
// LPT lanes per token (1, 2, 4 or 8, chosen from E), no branches that depend on the data.  A lane streams
// every LPT-th group of eight logits of its token's row (two 16-byte loads; the lanes of a token read
// adjacent groups, so a token's loads are contiguous), turns each logit into a 64-bit key
//     (order-preserving image of the float) << 32 | (0xFFFFFFFF - expert id)
// so that a plain unsigned comparison orders by (logit descending, expert id ascending), sorts the
// eight keys with a 19-comparator network and merges them into the running top-8 (element-wise max
// against the reversed list gives a bitonic sequence holding the 8 largest; 12 more comparators
// sort it).  The lanes of a token then merge their lists pairwise through shuffles with the same step.
// The weights are the softmax over the K winning logits, which equals the full softmax renormalised
// over the winners.  HBM traffic is 4E bytes in and 8K bytes out per token.
#include "director_common.cuh"

namespace director {

namespace {

constexpr int kRouteThreads = 128;

// Monotone map float -> uint32 (larger float => larger key); -0.0 is folded onto +0.0 first.
__device__ __forceinline__ uint32_t ordered_bits(float v) {
    const uint32_t u = __float_as_uint(v + 0.0f);
    return u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u);
}
__device__ __forceinline__ float bits_to_float(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// compare-exchange: afterwards a >= b
__device__ __forceinline__ void cx(unsigned long long& a, unsigned long long& b) {
    const unsigned long long hi = a > b ? a : b, lo = a > b ? b : a;
    a = hi;
    b = lo;
}

__device__ __forceinline__ void sort8_desc(unsigned long long (&k)[8]) {
    cx(k[0], k[1]); cx(k[2], k[3]); cx(k[4], k[5]); cx(k[6], k[7]);
    cx(k[0], k[2]); cx(k[1], k[3]); cx(k[4], k[6]); cx(k[5], k[7]);
    cx(k[1], k[2]); cx(k[5], k[6]); cx(k[0], k[4]); cx(k[3], k[7]);
    cx(k[1], k[5]); cx(k[2], k[6]);
    cx(k[1], k[4]); cx(k[3], k[6]);
    cx(k[2], k[4]); cx(k[3], k[5]);
    cx(k[3], k[4]);
}

// top[] and grp[] sorted descending -> top[] = the 8 largest of the 16, sorted descending
__device__ __forceinline__ void merge_top8(unsigned long long (&top)[8], const unsigned long long (&grp)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) top[i] = top[i] > grp[7 - i] ? top[i] : grp[7 - i];
    cx(top[0], top[4]); cx(top[1], top[5]); cx(top[2], top[6]); cx(top[3], top[7]);
    cx(top[0], top[2]); cx(top[1], top[3]); cx(top[4], top[6]); cx(top[5], top[7]);
    cx(top[0], top[1]); cx(top[2], top[3]); cx(top[4], top[5]); cx(top[6], top[7]);
}

// VEC: the row can be read with 16-byte loads (E % 4 == 0; rows are then 16-byte aligned).
template <bool VEC, int LPT>
__global__ void __launch_bounds__(kRouteThreads)
route_topk_kernel(const float* __restrict__ logits, int32_t* __restrict__ topk_idx, float* __restrict__ topk_w,
                  int T, int E, int K, int32_t* __restrict__ status) {
    const int tid = blockIdx.x * kRouteThreads + threadIdx.x;
    const int t_raw = tid / LPT, sub = tid % LPT;
    const bool live = t_raw < T;
    const int t = live ? t_raw : T - 1;                // surplus lanes redo the last token (keeps shuffles full)
    const float* row = logits + (size_t)t * E;

    unsigned long long top[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) top[i] = 0ull;      // below every real key
    uint32_t max_abs = 0u;                           // largest |logit| bit pattern: >= 0x7F800000 iff Inf/NaN present

    for (int e0 = 8 * sub; e0 < E; e0 += 8 * LPT) {
        float v[8];
        if (VEC && e0 + 8 <= E) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(row + e0));
            const float4 b = __ldg(reinterpret_cast<const float4*>(row + e0 + 4));
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = (e0 + i < E) ? __ldg(row + e0 + i) : 0.0f;
        }
        unsigned long long grp[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t raw = __float_as_uint(v[i]) & 0x7FFFFFFFu;
            const bool real = e0 + i < E;
            max_abs = real ? max(max_abs, raw) : max_abs;
            const uint32_t hi = raw > 0x7F800000u ? 1u : ordered_bits(v[i]);     // NaN orders below every number
            grp[i] = real ? ((unsigned long long)hi << 32) | (uint32_t)(0xFFFFFFFFu - (uint32_t)(e0 + i)) : 0ull;
        }
        sort8_desc(grp);
        merge_top8(top, grp);
    }
    // merge the lists of the token's lanes (butterfly: afterwards every lane holds the token's top 8)
#pragma unroll
    for (int step = 1; step < LPT; step <<= 1) {
        unsigned long long other[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) other[i] = __shfl_xor_sync(0xFFFFFFFFu, top[i], step);
        max_abs = max(max_abs, __shfl_xor_sync(0xFFFFFFFFu, max_abs, step));
        merge_top8(top, other);
    }
    if (!live || sub != 0) return;
    if (max_abs >= 0x7F800000u) director_set_status(status, DIRECTOR_ERR_NONFINITE);

    // softmax over the K winners relative to the largest
    const float l0 = bits_to_float((uint32_t)(top[0] >> 32));
    float p[8], sum = 0.0f;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        p[s] = s < K ? expf(bits_to_float((uint32_t)(top[s] >> 32)) - l0) : 0.0f;
        sum += p[s];
    }
    const float inv = 1.0f / sum;
    int32_t* oi = topk_idx + (size_t)t * K;
    float* ow = topk_w + (size_t)t * K;
    if (K == 8) {
        int4 i0, i1;
        float4 w0, w1;
        i0.x = (int)(0xFFFFFFFFu - (uint32_t)top[0]); i0.y = (int)(0xFFFFFFFFu - (uint32_t)top[1]);
        i0.z = (int)(0xFFFFFFFFu - (uint32_t)top[2]); i0.w = (int)(0xFFFFFFFFu - (uint32_t)top[3]);
        i1.x = (int)(0xFFFFFFFFu - (uint32_t)top[4]); i1.y = (int)(0xFFFFFFFFu - (uint32_t)top[5]);
        i1.z = (int)(0xFFFFFFFFu - (uint32_t)top[6]); i1.w = (int)(0xFFFFFFFFu - (uint32_t)top[7]);
        w0 = make_float4(p[0] * inv, p[1] * inv, p[2] * inv, p[3] * inv);
        w1 = make_float4(p[4] * inv, p[5] * inv, p[6] * inv, p[7] * inv);
        reinterpret_cast<int4*>(oi)[0] = i0; reinterpret_cast<int4*>(oi)[1] = i1;
        reinterpret_cast<float4*>(ow)[0] = w0; reinterpret_cast<float4*>(ow)[1] = w1;
    } else {
#pragma unroll
        for (int s = 0; s < 8; ++s)
            if (s < K) {
                oi[s] = (int)(0xFFFFFFFFu - (uint32_t)top[s]);
                ow[s] = p[s] * inv;
            }
    }
}

}  // namespace

int launch_route(director_ctx* ctx, int T, const float* logits, int32_t* topk_idx, float* topk_w, cudaStream_t st) {
    const int E = ctx->shape.E, K = ctx->shape.K;
    // lanes per token: one per group of eight experts, at most 8 (more lanes = more parallelism for the same work)
    const int groups = (E + 7) / 8;
    const int lpt = groups >= 8 ? 8 : groups >= 4 ? 4 : groups >= 2 ? 2 : 1;
    const long long threads = (long long)T * lpt;
    const dim3 grid((unsigned)((threads + kRouteThreads - 1) / kRouteThreads)), block(kRouteThreads);
    LaunchScope scope(ctx, st, "route_topk_kernel");
#define ROUTE_LAUNCH(VEC, LPT) \
    route_topk_kernel<VEC, LPT><<<grid, block, 0, st>>>(logits, topk_idx, topk_w, T, E, K, ctx->d_status)
    const bool vec = E % 4 == 0;
    if (lpt == 8) { if (vec) ROUTE_LAUNCH(true, 8); else ROUTE_LAUNCH(false, 8); }
    else if (lpt == 4) { if (vec) ROUTE_LAUNCH(true, 4); else ROUTE_LAUNCH(false, 4); }
    else if (lpt == 2) { if (vec) ROUTE_LAUNCH(true, 2); else ROUTE_LAUNCH(false, 2); }
    else { if (vec) ROUTE_LAUNCH(true, 1); else ROUTE_LAUNCH(false, 1); }
#undef ROUTE_LAUNCH
    return cuda_status(cudaGetLastError());
}

}  // namespace director
