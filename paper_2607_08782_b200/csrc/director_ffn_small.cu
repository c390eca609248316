// Expert FFN for decode-sized batches (at most kSmallFfnTokens tokens; Section II-A expert FFNs after dispatch).
//
// With a handful of tokens every segment holds at most a few rows and the FFN is a stream of the touched experts'
// weights through a few dot products: bound by HBM bandwidth, not by arithmetic (75.6 MB of weights against 75 MFLOP
// for one token of the Qwen3-shaped layer).  A tensor-core tile would compute 32 token columns for the one that
// exists and, worse, leaves the weight stream to as many SMs as there are (segment, weight block) items.  Here the
// work is cut per OUTPUT FEATURE instead: a warp owns two output features of one segment, streams their weight rows
// with 16-byte loads (all of a row's loads in flight at once), multiplies them with the segment's rows held in
// shared memory, and reduces over the warp.  Thousands of warps stream at once, whatever the number of segments.
//
//   gate/up:  Hg[r, f] = silu(x_r . Wg[e, f, :]) * (x_r . Wu[e, f, :])      r < n rows of the segment (n <= 4)
//   down:     Yp[r, h] = Hg_r . Wd[e, h, :]
//
// bf16 operands, fp32 accumulation in a fixed order (lane-strided partial sums, then a butterfly over the warp), so
// results are reproducible run to run and do not depend on the placement; Hg is rounded to bf16 between the two
// kernels exactly as in the tensor-core path.
#include "director_common.cuh"

#include <cuda_bf16.h>

namespace director {

namespace {

constexpr int kSmallWarps = 8;          // warps per CTA
constexpr int kFeaturesPerWarp = 2;     // output features a warp computes, one after the other
constexpr int kChunk = 4096;            // elements of the contraction dimension staged in shared memory at a time
constexpr int kRowsMax = kSmallFfnTokens;
static_assert(kRowsMax == 4, "the row-count switch below lists the cases 1..4");

struct SmallParams {
    const int32_t* seg_offsets;   // [G+1]
    const int32_t* slot_expert;   // [G]
    int G;
    const uint16_t* in;           // bf16 [rows, Kdim]
    const uint16_t* w0;           // MODE 0: gate [E, N, Kdim]; MODE 1: down [E, N, Kdim]
    const uint16_t* w1;           // MODE 0: up   [E, N, Kdim]
    int N;                        // output features per row: F (MODE 0), H (MODE 1)
    int Kdim;                     // contraction length: H (MODE 0), F (MODE 1)
    uint16_t* out;                // bf16 [rows, N]
    int32_t* status;
};

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

// Partial dot products of one weight row (two for MODE 0) with NR staged rows over the staged chunk.
template <int MODE, int NR>
__device__ __forceinline__ void accumulate_chunk(const uint16_t* __restrict__ wg, const uint16_t* __restrict__ wu,
                                                 const uint16_t* s_rows, int chunk_len, int lane, float (&ag)[kRowsMax],
                                                 float (&au)[kRowsMax]) {
    const int vecs = chunk_len >> 3;                       // 16-byte vectors in the chunk
    for (int c0 = lane; c0 < vecs; c0 += 128) {            // four vectors per lane and weight row in flight
        uint4 g[4], u[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = c0 + 32 * j;
            g[j] = c < vecs ? __ldcs(reinterpret_cast<const uint4*>(wg) + c) : make_uint4(0, 0, 0, 0);
            if (MODE == 0) u[j] = c < vecs ? __ldcs(reinterpret_cast<const uint4*>(wu) + c) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = c0 + 32 * j;
            if (c >= vecs) break;
            float gf[8], uf[8];
            unpack8(g[j], gf);
            if (MODE == 0) unpack8(u[j], uf);
#pragma unroll
            for (int r = 0; r < NR; ++r) {
                float xf[8];
                unpack8(*reinterpret_cast<const uint4*>(s_rows + (size_t)r * kChunk + 8 * c), xf);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    ag[r] = fmaf(gf[i], xf[i], ag[r]);
                    if (MODE == 0) au[r] = fmaf(uf[i], xf[i], au[r]);
                }
            }
        }
    }
}

// MODE 0: gate/up + SwiGLU.  MODE 1: down projection.
// grid.x: blocks of kSmallWarps * kFeaturesPerWarp output features; grid.y: ordinal of the non-empty segment.
template <int MODE>
__global__ void __launch_bounds__(kSmallWarps * 32)
small_ffn_kernel(const SmallParams p) {
    extern __shared__ __align__(16) uint16_t s_rows[];     // [n][kChunk] bf16
    __shared__ int s_slot;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // the blockIdx.y-th non-empty segment (slot with an expert and at least one row), found by warp 0
    if (warp == 0) {
        int seen = 0, found = -1;
        for (int g0 = 0; g0 < p.G && found < 0; g0 += 32) {
            const int g = g0 + lane;
            const bool full = g < p.G && __ldg(p.slot_expert + g) >= 0 && __ldg(p.seg_offsets + g + 1) > __ldg(p.seg_offsets + g);
            const unsigned m = __ballot_sync(0xFFFFFFFFu, full);
            const int here = __popc(m);
            if (seen + here > (int)blockIdx.y) {
                unsigned mm = m;
                for (int i = 0; i < (int)blockIdx.y - seen; ++i) mm &= mm - 1;   // drop the lower set bits
                found = g0 + __ffs(mm) - 1;
            }
            seen += here;
        }
        if (lane == 0) s_slot = found;
    }
    __syncthreads();
    const int g = s_slot;
    if (g < 0) return;                                      // fewer non-empty segments than grid.y
    const int row0 = __ldg(p.seg_offsets + g);
    int n = __ldg(p.seg_offsets + g + 1) - row0;
    if (n > kRowsMax) {                                     // cannot happen for a batch of at most kRowsMax tokens
        if (threadIdx.x == 0) director_set_status(p.status, DIRECTOR_ERR_BAD_INDEX);
        n = kRowsMax;
    }
    const int e = __ldg(p.slot_expert + g);

    const int f_base = (blockIdx.x * kSmallWarps + warp) * kFeaturesPerWarp;
    float ag[kFeaturesPerWarp][kRowsMax], au[kFeaturesPerWarp][kRowsMax];
#pragma unroll
    for (int q = 0; q < kFeaturesPerWarp; ++q)
#pragma unroll
        for (int r = 0; r < kRowsMax; ++r) ag[q][r] = au[q][r] = 0.0f;

    for (int k0 = 0; k0 < p.Kdim; k0 += kChunk) {
        const int len = min(kChunk, p.Kdim - k0);
        if (k0 > 0) __syncthreads();                        // everybody is done with the previous chunk
        for (int i = threadIdx.x; i < n * (len >> 3); i += blockDim.x) {
            const int r = i / (len >> 3), c = i - r * (len >> 3);
            *reinterpret_cast<uint4*>(s_rows + (size_t)r * kChunk + 8 * c) =
                __ldg(reinterpret_cast<const uint4*>(p.in + (size_t)(row0 + r) * p.Kdim + k0) + c);
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < kFeaturesPerWarp; ++q) {
            const int f = f_base + q;
            if (f >= p.N) break;
            const size_t w_off = ((size_t)e * p.N + f) * p.Kdim + k0;
            const uint16_t* wg = p.w0 + w_off;
            const uint16_t* wu = MODE == 0 ? p.w1 + w_off : nullptr;
            switch (n) {                                    // the row loop is unrolled for the segment's length
                case 1: accumulate_chunk<MODE, 1>(wg, wu, s_rows, len, lane, ag[q], au[q]); break;
                case 2: accumulate_chunk<MODE, 2>(wg, wu, s_rows, len, lane, ag[q], au[q]); break;
                case 3: accumulate_chunk<MODE, 3>(wg, wu, s_rows, len, lane, ag[q], au[q]); break;
                default: accumulate_chunk<MODE, kRowsMax>(wg, wu, s_rows, len, lane, ag[q], au[q]); break;
            }
        }
    }

    // butterfly over the warp; afterwards every lane holds the full sums.  Lane r writes row r.
#pragma unroll
    for (int q = 0; q < kFeaturesPerWarp; ++q) {
        const int f = f_base + q;
        if (f >= p.N) break;
        float mine = 0.0f;
#pragma unroll
        for (int r = 0; r < kRowsMax; ++r) {
            if (r >= n) break;
            float sg = ag[q][r], su = au[q][r];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                sg += __shfl_xor_sync(0xFFFFFFFFu, sg, o);
                if (MODE == 0) su += __shfl_xor_sync(0xFFFFFFFFu, su, o);
            }
            const float v = MODE == 0 ? __fdividef(sg * su, 1.0f + __expf(-sg)) : sg;
            if (lane == r) mine = v;
        }
        if (lane < n) p.out[(size_t)(row0 + lane) * p.N + f] = __bfloat16_as_ushort(__float2bfloat16_rn(mine));
    }
}

size_t small_smem_bytes(int rows) { return (size_t)rows * kChunk * 2; }

template <int MODE>
int launch_small(director_ctx* ctx, const char* name, const SmallParams& p, int rows_max, int max_segments, cudaStream_t st) {
    const dim3 grid((unsigned)((p.N + kSmallWarps * kFeaturesPerWarp - 1) / (kSmallWarps * kFeaturesPerWarp)),
                    (unsigned)max_segments);
    LaunchScope scope(ctx, st, name);
    small_ffn_kernel<MODE><<<grid, kSmallWarps * 32, small_smem_bytes(rows_max), st>>>(p);
    return cuda_status(cudaGetLastError());
}

}  // namespace

int ffn_small_init(director_ctx*) {
    const int bytes = (int)small_smem_bytes(kRowsMax);      // 32 KB
    if (cudaFuncSetAttribute(small_ffn_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess ||
        cudaFuncSetAttribute(small_ffn_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    return DIRECTOR_OK;
}

// in [rows, H] -> hidden [rows, Fw] -> out [rows, H] over a segment table whose segments hold at most kSmallFfnTokens
// rows (a batch of at most that many tokens).  max_segments: upper bound of the non-empty segments.
int ffn_pass_small(director_ctx* ctx, const void* in, const int32_t* seg_offsets, const int32_t* slot_expert, int G,
                   const void* w_gate, const void* w_up, const void* w_down, int Fw, void* hidden, void* out, int rows_max,
                   int max_segments, cudaStream_t st) {
    const int H = ctx->shape.H;
    const SmallParams p1{seg_offsets, slot_expert, G, static_cast<const uint16_t*>(in), static_cast<const uint16_t*>(w_gate),
                         static_cast<const uint16_t*>(w_up), Fw, H, static_cast<uint16_t*>(hidden), ctx->d_status};
    int rc = launch_small<0>(ctx, "small_ffn_swiglu_kernel", p1, rows_max, max_segments, st);
    if (rc != DIRECTOR_OK) return rc;
    const SmallParams p2{seg_offsets, slot_expert, G, static_cast<const uint16_t*>(hidden), static_cast<const uint16_t*>(w_down),
                         nullptr, H, Fw, static_cast<uint16_t*>(out), ctx->d_status};
    return launch_small<1>(ctx, "small_ffn_down_kernel", p2, rows_max, max_segments, st);
}

}  // namespace director
