// Expert FFN for decode-sized batches (at most kSmallFfnTokens tokens; Section II-A expert FFNs after dispatch).
//
// With a handful of tokens every segment holds at most a few rows and the FFN is a stream of the touched experts'
// weights through a few dot products: bound by HBM bandwidth, not by arithmetic (75.6 MB of weights against 75 MFLOP
// for one token of the Qwen3-shaped layer).  A tensor-core tile would compute 32 token columns for the one that
// exists and, worse, leaves the weight stream to as many SMs as there are (segment, weight block) items.  Here the
// work is cut per OUTPUT FEATURE instead: a CTA stages its segment's rows in shared memory and takes a block of
// output features sized so that the grid fills the GPU about twice; each warp streams the weight row(s) of one
// feature at a time with 16-byte loads (eight in flight per lane), multiplies them with the staged rows and reduces
// over the warp.  Every SM streams weights, whatever the number of segments.
//
//   gate/up:  Hg[r, f] = silu(x_r . Wg[e, f, :]) * (x_r . Wu[e, f, :])      r < n rows of the segment (n <= 4)
//   down:     Yp[r, h] = Hg_r . Wd[e, h, :]
//
// bf16 operands, fp32 accumulation in a fixed order (lane-strided partial sums, then a butterfly over the warp), so
// results are reproducible run to run and do not depend on the placement; Hg is rounded to bf16 between the two
// kernels exactly as in the tensor-core path.
#include "director_common.cuh"

#include <cuda_bf16.h>

#include <algorithm>

namespace director {

namespace {

constexpr int kSmallWarps = 8;          // warps per CTA
constexpr int kRowsMax = kSmallFfnTokens;
constexpr int kSmallMaxSmem = 200 * 1024;   // the segment's rows are staged whole: rows x contraction length x 2 bytes
inline size_t small_smem_bytes(int rows, int Kdim) { return (size_t)rows * Kdim * 2; }
static_assert(kRowsMax == 4, "the row-count switch below lists the cases 1..4");

struct SmallParams {
    const int32_t* seg_offsets;   // [G+1]
    const int32_t* slot_expert;   // [G]
    int G;
    const uint16_t* in;           // bf16 [rows, Kdim]
    const int32_t* gather_rows;   // nullptr, or: row i of the segment table is in[gather_rows[i]] (the un-permuted input)
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

// Dot products of one weight row (two for MODE 0: gate and up) with the NR staged rows.  Lane l takes the 16-byte
// vectors l, l + 32, ...; eight vectors per weight row are in flight at a time.
template <int MODE, int NR>
__device__ __forceinline__ void feature_dots(const uint16_t* __restrict__ wg, const uint16_t* __restrict__ wu,
                                             const uint16_t* s_rows, int row_pitch, int vecs, int lane,
                                             float (&ag)[kRowsMax], float (&au)[kRowsMax]) {
#pragma unroll
    for (int r = 0; r < kRowsMax; ++r) ag[r] = au[r] = 0.0f;
    constexpr int VB = MODE == 0 ? 8 : 8;                  // vectors per lane and weight row in flight
    for (int c0 = lane; c0 < vecs; c0 += 32 * VB) {
        uint4 g[VB], u[VB];
#pragma unroll
        for (int j = 0; j < VB; ++j) {
            const int c = c0 + 32 * j;
            g[j] = c < vecs ? __ldcs(reinterpret_cast<const uint4*>(wg) + c) : make_uint4(0, 0, 0, 0);
            if (MODE == 0) u[j] = c < vecs ? __ldcs(reinterpret_cast<const uint4*>(wu) + c) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int j = 0; j < VB; ++j) {
            const int c = c0 + 32 * j;
            if (c >= vecs) break;
            float gf[8], uf[8];
            unpack8(g[j], gf);
            if (MODE == 0) unpack8(u[j], uf);
#pragma unroll
            for (int r = 0; r < NR; ++r) {
                float xf[8];
                unpack8(*reinterpret_cast<const uint4*>(s_rows + (size_t)r * row_pitch + 8 * c), xf);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    ag[r] = fmaf(gf[i], xf[i], ag[r]);
                    if (MODE == 0) au[r] = fmaf(uf[i], xf[i], au[r]);
                }
            }
        }
    }
}

// Short contraction (at most 128 vectors per row, e.g. F = 768): one row gives a lane only a few loads, too few to
// cover the memory latency, so FB consecutive output features are streamed together (FB x ceil(vecs / 32) loads in
// flight per lane).  Down projection only.
template <int NR, int FB>
__device__ __forceinline__ void feature_dots_short(const uint16_t* __restrict__ w, int Kdim, int n_feat,
                                                   const uint16_t* s_rows, int vecs, int lane, float (&acc)[FB][kRowsMax]) {
    uint4 v[FB][4];
#pragma unroll
    for (int q = 0; q < FB; ++q)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = lane + 32 * j;
            v[q][j] = (c < vecs && q < n_feat) ? __ldcs(reinterpret_cast<const uint4*>(w + (size_t)q * Kdim) + c)
                                               : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
    for (int q = 0; q < FB; ++q)
#pragma unroll
        for (int r = 0; r < kRowsMax; ++r) acc[q][r] = 0.0f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int c = lane + 32 * j;
        if (c >= vecs) break;
#pragma unroll
        for (int r = 0; r < NR; ++r) {
            float xf[8];
            unpack8(*reinterpret_cast<const uint4*>(s_rows + (size_t)r * Kdim + 8 * c), xf);
#pragma unroll
            for (int q = 0; q < FB; ++q) {
                float wf[8];
                unpack8(v[q][j], wf);
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[q][r] = fmaf(wf[i], xf[i], acc[q][r]);
            }
        }
    }
}

// MODE 0: gate/up + SwiGLU.  MODE 1: down projection.
// grid.x: blocks of `features_per_cta` output features; grid.y: ordinal of the non-empty segment.
template <int MODE>
__global__ void __launch_bounds__(kSmallWarps * 32)
small_ffn_kernel(const SmallParams p, const int features_per_cta) {
    extern __shared__ __align__(16) uint16_t s_rows[];     // [n][Kdim] bf16: the segment's rows
    __shared__ int s_slot, s_lo, s_hi, s_ex;               // the CTA's segment: slot, row range, expert
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    chain_prologue();

    // The blockIdx.y-th non-empty segment (slot with an expert and at least one row), found by warp 0: the table is
    // read 256 slots at a time with all loads of a batch in flight together (one round trip to L2 per batch).
    if (warp == 0) {
        int seen = 0, found = -1, f_lo = 0, f_hi = 0, f_ex = -1;
        for (int b0 = 0; b0 < p.G && found < 0; b0 += 256) {
            int ex[8], lo[8], hi[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int g = b0 + 32 * i + lane;
                const bool in = g < p.G;
                ex[i] = in ? __ldg(p.slot_expert + g) : -1;
                lo[i] = in ? __ldg(p.seg_offsets + g) : 0;
                hi[i] = in ? __ldg(p.seg_offsets + g + 1) : 0;
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const unsigned m = __ballot_sync(0xFFFFFFFFu, ex[i] >= 0 && hi[i] > lo[i]);
                const int here = __popc(m);
                if (found < 0 && seen + here > (int)blockIdx.y) {
                    unsigned mm = m;
                    for (int k = 0; k < (int)blockIdx.y - seen; ++k) mm &= mm - 1;   // drop the lower set bits
                    const int src = __ffs(mm) - 1;                  // the lane that holds the segment (warp-uniform)
                    found = b0 + 32 * i + src;
                    f_lo = __shfl_sync(0xFFFFFFFFu, lo[i], src);
                    f_hi = __shfl_sync(0xFFFFFFFFu, hi[i], src);
                    f_ex = __shfl_sync(0xFFFFFFFFu, ex[i], src);
                }
                seen += here;
            }
        }
        if (lane == 0) { s_slot = found; s_lo = f_lo; s_hi = f_hi; s_ex = f_ex; }
    }
    __syncthreads();
    const int g = s_slot;
    if (g < 0) return;                                      // fewer non-empty segments than grid.y
    const int row0 = s_lo;
    int n = s_hi - row0;
    if (n > kRowsMax) {                                     // cannot happen for a batch of at most kRowsMax tokens
        if (threadIdx.x == 0) director_set_status(p.status, DIRECTOR_ERR_BAD_INDEX);
        n = kRowsMax;
    }
    const int e = s_ex;
    const int vecs = p.Kdim >> 3;                           // 16-byte vectors per row
    {
        // the first weight rows this CTA will stream (one feature per warp, two matrices for MODE 0) are asked into L2
        // now, so that their first round trip to HBM runs while the segment's rows are being staged below
        const int f0 = blockIdx.x * features_per_cta;
        const int n_first = min(kSmallWarps, min((int)(blockIdx.x + 1) * features_per_cta, p.N) - f0);
        const size_t lines = ((size_t)n_first * p.Kdim * 2 + 127) / 128;            // consecutive rows: one byte range
        const char* b0 = reinterpret_cast<const char*>(p.w0 + ((size_t)e * p.N + f0) * p.Kdim);
        const char* b1 = MODE == 0 ? reinterpret_cast<const char*>(p.w1 + ((size_t)e * p.N + f0) * p.Kdim) : nullptr;
        for (size_t l = threadIdx.x; l < lines; l += blockDim.x) {
            asm volatile("prefetch.global.L2 [%0];" ::"l"(b0 + 128 * l));
            if (MODE == 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(b1 + 128 * l));
        }
    }

    for (int i = threadIdx.x; i < n * vecs; i += blockDim.x) {
        const int r = i / vecs, c = i - r * vecs;
        const int src = p.gather_rows ? __ldg(p.gather_rows + row0 + r) : row0 + r;
        *reinterpret_cast<uint4*>(s_rows + (size_t)r * p.Kdim + 8 * c) =
            __ldg(reinterpret_cast<const uint4*>(p.in + (size_t)src * p.Kdim) + c);
    }
    __syncthreads();

    // the CTA's features, dealt to its warps in turn
    const int f_end = min((int)(blockIdx.x + 1) * features_per_cta, p.N);
    if (MODE == 1 && vecs <= 128) {
        // short rows: four consecutive features per warp and pass
        constexpr int FB = 4;
        for (int f = blockIdx.x * features_per_cta + FB * warp; f < f_end; f += FB * kSmallWarps) {
            const int n_feat = min(FB, f_end - f);
            const uint16_t* w = p.w0 + ((size_t)e * p.N + f) * p.Kdim;
            float acc[FB][kRowsMax];
            switch (n) {
                case 1: feature_dots_short<1, FB>(w, p.Kdim, n_feat, s_rows, vecs, lane, acc); break;
                case 2: feature_dots_short<2, FB>(w, p.Kdim, n_feat, s_rows, vecs, lane, acc); break;
                case 3: feature_dots_short<3, FB>(w, p.Kdim, n_feat, s_rows, vecs, lane, acc); break;
                default: feature_dots_short<kRowsMax, FB>(w, p.Kdim, n_feat, s_rows, vecs, lane, acc); break;
            }
#pragma unroll
            for (int q = 0; q < FB; ++q) {
                if (q >= n_feat) break;
                float mine = 0.0f;
#pragma unroll
                for (int r = 0; r < kRowsMax; ++r) {
                    if (r >= n) break;
                    float sg = acc[q][r];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) sg += __shfl_xor_sync(0xFFFFFFFFu, sg, o);
                    if (lane == r) mine = sg;
                }
                if (lane < n) p.out[(size_t)(row0 + lane) * p.N + f + q] = __bfloat16_as_ushort(__float2bfloat16_rn(mine));
            }
        }
        return;
    }
    for (int f = blockIdx.x * features_per_cta + warp; f < f_end; f += kSmallWarps) {
        const size_t w_off = ((size_t)e * p.N + f) * p.Kdim;
        const uint16_t* wg = p.w0 + w_off;
        const uint16_t* wu = MODE == 0 ? p.w1 + w_off : nullptr;
        float ag[kRowsMax], au[kRowsMax];
        switch (n) {                                        // the row loop is unrolled for the segment's length
            case 1: feature_dots<MODE, 1>(wg, wu, s_rows, p.Kdim, vecs, lane, ag, au); break;
            case 2: feature_dots<MODE, 2>(wg, wu, s_rows, p.Kdim, vecs, lane, ag, au); break;
            case 3: feature_dots<MODE, 3>(wg, wu, s_rows, p.Kdim, vecs, lane, ag, au); break;
            default: feature_dots<MODE, kRowsMax>(wg, wu, s_rows, p.Kdim, vecs, lane, ag, au); break;
        }
        // butterfly over the warp; afterwards every lane holds the full sums.  Lane r writes row r.
        float mine = 0.0f;
#pragma unroll
        for (int r = 0; r < kRowsMax; ++r) {
            if (r >= n) break;
            float sg = ag[r], su = au[r];
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

template <int MODE>
int launch_small(director_ctx* ctx, const char* name, const SmallParams& p, int rows_max, int max_segments, cudaStream_t st) {
    // as many features per CTA as keeps the grid at about two CTAs per SM per wave (at least one feature per warp)
    const long long total = (long long)p.N * max_segments;
    long long per_cta = (total + 2 * ctx->sm_count - 1) / (2 * ctx->sm_count);
    per_cta = std::max<long long>(kSmallWarps, std::min<long long>(per_cta, p.N));
    const long long quantum = (MODE == 1 && (p.Kdim >> 3) <= 128) ? 4 * kSmallWarps : kSmallWarps;   // features per pass of a CTA
    per_cta = (per_cta + quantum - 1) / quantum * quantum;
    const dim3 grid((unsigned)((p.N + per_cta - 1) / per_cta), (unsigned)max_segments);
    LaunchScope scope(ctx, st, name);
    return cuda_status(launch_chained(small_ffn_kernel<MODE>, grid, dim3(kSmallWarps * 32),
                                      (size_t)small_smem_bytes(rows_max, p.Kdim), st, p, (int)per_cta));
}

}  // namespace

int ffn_small_init(director_ctx*) {
    if (cudaFuncSetAttribute(small_ffn_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmallMaxSmem) != cudaSuccess ||
        cudaFuncSetAttribute(small_ffn_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmallMaxSmem) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    return DIRECTOR_OK;
}

// True if a batch of T tokens can take the weight-streaming kernels: few enough tokens, and the rows of a segment
// fit in shared memory for both projections of an FFN of width Fw.
bool ffn_small_applies(const director_ctx* ctx, int T, int Fw) {
    return T <= kSmallFfnTokens && small_smem_bytes(T, std::max(ctx->shape.H, Fw)) <= (size_t)kSmallMaxSmem;
}

// in [rows, H] -> hidden [rows, Fw] -> out [rows, H] over a segment table whose segments hold at most kSmallFfnTokens
// rows (a batch of at most that many tokens).  max_segments: upper bound of the non-empty segments.
// gather_rows != nullptr: `in` is the un-permuted layer input and row i of the segment table is in[gather_rows[i]]
// (the rows are staged in shared memory once per CTA either way, so the dispatch step needs no row copies).
int ffn_pass_small(director_ctx* ctx, const void* in, const int32_t* gather_rows, const int32_t* seg_offsets, const int32_t* slot_expert, int G,
                   const void* w_gate, const void* w_up, const void* w_down, int Fw, void* hidden, void* out, int rows_max,
                   int max_segments, cudaStream_t st) {
    const int H = ctx->shape.H;
    const SmallParams p1{seg_offsets, slot_expert, G, static_cast<const uint16_t*>(in), gather_rows, static_cast<const uint16_t*>(w_gate),
                         static_cast<const uint16_t*>(w_up), Fw, H, static_cast<uint16_t*>(hidden), ctx->d_status};
    int rc = launch_small<0>(ctx, "small_ffn_swiglu_kernel", p1, rows_max, max_segments, st);
    if (rc != DIRECTOR_OK) return rc;
    const SmallParams p2{seg_offsets, slot_expert, G, static_cast<const uint16_t*>(hidden), nullptr, static_cast<const uint16_t*>(w_down),
                         nullptr, H, Fw, static_cast<uint16_t*>(out), ctx->d_status};
    return launch_small<1>(ctx, "small_ffn_down_kernel", p2, rows_max, max_segments, st);
}

}  // namespace director
