// (a3) Grouped SwiGLU expert FFN on the 5th-generation tensor cores (Section II-A: every expert is
// an FFN sub-network; after dispatch each segment of rows runs its expert).
//
// Two grouped GEMMs over the ragged segments written by dispatch, both "TN" (A rows and B rows are
// K-contiguous), bf16 operands, fp32 accumulation in tensor memory:
//   GEMM-1  Hg[rows, F] = silu(Xp . Wgate[e]^T) * (Xp . Wup[e]^T)    (one 128x256 accumulator holds
//           128 gate columns next to the matching 128 up columns; SwiGLU is the epilogue)
//   GEMM-2  Yp[rows, H] = Hg . Wdown[e]^T                             (128x256 output tile)
//
// One persistent CTA per SM, warp-specialised:
//   warp 0     TMA producer: cp.async.bulk.tensor 2-D loads of a 128x64 A box and two 128x64 B boxes
//              per k-step into a 4-stage shared-memory ring (128-byte swizzle), mbarrier expect-tx.
//   warp 1     allocates the 512 TMEM columns; one lane issues tcgen05.mma (M128 N256 K16, 4 per
//              k-step) and tcgen05.commit to release ring stages / publish the accumulator.
//   warps 2-5  epilogue: tcgen05.ld the accumulator (one TMEM lane quadrant per warp, one row per
//              thread), SwiGLU or plain convert, predicated 16-byte stores (rows past the segment end
//              are computed but not stored).  Two accumulators (2 x 256 columns) let the epilogue of
//              tile i overlap the MMAs of tile i+1.
// Work items are (segment, n-block, m-block) in that nesting order, so CTAs running at the same time
// share the weight tile of one n-block through L2.  Segment sizes stay on the device: every CTA builds
// the tile prefix from seg_offsets in its prologue.  Every mbarrier wait is bounded; on expiry the CTA
// raises DIRECTOR_ERR_TIMEOUT, all roles drain and the CTA frees its TMEM and returns.
#include "director_common.cuh"
#include "director_umma.cuh"

#include <cuda_bf16.h>

#include <algorithm>

namespace director {

int ffn_swap_init(director_ctx* ctx);   // director_ffn_swap.cu
int ffn_pass_swap(director_ctx* ctx, const void* in, uint64_t in_rows, const int32_t* gather_rows, uint64_t rows,
                  const int32_t* seg_offsets, const int32_t* slot_expert, int G, const void* w_gate, const void* w_up,
                  const void* w_down, uint64_t n_experts, int Fw, void* hidden, void* out, unsigned int* counters,
                  const DenseFfn* dense, uint64_t max_seg_rows, const FusedCombine* fc, cudaStream_t st);
int ffn_small_init(director_ctx* ctx);  // director_ffn_small.cu
bool ffn_small_applies(const director_ctx* ctx, int T, int Fw);
int ffn_pass_small(director_ctx* ctx, const void* in, const int32_t* gather_rows, const int32_t* seg_offsets, const int32_t* slot_expert, int G,
                   const void* w_gate, const void* w_up, const void* w_down, int Fw, void* hidden, void* out, int rows_max,
                   int max_segments, cudaStream_t st);
int ffn_pair_init(director_ctx* ctx);   // director_ffn_pair.cu
int launch_gemm_pair(director_ctx* ctx, int mode, const char* name, const CUtensorMap& a, const CUtensorMap& b0,
                     const CUtensorMap& b1, const umma::GroupedGemmParams& p, cudaStream_t st);

namespace {

using namespace umma;

// Walks the work list for one role; `g` is the role's private segment cursor.
struct TileWalker {
    const int32_t* seg_off;
    const int32_t* mt_start;
    const int32_t* expert;
    int n_blocks, b_rows_per_expert, total, g = 0;
    __device__ bool get(int w, Tile& t, int n_out_rows) {
        if (w >= total) return false;
        while (w >= mt_start[g + 1] * n_blocks) ++g;
        const int mt = mt_start[g + 1] - mt_start[g];
        const int local = w - mt_start[g] * n_blocks;
        t.nb = local / mt;
        const int mb = local - t.nb * mt;
        t.row0 = seg_off[g] + mb * BLOCK_M;
        t.row_end = seg_off[g + 1];
        t.b_row = expert[g] * b_rows_per_expert + t.nb * n_out_rows;
        return true;
    }
};

// MODE 0: B = (gate rows, up rows) from two tensor maps, epilogue = SwiGLU, 128 output columns per tile.
// MODE 1: B = 256 consecutive rows of one tensor map, epilogue = convert, 256 output columns per tile.
template <int MODE>
__global__ void __launch_bounds__(FFN_THREADS, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b0,
                    const __grid_constant__ CUtensorMap tm_b1, const GroupedGemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;                 // 1024-byte aligned operand ring
    uint8_t* gen = smem_raw + (tiles - raw) + STAGES * STAGE_BYTES;  // generic pointer past the ring
    uint64_t* bars = reinterpret_cast<uint64_t*>(gen);             // full[4] empty[4] tfull[2] tempty[2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + 128);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + 132);
    int32_t* warp_sum = reinterpret_cast<int32_t*>(gen + 160);     // [6]
    int32_t* s_seg = reinterpret_cast<int32_t*>(gen + 256);        // [G+1]
    int32_t* s_mt = s_seg + (kMaxG + 1);                           // [G+1] tile prefix
    int32_t* s_exp = s_mt + (kMaxG + 1);                           // [G]

    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.G;

    // ---- prologue: tables, tile prefix, barriers, TMEM ----
    for (int g = threadIdx.x; g <= G; g += FFN_THREADS) s_seg[g] = __ldg(p.seg_offsets + g);
    for (int g = threadIdx.x; g < G; g += FFN_THREADS) s_exp[g] = __ldg(p.slot_expert + g);
    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    {
        const int per = (G + FFN_THREADS - 1) / FFN_THREADS;
        const int lo = min((int)threadIdx.x * per, G), hi = min(lo + per, G);
        int local = 0;
        for (int g = lo; g < hi; ++g) {
            const int len = s_seg[g + 1] - s_seg[g];
            local += (s_exp[g] >= 0 && len > 0) ? (len + BLOCK_M - 1) / BLOCK_M : 0;
        }
        int incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) warp_sum[warp] = incl;
        __syncthreads();
        int base = incl - local;
        for (int i = 0; i < warp; ++i) base += warp_sum[i];
        for (int g = lo; g < hi; ++g) {
            const int len = s_seg[g + 1] - s_seg[g];
            s_mt[g] = base;
            base += (s_exp[g] >= 0 && len > 0) ? (len + BLOCK_M - 1) / BLOCK_M : 0;
        }
        if (threadIdx.x == FFN_THREADS - 1) s_mt[G] = base;
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    constexpr int N_OUT = (MODE == 0) ? 128 : 256;   // output columns (= B rows per map load pair) per tile
    TileWalker walker{s_seg, s_mt, s_exp, p.n_blocks, p.b_rows_per_expert, s_mt[G] * p.n_blocks};
    Tile t;

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int w = blockIdx.x; ok && walker.get(w, t, N_OUT); w += gridDim.x) {
                for (int kb = 0; kb < p.k_steps; ++kb) {
                    if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag))) break;
                    const uint32_t a_dst = tiles + stage * STAGE_BYTES;
                    mbar_expect_tx(full_bar(stage), STAGE_BYTES);
                    tma_load_2d(a_dst, &tm_a, full_bar(stage), kb * BLOCK_K, t.row0);
                    tma_load_2d(a_dst + A_BYTES, &tm_b0, full_bar(stage), kb * BLOCK_K, t.b_row);
                    if (MODE == 0)
                        tma_load_2d(a_dst + A_BYTES + B_HALF_BYTES, &tm_b1, full_bar(stage), kb * BLOCK_K, t.b_row);
                    else
                        tma_load_2d(a_dst + A_BYTES + B_HALF_BYTES, &tm_b0, full_bar(stage), kb * BLOCK_K, t.b_row + 128);
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            int stage = 0, it = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int w = blockIdx.x; ok && walker.get(w, t, N_OUT); w += gridDim.x, ++it) {
                const int acc = it & 1;
                if (!(ok = mbar_wait(tempty_bar(acc), (((uint32_t)it >> 1) & 1u) ^ 1u, abort_flag))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * UMMA_N);
                for (int kb = 0; kb < p.k_steps; ++kb) {
                    if (!(ok = mbar_wait(full_bar(stage), phase, abort_flag))) break;
                    tc_fence_after();
                    const uint32_t a_src = tiles + stage * STAGE_BYTES;
                    const uint64_t a_desc = smem_desc(a_src), b_desc = smem_desc(a_src + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BLOCK_K / UMMA_K; ++k)   // advance 32 bytes (2 x 16-byte units) per UMMA_K
                        umma_bf16(d_tmem, a_desc + 2u * k, b_desc + 2u * k, (kb | k) != 0 ? 1u : 0u);
                    umma_commit(empty_bar(stage));               // stage reusable once these MMAs retire
                    if (++stage == STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit(tfull_bar(acc));             // accumulator complete
            }
        }
    } else {
        const int quad = warp & 3;                               // TMEM lane quadrant this warp may read
        uint16_t* out = static_cast<uint16_t*>(p.out);
        int it = 0;
        bool ok = true;
        for (int w = blockIdx.x; ok && walker.get(w, t, N_OUT); w += gridDim.x, ++it) {
            const int acc = it & 1;
            if (!(ok = mbar_wait(tfull_bar(acc), ((uint32_t)it >> 1) & 1u, abort_flag))) break;
            tc_fence_after();
            const int row = t.row0 + quad * 32 + lane;
            const bool live = row < t.row_end;
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * UMMA_N);
            uint16_t* orow = out + (size_t)row * p.out_pitch + (size_t)t.nb * N_OUT;
            if constexpr (MODE == 0) {
#pragma unroll 1
                for (int c = 0; c < 128; c += 32) {
                    uint32_t g[32], u[32];
                    tmem_ld32(taddr + c, g);
                    tmem_ld32(taddr + 128 + c, u);
                    tmem_ld_wait();
                    uint32_t o[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float g0 = __uint_as_float(g[2 * i]), g1 = __uint_as_float(g[2 * i + 1]);
                        const float u0 = __uint_as_float(u[2 * i]), u1 = __uint_as_float(u[2 * i + 1]);
                        const float h0 = __fdividef(g0 * u0, 1.0f + __expf(-g0));
                        const float h1 = __fdividef(g1 * u1, 1.0f + __expf(-g1));
                        o[i] = pack_bf16(h0, h1);
                    }
                    if (live) {
                        uint4* dst = reinterpret_cast<uint4*>(orow + c);
#pragma unroll
                        for (int i = 0; i < 4; ++i) dst[i] = make_uint4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
                    }
                }
            } else {
#pragma unroll 1
                for (int c = 0; c < 256; c += 32) {
                    uint32_t v[32];
                    tmem_ld32(taddr + c, v);
                    tmem_ld_wait();
                    if (live) {
                        uint4* dst = reinterpret_cast<uint4*>(orow + c);
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            dst[i] = make_uint4(pack_bf16(__uint_as_float(v[8 * i]), __uint_as_float(v[8 * i + 1])),
                                                pack_bf16(__uint_as_float(v[8 * i + 2]), __uint_as_float(v[8 * i + 3])),
                                                pack_bf16(__uint_as_float(v[8 * i + 4]), __uint_as_float(v[8 * i + 5])),
                                                pack_bf16(__uint_as_float(v[8 * i + 6]), __uint_as_float(v[8 * i + 7])));
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty_bar(acc));
        }
    }

    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag) director_set_status(p.status, DIRECTOR_ERR_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 matrix [rows, cols] row-major; box = 64 columns (128 bytes) x 128 rows, 128-byte swizzle;
// out-of-range rows are filled with zeros.
bool make_map(director_ctx* ctx, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols) {
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {BLOCK_K, 128};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
        map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

template <int MODE>
int launch_gemm(director_ctx* ctx, const char* name, const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1,
                const GroupedGemmParams& p, cudaStream_t st) {
    if (ctx->ffn_variant >= 1) return launch_gemm_pair(ctx, MODE, name, a, b0, b1, p, st);
    LaunchScope scope(ctx, st, name);
    grouped_gemm_kernel<MODE><<<ctx->sm_count, FFN_THREADS, SMEM_BYTES, st>>>(a, b0, b1, p);
    return cuda_status(cudaGetLastError());
}

// One SwiGLU FFN pass over a segment table: in [rows, H] -> hidden [rows, Fw] -> out [rows, H].
// max_seg_rows: an upper bound on any segment's length (a token goes to an expert at most once, so the batch size).
int ffn_pass(director_ctx* ctx, const void* in, uint64_t in_rows, const int32_t* gather_rows, uint64_t rows,
             const int32_t* seg_offsets, const int32_t* slot_expert, int G, const void* w_gate, const void* w_up,
             const void* w_down, uint64_t n_experts, int Fw, void* hidden, void* out, unsigned int* counters,
             uint64_t max_seg_rows, cudaStream_t st) {
    if (ctx->ffn_variant == 2) {
        const int rc = ffn_pass_swap(ctx, in, in_rows, gather_rows, rows, seg_offsets, slot_expert, G, w_gate, w_up, w_down,
                                     n_experts, Fw, hidden, out, counters, nullptr, max_seg_rows, nullptr, st);
        if (rc != DIRECTOR_ERR_UNSUPPORTED) return rc;   // weight arrays not expressible as one map: tile scheme 0
    }
    if (gather_rows != nullptr) return DIRECTOR_ERR_UNSUPPORTED;   // only the weight-stationary scheme gathers
    const int H = ctx->shape.H;
    CUtensorMap m_in, m_g, m_u, m_h, m_d;
    if (!make_map(ctx, &m_in, in, rows, H) || !make_map(ctx, &m_g, w_gate, n_experts * Fw, H) ||
        !make_map(ctx, &m_u, w_up, n_experts * Fw, H) || !make_map(ctx, &m_h, hidden, rows, Fw) ||
        !make_map(ctx, &m_d, w_down, n_experts * H, Fw))
        return DIRECTOR_ERR_CUDA;
    GroupedGemmParams p1{seg_offsets, slot_expert, G, Fw / 128, H / BLOCK_K, Fw, Fw, hidden, ctx->d_status};
    int rc = launch_gemm<0>(ctx, "grouped_gemm_swiglu_kernel", m_in, m_g, m_u, p1, st);
    if (rc != DIRECTOR_OK) return rc;
    GroupedGemmParams p2{seg_offsets, slot_expert, G, H / 256, Fw / BLOCK_K, H, H, out, ctx->d_status};
    return launch_gemm<1>(ctx, "grouped_gemm_down_kernel", m_h, m_d, m_d, p2, st);
}

__global__ void one_segment_kernel(int32_t* seg, int T) {
    seg[0] = 0;
    seg[1] = T;
}

}  // namespace

int ffn_init(director_ctx* ctx) {
    if (ffn_pair_init(ctx) != DIRECTOR_OK || ffn_swap_init(ctx) != DIRECTOR_OK || ffn_small_init(ctx) != DIRECTOR_OK)
        return DIRECTOR_ERR_CUDA;
    if (cudaFuncSetAttribute(grouped_gemm_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(grouped_gemm_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    return DIRECTOR_OK;
}

// True if a batch of T tokens takes the weight-streaming FFN kernels (tile scheme 2 only): the one-call entry points
// then skip the row copies of the dispatch step, since those kernels stage their rows from x themselves.
bool ffn_streams_weights(const director_ctx* ctx, int T) {
    const director_shape& s = ctx->shape;
    return ctx->ffn_variant == 2 && ctx->ffn_small && ffn_small_applies(ctx, T, s.F) &&
           (s.S == 0 || ffn_small_applies(ctx, T, s.S * s.F));
}

// row_token == nullptr: the routed experts read the permuted rows xp.  Otherwise they gather row i as
// x[row_token[i]] and xp is not used.
int launch_expert_ffn(director_ctx* ctx, int T, const void* xp, const int32_t* row_token, const int32_t* seg_offsets,
                      const void* w_gate, const void* w_up, const void* w_down, void* yp, const void* x,
                      const void* ws_gate, const void* ws_up, const void* ws_down, void* y_shared, cudaStream_t st) {
    StageScope stage(ctx, st, "stage_expert_ffn");
    const director_shape& s = ctx->shape;
    const uint64_t A = (uint64_t)T * s.K;
    const bool shared = s.S > 0 && x != nullptr && y_shared != nullptr;
    if (ffn_streams_weights(ctx, T)) {
        // decode-sized batch: every segment has at most T rows; stream the touched weights once, feature by feature
        // (with row_token the rows are staged straight from x: x must then be given even without shared experts)
        if (row_token != nullptr && x == nullptr) return DIRECTOR_ERR_INVALID_ARG;
        int rc = ffn_pass_small(ctx, row_token ? x : xp, row_token, seg_offsets, ctx->d_slot_expert, ctx->G, w_gate, w_up, w_down,
                                s.F, ctx->d_hidden, yp, T, (int)std::min<uint64_t>((uint64_t)ctx->G, A), st);
        if (rc != DIRECTOR_OK || !shared) return rc;
        {
            LaunchScope scope(ctx, st, "one_segment_kernel");
            one_segment_kernel<<<1, 1, 0, st>>>(ctx->d_one_seg, T);
            if ((rc = cuda_status(cudaGetLastError())) != DIRECTOR_OK) return rc;
        }
        return ffn_pass_small(ctx, x, nullptr, ctx->d_one_seg, ctx->d_zero_expert, 1, ws_gate, ws_up, ws_down, s.S * s.F,
                              ctx->d_hidden_shared, y_shared, T, 1, st);
    }
    // work-item counters of the (up to four) GEMM launches below
    if (cudaMemsetAsync(ctx->d_sched, 0, 4 * sizeof(unsigned int), st) != cudaSuccess) return DIRECTOR_ERR_CUDA;
    if (shared && row_token == nullptr && ctx->ffn_variant == 2) {
        // routed and shared experts in the same two launches: the shared experts' work items follow the routed ones
        const DenseFfn dense{x, (uint64_t)T, ws_gate, ws_up, ws_down, s.S * s.F, ctx->d_hidden_shared, y_shared};
        const int rc = ffn_pass_swap(ctx, xp, A, nullptr, A, seg_offsets, ctx->d_slot_expert, ctx->G, w_gate, w_up, w_down,
                                     s.E, s.F, ctx->d_hidden, yp, ctx->d_sched, &dense, (uint64_t)T, nullptr, st);
        if (rc != DIRECTOR_ERR_UNSUPPORTED) return rc;    // a weight pair not expressible as one map: separate passes
    }
    int rc = row_token ? ffn_pass(ctx, x, (uint64_t)T, row_token, A, seg_offsets, ctx->d_slot_expert, ctx->G, w_gate, w_up,
                                  w_down, s.E, s.F, ctx->d_hidden, yp, ctx->d_sched, (uint64_t)T, st)
                       : ffn_pass(ctx, xp, A, nullptr, A, seg_offsets, ctx->d_slot_expert, ctx->G, w_gate, w_up, w_down,
                                  s.E, s.F, ctx->d_hidden, yp, ctx->d_sched, (uint64_t)T, st);
    if (rc != DIRECTOR_OK || !shared) return rc;
    {
        LaunchScope scope(ctx, st, "one_segment_kernel");
        one_segment_kernel<<<1, 1, 0, st>>>(ctx->d_one_seg, T);
        if ((rc = cuda_status(cudaGetLastError())) != DIRECTOR_OK) return rc;
    }
    // The S shared experts as one FFN of width S*F over all T rows of x (a single segment, "expert" 0).
    return ffn_pass(ctx, x, (uint64_t)T, nullptr, (uint64_t)T, ctx->d_one_seg, ctx->d_zero_expert, 1, ws_gate, ws_up,
                    ws_down, 1, s.S * s.F, ctx->d_hidden_shared, y_shared, ctx->d_sched + 2, (uint64_t)T, st);
}

namespace {

// Zeroes the fp32 accumulator of y and writes every permuted row's gating weight (row_weight[inv_row[t,s]] = w[t,s]).
__global__ void __launch_bounds__(256)
combine_prepare_kernel(float4* __restrict__ y_acc, long long n_vec, const int32_t* __restrict__ inv_row,
                       const float* __restrict__ topk_w, float* __restrict__ row_weight, long long A) {
    chain_prologue();
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x, stride = (long long)gridDim.x * blockDim.x;
    for (long long i = i0; i < n_vec; i += stride) y_acc[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    for (long long i = i0; i < A; i += stride) {
        const int row = __ldg(inv_row + i);
        if (row >= 0) row_weight[row] = __ldg(topk_w + i);
    }
}

// y = bf16(y_acc + y_shared): the one rounding of the combining form.
__global__ void __launch_bounds__(256)
combine_finish_kernel(const float4* __restrict__ y_acc, const uint2* __restrict__ y_shared, uint2* __restrict__ y,
                      long long n_vec) {
    chain_prologue();
    const long long i0 = (long long)blockIdx.x * blockDim.x + threadIdx.x, stride = (long long)gridDim.x * blockDim.x;
    for (long long i = i0; i < n_vec; i += stride) {
        float4 a = __ldcs(y_acc + i);
        if (y_shared != nullptr) {
            const uint2 sh = __ldg(y_shared + i);
            a.x += __uint_as_float(sh.x << 16);
            a.y += __uint_as_float(sh.x & 0xFFFF0000u);
            a.z += __uint_as_float(sh.y << 16);
            a.w += __uint_as_float(sh.y & 0xFFFF0000u);
        }
        uint2 o;
        o.x = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(a.x)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(a.y)) << 16);
        o.y = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(a.z)) | ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(a.w)) << 16);
        y[i] = o;
    }
}

}  // namespace

// (a3) and (a4) in one: both projections on the tensor-core kernels, the down projection combining in its epilogue.
// y_acc: fp32 [T, H] scratch, row_weight: fp32 [T*K] scratch (both caller-owned).  Tile scheme 2 only.
int launch_expert_ffn_combine(director_ctx* ctx, int T, const void* xp, const int32_t* seg_offsets, const int32_t* row_token,
                              const int32_t* inv_row, const float* topk_w, const void* w_gate, const void* w_up,
                              const void* w_down, const void* x, const void* ws_gate, const void* ws_up,
                              const void* ws_down, float* y_acc, float* row_weight, void* y, cudaStream_t st) {
    if (ctx->ffn_variant != 2) return DIRECTOR_ERR_UNSUPPORTED;
    const director_shape& s = ctx->shape;
    const uint64_t A = (uint64_t)T * s.K;
    const bool shared = s.S > 0 && x != nullptr;
    const long long n_vec = (long long)T * s.H / 4;
    const unsigned grid = (unsigned)std::min<long long>((n_vec + 255) / 256, 8LL * ctx->sm_count);
    {
        StageScope stage(ctx, st, "stage_expert_ffn");
        {
            LaunchScope scope(ctx, st, "fused_combine_prepare_kernel");
            int rc = cuda_status(launch_chained(combine_prepare_kernel, dim3(grid), dim3(256), 0, st,
                                                reinterpret_cast<float4*>(y_acc), n_vec, inv_row, topk_w, row_weight, (long long)A));
            if (rc != DIRECTOR_OK) return rc;
        }
        if (cudaMemsetAsync(ctx->d_sched, 0, 4 * sizeof(unsigned int), st) != cudaSuccess) return DIRECTOR_ERR_CUDA;
        const FusedCombine fc{row_token, row_weight, y_acc};
        const DenseFfn dense{x, (uint64_t)T, ws_gate, ws_up, ws_down, s.S * s.F, ctx->d_hidden_shared, ctx->e_y_shared};
        const int rc = ffn_pass_swap(ctx, xp, A, nullptr, A, seg_offsets, ctx->d_slot_expert, ctx->G, w_gate, w_up, w_down,
                                     s.E, s.F, ctx->d_hidden, nullptr, ctx->d_sched, shared ? &dense : nullptr, (uint64_t)T,
                                     &fc, st);
        if (rc != DIRECTOR_OK) return rc;
    }
    StageScope stage(ctx, st, "stage_combine");
    LaunchScope scope(ctx, st, "fused_combine_finish_kernel");
    return cuda_status(launch_chained(combine_finish_kernel, dim3(grid), dim3(256), 0, st,
                                      reinterpret_cast<const float4*>(y_acc),
                                      shared ? static_cast<const uint2*>(ctx->e_y_shared) : static_cast<const uint2*>(nullptr),
                                      static_cast<uint2*>(y), n_vec));
}

}  // namespace director
