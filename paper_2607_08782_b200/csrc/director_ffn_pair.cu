// CTA-pair variant of the grouped expert-FFN GEMMs (Section II-A expert FFNs): two CTAs of a cluster,
// one per SM of a pair, compute a 256 x 256 tile with tcgen05.mma cta_group::2.
//
// Why: a 128x256 tile per SM needs 48 KB of operands per k-step (A 16 KB + B 32 KB); with the tensor
// pipe consuming a k-step in 512 cycles that is 96 B/clk of L2 -> shared-memory traffic per SM, more
// than an SM can draw.  In a pair each CTA loads its own 128 rows of A but only half of B (128 of the
// 256 rows): 32 KB per k-step per SM.  The instruction reads both halves of B and both A tiles from
// the two CTAs' shared memory; each CTA's tensor memory receives its own 128 x 256 accumulator.
//
//   CTA 0 (leader): loads A(m-block 2p) and B rows [0,128)   (gate tile / first half of the down tile)
//   CTA 1         : loads A(m-block 2p+1) and B rows [128,256) (up tile / second half)
// The leader's MMA thread issues every instruction and commits to mbarriers in both CTAs (the commit's
// own cluster multicast; no TMA load uses multicast).  Each CTA's producer announces its bytes on the
// LEADER's "full" barrier (remote arrive.expect_tx) and points its TMA loads (cta_group::2 form) at it.
// Each CTA's epilogue drains its own accumulator and releases it on the leader's barrier.
// An odd last m-block of a segment leaves CTA 1 computing rows it never stores.
//
// Every wait is bounded (see mbar_wait); a CTA that gives up raises DIRECTOR_ERR_TIMEOUT, its roles
// drain, and both CTAs meet at the closing cluster barrier before freeing tensor memory.
#include "director_common.cuh"
#include "director_umma.cuh"

namespace director {

using namespace umma;

namespace {

constexpr int P_STAGES = 6;
constexpr int P_STAGE_BYTES = A_BYTES + B_HALF_BYTES;          // 32 KB per CTA per k-step
constexpr int P_SMEM_BYTES = P_STAGES * P_STAGE_BYTES + 1024 + 256 + TABLE_INTS * 4;

// kind::f16 instruction descriptor for the pair: M = 256 (128 rows per CTA), N = 256.
constexpr uint32_t P_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);

__device__ __forceinline__ void umma_pair_bf16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(P_IDESC), "r"(accumulate) : "memory");
}
struct PairWalker {
    const int32_t* seg_off;
    const int32_t* mp_start;     // prefix of m-block PAIRS per segment
    const int32_t* expert;
    int n_blocks, b_rows_per_expert, total, g = 0;
    // tile of CTA `rank` for cluster work item w
    __device__ bool get(int w, Tile& t, int n_out_rows, int rank) {
        if (w >= total) return false;
        while (w >= mp_start[g + 1] * n_blocks) ++g;
        const int mp = mp_start[g + 1] - mp_start[g];
        const int local = w - mp_start[g] * n_blocks;
        t.nb = local / mp;
        const int pair = local - t.nb * mp;
        t.row0 = seg_off[g] + (2 * pair + rank) * BLOCK_M;      // may lie past the segment end (odd tail)
        t.row_end = seg_off[g + 1];
        t.b_row = expert[g] * b_rows_per_expert + t.nb * n_out_rows;
        return true;
    }
};

template <int MODE>
__global__ void __launch_bounds__(FFN_THREADS, 1)
grouped_gemm_pair_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b0,
                         const __grid_constant__ CUtensorMap tm_b1, const GroupedGemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    uint8_t* gen = smem_raw + (tiles - raw) + P_STAGES * P_STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(gen);             // full[6] empty[6] tfull[2] tempty[2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + 160);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + 164);
    int32_t* warp_sum = reinterpret_cast<int32_t*>(gen + 192);     // [6]
    int32_t* s_seg = reinterpret_cast<int32_t*>(gen + 256);
    int32_t* s_mp = s_seg + (kMaxG + 1);
    int32_t* s_exp = s_mp + (kMaxG + 1);

    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (P_STAGES + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * P_STAGES + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * P_STAGES + 2 + a); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = p.G;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;

    for (int g = threadIdx.x; g <= G; g += FFN_THREADS) s_seg[g] = __ldg(p.seg_offsets + g);
    for (int g = threadIdx.x; g < G; g += FFN_THREADS) s_exp[g] = __ldg(p.slot_expert + g);
    if (threadIdx.x == 0) {
        *abort_flag = 0;
        for (int s = 0; s < P_STAGES; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    {
        auto pairs_of = [&](int g) {
            const int len = s_seg[g + 1] - s_seg[g];
            return (s_exp[g] >= 0 && len > 0) ? (len + 2 * BLOCK_M - 1) / (2 * BLOCK_M) : 0;
        };
        const int per = (G + FFN_THREADS - 1) / FFN_THREADS;
        const int lo = min((int)threadIdx.x * per, G), hi = min(lo + per, G);
        int local = 0;
        for (int g = lo; g < hi; ++g) local += pairs_of(g);
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
        for (int g = lo; g < hi; ++g) { s_mp[g] = base; base += pairs_of(g); }
        if (threadIdx.x == FFN_THREADS - 1) s_mp[G] = base;
    }
    if (warp == 1) {   // the same warp in both CTAs allocates the pair's tensor memory
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();            // both CTAs' barriers are initialised before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    constexpr int N_OUT = (MODE == 0) ? 128 : 256;
    PairWalker walker{s_seg, s_mp, s_exp, p.n_blocks, p.b_rows_per_expert, s_mp[G] * p.n_blocks};
    Tile t;

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            const CUtensorMap* b_map = (MODE == 0 && rank == 1) ? &tm_b1 : &tm_b0;
            const int b_off = (MODE == 1 && rank == 1) ? 128 : 0;
            for (int w = cluster_id; ok && walker.get(w, t, N_OUT, (int)rank); w += n_clusters) {
                for (int kb = 0; kb < p.k_steps; ++kb) {
                    if (!(ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag))) break;
                    const uint32_t leader_full = map_to_cta(full_bar(stage), 0);
                    const uint32_t a_dst = tiles + stage * P_STAGE_BYTES;
                    mbar_expect_tx_cluster(leader_full, P_STAGE_BYTES);
                    tma_load_2d_pair(a_dst, &tm_a, leader_full, kb * BLOCK_K, t.row0);
                    tma_load_2d_pair(a_dst + A_BYTES, b_map, leader_full, kb * BLOCK_K, t.b_row + b_off);
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && leader) {
            int stage = 0, it = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int w = cluster_id; ok && walker.get(w, t, N_OUT, 0); w += n_clusters, ++it) {
                const int acc = it & 1;
                if (!(ok = mbar_wait(tempty_bar(acc), (((uint32_t)it >> 1) & 1u) ^ 1u, abort_flag))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * UMMA_N);
                for (int kb = 0; kb < p.k_steps; ++kb) {
                    if (!(ok = mbar_wait(full_bar(stage), phase, abort_flag))) break;
                    tc_fence_after();
                    const uint32_t a_src = tiles + stage * P_STAGE_BYTES;
                    const uint64_t a_desc = smem_desc(a_src), b_desc = smem_desc(a_src + A_BYTES);
#pragma unroll
                    for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                        umma_pair_bf16(d_tmem, a_desc + 2u * k, b_desc + 2u * k, (kb | k) != 0 ? 1u : 0u);
                    umma_commit_both(empty_bar(stage));
                    if (++stage == P_STAGES) { stage = 0; phase ^= 1u; }
                }
                if (ok) umma_commit_both(tfull_bar(acc));
            }
        }
    } else {
        const int quad = warp & 3;
        uint16_t* out = static_cast<uint16_t*>(p.out);
        int it = 0;
        bool ok = true;
        for (int w = cluster_id; ok && walker.get(w, t, N_OUT, (int)rank); w += n_clusters, ++it) {
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
                        o[i] = pack_bf16(__fdividef(g0 * u0, 1.0f + __expf(-g0)), __fdividef(g1 * u1, 1.0f + __expf(-g1)));
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
            if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));   // release on the leader's barrier
        }
    }

    // ---- teardown: nobody leaves while the peer may still signal into this CTA ----
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (threadIdx.x == 0 && *abort_flag) director_set_status(p.status, DIRECTOR_ERR_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

template <int MODE>
int launch_pair(director_ctx* ctx, const char* name, const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1,
                const GroupedGemmParams& p, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * ctx->pair_clusters));
    cfg.blockDim = dim3(FFN_THREADS);
    cfg.dynamicSmemBytes = P_SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    LaunchScope scope(ctx, st, name);
    return cuda_status(cudaLaunchKernelEx(&cfg, grouped_gemm_pair_kernel<MODE>, a, b0, b1, p));
}

}  // namespace

int ffn_pair_init(director_ctx* ctx) {
    if (cudaFuncSetAttribute(grouped_gemm_pair_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(grouped_gemm_pair_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, P_SMEM_BYTES) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    // how many CTA pairs the device can hold at once: the persistent grid must not exceed it, or the
    // surplus clusters would only start when the first ones are done
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(ctx->sm_count & ~1));
    cfg.blockDim = dim3(FFN_THREADS);
    cfg.dynamicSmemBytes = P_SMEM_BYTES;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, grouped_gemm_pair_kernel<0>, &cfg) != cudaSuccess || n < 1) {
        cudaGetLastError();
        n = ctx->sm_count / 2;
    }
    ctx->pair_clusters = n < ctx->sm_count / 2 ? n : ctx->sm_count / 2;
    return DIRECTOR_OK;
}

int launch_gemm_pair(director_ctx* ctx, int mode, const char* name, const CUtensorMap& a, const CUtensorMap& b0,
                     const CUtensorMap& b1, const umma::GroupedGemmParams& p, cudaStream_t st) {
    return mode == 0 ? launch_pair<0>(ctx, name, a, b0, b1, p, st) : launch_pair<1>(ctx, name, a, b0, b1, p, st);
}

}  // namespace director
