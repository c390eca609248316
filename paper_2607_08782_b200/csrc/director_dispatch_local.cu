// (a2)/(a5) under the locality-first replica rule, and the de-duplicated dispatch volume.
//
// The paper replicates hot experts to cut the dispatch volume of Eq. 3 (Section III) but leaves open which
// replica a token uses.  Besides the default round-robin rule this library offers "locality first": token t on
// rank src(t) uses the replica of expert e on its own rank when there is one; otherwise the assignment
// "travels": it is the m-th travelling assignment of e in ascending token id and goes to replica m mod r_e.
// A segment (rank, expert) holds its assignments in ascending token id.
//
// Unlike round-robin, an assignment's place inside its segment no longer follows from its rank among the
// expert's assignments, so the counting sort takes two scans:
//   travel_count_scan_kernel  per 256-token tile and expert: number of travelling assignments; the last CTA
//                             turns the counts into exclusive per-tile prefixes (-> m).
//   slot_count_scan_kernel    every assignment's replica (written to dest_rank and, as a replica index, to
//                             inv_row); per tile and replica: number of assignments; the last CTA scans them
//                             over the tiles and the slot lengths into seg_offsets.
//   local_index_kernel        row = seg_offsets[slot] + tile prefix + stable rank inside the tile.
// All counts come from lane bitmasks and popcounts: integer only, order independent, deterministic.
#include "director_common.cuh"
#include "director_sort.cuh"

namespace director {

using namespace sort;

namespace {

constexpr int kW = kTileWarps;   // warps per tile

__device__ __forceinline__ int home_rank(const int32_t* __restrict__ src_rank, int t, int T, int R, int32_t* status) {
    int src = src_rank ? __ldg(src_rank + t) : (int)(((long long)t * R) / T);
    if ((unsigned)src >= (unsigned)R) {
        director_set_status(status, DIRECTOR_ERR_BAD_INDEX);
        src = -1;                         // such a token has no home: all its assignments travel
    }
    return src;
}

__device__ __forceinline__ bool hosted_at(const unsigned long long* __restrict__ host_mask, int e, int src) {
    return src >= 0 && ((__ldg(host_mask + e) >> src) & 1ull);
}

// travel[e][w]: bit l set iff token (tile*256 + w*32 + l) chose expert e and its home rank does not host e.
__device__ __forceinline__ void build_travel_masks(uint32_t (*travel)[kW], const int32_t* __restrict__ topk_idx,
                                                   const int32_t* __restrict__ src_rank,
                                                   const unsigned long long* __restrict__ host_mask, int tile, int T,
                                                   int E, int K, int R, int32_t* status) {
    for (int i = threadIdx.x; i < E * kW; i += blockDim.x) (&travel[0][0])[i] = 0u;
    __syncthreads();
    const int t = tile * kTokenTile + threadIdx.x;
    if (t < T) {
        const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
        const int src = home_rank(src_rank, t, T, R, status);
        for (int s = 0; s < K; ++s) {
            const int e = __ldg(topk_idx + (size_t)t * K + s);
            if ((unsigned)e >= (unsigned)E) { director_set_status(status, DIRECTOR_ERR_BAD_INDEX); continue; }
            if (!hosted_at(host_mask, e, src)) atomicOr(&travel[e][w], 1u << lane);
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kTokenTile)
travel_count_scan_kernel(const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ src_rank,
                         const unsigned long long* __restrict__ host_mask, int T, int E, int K, int R, int n_tiles,
                         int32_t* __restrict__ tile_travel, unsigned int* __restrict__ ticket,
                         int32_t* __restrict__ status) {
    __shared__ uint32_t travel[kMaxE][kW];
    __shared__ bool is_last;
    const int tile = blockIdx.x;
    build_travel_masks(travel, topk_idx, src_rank, host_mask, tile, T, E, K, R, status);
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        int c = 0;
#pragma unroll
        for (int w = 0; w < kW; ++w) c += __popc(travel[e][w]);
        tile_travel[(size_t)tile * E + e] = c;
    }
    if (!last_cta_done(ticket, n_tiles, &is_last)) return;
    for (int e = threadIdx.x; e < E; e += blockDim.x) scan_column(tile_travel, n_tiles, E, e);
    if (threadIdx.x == 0) *ticket = 0u;
}

// Replica index (position in rep_slot) of the assignment (token in warp w / lane, expert e, home rank src).
__device__ __forceinline__ int replica_of(const uint32_t (*travel)[kW], const uint16_t (*travel_prefix)[kW],
                                          const unsigned long long* __restrict__ host_mask,
                                          const int32_t* __restrict__ rep_start,
                                          const int32_t* __restrict__ tile_travel, int tile, int E, int e, int src, int w,
                                          int lane) {
    const int r0 = __ldg(rep_start + e);
    if (src >= 0) {
        const unsigned long long hm = __ldg(host_mask + e);
        if ((hm >> src) & 1ull) return r0 + __popcll(hm & ((1ull << src) - 1ull));   // replicas are in ascending rank
    }
    const int r_e = __ldg(rep_start + e + 1) - r0;
    const int m = __ldg(tile_travel + (size_t)tile * E + e) + tile_rank(travel, travel_prefix, e, w, lane);
    return r0 + m % r_e;
}

// dynamic shared memory of slot_count_scan_kernel: travel[E][kW] u32 | rep[NR][kW] u32 | slot_len[G] i32 |
// travel_prefix[E][kW] u16
__host__ __device__ inline size_t slot_count_smem_bytes(int E, int NR, int G) {
    return (size_t)E * kW * 4 + (size_t)NR * kW * 4 + (size_t)G * 4 + (size_t)E * kW * 2;
}

__global__ void __launch_bounds__(kTokenTile)
slot_count_scan_kernel(const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ src_rank,
                       const unsigned long long* __restrict__ host_mask, int T, int E, int K, int R, int C_max, int G,
                       int NR, int n_tiles, const int32_t* __restrict__ rep_start, const int32_t* __restrict__ rep_slot,
                       const int32_t* __restrict__ tile_travel, int32_t* __restrict__ tile_rep,
                       int32_t* __restrict__ rep_index /* [T,K] */, int32_t* __restrict__ dest_rank,
                       int32_t* __restrict__ seg_offsets_a, int32_t* __restrict__ seg_offsets_b,
                       unsigned int* __restrict__ ticket, int32_t* __restrict__ status) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint32_t (*travel)[kW] = reinterpret_cast<uint32_t (*)[kW]>(smem_raw);
    uint32_t (*rep)[kW] = reinterpret_cast<uint32_t (*)[kW]>(smem_raw + (size_t)E * kW * 4);
    int32_t* slot_len = reinterpret_cast<int32_t*>(smem_raw + (size_t)(E + NR) * kW * 4);
    uint16_t (*travel_prefix)[kW] = reinterpret_cast<uint16_t (*)[kW]>(smem_raw + (size_t)(E + NR) * kW * 4 + (size_t)G * 4);
    __shared__ int32_t warp_sum[kW];
    __shared__ bool is_last;

    const int tile = blockIdx.x;
    for (int i = threadIdx.x; i < NR * kW; i += blockDim.x) (&rep[0][0])[i] = 0u;
    build_travel_masks(travel, topk_idx, src_rank, host_mask, tile, T, E, K, R, status);
    build_warp_prefix(travel, travel_prefix, E);
    const int t = tile * kTokenTile + threadIdx.x;
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (t < T) {
        const int src = home_rank(src_rank, t, T, R, status);
        for (int s = 0; s < K; ++s) {
            const int e = __ldg(topk_idx + (size_t)t * K + s);
            int ri = -1, dest = -1;
            if ((unsigned)e < (unsigned)E) {
                ri = replica_of(travel, travel_prefix, host_mask, rep_start, tile_travel, tile, E, e, src, w, lane);
                dest = __ldg(rep_slot + ri) / C_max;
                atomicOr(&rep[ri][w], 1u << lane);      // a token picks an expert once: one bit per (replica, token)
            }
            rep_index[(size_t)t * K + s] = ri;
            dest_rank[(size_t)t * K + s] = dest;
        }
    }
    __syncthreads();
    for (int ri = threadIdx.x; ri < NR; ri += blockDim.x) {
        int c = 0;
#pragma unroll
        for (int ww = 0; ww < kW; ++ww) c += __popc(rep[ri][ww]);
        tile_rep[(size_t)tile * NR + ri] = c;
    }
    if (!last_cta_done(ticket, n_tiles, &is_last)) return;

    // ---- last CTA: per-replica exclusive scan over tiles, slot lengths, slot scan ----
    for (int g = threadIdx.x; g < G; g += blockDim.x) slot_len[g] = 0;
    __syncthreads();
    for (int ri = threadIdx.x; ri < NR; ri += blockDim.x) slot_len[__ldg(rep_slot + ri)] = scan_column(tile_rep, n_tiles, NR, ri);
    __syncthreads();
    scan_slots(slot_len, G, warp_sum, seg_offsets_a, seg_offsets_b, ticket);
}

// dynamic shared memory of local_index_kernel: rep[NR][kW] u32 | rep_prefix[NR][kW] u16
__host__ __device__ inline size_t local_index_smem_bytes(int NR) { return (size_t)NR * kW * 6; }

__global__ void __launch_bounds__(kTokenTile)
local_index_kernel(int T, int K, int NR, const int32_t* __restrict__ rep_slot, const int32_t* __restrict__ tile_rep,
                   const int32_t* __restrict__ seg_offsets, int32_t* __restrict__ row_token,
                   int32_t* __restrict__ inv_row /* in: replica index, out: row */) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint32_t (*rep)[kW] = reinterpret_cast<uint32_t (*)[kW]>(smem_raw);
    uint16_t (*rep_prefix)[kW] = reinterpret_cast<uint16_t (*)[kW]>(smem_raw + (size_t)NR * kW * 4);
    const int tile = blockIdx.x;
    for (int i = threadIdx.x; i < NR * kW; i += blockDim.x) (&rep[0][0])[i] = 0u;
    __syncthreads();
    const int t = tile * kTokenTile + threadIdx.x;
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int ri[kMaxK];
#pragma unroll
    for (int s = 0; s < kMaxK; ++s) {
        ri[s] = (t < T && s < K) ? inv_row[(size_t)t * K + s] : -1;
        if (ri[s] >= 0) atomicOr(&rep[ri[s]][w], 1u << lane);
    }
    __syncthreads();
    build_warp_prefix(rep, rep_prefix, NR);
    if (t >= T) return;
#pragma unroll
    for (int s = 0; s < kMaxK; ++s) {
        if (s >= K) break;
        int row = -1;
        if (ri[s] >= 0) {
            row = __ldg(seg_offsets + __ldg(rep_slot + ri[s])) + __ldg(tile_rep + (size_t)tile * NR + ri[s]) +
                  tile_rank(rep, rep_prefix, ri[s], w, lane);
            row_token[row] = t;
        }
        inv_row[(size_t)t * K + s] = row;
    }
}

// Placement cost per assignment (any source-rank map): W, Eq. 1 load, Eq. 3 volume under the locality-first rule.
__global__ void __launch_bounds__(kTokenTile)
local_cost_kernel(const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ src_rank,
                  const unsigned long long* __restrict__ host_mask, int T, int E, int K, int R, int C_max,
                  const int32_t* __restrict__ rep_start, const int32_t* __restrict__ rep_slot,
                  const int32_t* __restrict__ tile_travel, unsigned long long* __restrict__ workload,
                  unsigned long long* __restrict__ rank_load, unsigned long long* __restrict__ dispatch_tokens,
                  unsigned long long* __restrict__ dispatch_bytes, unsigned long long bytes_per_token,
                  int32_t* __restrict__ status) {
    __shared__ uint32_t travel[kMaxE][kW];
    __shared__ uint16_t travel_prefix[kMaxE][kW];
    __shared__ uint32_t h_rr[kMaxR * kMaxR];        // [src][dest]
    __shared__ uint32_t h_load[kMaxR];
    const int tile = blockIdx.x;
    for (int i = threadIdx.x; i < R * R; i += blockDim.x) h_rr[i] = 0u;
    for (int i = threadIdx.x; i < R; i += blockDim.x) h_load[i] = 0u;
    build_travel_masks(travel, topk_idx, src_rank, host_mask, tile, T, E, K, R, status);
    build_warp_prefix(travel, travel_prefix, E);
    const int t = tile * kTokenTile + threadIdx.x;
    if (t < T) {
        const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
        const int src = home_rank(src_rank, t, T, R, status);
        for (int s = 0; s < K && src >= 0; ++s) {
            const int e = __ldg(topk_idx + (size_t)t * K + s);
            if ((unsigned)e >= (unsigned)E) continue;
            const int ri = replica_of(travel, travel_prefix, host_mask, rep_start, tile_travel, tile, E, e, src, w, lane);
            const int dest = __ldg(rep_slot + ri) / C_max;
            atomicAdd(&h_rr[src * R + dest], 1u);
            atomicAdd(&h_load[dest], 1u);
            atomicAdd(workload + (size_t)src * E + e, 1ull);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < R * R; i += blockDim.x) {
        const uint32_t c = h_rr[i];
        if (c) {
            atomicAdd(dispatch_tokens + i, (unsigned long long)c);
            atomicAdd(dispatch_bytes + i, (unsigned long long)c * bytes_per_token);
        }
    }
    for (int i = threadIdx.x; i < R; i += blockDim.x)
        if (h_load[i]) atomicAdd(rank_load + i, (unsigned long long)h_load[i]);
}

// De-duplicated dispatch volume: U[j][k] = tokens of rank j with at least one assignment executed on rank k
// (a token whose several experts share a rank is sent there once).  One thread per token.
__global__ void __launch_bounds__(kTokenTile)
dedup_volume_kernel(const int32_t* __restrict__ dest_rank, const int32_t* __restrict__ src_rank, int T, int K, int R,
                    unsigned long long* __restrict__ dedup_tokens, int32_t* __restrict__ status) {
    __shared__ uint32_t h_rr[kMaxR * kMaxR];
    for (int i = threadIdx.x; i < R * R; i += blockDim.x) h_rr[i] = 0u;
    __syncthreads();
    const int t = blockIdx.x * kTokenTile + threadIdx.x;
    if (t < T) {
        const int src = home_rank(src_rank, t, T, R, status);
        unsigned long long seen = 0ull;
        for (int s = 0; s < K; ++s) {
            const int d = __ldg(dest_rank + (size_t)t * K + s);
            if (d < 0) continue;                                   // an assignment dispatch skipped (bad expert id)
            if (d >= R) { director_set_status(status, DIRECTOR_ERR_BAD_INDEX); continue; }
            seen |= 1ull << d;
        }
        while (seen && src >= 0) {
            const int d = __ffsll((long long)seen) - 1;
            seen &= seen - 1ull;
            atomicAdd(&h_rr[src * R + d], 1u);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < R * R; i += blockDim.x)
        if (h_rr[i]) atomicAdd(dedup_tokens + i, (unsigned long long)h_rr[i]);
}

int launch_travel_scan(director_ctx* ctx, const char* name, int T, const int32_t* topk_idx, const int32_t* src_rank,
                       cudaStream_t st) {
    const director_shape& s = ctx->shape;
    const int n_tiles = (T + kTokenTile - 1) / kTokenTile;
    LaunchScope scope(ctx, st, name);
    travel_count_scan_kernel<<<n_tiles, kTokenTile, 0, st>>>(topk_idx, src_rank, ctx->d_host_mask, T, s.E, s.K, s.R,
                                                             n_tiles, ctx->d_tile_counts, ctx->d_ticket, ctx->d_status);
    return cuda_status(cudaGetLastError());
}

}  // namespace

int dispatch_local_init(director_ctx* ctx) {
    // The attribute belongs to the kernel, not to the context: opt in once for the largest supported shape
    // (E = 256, G = 1024 replicas: 56 KB), so that a context of a smaller shape never lowers another one's limit.
    (void)ctx;
    if (cudaFuncSetAttribute(slot_count_scan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)slot_count_smem_bytes(kMaxE, kMaxG, kMaxG)) != cudaSuccess ||
        cudaFuncSetAttribute(local_index_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)local_index_smem_bytes(kMaxG)) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    return DIRECTOR_OK;
}

int launch_dispatch_local_first(director_ctx* ctx, int T, const void* x, const int32_t* topk_idx,
                                const int32_t* src_rank, void* xp, int32_t* row_token, int32_t* inv_row,
                                int32_t* dest_rank, int32_t* seg_offsets, cudaStream_t st) {
    const director_shape& s = ctx->shape;
    const int n_tiles = (T + kTokenTile - 1) / kTokenTile;
    const int NR = ctx->n_replicas;
    int rc = launch_travel_scan(ctx, "dispatch_travel_count_scan_kernel", T, topk_idx, src_rank, st);
    if (rc != DIRECTOR_OK) return rc;
    {
        LaunchScope scope(ctx, st, "dispatch_slot_count_scan_kernel");
        slot_count_scan_kernel<<<n_tiles, kTokenTile, slot_count_smem_bytes(s.E, NR, ctx->G), st>>>(
            topk_idx, src_rank, ctx->d_host_mask, T, s.E, s.K, s.R, s.C_max, ctx->G, NR, n_tiles, ctx->d_rep_start,
            ctx->d_rep_slot, ctx->d_tile_counts, ctx->d_tile_rep, inv_row, dest_rank, seg_offsets, ctx->d_seg_offsets,
            ctx->d_ticket, ctx->d_status);
        if (cudaGetLastError() != cudaSuccess) return DIRECTOR_ERR_CUDA;
    }
    {
        LaunchScope scope(ctx, st, "dispatch_local_index_kernel");
        local_index_kernel<<<n_tiles, kTokenTile, local_index_smem_bytes(NR), st>>>(
            T, s.K, NR, ctx->d_rep_slot, ctx->d_tile_rep, seg_offsets, row_token, inv_row);
        if (cudaGetLastError() != cudaSuccess) return DIRECTOR_ERR_CUDA;
    }
    if (xp != nullptr) rc = launch_scatter_rows(ctx, T, x, inv_row, xp, st);
    return rc;
}

int launch_cost_local_first(director_ctx* ctx, int T, const int32_t* topk_idx, const int32_t* src_rank,
                            int64_t* workload, int64_t* rank_load, int64_t* dispatch_tokens, uint64_t* dispatch_bytes,
                            cudaStream_t st) {
    const director_shape& s = ctx->shape;
    const int n_tiles = (T + kTokenTile - 1) / kTokenTile;
    if (cudaMemsetAsync(workload, 0, sizeof(int64_t) * s.R * s.E, st) != cudaSuccess ||
        cudaMemsetAsync(rank_load, 0, sizeof(int64_t) * s.R, st) != cudaSuccess ||
        cudaMemsetAsync(dispatch_tokens, 0, sizeof(int64_t) * s.R * s.R, st) != cudaSuccess ||
        cudaMemsetAsync(dispatch_bytes, 0, sizeof(uint64_t) * s.R * s.R, st) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    int rc = launch_travel_scan(ctx, "cost_travel_count_scan_kernel", T, topk_idx, src_rank, st);
    if (rc != DIRECTOR_OK) return rc;
    LaunchScope scope(ctx, st, "cost_local_kernel");
    local_cost_kernel<<<n_tiles, kTokenTile, 0, st>>>(
        topk_idx, src_rank, ctx->d_host_mask, T, s.E, s.K, s.R, s.C_max, ctx->d_rep_start, ctx->d_rep_slot,
        ctx->d_tile_counts, reinterpret_cast<unsigned long long*>(workload),
        reinterpret_cast<unsigned long long*>(rank_load), reinterpret_cast<unsigned long long*>(dispatch_tokens),
        reinterpret_cast<unsigned long long*>(dispatch_bytes), (unsigned long long)s.H * 2ull, ctx->d_status);
    return cuda_status(cudaGetLastError());
}

int launch_dedup_volume(director_ctx* ctx, int T, const int32_t* dest_rank, const int32_t* src_rank,
                        int64_t* dedup_tokens, cudaStream_t st) {
    const director_shape& s = ctx->shape;
    const int n_tiles = (T + kTokenTile - 1) / kTokenTile;
    if (cudaMemsetAsync(dedup_tokens, 0, sizeof(int64_t) * s.R * s.R, st) != cudaSuccess) return DIRECTOR_ERR_CUDA;
    LaunchScope scope(ctx, st, "dedup_volume_kernel");
    dedup_volume_kernel<<<n_tiles, kTokenTile, 0, st>>>(dest_rank, src_rank, T, s.K, s.R,
                                                        reinterpret_cast<unsigned long long*>(dedup_tokens),
                                                        ctx->d_status);
    return cuda_status(cudaGetLastError());
}

}  // namespace director
