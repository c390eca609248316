// Building blocks of the on-device counting sorts (dispatch under either replica rule, placement cost):
// lane-bitmask ranks inside a 256-token tile, the last-CTA-done ticket, column scans over the tiles and the
// block scan of the slot lengths into seg_offsets.  Integer only; every count comes from popcounts of bitmasks
// built with order-independent atomicOr, so results do not depend on scheduling.
#pragma once

#include "director_common.cuh"

namespace director {
namespace sort {

constexpr int kTileWarps = kTokenTile / 32;

// prefix[i][w] = number of set bits of mask[i][0..w): the stable rank offset of warp w's tokens inside the tile.
__device__ __forceinline__ void build_warp_prefix(const uint32_t (*mask)[kTileWarps], uint16_t (*prefix)[kTileWarps], int n) {
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        int run = 0;
#pragma unroll
        for (int w = 0; w < kTileWarps; ++w) { prefix[i][w] = (uint16_t)run; run += __popc(mask[i][w]); }
    }
    __syncthreads();
}

// Stable rank of the token (warp w, lane) among the tile's tokens whose bit is set in row i.
__device__ __forceinline__ int tile_rank(const uint32_t (*mask)[kTileWarps], const uint16_t (*prefix)[kTileWarps], int i,
                                         int w, int lane) {
    return prefix[i][w] + __popc(mask[i][w] & ((1u << lane) - 1u));
}

// True in exactly one CTA of the grid: the last one to get here (atomic ticket, nobody spins).  The caller resets
// the ticket once it is done.
__device__ __forceinline__ bool last_cta_done(unsigned int* ticket, int n_ctas, bool* flag) {
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) *flag = (atomicAdd(ticket, 1u) == (unsigned)(n_ctas - 1));
    __syncthreads();
    if (*flag) __threadfence();
    return *flag;
}

// In-place exclusive scan of column `col` of counts[n_tiles][ncol] over the tiles; returns the column total.
// Chunks of 16 tiles: all loads of a chunk are issued before the first store, so the loop runs at memory
// throughput instead of one L2 round trip per tile.
__device__ __forceinline__ int scan_column(int32_t* counts, int n_tiles, int ncol, int col) {
    int run = 0;
    for (int i0 = 0; i0 < n_tiles; i0 += 16) {
        int c[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) c[k] = (i0 + k < n_tiles) ? __ldcg(counts + (size_t)(i0 + k) * ncol + col) : 0;
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            if (i0 + k < n_tiles) counts[(size_t)(i0 + k) * ncol + col] = run;
            run += c[k];
        }
    }
    return run;
}

// Exclusive scan of slot_len[0..G) (shared memory) by the whole block into seg_offsets_a (and _b if not null);
// entry G receives the total.  warp_sum: shared scratch of blockDim.x / 32 ints.  Ends with the ticket reset by
// the last thread (the scan is the closing act of a last-CTA section).
__device__ __forceinline__ void scan_slots(const int32_t* slot_len, int G, int32_t* warp_sum,
                                           int32_t* __restrict__ seg_offsets_a, int32_t* __restrict__ seg_offsets_b,
                                           unsigned int* ticket) {
    const int per = (G + blockDim.x - 1) / blockDim.x;          // each thread owns a contiguous chunk
    const int lo = min((int)threadIdx.x * per, G), hi = min(lo + per, G);
    int local = 0;
    for (int g = lo; g < hi; ++g) local += slot_len[g];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    int incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) warp_sum[w] = incl;
    __syncthreads();
    int base = incl - local;
    for (int i = 0; i < w; ++i) base += warp_sum[i];
    for (int g = lo; g < hi; ++g) {
        seg_offsets_a[g] = base;
        if (seg_offsets_b) seg_offsets_b[g] = base;
        base += slot_len[g];
    }
    if (threadIdx.x == blockDim.x - 1) {
        // the last thread's running total is the grand total T*K (minus skipped bad indices)
        seg_offsets_a[G] = base;
        if (seg_offsets_b) seg_offsets_b[G] = base;
        *ticket = 0u;                                            // ready for the next call on this stream
    }
}

}  // namespace sort
}  // namespace director
