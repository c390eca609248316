// (a2) Placement-aware dispatch and (a5) placement cost.
//
// Dispatch (Section II-B: the first all-to-all moves every token to the ranks that host its experts) is an
// on-device stable counting sort of the T*K (token, choice) assignments by (destination rank,
// expert id, token id), followed by the row copies.  The same counting front-end feeds the
// placement-cost histograms (Section VI-A: workload matrix W, Eq. 1 load, Eq. 3 dispatch volume).
//
// Kernels
//   dispatch_plan_kernel  the whole index computation in ONE cooperative launch (batches whose 256-token
//                      tiles are all resident at once, i.e. up to ~300 K tokens): per-tile expert counts
//                      from lane bitmasks, a grid-wide barrier, then EVERY CTA sums the count columns it
//                      needs (tiles before its own -> its prefix, all tiles -> the totals), splits the totals
//                      over the replicas, scans the slot lengths and writes its own tokens' inv_row /
//                      dest_rank / row_token - the bitmasks never leave shared memory and no CTA waits for
//                      a single scanning CTA.  Larger batches and the allocation-free entry point use the
//                      two kernels below.
//   count_scan_kernel  per 256-token tile: per-expert counts from lane bitmasks; the last CTA to
//                      finish (atomic ticket, no spinning) turns them into exclusive per-tile
//                      prefixes, splits every expert's total over its replicas and scans the
//                      slot lengths into seg_offsets.
//   index_kernel       recomputes each assignment's stable rank inside its tile from the bitmasks,
//                      adds the tile prefix, applies the round-robin replica rule and writes
//                      inv_row / dest_rank / row_token.
//   scatter_rows_kernel  one warp per (token, 2 KB column slice): one coalesced 16-byte-per-lane read
//                      of x, K writes into xp.  HBM-bound: 2H + 2HK bytes per token.
//   cost_kernel        same ranks -> destination rank; shared-memory histograms flushed with
//                      integer atomics (order independent, hence deterministic).
#include "director_common.cuh"
#include "director_sort.cuh"

namespace director {

using namespace sort;

namespace {

// Lane bitmasks: mask[e][w] has bit l set iff token (tile*256 + w*32 + l) chose expert e.
__device__ __forceinline__ void build_masks(uint32_t (*mask)[kTileWarps], const int32_t* __restrict__ topk_idx,
                                            int tile, int T, int E, int K, int32_t* status) {
    for (int i = threadIdx.x; i < E * kTileWarps; i += blockDim.x) (&mask[0][0])[i] = 0u;
    __syncthreads();
    const int t = tile * kTokenTile + threadIdx.x;
    if (t < T) {
        const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
        for (int s = 0; s < K; ++s) {
            const int e = __ldg(topk_idx + (size_t)t * K + s);
            if ((unsigned)e < (unsigned)E) atomicOr(&mask[e][w], 1u << lane);
            else director_set_status(status, DIRECTOR_ERR_BAD_INDEX);
        }
    }
    __syncthreads();
}

__global__ void __launch_bounds__(kTokenTile)
count_scan_kernel(const int32_t* __restrict__ topk_idx, int T, int E, int K, int G, int n_tiles,
                  const int32_t* __restrict__ rep_start, const int32_t* __restrict__ rep_slot,
                  int32_t* __restrict__ tile_counts, int32_t* __restrict__ seg_offsets_a,
                  int32_t* __restrict__ seg_offsets_b, unsigned int* __restrict__ ticket,
                  int32_t* __restrict__ status) {
    __shared__ uint32_t mask[kMaxE][kTileWarps];
    __shared__ int32_t slot_len[kMaxG];
    __shared__ int32_t warp_sum[kTileWarps];
    __shared__ bool is_last;

    const int tile = blockIdx.x;
    build_masks(mask, topk_idx, tile, T, E, K, status);
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        int c = 0;
#pragma unroll
        for (int w = 0; w < kTileWarps; ++w) c += __popc(mask[e][w]);
        tile_counts[(size_t)tile * E + e] = c;
    }
    if (!last_cta_done(ticket, n_tiles, &is_last)) return;

    // ---- last CTA: per-expert exclusive scan over tiles, replica split, slot scan ----
    for (int g = threadIdx.x; g < G; g += blockDim.x) slot_len[g] = 0;
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        const int run = scan_column(tile_counts, n_tiles, E, e);
        const int r0 = rep_start[e], r_e = rep_start[e + 1] - r0;
        if (r_e < 1 && run > 0) director_set_status(status, DIRECTOR_ERR_BAD_INDEX);   // a routed-to expert without a host
        for (int q = 0; q < r_e; ++q) {             // replica q gets ceil((N_e - q) / r_e) rows
            const int slot = rep_slot[r0 + q];
            if ((unsigned)slot < (unsigned)G) slot_len[slot] = (run > q) ? (run - q + r_e - 1) / r_e : 0;
            else director_set_status(status, DIRECTOR_ERR_BAD_INDEX);
        }
    }
    __syncthreads();
    scan_slots(slot_len, G, warp_sum, seg_offsets_a, seg_offsets_b, ticket);
}

__global__ void __launch_bounds__(kTokenTile)
index_kernel(const int32_t* __restrict__ topk_idx, int T, int E, int K, int C_max, int G,
             const int32_t* __restrict__ rep_start, const int32_t* __restrict__ rep_slot,
             const int32_t* __restrict__ tile_prefix, const int32_t* __restrict__ seg_offsets,
             int32_t* __restrict__ row_token, int32_t* __restrict__ inv_row, int32_t* __restrict__ dest_rank,
             int32_t* __restrict__ status) {
    __shared__ uint32_t mask[kMaxE][kTileWarps];
    __shared__ uint16_t warp_prefix[kMaxE][kTileWarps];
    const int tile = blockIdx.x;
    build_masks(mask, topk_idx, tile, T, E, K, status);
    build_warp_prefix(mask, warp_prefix, E);
    const int t = tile * kTokenTile + threadIdx.x;
    if (t >= T) return;
    const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int s = 0; s < K; ++s) {
        const int e = __ldg(topk_idx + (size_t)t * K + s);
        int row = -1, dest = -1;
        if ((unsigned)e < (unsigned)E) {
            const int n = __ldg(tile_prefix + (size_t)tile * E + e) + tile_rank(mask, warp_prefix, e, w, lane);
            const int r0 = __ldg(rep_start + e), r_e = __ldg(rep_start + e + 1) - r0;
            // the context's tables are validated when the placement is set; caller-built tables (the allocation-free
            // entry point) are not, so an expert without a host or a slot outside the table is skipped and flagged
            const int slot = r_e >= 1 ? __ldg(rep_slot + r0 + n % r_e) : -1;
            if ((unsigned)slot < (unsigned)G) {
                row = __ldg(seg_offsets + slot) + n / r_e;
                dest = slot / C_max;
                row_token[row] = t;
            } else {
                director_set_status(status, DIRECTOR_ERR_BAD_INDEX);
            }
        }
        inv_row[(size_t)t * K + s] = row;
        dest_rank[(size_t)t * K + s] = dest;
    }
}

// Grid-wide barrier of a cooperative launch (all CTAs resident).  bar[0] counts arrivals, bar[1] departures; the last
// CTA to leave zeroes both for the next launch.  The wait is bounded: on expiry the CTA reports false.
__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long plan_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ bool grid_barrier(unsigned int* bar, unsigned int n_ctas, int* s_flag) {
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        atomicAdd(bar, 1u);
        int ok = 1;
        if (ld_acquire_gpu(bar) < n_ctas) {
            const unsigned long long t0 = plan_timer_ns();
            unsigned int spins = 0;
            while (ld_acquire_gpu(bar) < n_ctas) {
                __nanosleep(32);
                if ((++spins & 255u) == 0u && plan_timer_ns() - t0 > 2000000000ull) { ok = 0; break; }
            }
        }
        *s_flag = ok;
    }
    __syncthreads();
    return *s_flag != 0;
}
__device__ __forceinline__ void grid_barrier_leave(unsigned int* bar, unsigned int n_ctas) {
    if (threadIdx.x == 0 && atomicAdd(bar + 1, 1u) == n_ctas - 1u) {
        bar[0] = 0u;                // everybody has passed the wait: ready for the next launch on this stream
        bar[1] = 0u;
    }
}

__global__ void __launch_bounds__(kTokenTile)
dispatch_plan_kernel(const int32_t* __restrict__ topk_idx, int T, int E, int K, int C_max, int G, int n_tiles,
                     const int32_t* __restrict__ rep_start, const int32_t* __restrict__ rep_slot,
                     int32_t* __restrict__ tile_counts, int32_t* __restrict__ seg_offsets_a,
                     int32_t* __restrict__ seg_offsets_b, int32_t* __restrict__ row_token, int32_t* __restrict__ inv_row,
                     int32_t* __restrict__ dest_rank, unsigned int* __restrict__ bar, int32_t* __restrict__ status) {
    __shared__ uint32_t mask[kMaxE][kTileWarps];
    __shared__ uint16_t warp_prefix[kMaxE][kTileWarps];
    __shared__ int32_t s_pre[kMaxE], s_tot[kMaxE];
    __shared__ int32_t s_seg[kMaxG + 1];          // slot lengths, then their exclusive prefix
    __shared__ int32_t warp_sum[kTileWarps];
    __shared__ int s_flag;

    const int tile = blockIdx.x;
    build_masks(mask, topk_idx, tile, T, E, K, status);
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        int c = 0;
#pragma unroll
        for (int w = 0; w < kTileWarps; ++w) c += __popc(mask[e][w]);
        tile_counts[(size_t)tile * E + e] = c;
        s_pre[e] = 0;
        s_tot[e] = 0;
    }
    for (int g = threadIdx.x; g <= G; g += blockDim.x) s_seg[g] = 0;
    build_warp_prefix(mask, warp_prefix, E);
    if (!grid_barrier(bar, (unsigned)n_tiles, &s_flag)) {
        if (threadIdx.x == 0) director_set_status(status, DIRECTOR_ERR_TIMEOUT);
        return;
    }
    // every CTA of this grid is running: a programmatically dependent kernel (the row copies) may be scheduled into
    // the free SMs now; it still waits for this grid to finish before it reads the indices
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // ---- every CTA: column sums over the tiles (tiles before mine -> my prefix; all tiles -> the totals) ----
    // 256 threads = `parts` groups of E_pad threads; group p sums tiles p, p + parts, ... of its expert's column;
    // the partial sums meet in shared memory (integer adds: the order does not matter).
    int e_pad = 1;
    while (e_pad < E) e_pad <<= 1;
    const int parts = kTokenTile / e_pad;                       // E <= 256 = blockDim
    const int e_mine = threadIdx.x & (e_pad - 1), part = threadIdx.x / e_pad;
    if (e_mine < E) {
        int pre = 0, tot = 0;
        for (int i0 = part; i0 < n_tiles; i0 += 8 * parts) {    // eight independent loads in flight per thread
            int c[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int i = i0 + k * parts;
                c[k] = i < n_tiles ? __ldcg(tile_counts + (size_t)i * E + e_mine) : 0;
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                tot += c[k];
                if (i0 + k * parts < tile) pre += c[k];
            }
        }
        if (parts > 1) {
            if (pre) atomicAdd(&s_pre[e_mine], pre);
            if (tot) atomicAdd(&s_tot[e_mine], tot);
        } else {
            s_pre[e_mine] = pre;
            s_tot[e_mine] = tot;
        }
    }
    __syncthreads();
    for (int e = threadIdx.x; e < E; e += blockDim.x) {
        const int run = s_tot[e];
        const int r0 = __ldg(rep_start + e), r_e = __ldg(rep_start + e + 1) - r0;
        if (r_e < 1 && run > 0 && tile == 0) director_set_status(status, DIRECTOR_ERR_BAD_INDEX);
        for (int q = 0; q < r_e; ++q) {             // replica q gets ceil((N_e - q) / r_e) rows
            const int slot = __ldg(rep_slot + r0 + q);
            if ((unsigned)slot < (unsigned)G) s_seg[slot] = (run > q) ? (run - q + r_e - 1) / r_e : 0;
        }
    }
    __syncthreads();
    {   // exclusive scan of the slot lengths, in place; entry G receives the total
        const int per = (G + blockDim.x - 1) / blockDim.x;
        const int lo = min((int)threadIdx.x * per, G), hi = min(lo + per, G);
        int local = 0;
        for (int g = lo; g < hi; ++g) local += s_seg[g];
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
            const int len = s_seg[g];
            s_seg[g] = base;
            base += len;
        }
        if (threadIdx.x == blockDim.x - 1) s_seg[G] = base;
        __syncthreads();
    }
    if (tile == 0) {
        for (int g = threadIdx.x; g <= G; g += blockDim.x) {
            seg_offsets_a[g] = s_seg[g];
            if (seg_offsets_b) seg_offsets_b[g] = s_seg[g];
        }
    }

    // ---- my tile's assignments ----
    const int t = tile * kTokenTile + threadIdx.x;
    if (t < T) {
        const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
        for (int s = 0; s < K; ++s) {
            const int e = __ldg(topk_idx + (size_t)t * K + s);
            int row = -1, dest = -1;
            if ((unsigned)e < (unsigned)E) {
                const int n = s_pre[e] + tile_rank(mask, warp_prefix, e, w, lane);
                const int r0 = __ldg(rep_start + e), r_e = __ldg(rep_start + e + 1) - r0;
                const int slot = r_e >= 1 ? __ldg(rep_slot + r0 + n % r_e) : -1;
                if ((unsigned)slot < (unsigned)G) {
                    row = s_seg[slot] + n / r_e;
                    dest = slot / C_max;
                    row_token[row] = t;
                } else {
                    director_set_status(status, DIRECTOR_ERR_BAD_INDEX);
                }
            }
            inv_row[(size_t)t * K + s] = row;
            dest_rank[(size_t)t * K + s] = dest;
        }
    }
    grid_barrier_leave(bar, (unsigned)n_tiles);
}

// One warp copies a 2 KB slice (4 x 16 bytes per lane) of row t of x to its K destination rows.
constexpr int kSliceVec = 4;                       // uint4 per lane
constexpr int kSliceBytes = 32 * 16 * kSliceVec;   // 2048
constexpr int kScatterWarps = 8;

__global__ void __launch_bounds__(kScatterWarps * 32)
scatter_rows_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ inv_row, uint4* __restrict__ xp,
                    int T, int K, int row_vec /* uint4 per row */, int slices_per_row) {
    const int lane = threadIdx.x & 31;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");     // the kernel after this one may be scheduled
    const long long item = (long long)blockIdx.x * kScatterWarps + (threadIdx.x >> 5);
    if (item >= (long long)T * slices_per_row) return;
    const int t = (int)(item / slices_per_row);
    const int v0 = (int)(item % slices_per_row) * (32 * kSliceVec) + lane;
    const uint4* src = x + (size_t)t * row_vec;
    uint4 v[kSliceVec];
    // x is an input of the whole dispatch: its slice is fetched before the wait below, while the index kernel
    // that this launch programmatically depends on may still be finishing
#pragma unroll
    for (int i = 0; i < kSliceVec; ++i)
        if (v0 + 32 * i < row_vec) v[i] = __ldcs(src + v0 + 32 * i);
    // launched with programmatic stream serialization: returns once the preceding kernel of the stream has
    // completed and its writes (inv_row) are visible; a no-op under an ordinary launch
    asm volatile("griddepcontrol.wait;" ::: "memory");
    int my_row = (lane < K) ? __ldcg(inv_row + (size_t)t * K + lane) : -1;
    for (int s = 0; s < K; ++s) {
        const int row = __shfl_sync(0xFFFFFFFFu, my_row, s);
        if (row < 0) continue;
        uint4* dst = xp + (size_t)row * row_vec;
#pragma unroll
        for (int i = 0; i < kSliceVec; ++i)
            if (v0 + 32 * i < row_vec) dst[v0 + 32 * i] = v[i];
    }
}

// Placement cost: per assignment (src rank j, expert e, destination rank k).
__global__ void __launch_bounds__(kTokenTile)
cost_kernel(const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ src_rank, int T, int E, int K, int R,
            int C_max, const int32_t* __restrict__ rep_start, const int32_t* __restrict__ rep_slot,
            const int32_t* __restrict__ tile_prefix, unsigned long long* __restrict__ workload,
            unsigned long long* __restrict__ rank_load, unsigned long long* __restrict__ dispatch_tokens,
            unsigned long long* __restrict__ dispatch_bytes, unsigned long long bytes_per_token,
            int32_t* __restrict__ status) {
    __shared__ uint32_t mask[kMaxE][kTileWarps];
    __shared__ uint16_t warp_prefix[kMaxE][kTileWarps];
    __shared__ uint32_t h_rr[kMaxR * kMaxR];        // [src][dest]
    __shared__ uint32_t h_load[kMaxR];
    const int tile = blockIdx.x;
    for (int i = threadIdx.x; i < R * R; i += blockDim.x) h_rr[i] = 0u;
    for (int i = threadIdx.x; i < R; i += blockDim.x) h_load[i] = 0u;
    build_masks(mask, topk_idx, tile, T, E, K, status);
    build_warp_prefix(mask, warp_prefix, E);
    const int t = tile * kTokenTile + threadIdx.x;
    if (t < T) {
        const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
        int src = src_rank ? __ldg(src_rank + t) : (int)(((long long)t * R) / T);
        if ((unsigned)src >= (unsigned)R) { director_set_status(status, DIRECTOR_ERR_BAD_INDEX); src = -1; }
        for (int s = 0; s < K && src >= 0; ++s) {
            const int e = __ldg(topk_idx + (size_t)t * K + s);
            if ((unsigned)e >= (unsigned)E) continue;
            const int n = __ldg(tile_prefix + (size_t)tile * E + e) + tile_rank(mask, warp_prefix, e, w, lane);
            const int r0 = __ldg(rep_start + e), r_e = __ldg(rep_start + e + 1) - r0;
            const int dest = __ldg(rep_slot + r0 + n % r_e) / C_max;
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

// ---- placement cost, fast path for the default block partition of tokens over source ranks ----
//
// With src(t) = floor(t*R/T) the tokens of a source rank are a contiguous range, and the n-th assignment of
// an expert is numbered in ascending token order, so the assignments that rank j sends to expert e occupy a
// contiguous range [a, b) of n.  Round-robin over r replicas gives replica q exactly
//     f(b) - f(a),  f(x) = max(0, ceil((x - q) / r))
// of them.  The whole cost therefore follows from the workload matrix W alone: one histogram kernel and one
// warp-per-expert kernel, no per-assignment ranks.  Under the locality-first rule the ranks that host e keep their
// own W[j][e] assignments and the same closed form runs over the remaining (travelling) ranks' counts.

constexpr int kHistSmemInts = 4096;

__global__ void __launch_bounds__(kTokenTile)
workload_hist_kernel(const int32_t* __restrict__ topk_idx, int T, int E, int K, int R,
                     unsigned long long* __restrict__ workload, unsigned long long* __restrict__ rank_load,
                     unsigned long long* __restrict__ dispatch_tokens, unsigned long long* __restrict__ dispatch_bytes,
                     int32_t* __restrict__ status) {
    __shared__ uint32_t hist[kHistSmemInts];
    if (blockIdx.x == 0) {      // the other outputs are accumulated by the next kernel: clear them here
        for (int i = threadIdx.x; i < R * R; i += blockDim.x) { dispatch_tokens[i] = 0ull; dispatch_bytes[i] = 0ull; }
        for (int i = threadIdx.x; i < R; i += blockDim.x) rank_load[i] = 0ull;
    }
    const int t0 = blockIdx.x * kTokenTile, t1 = min(t0 + kTokenTile, T) - 1;
    const int src_lo = (int)(((long long)t0 * R) / T), src_hi = (int)(((long long)t1 * R) / T);
    const int n_src = src_hi - src_lo + 1;
    const bool use_smem = n_src * E <= kHistSmemInts;
    if (use_smem) {
        for (int i = threadIdx.x; i < n_src * E; i += blockDim.x) hist[i] = 0u;
        __syncthreads();
    }
    const int t = t0 + threadIdx.x;
    if (t < T) {
        const int src = (int)(((long long)t * R) / T);
        for (int s = 0; s < K; ++s) {
            const int e = __ldg(topk_idx + (size_t)t * K + s);
            if ((unsigned)e >= (unsigned)E) { director_set_status(status, DIRECTOR_ERR_BAD_INDEX); continue; }
            if (use_smem) atomicAdd(&hist[(src - src_lo) * E + e], 1u);
            else atomicAdd(workload + (size_t)src * E + e, 1ull);
        }
    }
    if (use_smem) {
        __syncthreads();
        for (int i = threadIdx.x; i < n_src * E; i += blockDim.x)
            if (hist[i]) atomicAdd(workload + (size_t)src_lo * E + i, (unsigned long long)hist[i]);
    }
}

// One warp per expert, lanes over the source ranks: prefix-scan the expert's column of W over the ranks
// (the start a_j of rank j's range of n), split each range over the replicas, add into the outputs
// (zeroed by workload_hist_kernel) with 64-bit global atomics.
constexpr int kCostWarps = 8;

__global__ void __launch_bounds__(kCostWarps * 32)
cost_from_workload_kernel(const unsigned long long* __restrict__ workload, int E, int R, int C_max,
                          const int32_t* __restrict__ rep_start, const int32_t* __restrict__ rep_slot,
                          const unsigned long long* __restrict__ host_mask /* non-null: locality-first rule */,
                          unsigned long long* __restrict__ rank_load, unsigned long long* __restrict__ dispatch_tokens,
                          unsigned long long* __restrict__ dispatch_bytes, unsigned long long bytes_per_token) {
    const int e = blockIdx.x * kCostWarps + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (e >= E) return;
    const int r0 = __ldg(rep_start + e);
    const uint32_t r = (uint32_t)(__ldg(rep_start + e + 1) - r0);
    const unsigned long long hm = host_mask ? __ldg(host_mask + e) : 0ull;
    uint32_t carry = 0;                                        // assignments of e sent by ranks before this chunk
    for (int j0 = 0; j0 < R; j0 += 32) {
        const int j = j0 + lane;
        uint32_t w = j < R ? (uint32_t)workload[(size_t)j * E + e] : 0u;   // counts fit 32 bits: T*K < 2^31
        if (j < R && ((hm >> j) & 1ull)) {
            // locality first: a rank that hosts e serves its own tokens; only the others' assignments are numbered
            if (w) {
                atomicAdd(dispatch_tokens + (size_t)j * R + j, (unsigned long long)w);
                atomicAdd(dispatch_bytes + (size_t)j * R + j, (unsigned long long)w * bytes_per_token);
                atomicAdd(rank_load + j, (unsigned long long)w);
            }
            w = 0u;
        }
        uint32_t incl = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += v;
        }
        const uint32_t b = carry + incl, a = b - w;            // rank j sends assignments n in [a, b)
        if (w) {
            for (uint32_t q = 0; q < r; ++q) {
                const uint32_t fb = b > q ? (b - q + r - 1) / r : 0u, fa = a > q ? (a - q + r - 1) / r : 0u;
                if (fb > fa) {
                    const int dest = __ldg(rep_slot + r0 + q) / C_max;
                    const unsigned long long n = fb - fa;
                    atomicAdd(dispatch_tokens + (size_t)j * R + dest, n);
                    atomicAdd(dispatch_bytes + (size_t)j * R + dest, n * bytes_per_token);
                    atomicAdd(rank_load + dest, n);
                }
            }
        }
        carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
}

// ---- batched placement cost: many candidate placements against one workload matrix ----
//
// Section VI-C: the placement search evaluates candidate after candidate against the same predicted workload.
// With W fixed, a candidate's per-rank load (Eq. 1) and dispatch volume (Eq. 3) follow from its placement matrix
// alone by the closed form above, so a whole batch of candidates is one launch: one warp per (candidate, expert).
// A candidate is given as its raw matrix X[E][R]; the replicas of an expert are its set ranks in ascending order.

__global__ void __launch_bounds__(kCostWarps * 32)
cost_batch_kernel(const unsigned long long* __restrict__ workload, int E, int R, const uint8_t* __restrict__ X,
                  int local_first, unsigned long long* __restrict__ rank_load,
                  unsigned long long* __restrict__ dispatch_tokens) {
    const int e = blockIdx.x * kCostWarps + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    const int c = blockIdx.y;
    if (e >= E) return;
    const uint8_t* xrow = X + ((size_t)c * E + e) * R;
    // replica set of e under candidate c as two 32-bit rank masks
    const uint32_t m0 = __ballot_sync(0xFFFFFFFFu, lane < R && xrow[lane] != 0);
    const uint32_t m1 = __ballot_sync(0xFFFFFFFFu, lane + 32 < R && xrow[lane + 32] != 0);
    const uint32_t r = (uint32_t)(__popc(m0) + __popc(m1));
    if (r == 0) return;                                         // unhosted expert: candidate is flagged invalid elsewhere
    unsigned long long* load_c = rank_load + (size_t)c * R;
    unsigned long long* disp_c = dispatch_tokens + (size_t)c * R * R;
    uint32_t carry = 0;
    for (int j0 = 0; j0 < R; j0 += 32) {
        const int j = j0 + lane;
        uint32_t w = j < R ? (uint32_t)workload[(size_t)j * E + e] : 0u;
        if (local_first && (((j0 == 0 ? m0 : m1) >> lane) & 1u)) {     // this rank hosts e: its tokens stay
            if (w) {
                atomicAdd(disp_c + (size_t)j * R + j, (unsigned long long)w);
                atomicAdd(load_c + j, (unsigned long long)w);
            }
            w = 0u;
        }
        uint32_t incl = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += v;
        }
        const uint32_t b = carry + incl, a = b - w;
        if (w) {
            uint32_t rem0 = m0, rem1 = m1;
            for (uint32_t q = 0; q < r; ++q) {                  // q-th replica = q-th set rank
                int dest;
                if (rem0) { dest = __ffs(rem0) - 1; rem0 &= rem0 - 1; }
                else { dest = 32 + __ffs(rem1) - 1; rem1 &= rem1 - 1; }
                const uint32_t fb = b > q ? (b - q + r - 1) / r : 0u, fa = a > q ? (a - q + r - 1) / r : 0u;
                if (fb > fa) {
                    atomicAdd(disp_c + (size_t)j * R + dest, (unsigned long long)(fb - fa));
                    atomicAdd(load_c + dest, (unsigned long long)(fb - fa));
                }
            }
        }
        carry += __shfl_sync(0xFFFFFFFFu, incl, 31);
    }
}

// One CTA per candidate: validity (every expert hosted, at most C_max experts per rank) and the reductions the
// objective is built from: max_j lambda_j (Eq. 2), max_j sum_{k != j} D[j][k] (Eq. 4), total cross-rank tokens.
__global__ void __launch_bounds__(64)
cost_batch_summary_kernel(int E, int R, int C_max, const uint8_t* __restrict__ X,
                          const unsigned long long* __restrict__ rank_load,
                          const unsigned long long* __restrict__ dispatch_tokens, long long* __restrict__ summary) {
    __shared__ long long s_load[kMaxR], s_send[kMaxR];
    __shared__ int s_bad;
    const int c = blockIdx.x, j = threadIdx.x;
    if (j == 0) s_bad = 0;
    __syncthreads();
    const uint8_t* Xc = X + (size_t)c * E * R;
    if (j < R) {
        int hosted = 0;
        for (int e = 0; e < E; ++e) hosted += Xc[(size_t)e * R + j] != 0;
        if (hosted > C_max) atomicOr(&s_bad, 1);
        long long send = 0;
        for (int k = 0; k < R; ++k)
            if (k != j) send += (long long)dispatch_tokens[((size_t)c * R + j) * R + k];
        s_send[j] = send;
        s_load[j] = (long long)rank_load[(size_t)c * R + j];
    }
    for (int e = j; e < E; e += blockDim.x) {
        int any = 0;
        for (int k = 0; k < R; ++k) any |= Xc[(size_t)e * R + k];
        if (!any) atomicOr(&s_bad, 1);
    }
    __syncthreads();
    if (j == 0) {
        long long max_load = 0, max_send = 0, cross = 0;
        for (int k = 0; k < R; ++k) {
            max_load = max(max_load, s_load[k]);
            max_send = max(max_send, s_send[k]);
            cross += s_send[k];
        }
        summary[4 * c + 0] = max_load;
        summary[4 * c + 1] = max_send;
        summary[4 * c + 2] = cross;
        summary[4 * c + 3] = s_bad ? 0 : 1;
    }
}

int launch_count_scan(director_ctx* ctx, const char* name, int T, const int32_t* topk_idx, int32_t* seg_a, int32_t* seg_b,
                      cudaStream_t st) {
    const director_shape& s = ctx->shape;
    const int n_tiles = (T + kTokenTile - 1) / kTokenTile;
    LaunchScope scope(ctx, st, name);
    count_scan_kernel<<<n_tiles, kTokenTile, 0, st>>>(topk_idx, T, s.E, s.K, ctx->G, n_tiles, ctx->d_rep_start,
                                                      ctx->d_rep_slot, ctx->d_tile_counts, seg_a, seg_b,
                                                      ctx->d_ticket, ctx->d_status);
    return cuda_status(cudaGetLastError());
}

}  // namespace

// Largest number of 256-token tiles the one-launch index kernel can take: all its CTAs must be resident at once.
int dispatch_init(director_ctx* ctx) {
    int per_sm = 0, coop = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, dispatch_plan_kernel, kTokenTile, 0) != cudaSuccess ||
        cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, ctx->device) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    ctx->plan_max_tiles = coop ? per_sm * ctx->sm_count : 0;
    return DIRECTOR_OK;
}

int launch_scatter_rows(director_ctx* ctx, int T, const void* x, const int32_t* inv_row, void* xp, cudaStream_t st) {
    StageScope stage(ctx, st, "stage_dispatch");
    const director_shape& s = ctx->shape;
    const int row_vec = s.H * 2 / 16;
    const int slices = (s.H * 2 + kSliceBytes - 1) / kSliceBytes;
    const long long items = (long long)T * slices;
    const unsigned grid = (unsigned)((items + kScatterWarps - 1) / kScatterWarps);
    LaunchScope scope(ctx, st, "dispatch_scatter_rows_kernel");
    // programmatic dependent launch: the copy kernel's CTAs may be set up, and read their slices of x, while the
    // kernel before it in the stream (the index kernel) drains; they wait for it before touching inv_row
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kScatterWarps * 32);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cuda_status(cudaLaunchKernelEx(&cfg, scatter_rows_kernel, static_cast<const uint4*>(x), inv_row,
                                          static_cast<uint4*>(xp), T, (int)s.K, row_vec, slices));
}

int launch_dispatch(director_ctx* ctx, int T, const void* x, const int32_t* topk_idx, const int32_t* src_rank, void* xp,
                    int32_t* row_token, int32_t* inv_row, int32_t* dest_rank, int32_t* seg_offsets, cudaStream_t st) {
    StageScope stage(ctx, st, "stage_dispatch");
    if (ctx->replica_policy == DIRECTOR_REPLICA_LOCAL_FIRST)
        return launch_dispatch_local_first(ctx, T, x, topk_idx, src_rank, xp, row_token, inv_row, dest_rank,
                                           seg_offsets, st);
    const director_shape& s = ctx->shape;
    const int n_tiles = (T + kTokenTile - 1) / kTokenTile;
    int rc;
    if (n_tiles <= ctx->plan_max_tiles) {
        // one cooperative launch: counts, grid barrier, per-CTA scans, indices
        int E = s.E, K = s.K, C_max = s.C_max, G = ctx->G, nt = n_tiles, Tv = T;
        const int32_t* rs = ctx->d_rep_start;
        const int32_t* rl = ctx->d_rep_slot;
        int32_t* tc = ctx->d_tile_counts;
        int32_t* seg_b = ctx->d_seg_offsets;
        unsigned int* bar = ctx->d_ticket + 1;
        int32_t* status = ctx->d_status;
        void* args[] = {&topk_idx, &Tv, &E, &K, &C_max, &G, &nt, &rs, &rl, &tc, &seg_offsets, &seg_b,
                        &row_token, &inv_row, &dest_rank, &bar, &status};
        {
            LaunchScope scope(ctx, st, "dispatch_plan_kernel");
            rc = cuda_status(cudaLaunchCooperativeKernel(reinterpret_cast<const void*>(dispatch_plan_kernel), dim3(n_tiles),
                                                         dim3(kTokenTile), args, 0, st));
        }
        if (rc != DIRECTOR_OK) return rc;
        if (xp != nullptr) rc = launch_scatter_rows(ctx, T, x, inv_row, xp, st);
        return rc;
    }
    rc = launch_count_scan(ctx, "dispatch_count_scan_kernel", T, topk_idx, seg_offsets, ctx->d_seg_offsets, st);
    if (rc != DIRECTOR_OK) return rc;
    {
        LaunchScope scope(ctx, st, "dispatch_index_kernel");
        index_kernel<<<n_tiles, kTokenTile, 0, st>>>(topk_idx, T, s.E, s.K, s.C_max, ctx->G, ctx->d_rep_start, ctx->d_rep_slot,
                                                     ctx->d_tile_counts, seg_offsets, row_token, inv_row, dest_rank,
                                                     ctx->d_status);
        rc = cuda_status(cudaGetLastError());
        if (rc != DIRECTOR_OK) return rc;
    }
    // xp == nullptr: indices only (the expert FFN then gathers its rows from x itself)
    if (xp != nullptr) rc = launch_scatter_rows(ctx, T, x, inv_row, xp, st);
    return rc;
}

int launch_cost_batch(director_ctx* ctx, const int64_t* workload, int n, const uint8_t* X, int64_t* rank_load,
                      int64_t* dispatch_tokens, int64_t* summary, cudaStream_t st) {
    const director_shape& s = ctx->shape;
    if (cudaMemsetAsync(rank_load, 0, sizeof(int64_t) * (size_t)n * s.R, st) != cudaSuccess ||
        cudaMemsetAsync(dispatch_tokens, 0, sizeof(int64_t) * (size_t)n * s.R * s.R, st) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    {
        LaunchScope scope(ctx, st, "cost_batch_kernel");
        cost_batch_kernel<<<dim3((s.E + kCostWarps - 1) / kCostWarps, n), kCostWarps * 32, 0, st>>>(
            reinterpret_cast<const unsigned long long*>(workload), s.E, s.R, X,
            ctx->replica_policy == DIRECTOR_REPLICA_LOCAL_FIRST ? 1 : 0,
            reinterpret_cast<unsigned long long*>(rank_load), reinterpret_cast<unsigned long long*>(dispatch_tokens));
        if (cudaGetLastError() != cudaSuccess) return DIRECTOR_ERR_CUDA;
    }
    LaunchScope scope(ctx, st, "cost_batch_summary_kernel");
    cost_batch_summary_kernel<<<n, 64, 0, st>>>(s.E, s.R, s.C_max, X, reinterpret_cast<const unsigned long long*>(rank_load),
                                                reinterpret_cast<const unsigned long long*>(dispatch_tokens),
                                                reinterpret_cast<long long*>(summary));
    return cuda_status(cudaGetLastError());
}

int launch_cost(director_ctx* ctx, int T, const int32_t* topk_idx, const int32_t* src_rank, int64_t* workload,
                int64_t* rank_load, int64_t* dispatch_tokens, uint64_t* dispatch_bytes, cudaStream_t st) {
    StageScope stage(ctx, st, "stage_placement_cost");
    const director_shape& s = ctx->shape;
    const int n_tiles = (T + kTokenTile - 1) / kTokenTile;
    const bool local_first = ctx->replica_policy == DIRECTOR_REPLICA_LOCAL_FIRST;
    if (local_first && src_rank != nullptr)
        return launch_cost_local_first(ctx, T, topk_idx, src_rank, workload, rank_load, dispatch_tokens, dispatch_bytes, st);
    cudaError_t e;
    if ((e = cudaMemsetAsync(workload, 0, sizeof(int64_t) * s.R * s.E, st)) != cudaSuccess) return cuda_status(e);
    if (src_rank == nullptr) {
        {
            LaunchScope scope(ctx, st, "cost_workload_hist_kernel");
            workload_hist_kernel<<<n_tiles, kTokenTile, 0, st>>>(topk_idx, T, s.E, s.K, s.R,
                                                                 reinterpret_cast<unsigned long long*>(workload),
                                                                 reinterpret_cast<unsigned long long*>(rank_load),
                                                                 reinterpret_cast<unsigned long long*>(dispatch_tokens),
                                                                 reinterpret_cast<unsigned long long*>(dispatch_bytes),
                                                                 ctx->d_status);
            if (cudaGetLastError() != cudaSuccess) return DIRECTOR_ERR_CUDA;
        }
        LaunchScope scope(ctx, st, "cost_from_workload_kernel");
        cost_from_workload_kernel<<<(s.E + kCostWarps - 1) / kCostWarps, kCostWarps * 32, 0, st>>>(reinterpret_cast<const unsigned long long*>(workload), s.E, s.R,
                                                     s.C_max, ctx->d_rep_start, ctx->d_rep_slot,
                                                     local_first ? ctx->d_host_mask : nullptr,
                                                     reinterpret_cast<unsigned long long*>(rank_load),
                                                     reinterpret_cast<unsigned long long*>(dispatch_tokens),
                                                     reinterpret_cast<unsigned long long*>(dispatch_bytes),
                                                     (unsigned long long)s.H * 2ull);
        return cuda_status(cudaGetLastError());
    }
    if ((e = cudaMemsetAsync(rank_load, 0, sizeof(int64_t) * s.R, st)) != cudaSuccess) return cuda_status(e);
    if ((e = cudaMemsetAsync(dispatch_tokens, 0, sizeof(int64_t) * s.R * s.R, st)) != cudaSuccess) return cuda_status(e);
    if ((e = cudaMemsetAsync(dispatch_bytes, 0, sizeof(uint64_t) * s.R * s.R, st)) != cudaSuccess) return cuda_status(e);
    int rc = launch_count_scan(ctx, "cost_count_scan_kernel", T, topk_idx, ctx->d_seg_offsets, nullptr, st);
    if (rc != DIRECTOR_OK) return rc;
    LaunchScope scope(ctx, st, "cost_kernel");
    cost_kernel<<<n_tiles, kTokenTile, 0, st>>>(topk_idx, src_rank, T, s.E, s.K, s.R, s.C_max, ctx->d_rep_start,
                                                ctx->d_rep_slot, ctx->d_tile_counts,
                                                reinterpret_cast<unsigned long long*>(workload),
                                                reinterpret_cast<unsigned long long*>(rank_load),
                                                reinterpret_cast<unsigned long long*>(dispatch_tokens),
                                                reinterpret_cast<unsigned long long*>(dispatch_bytes),
                                                (unsigned long long)s.H * 2ull, ctx->d_status);
    return cuda_status(cudaGetLastError());
}

}  // namespace director

// ---------------------------------------------------------------------------------------------
// Allocation-free variant of the dispatch index computation.
//
// Some hosts of this library may not call cudaMalloc at all: a plugin running inside an engine
// that owns the whole device heap, a real-time loop that must not take the allocator lock, a
// process whose memory budget was handed out up front.  Such callers cannot create a
// director_ctx (creation allocates the workspace).  For them the counting sort keeps its
// scratch - the launch ticket, a status word and the per-tile expert counts - in the fixed
// array below, which every device that loads the library carries until the process exits.
// ---------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticScratchInts = 262144;   // 1 MiB
constexpr int kStaticHeaderInts = 64;        // [0] launch ticket, [1] status word, rest reserved
static __device__ __align__(256) int32_t g_static_scratch[kStaticScratchInts];

constexpr int kStaticMaxDevices = 64;
int32_t* g_static_scratch_addr[kStaticMaxDevices] = {};   // device address of the array, per device

}  // namespace

extern "C" int director_dispatch_index_static(int32_t T, int32_t K, int32_t E, int32_t R, int32_t C_max,
                                              const int32_t* topk_idx, const int32_t* rep_start,
                                              const int32_t* rep_slot, int32_t* row_token, int32_t* inv_row,
                                              int32_t* dest_rank, int32_t* seg_offsets, int32_t* device_status,
                                              void* stream) {
    using namespace director;
    if (T < 1 || K < 1 || K > kMaxK || E < K || E > kMaxE || R < 1 || R > kMaxR || C_max < 1 || C_max > kMaxC)
        return DIRECTOR_ERR_INVALID_ARG;
    if ((long long)T * K >= (1ll << 31)) return DIRECTOR_ERR_INVALID_ARG;
    if (!topk_idx || !rep_start || !rep_slot || !row_token || !inv_row || !dest_rank || !seg_offsets)
        return DIRECTOR_ERR_INVALID_ARG;
    const int n_tiles = (T + kTokenTile - 1) / kTokenTile;
    if ((long long)n_tiles * E > kStaticScratchInts - kStaticHeaderInts) return DIRECTOR_ERR_STATIC_LIMIT;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DIRECTOR_ERR_CUDA;
    if (dev < 0 || dev >= kStaticMaxDevices) return DIRECTOR_ERR_UNSUPPORTED;
    if (g_static_scratch_addr[dev] == nullptr) {
        // One-time set-up on this device (the first call on a device should precede any stream capture).
        // In host code the array's name is only a handle; the kernels need its device address.
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return DIRECTOR_ERR_CUDA;
        g_static_scratch_addr[dev] = static_cast<int32_t*>(p);
    }
    int32_t* scratch = g_static_scratch_addr[dev];
    unsigned int* ticket = reinterpret_cast<unsigned int*>(scratch);
    int32_t* status = device_status ? device_status : scratch + 1;
    int32_t* tile_counts = scratch + kStaticHeaderInts;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    // The array keeps whatever the previous call left: the ticket must start at zero (the tile
    // counts are fully rewritten by the first kernel before they are read).
    if (cudaMemsetAsync(scratch, 0, kStaticHeaderInts * sizeof(int32_t), st) != cudaSuccess) return DIRECTOR_ERR_CUDA;
    const int G = R * C_max;
    count_scan_kernel<<<n_tiles, kTokenTile, 0, st>>>(topk_idx, T, E, K, G, n_tiles, rep_start, rep_slot, tile_counts,
                                                      seg_offsets, nullptr, ticket, status);
    if (cudaGetLastError() != cudaSuccess) return DIRECTOR_ERR_CUDA;
    index_kernel<<<n_tiles, kTokenTile, 0, st>>>(topk_idx, T, E, K, C_max, G, rep_start, rep_slot, tile_counts, seg_offsets,
                                                 row_token, inv_row, dest_rank, status);
    return cuda_status(cudaGetLastError());
}
