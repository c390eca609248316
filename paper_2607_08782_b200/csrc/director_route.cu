// (a1) Top-k softmax gating (Section II-A): the gate scores every expert for a token, the k best are kept and
// their scores weight the sum of the experts' outputs.
//
// LPT lanes per token (1, 2, 4 or 8, chosen from E and T), no data-dependent branches on the common path.
// A lane streams every LPT-th group of eight logits of its token's row (two 16-byte loads, the next group
// prefetched; the lanes of a token read adjacent groups, so a token's loads are contiguous).
//
// Fast path, 32-bit keys: key = (top 24 bits of the order-preserving image of the float) << 8 | (255 - expert).
// A compare-exchange on such keys is one integer max and one integer min.  The lane sorts its eight keys with a
// 19-comparator network and merges them into its running top-8 (element-wise max against the reversed list
// gives a bitonic sequence holding the 8 largest; 12 more comparators sort it); for K = 8 the largest key ever
// rejected is tracked too (for K < 8 the runner-up is simply the list's entry K).  The token's lanes then merge
// their lists pairwise through shuffles.  Dropping the float's low 8 bits cannot change the answer if the K
// winners and the runner-up all differ in the 24 bits kept - then their order is the order of the exact values
// and everything else is strictly smaller.  That is checked, and the rare token that fails the check (two
// candidates within 2^-15 of each other, or real ties) is redone by one lane with exact 64-bit keys (logit image
// << 8 | 255 - expert), which order by (logit descending, expert id ascending).  Winners' exact logits are
// re-read by index for the weights.  The loop is bound by the integer pipe: ~13 integer instructions per logit.
// The weights are the softmax over the K winning logits, which equals the full softmax renormalised over the
// winners.  HBM traffic is 4E bytes in and 8K bytes out per token.
#include "director_common.cuh"

#include <algorithm>

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

typedef unsigned long long rkey;

__device__ __forceinline__ rkey make_key(uint32_t ordered, uint32_t expert) {
    return ((unsigned long long)ordered << 8) | (255u - expert);
}
__device__ __forceinline__ unsigned long long key_bits(rkey k) { return k; }
__device__ __forceinline__ rkey key_floor() { return 0ull; }   // below every real key

// compare-exchange: afterwards a >= b
__device__ __forceinline__ void cx(rkey& a, rkey& b) {
    const bool swap = b > a;
    const rkey hi = swap ? b : a, lo = swap ? a : b;
    a = hi;
    b = lo;
}

__device__ __forceinline__ void sort8_desc(rkey (&k)[8]) {
    cx(k[0], k[1]); cx(k[2], k[3]); cx(k[4], k[5]); cx(k[6], k[7]);
    cx(k[0], k[2]); cx(k[1], k[3]); cx(k[4], k[6]); cx(k[5], k[7]);
    cx(k[1], k[2]); cx(k[5], k[6]); cx(k[0], k[4]); cx(k[3], k[7]);
    cx(k[1], k[5]); cx(k[2], k[6]);
    cx(k[1], k[4]); cx(k[3], k[6]);
    cx(k[2], k[4]); cx(k[3], k[5]);
    cx(k[3], k[4]);
}

// top[] and grp[] sorted descending -> top[] = the 8 largest of the 16, sorted descending
__device__ __forceinline__ void merge_top8(rkey (&top)[8], const rkey (&grp)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) top[i] = top[i] > grp[7 - i] ? top[i] : grp[7 - i];
    cx(top[0], top[4]); cx(top[1], top[5]); cx(top[2], top[6]); cx(top[3], top[7]);
    cx(top[0], top[2]); cx(top[1], top[3]); cx(top[4], top[6]); cx(top[5], top[7]);
    cx(top[0], top[1]); cx(top[2], top[3]); cx(top[4], top[5]); cx(top[6], top[7]);
}

// ---- 32-bit fast path ----
__device__ __forceinline__ void cx32(uint32_t& a, uint32_t& b) {
    const uint32_t hi = max(a, b), lo = min(a, b);
    a = hi;
    b = lo;
}
__device__ __forceinline__ void sort8_desc32(uint32_t (&k)[8]) {
    cx32(k[0], k[1]); cx32(k[2], k[3]); cx32(k[4], k[5]); cx32(k[6], k[7]);
    cx32(k[0], k[2]); cx32(k[1], k[3]); cx32(k[4], k[6]); cx32(k[5], k[7]);
    cx32(k[1], k[2]); cx32(k[5], k[6]); cx32(k[0], k[4]); cx32(k[3], k[7]);
    cx32(k[1], k[5]); cx32(k[2], k[6]);
    cx32(k[1], k[4]); cx32(k[3], k[6]);
    cx32(k[2], k[4]); cx32(k[3], k[5]);
    cx32(k[3], k[4]);
}
// as merge_top8; with REJ the rejected keys are folded into `rej` (the largest key not in top[]), which only a
// gate that keeps all eight list entries (K = 8) needs: for K < 8 the runner-up is top[K]
template <bool REJ>
__device__ __forceinline__ void merge_top8_32(uint32_t (&top)[8], const uint32_t (&grp)[8], uint32_t& rej) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        if (REJ) rej = max(rej, min(top[i], grp[7 - i]));
        top[i] = max(top[i], grp[7 - i]);
    }
    cx32(top[0], top[4]); cx32(top[1], top[5]); cx32(top[2], top[6]); cx32(top[3], top[7]);
    cx32(top[0], top[2]); cx32(top[1], top[3]); cx32(top[4], top[6]); cx32(top[5], top[7]);
    cx32(top[0], top[1]); cx32(top[2], top[3]); cx32(top[4], top[5]); cx32(top[6], top[7]);
}

// Exact top-8 of a whole row by one thread with 64-bit keys (the fallback of the fast path).
__device__ __noinline__ void exact_top8(const float* __restrict__ row, int E, rkey (&top)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) top[i] = key_floor();
    for (int e0 = 0; e0 < E; e0 += 8) {
        rkey grp[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const bool real = e0 + i < E;
            const float v = real ? __ldg(row + e0 + i) : 0.0f;
            const uint32_t raw = __float_as_uint(v) & 0x7FFFFFFFu;
            const uint32_t hi = raw > 0x7F800000u ? 1u : ordered_bits(v);     // NaN orders below every number
            grp[i] = real ? make_key(hi, (uint32_t)(e0 + i)) : key_floor();
        }
        sort8_desc(grp);
        merge_top8(top, grp);
    }
}

// The gate of one token, computed by LPT adjacent lanes (sub = 0 .. LPT-1) that all call this together.
// Returns true in the lane that holds the result (sub == 0): win_idx[0..K) / win_w[0..K) are the chosen experts
// in descending logit order and their renormalised softmax weights.
// VEC: the row can be read with 16-byte loads (E % 4 == 0; rows are then 16-byte aligned).  K8: K == 8.
// The loop is bound by the integer pipe (min/max/logic run at half the issue rate), so the key of a logit costs
// three integer instructions (shift, two 3-input logic ops); folding -0.0 onto +0.0 and the Inf/NaN detector
// (x * 0 is NaN exactly for Inf and NaN) are floating-point instructions that issue beside them.
// PRE > 0: the lane's (at most PRE) groups are all loaded before the first is sorted - one memory round trip instead of
// one per group - for launches too small to hide a load's latency behind other warps; PRE == 0: the loads of the
// lane's next group are in flight while the current one is sorted (fewer registers).
template <bool VEC, int LPT, bool K8, int PRE = 0>
__device__ __forceinline__ bool route_token(const float* __restrict__ row, int E, int K, int sub, bool live,
                                            int32_t* __restrict__ status, int (&win_idx)[8], float (&win_w)[8]) {
    uint32_t top[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) top[i] = 0u;        // below every real key
    uint32_t rej = 0u;                               // largest key seen that is not in top[] (K8 only)
    float nonfinite = 0.0f;                          // becomes NaN iff an Inf or NaN logit was read

    auto load_group = [&](int e0, float (&v)[8]) {
        if (VEC && e0 + 8 <= E) {
            const float4 a = __ldg(reinterpret_cast<const float4*>(row + e0));
            const float4 b = __ldg(reinterpret_cast<const float4*>(row + e0 + 4));
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = (e0 + i < E) ? __ldg(row + e0 + i) : 0.0f;
        }
    };
    // keys of one group, sorted and merged into the running top-8
    auto take_group = [&](int e0, const float (&v)[8]) {
        uint32_t grp[8];
        // low byte of the key: 255 - expert = (248 - e0) | (7 - i), e0 being a multiple of 8
        const uint32_t group_field = 248u - (uint32_t)e0;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            nonfinite = fmaf(v[i], 0.0f, nonfinite);
            const uint32_t key = (ordered_bits(v[i]) & 0xFFFFFF00u) | group_field | (uint32_t)(7 - i);
            grp[i] = key;
        }
        if (e0 + 8 > E) {                            // ragged last group: positions past the row are no candidates
#pragma unroll
            for (int i = 0; i < 8; ++i) grp[i] = (e0 + i < E) ? grp[i] : 0u;
        }
        sort8_desc32(grp);
        merge_top8_32<K8>(top, grp, rej);
    };
    if constexpr (PRE > 0) {
        float va[PRE][8];
#pragma unroll
        for (int g = 0; g < PRE; ++g)
            if (8 * (sub + g * LPT) < E) load_group(8 * (sub + g * LPT), va[g]);
#pragma unroll
        for (int g = 0; g < PRE; ++g)
            if (8 * (sub + g * LPT) < E) take_group(8 * (sub + g * LPT), va[g]);
    } else {
        float v[8], v_next[8];
        if (8 * sub < E) load_group(8 * sub, v);
        for (int e0 = 8 * sub; e0 < E; e0 += 8 * LPT) {
            const int e_next = e0 + 8 * LPT;
            if (e_next < E) load_group(e_next, v_next);
            take_group(e0, v);
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = v_next[i];
        }
    }
    // merge the lists of the token's lanes (butterfly: afterwards every lane holds the token's top 8)
#pragma unroll
    for (int step = 1; step < LPT; step <<= 1) {
        uint32_t other[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) other[i] = __shfl_xor_sync(0xFFFFFFFFu, top[i], step);
        if (K8) rej = max(rej, __shfl_xor_sync(0xFFFFFFFFu, rej, step));
        nonfinite += __shfl_xor_sync(0xFFFFFFFFu, nonfinite, step);
        merge_top8_32<K8>(top, other, rej);
    }
    if (!live || sub != 0) return false;
    if (nonfinite != nonfinite) director_set_status(status, DIRECTOR_ERR_NONFINITE);

    // the truncated keys decide exactly iff the K winners and the runner-up differ pairwise in the bits kept
    bool exact = true;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        const uint32_t next = s < 7 ? top[s + 1] : rej;
        if (s < K) exact = exact && ((top[s] >> 8) != (next >> 8));
    }
    uint32_t win_bits[8];
    if (exact) {
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            win_idx[s] = 255 - (int)(top[s] & 0xFFu);
            win_bits[s] = s < K ? ordered_bits(__ldg(row + win_idx[s])) : 0u;
        }
    } else {
        rkey top64[8];
        exact_top8(row, E, top64);
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            const unsigned long long kb = key_bits(top64[s]);
            win_bits[s] = (uint32_t)(kb >> 8);
            win_idx[s] = 255 - (int)(kb & 0xFFull);
        }
    }
    // softmax over the K winners relative to the largest
    const float l0 = bits_to_float(win_bits[0]);
    float p[8], sum = 0.0f;
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        p[s] = s < K ? expf(bits_to_float(win_bits[s]) - l0) : 0.0f;
        sum += p[s];
    }
    const float inv = 1.0f / sum;
#pragma unroll
    for (int s = 0; s < 8; ++s) win_w[s] = p[s] * inv;
    return true;
}

__device__ __forceinline__ void store_gate(int32_t* __restrict__ oi, float* __restrict__ ow, int K, const int (&win_idx)[8],
                                           const float (&win_w)[8]) {
    if (K == 8) {
        reinterpret_cast<int4*>(oi)[0] = make_int4(win_idx[0], win_idx[1], win_idx[2], win_idx[3]);
        reinterpret_cast<int4*>(oi)[1] = make_int4(win_idx[4], win_idx[5], win_idx[6], win_idx[7]);
        reinterpret_cast<float4*>(ow)[0] = make_float4(win_w[0], win_w[1], win_w[2], win_w[3]);
        reinterpret_cast<float4*>(ow)[1] = make_float4(win_w[4], win_w[5], win_w[6], win_w[7]);
    } else {
#pragma unroll
        for (int s = 0; s < 8; ++s)
            if (s < K) {
                oi[s] = win_idx[s];
                ow[s] = win_w[s];
            }
    }
}

template <bool VEC, int LPT, bool K8>
__global__ void __launch_bounds__(kRouteThreads)
route_topk_kernel(const float* __restrict__ logits, int32_t* __restrict__ topk_idx, float* __restrict__ topk_w,
                  int T, int E, int K, int32_t* __restrict__ status) {
    const int tid = blockIdx.x * kRouteThreads + threadIdx.x;
    const int t_raw = tid / LPT, sub = tid % LPT;
    const bool live = t_raw < T;
    const int t = live ? t_raw : T - 1;                // surplus lanes redo the last token (keeps shuffles full)
    int win_idx[8];
    float win_w[8];
    if (route_token<VEC, LPT, K8>(logits + (size_t)t * E, E, K, sub, live, status, win_idx, win_w))
        store_gate(topk_idx + (size_t)t * K, topk_w + (size_t)t * K, K, win_idx, win_w);
}

// ---- decode-sized batches: gate, dispatch indices and placement cost in one CTA ----
//
// For T <= 256 the whole batch is one tile of the counting sort, every stage of the front end moves a few KB and
// the five launches (route, count/scan, index, workload histogram, cost) cost more than their work.  One CTA of
// 1024 threads does them back to back: eight lanes per token compute the gate (all of a lane's logits are loaded
// before the first is sorted: with a single CTA there is nothing else to hide a load behind); then thread t < T is token t for the
// counting sort (lane bitmasks per expert, popcounts; a single tile, so the tile prefix is zero), the slot lengths
// are scanned by the block, and the histograms are accumulated per assignment in shared memory.  Same integer
// arithmetic as the separate kernels, hence the same bits.  Round-robin replica rule, block partition of the
// tokens over the source ranks.
constexpr int kFrontThreads = 1024;
constexpr int kFrontLpt = 8;                              // at most four groups of logits per lane (E <= 256)
constexpr int kFrontTokens = 256;                         // largest batch: two passes of 128 tokens through the gate
constexpr int kFrontWarps = kFrontTokens / 32;            // 8 warps of token threads

template <bool VEC, bool K8>
__global__ void __launch_bounds__(kFrontThreads)
front_small_kernel(const float* __restrict__ logits, int T, int E, int K, int R, int C_max, int G, int n_replicas,
                   const int32_t* __restrict__ rep_start, const int32_t* __restrict__ rep_slot,
                   int32_t* __restrict__ topk_idx, float* __restrict__ topk_w, int32_t* __restrict__ row_token,
                   int32_t* __restrict__ inv_row, int32_t* __restrict__ dest_rank, int32_t* __restrict__ seg_offsets_a,
                   int32_t* __restrict__ seg_offsets_b, unsigned long long* __restrict__ workload,
                   unsigned long long* __restrict__ rank_load, unsigned long long* __restrict__ dispatch_tokens,
                   unsigned long long* __restrict__ dispatch_bytes, unsigned long long bytes_per_token,
                   int32_t* __restrict__ status) {
    __shared__ uint32_t mask[kMaxE][kFrontWarps];
    __shared__ uint16_t warp_prefix[kMaxE][kFrontWarps];
    __shared__ uint8_t s_idx[kFrontTokens][kMaxK];
    __shared__ int32_t s_seg[kMaxG + 1];              // slot lengths, then their exclusive scan
    __shared__ int32_t warp_sum[kFrontThreads / 32];
    __shared__ uint32_t h_rr[kMaxR * kMaxR];          // [src][dest]
    __shared__ uint32_t h_load[kMaxR];
    __shared__ int32_t s_rep_start[kMaxE + 1];        // the placement tables, fetched while the gate runs
    __shared__ int16_t s_rep_slot[kMaxG];
    const int tid = threadIdx.x;
    const int nthr = blockDim.x;                       // a multiple of 32, at least max(G, T, 4 lanes per token of a pass)
    chain_prologue();
    for (int i = tid; i <= E; i += nthr) s_rep_start[i] = __ldg(rep_start + i);
    for (int i = tid; i < n_replicas; i += nthr) s_rep_slot[i] = (int16_t)__ldg(rep_slot + i);

    for (int i = tid; i < E * kFrontWarps; i += nthr) (&mask[0][0])[i] = 0u;
    for (int i = tid; i <= G; i += nthr) s_seg[i] = 0;
    for (int i = tid; i < R * R; i += nthr) h_rr[i] = 0u;
    for (int i = tid; i < R; i += nthr) h_load[i] = 0u;
    for (int i = tid; i < R * E; i += nthr) workload[i] = 0ull;
    for (int i = tid; i < R; i += nthr) rank_load[i] = 0ull;
    for (int i = tid; i < R * R; i += nthr) { dispatch_tokens[i] = 0ull; dispatch_bytes[i] = 0ull; }

    // ---- gate (a1) ----
    for (int t0 = 0; t0 < T; t0 += nthr / kFrontLpt) {
        const int t_raw = t0 + tid / kFrontLpt, sub = tid % kFrontLpt;
        const bool live = t_raw < T;
        const int t = live ? t_raw : T - 1;
        int win_idx[8];
        float win_w[8];
        if (route_token<VEC, kFrontLpt, K8, 4>(logits + (size_t)t * E, E, K, sub, live, status, win_idx, win_w)) {
            store_gate(topk_idx + (size_t)t * K, topk_w + (size_t)t * K, K, win_idx, win_w);
#pragma unroll
            for (int s = 0; s < 8; ++s)
                if (s < K) s_idx[t][s] = (uint8_t)win_idx[s];
        }
    }
    __syncthreads();

    // ---- counting sort of the single tile (a2 indices) ----
    const int w = tid >> 5, lane = tid & 31;
    const bool token_thread = tid < T;                 // T <= 256: thread t is token t from here on
    if (token_thread)
        for (int s = 0; s < K; ++s) atomicOr(&mask[s_idx[tid][s]][w], 1u << lane);
    __syncthreads();
    for (int e = tid; e < E; e += nthr) {
        int run = 0;
#pragma unroll
        for (int ww = 0; ww < kFrontWarps; ++ww) { warp_prefix[e][ww] = (uint16_t)run; run += __popc(mask[e][ww]); }
        const int r0 = s_rep_start[e], r_e = s_rep_start[e + 1] - r0;
        for (int q = 0; q < r_e; ++q)                   // replica q gets ceil((N_e - q) / r_e) rows
            s_seg[s_rep_slot[r0 + q]] = (run > q) ? (run - q + r_e - 1) / r_e : 0;
    }
    __syncthreads();
    // exclusive scan of the G <= 1024 slot lengths: thread g owns slot g
    {
        const int len = tid < G ? s_seg[tid] : 0;
        int incl = len;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xFFFFFFFFu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) warp_sum[w] = incl;
        __syncthreads();
        int base = incl - len;
        for (int i = 0; i < w; ++i) base += warp_sum[i];
        __syncthreads();                                // every thread has read its slot length
        if (tid < G) s_seg[tid] = base;
        if (tid == G - 1) s_seg[G] = base + len;
        __syncthreads();
        for (int g = tid; g <= G; g += nthr) {
            seg_offsets_a[g] = s_seg[g];
            if (seg_offsets_b) seg_offsets_b[g] = s_seg[g];
        }
    }

    // ---- rows (a2) and histograms (a5) per assignment ----
    if (token_thread) {
        const int t = tid;
        const int src = (int)(((long long)t * R) / T);
        for (int s = 0; s < K; ++s) {
            const int e = s_idx[t][s];
            const int n = warp_prefix[e][w] + __popc(mask[e][w] & ((1u << lane) - 1u));
            const int r0 = s_rep_start[e], r_e = s_rep_start[e + 1] - r0;
            const int slot = s_rep_slot[r0 + n % r_e];
            const int row = s_seg[slot] + n / r_e;
            const int dest = slot / C_max;
            row_token[row] = t;
            inv_row[(size_t)t * K + s] = row;
            dest_rank[(size_t)t * K + s] = dest;
            atomicAdd(&h_rr[src * R + dest], 1u);
            atomicAdd(&h_load[dest], 1u);
            atomicAdd(workload + (size_t)src * E + e, 1ull);     // zeroed above, before the first barrier
        }
    }
    __syncthreads();
    for (int i = tid; i < R * R; i += nthr) {
        const unsigned long long c = h_rr[i];
        dispatch_tokens[i] = c;
        dispatch_bytes[i] = c * bytes_per_token;
    }
    for (int i = tid; i < R; i += nthr) rank_load[i] = h_load[i];
}

}  // namespace

bool front_small_applies(const director_ctx* ctx, int T) {
    return T <= kFrontTokens && ctx->replica_policy == DIRECTOR_REPLICA_ROUND_ROBIN;
}

// Gate + dispatch indices + placement cost of a batch of at most 256 tokens in one launch.
int launch_front_small(director_ctx* ctx, int T, const float* logits, int32_t* topk_idx, float* topk_w,
                       int32_t* row_token, int32_t* inv_row, int32_t* dest_rank, int32_t* seg_offsets, int64_t* workload,
                       int64_t* rank_load, int64_t* dispatch_tokens, uint64_t* dispatch_bytes, cudaStream_t st) {
    StageScope stage(ctx, st, "stage_front_small");
    const director_shape& s = ctx->shape;
    LaunchScope scope(ctx, st, "front_small_kernel");
    // a thread per segment slot (the scan) and per token, four lanes per token in a pass of the gate; no more warps
    // than that: the kernel is a chain of barriers, and a barrier costs by the warp
    const int threads = std::min(kFrontThreads, (std::max(std::max(ctx->G, kFrontLpt * T), 128) + 31) / 32 * 32);
#define FRONT_LAUNCH(VEC, K8)                                                                                          \
    launch_chained(front_small_kernel<VEC, K8>, dim3(1), dim3(threads), 0, st,                                          \
        logits, T, (int)s.E, (int)s.K, (int)s.R, (int)s.C_max, ctx->G, ctx->n_replicas, ctx->d_rep_start, ctx->d_rep_slot, topk_idx, topk_w, \
        row_token,                                                                                                     \
        inv_row, dest_rank, seg_offsets, ctx->d_seg_offsets, reinterpret_cast<unsigned long long*>(workload),          \
        reinterpret_cast<unsigned long long*>(rank_load), reinterpret_cast<unsigned long long*>(dispatch_tokens),      \
        reinterpret_cast<unsigned long long*>(dispatch_bytes), (unsigned long long)s.H * 2ull, ctx->d_status)
    const bool vec = s.E % 4 == 0, k8 = s.K == 8;
    if (vec) { if (k8) FRONT_LAUNCH(true, true); else FRONT_LAUNCH(true, false); }
    else { if (k8) FRONT_LAUNCH(false, true); else FRONT_LAUNCH(false, false); }
#undef FRONT_LAUNCH
    return cuda_status(cudaGetLastError());
}

int launch_route(director_ctx* ctx, int T, const float* logits, int32_t* topk_idx, float* topk_w, cudaStream_t st) {
    StageScope stage(ctx, st, "stage_route");
    const int E = ctx->shape.E, K = ctx->shape.K;
    // lanes per token: splitting a token over more lanes adds merge work, so use the fewest lanes (at most one per
    // group of eight experts, at most 8) that give the GPU about 128 K threads and each lane at most four groups
    const int groups = (E + 7) / 8;
    int lpt = 1;
    while (lpt < 8 && 2 * lpt <= groups && ((long long)T * lpt < 131072 || groups > 4 * lpt)) lpt *= 2;
    if (T >= (1 << 19)) lpt = 1;   // far above the launch-latency regime a lane per token executes the fewest instructions
    const long long threads = (long long)T * lpt;
    const dim3 grid((unsigned)((threads + kRouteThreads - 1) / kRouteThreads)), block(kRouteThreads);
    LaunchScope scope(ctx, st, "route_topk_kernel");
#define ROUTE_LAUNCH(VEC, LPT)                                                                                         \
    do {                                                                                                               \
        if (K == 8) route_topk_kernel<VEC, LPT, true><<<grid, block, 0, st>>>(logits, topk_idx, topk_w, T, E, K, ctx->d_status); \
        else route_topk_kernel<VEC, LPT, false><<<grid, block, 0, st>>>(logits, topk_idx, topk_w, T, E, K, ctx->d_status);       \
    } while (0)
    const bool vec = E % 4 == 0;
    if (lpt == 8) { if (vec) ROUTE_LAUNCH(true, 8); else ROUTE_LAUNCH(false, 8); }
    else if (lpt == 4) { if (vec) ROUTE_LAUNCH(true, 4); else ROUTE_LAUNCH(false, 4); }
    else if (lpt == 2) { if (vec) ROUTE_LAUNCH(true, 2); else ROUTE_LAUNCH(false, 2); }
    else { if (vec) ROUTE_LAUNCH(true, 1); else ROUTE_LAUNCH(false, 1); }
#undef ROUTE_LAUNCH
    return cuda_status(cudaGetLastError());
}

}  // namespace director
