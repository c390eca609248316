// Weight-stationary ("swapped") CTA-pair variant of the grouped expert-FFN GEMMs (Section II-A expert
// FFNs after dispatch).
//
// Segments are ragged: their lengths follow the routing skew, so tiling the TOKEN dimension in steps
// of 128 or 256 rows (the M of the tensor-core instruction) pads every segment tail with rows that are
// computed and thrown away (9-27 % extra work on the paper-shaped workloads).  Here the roles are
// swapped: the weight rows are the M operand (always full: 128 rows per CTA, 256 per CTA pair) and the
// tokens are the N operand, whose size is a runtime field of the instruction descriptor in steps of 32.
// A segment tail then costs only its length rounded up to 32 tokens.
//
//   D[weight row, token] = sum_k W[weight row, k] * X[token, k]        (both operands K-major)
//
// CTA pair, tcgen05.mma cta_group::2, M = 256, N = tokens in the tile (32..256):
//   CTA r supplies 128 weight rows (A) and half of the tile's tokens (B rows [r*N/2, (r+1)*N/2)).
//   GEMM-1: CTA r's weight rows are 64 gate rows INTERLEAVED with the matching 64 up rows (a 3-D TMA box
//           over {k, gate|up, f} builds the interleave on the fly from the two separate weight arrays), so
//           TMEM lane 2j holds gate_f and lane 2j+1 holds up_f: SwiGLU is a lane-pair shuffle.
//   GEMM-2: CTA r's weight rows are 128 consecutive rows of W_down.
// The accumulator is [weight rows x tokens]; the epilogue writes it transposed (2-byte stores, one
// token per instruction, 32-64 contiguous bytes per warp) into the row-major [tokens, features] outputs.
// Barrier protocol, bounded waits and teardown are those of the plain CTA-pair kernel.
//
// Roles: warp 0 of both CTAs loads operands (TMA), warp 1 of the leader CTA issues the MMAs, lane 0 of warp 2 of the
// leader claims work items, the remaining warps drain accumulators.  The producer and the MMA warp run their loops
// as WHOLE warps in lock step, with one lead lane polling the barriers and issuing: loop state stays warp-uniform,
// which keeps the issue cost of a k-step well under the 512 cycles a full tile occupies the tensor pipe, so that a
// ragged tile (fewer tokens, shorter MMAs) really takes less time than a full one.
#include "director_common.cuh"
#include "director_umma.cuh"

#include <cuda_bf16.h>

namespace director {

using namespace umma;

namespace {

constexpr int S_HEADER_BYTES = 384;                            // barriers, scheduler ring, TMEM slot, scratch (ring of <= 8 stages)
constexpr int S_MAX_SMEM = 232448;                             // opt-in shared memory per CTA on sm_100
// Two shapes of the operand ring.  The ordinary one: stages of 16 KB weights + 16 KB tokens (128 token rows per CTA,
// tiles of up to 256 tokens), six or seven of them.  The small-batch one (more than eight stages): the token box
// shrinks to 32 rows per CTA (tiles of up to 64 tokens), a stage to 20 KB, and ten stages fit - with a batch of at
// most 64 tokens no segment is longer than that, the weights are streamed from HBM once, and what the launch needs
// is weight bytes in flight, not token rows it does not have.
constexpr int S_SMALL_STAGES = 10;
constexpr int swap_tok_rows(int stages) { return stages > 8 ? 32 : 128; }          // token rows per CTA in a stage
constexpr int swap_stage_bytes(int stages) { return A_BYTES + swap_tok_rows(stages) * 128; }
constexpr int swap_bar_slots(int stages) { return stages > 8 ? 16 : 8; }           // capacity of the full / empty barrier arrays
constexpr int swap_header_bytes(int stages) { return S_HEADER_BYTES + (swap_bar_slots(stages) - 8) * 16; }
// Shared memory of a launch: alignment slack, the operand ring, the header, and the segment tables of its G slots
// (segment starts, work-item prefix as int32, expert ids as int16; segment ends as int32 when the segments are
// walked in expert order rather than slot order).
constexpr int swap_smem_bytes(int stages, int G, bool ordered = false) {
    return 1024 + stages * swap_stage_bytes(stages) + swap_header_bytes(stages) + (G + 1) * (ordered ? 14 : 10) + 6;
}
// The operand stream is latency-bound (a stage comes back ~2.5 us after it is released), so the ring is as deep as
// shared memory allows: seven stages when the segment tables are small enough, else six.
inline int swap_stages(int G, bool ordered = false) { return swap_smem_bytes(7, G, ordered) <= S_MAX_SMEM ? 7 : 6; }
// Walking the segments in expert order costs four more bytes of shared memory per segment; it is done when that
// does not cost the ring its seventh stage.
inline bool swap_can_order(int G) { return swap_stages(G, true) == swap_stages(G, false); }
static_assert(swap_smem_bytes(6, kMaxG, true) <= S_MAX_SMEM, "six stages do not fit with the largest segment table");
static_assert(swap_smem_bytes(S_SMALL_STAGES, kMaxG, true) <= S_MAX_SMEM, "the small-batch ring does not fit with the largest segment table");
constexpr int TOKEN_TILE = 256;                                // tokens per full tile (N of the pair's MMA); accumulator buffers are this many TMEM columns apart
constexpr int TOKEN_STEP = 32;                                 // granularity of N
// Epilogue warps per TMEM lane quadrant.  The SwiGLU epilogue of GEMM-1 is long (shuffle, exp, reciprocal,
// convert and a 2-byte store per element) and a lone warp per scheduler cannot hide its own latencies, so it
// gets two warps per quadrant, each taking every other 32-token chunk.  GEMM-2's epilogue is a plain convert
// and store; one warp per quadrant with a large register budget (all 32 stores of a chunk in flight) is faster.
constexpr int EPI_GROUPS_GEMM1 = 2;
constexpr int EPI_GROUPS_GEMM2 = 1;

// kind::f16 descriptor for the pair without the N field: D=f32, A=B=bf16, K-major, M=256.
// One lane of a converged warp (the same lane every time).
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xFFFFFFFF;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}
// Bounded barrier wait for a loop that a whole warp runs in lock step.  The spin, the poll of the CTA's abort flag
// and the time limit sit inside one block of PTX, so the code around the call has no data-dependent branch: loop
// counters, shared-memory addresses and matrix descriptors stay warp-uniform, and the instructions that want them in
// uniform registers (tcgen05.mma, tcgen05.commit, the TMA loads) get them without a move per operand.  With one
// thread running such a loop inside `if (lane == 0)`, issuing a k-step took ~510 cycles whatever the tile's width - as
// long as the tensor pipe needs for a FULL tile, so that a ragged tile cost as much as a full one.
// Only the lane with `polls` != 0 waits (31 more lanes polling the same barrier add nothing but power); the others fall
// through and meet it at the warp's next converging instruction.  `bad` != 0 skips the wait (an earlier wait of this
// lane expired: the loop runs out without waiting or issuing); returns the new `bad`.  An expiry raises the CTA's
// abort flag.
__device__ __forceinline__ uint32_t mbar_wait_conv(uint32_t bar, uint32_t parity, uint32_t abort_addr, uint32_t bad,
                                                   uint32_t polls) {
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        ".reg .u64 t0, t1;\n\t"
        ".reg .u32 ab, n;\n\t"
        "setp.ne.u32 q, %0, 0;\n\t"
        "@q bra DONE;\n\t"
        "setp.eq.u32 q, %5, 0;\n\t"
        "@q bra DONE;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "@p bra DONE;\n\t"
        "mov.u64 t0, %globaltimer;\n\t"
        "mov.u32 n, 0;\n\t"
        "SPIN:\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "@p bra DONE;\n\t"
        "add.u32 n, n, 1;\n\t"
        "and.b32 ab, n, 63;\n\t"
        "setp.ne.u32 q, ab, 0;\n\t"
        "@q bra SPIN;\n\t"                       // flag and clock are looked at once in 64 polls
        "ld.volatile.shared.u32 ab, [%3];\n\t"
        "setp.ne.u32 q, ab, 0;\n\t"
        "@q bra FAIL;\n\t"
        "mov.u64 t1, %globaltimer;\n\t"
        "sub.u64 t1, t1, t0;\n\t"
        "setp.lt.u64 q, t1, %4;\n\t"
        "@q bra SPIN;\n\t"
        "FAIL:\n\t"
        "mov.u32 ab, 1;\n\t"
        "st.volatile.shared.u32 [%3], ab;\n\t"
        "mov.u32 %0, 1;\n\t"
        "DONE:\n\t"
        "}"
        : "+r"(bad) : "r"(bar), "r"(parity), "r"(abort_addr), "l"(WAIT_LIMIT_NS), "r"(polls) : "memory");
    return bad;
}

constexpr uint32_t S_IDESC_BASE = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 4) << 24);

__device__ __forceinline__ void umma_pair_n(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t cluster_bar, int x, int y,
                                                 int z) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(cluster_bar), "r"(x), "r"(y), "r"(z) : "memory");
}

__device__ __forceinline__ void st_cluster_v4(uint32_t cluster_addr, int4 v) {
    asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}
// remote arrive that publishes this thread's earlier (remote) stores to the waiting CTA
__device__ __forceinline__ void mbar_arrive_cluster_release(uint32_t cluster_bar) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_acquire_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_acquire_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_acquire_cluster(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    uint32_t n = 0;
    while (!mbar_try_acquire_cluster(bar, parity)) {
        if ((++n & 63u) == 0u) {
            if (*abort_flag) return false;
            if (global_ns() - t0 > WAIT_LIMIT_NS) { *abort_flag = 1; return false; }
        }
    }
    return true;
}

constexpr int SCHED_SLOTS = 4;      // ring through which the scheduler thread hands work items to the other roles
constexpr int CLAIM_LEAD = 32;     // k-steps of claimed work the scheduler keeps ahead of its CTA's producer

struct SwapParams {
    const int32_t* seg_offsets;
    const int32_t* slot_expert;
    // Optional: the order in which the segments are walked, [G] slot ids sorted by (expert, slot), unused slots last.
    // Replica segments of one expert then follow each other in the work-item order and share every weight block, so
    // the second replica finds the expert's weights in L2 instead of streaming them from HBM again.  nullptr: slot order.
    const int32_t* slot_order;
    int G;
    int w_blocks;              // weight-row blocks per expert (128 f per pair in GEMM-1, 256 h in GEMM-2)
    int k_steps;
    int w_rows_per_expert;     // F (GEMM-1, in units of f) or H (GEMM-2)
    int out_pitch;             // bf16 elements per output row
    int gate_first;            // GEMM-1: 1 if even lanes hold gate rows, 0 if they hold up rows
    void* out;
    int32_t* status;
    unsigned int* counter;     // next unclaimed work item of this launch (zero when the kernel starts)
    const int32_t* row_token;  // GATHER / combining epilogue: token of every permuted row
    const float* row_weight;   // combining epilogue only: gating weight of every permuted row
    // Optional second problem of the same launch: one dense segment of `dense_rows` rows against a single weight
    // set (the shared experts run as one wide FFN over all tokens).  Its items follow the grouped problem's in the
    // work-item order, so the two share the launch, its prologue and its tail.  dense_rows == 0: absent.
    int dense_rows;
    int dense_w_blocks;
    int dense_k_steps;
    int dense_out_pitch;
    int dense_gate_first;
    void* dense_out;
    // Optional: every CTA writes a record of kGemmClockWords 64-bit words about itself (see director_gemm_counters):
    // SM cycles and nanoseconds spent in the kernel (clock64 and the global timer read by one thread at both ends:
    // cycles / ns is the SM clock the kernel really ran at, which a host-side sampler with millisecond resolution
    // cannot see), and where the MMA-issuing thread and one epilogue warp spent their cycles.  nullptr: nothing is read.
    unsigned long long* clock_out;
};

struct SwapTile {
    int prob;      // 0: grouped problem, 1: dense problem
    int row0;      // first token row of the tile
    int valid;     // tokens of the tile that belong to the segment (1..256)
    int n;         // valid rounded up to a multiple of 32: N of the MMA
    int w_row;     // first weight row of the pair's block (f index for GEMM-1, W_down row for GEMM-2)
    int wb;
    int tail;      // 1: the tile follows full tiles of its segment (its ragged end), 0: the segment's first tile
};

// Work items in their hand-out order.  Consecutive segments of the walk that hold the same expert (the replicas of
// an expert, adjacent when the segments are walked in expert order) form a group, and the items of a group are
// ordered weight block first: for every weight block, the token tiles of all the group's segments.  The clusters
// that run together therefore work on one weight block of one expert, whichever replica the tokens belong to, and
// every weight tile is fetched from HBM once per step, not once per replica.
struct SwapWalker {
    const int32_t* seg_off;     // first row of the i-th segment of the walk
    const int32_t* seg_end;     // one past its last row
    const int32_t* tt_start;    // prefix of token tiles per segment
    const int16_t* expert;
    int w_blocks, w_rows_per_expert, rows_per_block, total, G;
    int tile_rows;              // tokens per full tile
    bool grouped;               // false: every segment is its own group (the walk is in slot order)
    int gs = 0, ge = 0;         // current group: segments [gs, ge) of the walk
    __device__ bool get(int w, SwapTile& t) {
        if (w >= total) return false;
        int g, nt, local;
        if (!grouped) {
            // one segment per group: the short form of the search below (decoding an item is on the scheduler
            // thread's critical path when items are short, as in the down projection of a small batch)
            g = gs;
            while (w >= tt_start[g + 1] * w_blocks) ++g;
            gs = g;
            nt = tt_start[g + 1] - tt_start[g];
            local = w - tt_start[g] * w_blocks;
            t.wb = local / nt;
            local -= t.wb * nt;
        } else {
            while (w >= tt_start[ge] * w_blocks) {          // w only grows: groups are entered in order
                gs = ge;
                ge = gs + 1;
                while (ge < G && expert[ge] == expert[gs]) ++ge;
            }
            nt = tt_start[ge] - tt_start[gs];               // token tiles of the group
            local = w - tt_start[gs] * w_blocks;
            t.wb = local / nt;
            local -= t.wb * nt;                             // tile inside the group
            g = gs;
            while (tt_start[g + 1] - tt_start[gs] <= local) ++g;   // its segment
            local -= tt_start[g] - tt_start[gs];
        }
        t.prob = 0;
        t.tail = local > 0 ? 1 : 0;
        t.row0 = seg_off[g] + local * tile_rows;
        t.valid = min(tile_rows, seg_end[g] - t.row0);
        t.n = (t.valid + TOKEN_STEP - 1) / TOKEN_STEP * TOKEN_STEP;
        t.w_row = expert[g] * w_rows_per_expert + t.wb * rows_per_block;
        return true;
    }
};

// MODE 0: gate/up + SwiGLU (A from the 3-D interleaving map).  MODE 1: down projection (A from a 2-D map).
// ALT selects the alternative form of a launch.  GEMM-2 (MODE 1): the combining epilogue - instead of storing the
// bf16 rows of Yp, every accumulator element is multiplied by its row's gating weight and added (red.global.add.f32)
// into an fp32 [tokens, H] accumulator of y at its row's token, so the un-permute / combine step shrinks to one
// rounding pass.  The K contributions of a token arrive in no fixed order: results are reproducible to fp32
// rounding only, which is why this form is opt-in.  The dense problem (shared experts) stores bf16 as usual.
// GEMM-1 (MODE 0), GATHER: the token rows are not read from a permuted copy but gathered straight from the layer
// input x through row_token - tm_x then describes x with a one-row box and the whole producer warp issues the
// loads, four rows per lane - so the dispatch step needs no row copies at all.
template <int MODE, int EPI_GROUPS, bool ALT, int S_STAGES>
__global__ void __launch_bounds__(96 + 128 * EPI_GROUPS, 1)
grouped_gemm_swap_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_x,
                         const __grid_constant__ CUtensorMap tm_w2 /* dense problem */,
                         const __grid_constant__ CUtensorMap tm_x2, const SwapParams p) {
    constexpr bool GATHER = ALT && MODE == 0;               // token rows gathered from x
    constexpr bool COMBINE = ALT && MODE == 1;              // combining epilogue
    extern __shared__ uint8_t smem_raw[];
    chain_prologue();
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;
    constexpr int STAGE_BYTES = swap_stage_bytes(S_STAGES);        // weights + this CTA's token rows of one k-step
    constexpr int TILE_ROWS = 2 * swap_tok_rows(S_STAGES);         // tokens per full tile
    constexpr int BAR_SLOTS = swap_bar_slots(S_STAGES);
    constexpr int HEADER_BYTES = swap_header_bytes(S_STAGES);
    constexpr int HX = (BAR_SLOTS - 8) * 16;                       // what the larger barrier arrays shift the rest of the header by
    uint8_t* gen = smem_raw + (tiles - raw) + S_STAGES * STAGE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(gen);             // full[BAR_SLOTS] empty[BAR_SLOTS] tfull[2] tempty[2]
    // sched_full[4] at +160, sched_empty[4] at +192 (sched_empty: the scheduler CTA's are the ones used)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(gen + HX + 224);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + HX + 228);
    int4* sched_item = reinterpret_cast<int4*>(gen + HX + 304);    // [4] decoded work items {row0, valid, w_row, wb}
    int32_t* warp_sum = reinterpret_cast<int32_t*>(gen + HX + 248);     // [11]
    volatile int* prod_k = reinterpret_cast<volatile int*>(gen + HX + 292);  // k-steps the scheduler CTA's producer has issued so far
    const int G = p.G;
    int32_t* s_seg = reinterpret_cast<int32_t*>(gen + HEADER_BYTES);
    int32_t* s_tt = s_seg + (G + 1);
    int16_t* s_exp = reinterpret_cast<int16_t*>(s_tt + (G + 1));
    // in slot order a segment ends where the next one starts; in expert order the ends are a table of their own
    const bool ordered = p.slot_order != nullptr;
    int32_t* s_hi = reinterpret_cast<int32_t*>(gen + HEADER_BYTES + (((G + 1) * 10 + 3) & ~3));   // 4-byte aligned, behind s_exp
    const int32_t* s_end = ordered ? s_hi : s_seg + 1;

    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * BAR_SLOTS + 8u * s; };
    auto tfull_bar = [&](int a) { return bar0 + HX + 128u + 8u * a; };
    auto tempty_bar = [&](int a) { return bar0 + HX + 144u + 8u * a; };
    auto sched_full = [&](int q) { return bar0 + HX + 160u + 8u * q; };
    auto sched_empty = [&](int q) { return bar0 + HX + 192u + 8u * q; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    // optional self-measurement (see SwapParams::clock_out): nothing is read unless a record is asked for
    const bool stats = p.clock_out != nullptr;
    uint32_t stat_a = 0, stat_b = 0, stat_c = 0, stat_d = 0;       // 32-bit cycle sums: enough for two seconds
    unsigned long long* const t_start = reinterpret_cast<unsigned long long*>(gen + HX + 232);   // {clock64, ns} at the start
    if (stats && threadIdx.x == 0) { t_start[0] = (unsigned long long)clock64(); t_start[1] = global_ns(); }

    constexpr int n_threads = 96 + 128 * EPI_GROUPS;               // producer, MMA and scheduler warps + epilogue warps
    if (ordered) {
        for (int i = threadIdx.x; i < G; i += n_threads) {
            const int g = __ldg(p.slot_order + i);
            s_seg[i] = __ldg(p.seg_offsets + g);
            s_hi[i] = __ldg(p.seg_offsets + g + 1);
            s_exp[i] = (int16_t)__ldg(p.slot_expert + g);
        }
    } else {
        for (int g = threadIdx.x; g <= G; g += n_threads) s_seg[g] = __ldg(p.seg_offsets + g);
        for (int g = threadIdx.x; g < G; g += n_threads) s_exp[g] = (int16_t)__ldg(p.slot_expert + g);
    }
    if (threadIdx.x == 0) {
        *abort_flag = 0;
        *prod_k = 0;
        for (int s = 0; s < S_STAGES; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 8 * EPI_GROUPS); }
        // a slot is free again once every reader has read it: MMA thread, both producers, all epilogue warps
        for (int q = 0; q < SCHED_SLOTS; ++q) { mbar_init(sched_full(q), 1); mbar_init(sched_empty(q), 3 + 8 * EPI_GROUPS); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    {
        auto tiles_of = [&](int g) {
            const int len = s_end[g] - s_seg[g];
            return (s_exp[g] >= 0 && len > 0) ? (len + TILE_ROWS - 1) / TILE_ROWS : 0;
        };
        const int per = (G + n_threads - 1) / n_threads;
        const int lo = min((int)threadIdx.x * per, G), hi = min(lo + per, G);
        int local = 0;
        for (int g = lo; g < hi; ++g) local += tiles_of(g);
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
        for (int g = lo; g < hi; ++g) { s_tt[g] = base; base += tiles_of(g); }
        if (threadIdx.x == n_threads - 1) s_tt[G] = base;
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    constexpr int ROWS_PER_BLOCK = (MODE == 0) ? 128 : 256;   // weight rows (f or h) per pair block
    SwapWalker walker{s_seg, s_end, s_tt, s_exp, p.w_blocks, p.w_rows_per_expert, ROWS_PER_BLOCK, s_tt[G] * p.w_blocks, G, TILE_ROWS, ordered};
    SwapTile t;

    // Work items (segment, weight block, token tile) are handed out dynamically, in their natural order, from a
    // global counter.  A scheduler thread - lane 0 of a warp of its own in the leader CTA, next to the MMA warp that
    // reads its ring most urgently - claims items and publishes them through a small ring in both CTAs' shared
    // memory, already decoded into tile coordinates; every other role (both producers, the MMA warp, all epilogue
    // warps) reads the ring.  Claiming and publishing take ~2000 cycles per item (a global atomic, a remote
    // store and a remote arrive with cluster-scope release); on a thread of its own that latency is off the load
    // path.  Tail tiles are cheaper than full ones, so fixed assignments leave 6-15 % of imbalance between clusters;
    // and since the items are still taken in order, clusters running at the same time keep working on neighbouring
    // items and share their weight tiles in L2.
    const int dense_tiles = (p.dense_rows + TILE_ROWS - 1) / TILE_ROWS;
    const int total_items = walker.total + dense_tiles * p.dense_w_blocks;
    constexpr uint32_t SCHED_RANK = 0;                             // CTA of the pair that owns the ring's barriers
    const bool sched_local = rank == SCHED_RANK;
    // consumer side of the ring: wait for item i, read it, hand the slot back
    // (valid == 0 marks the item past the end)
    auto take_item = [&](int i, SwapTile& tile) -> bool {
        const int q = i & (SCHED_SLOTS - 1);
        const uint32_t par = ((uint32_t)i / SCHED_SLOTS) & 1u;
        const bool ok = sched_local ? mbar_wait(sched_full(q), par, abort_flag)
                                    : mbar_wait_acquire_cluster(sched_full(q), par, abort_flag);
        if (ok) {
            const int4 v = sched_item[q];
            tile.row0 = v.x;
            tile.valid = v.y;
            tile.n = (v.y + TOKEN_STEP - 1) / TOKEN_STEP * TOKEN_STEP;
            tile.w_row = v.z;
            tile.wb = v.w & 0x1FFFFFFF;
            tile.tail = (v.w >> 29) & 1;
            tile.prob = (v.w >> 30) & 1;
        }
        return ok;
    };
    auto release_item = [&](int i) {
        const int q = i & (SCHED_SLOTS - 1);
        if (sched_local) mbar_arrive(sched_empty(q));
        else mbar_arrive_cluster(map_to_cta(sched_empty(q), SCHED_RANK));
    };
    // the same for a warp that runs its loop in lock step: every lane waits for and reads the slot; the outcome and the
    // item's fields are made warp-uniform (one lane releases the slot afterwards)
    auto take_item_warp = [&](int i, SwapTile& tile) -> bool {
        const bool ok = __all_sync(0xFFFFFFFFu, take_item(i, tile));
        tile.row0 = __shfl_sync(0xFFFFFFFFu, tile.row0, 0);
        tile.valid = __shfl_sync(0xFFFFFFFFu, tile.valid, 0);
        tile.n = __shfl_sync(0xFFFFFFFFu, tile.n, 0);
        tile.w_row = __shfl_sync(0xFFFFFFFFu, tile.w_row, 0);
        tile.wb = __shfl_sync(0xFFFFFFFFu, tile.wb, 0);
        tile.prob = __shfl_sync(0xFFFFFFFFu, tile.prob, 0);
        tile.tail = __shfl_sync(0xFFFFFFFFu, tile.tail, 0);
        return ok;
    };
    const uint32_t abort_addr = smem_u32(const_cast<const int*>(abort_flag));

    if (warp == 0 && GATHER) {
        // whole warp: lane 0 loads the weight tile, every lane gathers four token rows per k-step
        int stage = 0;
        uint32_t phase = 0;
        int ok = 1;
        for (int i = 0; ok; ++i) {
            if (lane == 0) {
                ok = take_item(i, t) ? 1 : 0;
                if (ok) release_item(i);
                if (ok && sched_local) *prod_k = (i + 1) * p.k_steps;   // counted when the item is taken
            }
            ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
            t.row0 = __shfl_sync(0xFFFFFFFFu, t.row0, 0);
            t.valid = __shfl_sync(0xFFFFFFFFu, t.valid, 0);
            t.n = __shfl_sync(0xFFFFFFFFu, t.n, 0);
            t.w_row = __shfl_sync(0xFFFFFFFFu, t.w_row, 0);
            t.wb = __shfl_sync(0xFFFFFFFFu, t.wb, 0);
            t.prob = 0;                                                 // a gathering launch has no dense problem
            if (!ok || t.valid == 0) break;
            const int half = t.n >> 1;                                  // token rows this CTA supplies (multiple of 16)
            const int x_row = t.row0 + (int)rank * half;
            const int w_row = t.w_row + (int)rank * (ROWS_PER_BLOCK / 2);
            const bool active = 4 * lane < half;
            int tok[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {                               // rows past the tile's last token repeat it
                const int row = min(x_row + 4 * lane + r, t.row0 + t.valid - 1);
                tok[r] = active ? __ldg(p.row_token + row) : 0;
            }
            const uint32_t tx = (uint32_t)(A_BYTES + half * 128);
            for (int kb = 0; kb < p.k_steps; ++kb) {
                if (lane == 0) ok = mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag) ? 1 : 0;
                ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
                if (!ok) break;
                const uint32_t leader_full = map_to_cta(full_bar(stage), 0);
                const uint32_t a_dst = tiles + stage * STAGE_BYTES;
                if (lane == 0) {
                    mbar_expect_tx_cluster(leader_full, tx);
                    tma_load_3d_pair(a_dst, &tm_w, leader_full, kb * BLOCK_K, 0, w_row);
                }
                if (active) {
#pragma unroll
                    for (int r = 0; r < 4; ++r)
                        tma_load_2d_pair(a_dst + A_BYTES + (4 * lane + r) * 128, &tm_x, leader_full, kb * BLOCK_K, tok[r]);
                }
                if (++stage == S_STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 0) {
        // Operand producer, both CTAs: the whole warp walks the items and the ring in lock step (warp-uniform loop
        // state, see mbar_wait_conv); one elected lane arms the leader's barrier and issues the two loads of a k-step.
        const uint32_t lead_lane = elect_one() ? 1u : 0u;          // polls the barriers and issues the loads
        int stage = 0, issued_k = 0;
        uint32_t phase = 0, bad = 0;
        for (int i = 0;; ++i) {
            if (!take_item_warp(i, t)) break;
            if (lane == 0) release_item(i);
            if (t.valid == 0) break;
            const int x_row = t.row0 + (int)rank * (t.n >> 1);          // this CTA's half of the tile's tokens
            const int w_row = t.w_row + (int)rank * (ROWS_PER_BLOCK / 2);
            const CUtensorMap* mw = t.prob ? &tm_w2 : &tm_w;
            const CUtensorMap* mx = t.prob ? &tm_x2 : &tm_x;
            const int k_steps = t.prob ? p.dense_k_steps : p.k_steps;
            for (int kb = 0; kb < k_steps; ++kb) {
                const uint32_t leader_full = map_to_cta(full_bar(stage), 0);
                const uint32_t a_dst = tiles + stage * STAGE_BYTES;
                bad = mbar_wait_conv(empty_bar(stage), phase ^ 1u, abort_addr, bad, lead_lane);
                ++issued_k;
                if (lead_lane && !bad) {
                    mbar_expect_tx_cluster(leader_full, STAGE_BYTES);
                    if (MODE == 0) tma_load_3d_pair(a_dst, mw, leader_full, kb * BLOCK_K, 0, w_row);
                    else tma_load_2d_pair(a_dst, mw, leader_full, kb * BLOCK_K, w_row);
                    tma_load_2d_pair(a_dst + A_BYTES, mx, leader_full, kb * BLOCK_K, x_row);
                    if (sched_local) *prod_k = issued_k;                 // the scheduler claims work against this count
                }
                if (++stage == S_STAGES) { stage = 0; phase ^= 1u; }
            }
            if (__any_sync(0xFFFFFFFFu, bad != 0u)) break;
        }
    } else if (warp == 1) {
        // MMA issuer, leader CTA: the whole warp runs the loops in lock step, one elected lane issues the four
        // MMAs of a k-step and the commit that frees the stage.
        if (leader) {
            const uint32_t lead_lane = elect_one() ? 1u : 0u;      // polls the barriers, issues the MMAs and commits
            int stage = 0;
            uint32_t phase = 0, bad = 0;
            for (int it = 0;; ++it) {
                if (!take_item_warp(it, t)) break;
                if (lane == 0) release_item(it);
                if (t.valid == 0) break;
                const int acc = it & 1;
                const uint32_t c_item = stats ? (uint32_t)clock() : 0u;
                bad = mbar_wait_conv(tempty_bar(acc), (((uint32_t)it >> 1) & 1u) ^ 1u, abort_addr, bad, lead_lane);
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * TOKEN_TILE);
                const uint32_t idesc = S_IDESC_BASE | ((uint32_t)(t.n >> 3) << 17);
                const int k_steps = t.prob ? p.dense_k_steps : p.k_steps;
                const uint32_t c_loop = stats ? (uint32_t)clock() : 0u;
                // The ragged end of a segment that also has full tiles, in a LONG contraction, is paced to a full tile's
                // speed (512 cycles per k-step).  Finishing early buys nothing there - items are few and long, the part
                // is power-limited - while a cluster that runs ahead of the clusters it shares its weight block with,
                // and then starts its next item out of step with its neighbours, stops meeting them in L2: with unpaced
                // ragged tiles a Mixtral-shaped down projection read 2.19 GB from DRAM instead of 1.59 GB, and the
                // layer step was 2.8 % slower.  Segments without a full tile (small batches) are never paced.
                const bool paced = MODE == 1 && S_STAGES <= 8 && k_steps >= 128 && t.tail && t.n < TOKEN_TILE;
                const uint32_t c_pace = (uint32_t)clock();
                stat_a += c_loop - c_item;                  // waited for the accumulator buffer
                stat_c += (uint32_t)k_steps;
                stat_d += 1;
                for (int kb = 0; kb < k_steps; ++kb) {
                    const uint32_t a_src = tiles + stage * STAGE_BYTES;
                    const uint64_t a_desc = smem_desc(a_src), b_desc = smem_desc(a_src + A_BYTES);
                    bad = mbar_wait_conv(full_bar(stage), phase, abort_addr, bad, lead_lane);
                    tc_fence_after();
                    if (lead_lane && !bad) {
                        if (paced) {                       // see `paced` above: no k-step before its full-tile slot
                            while ((uint32_t)clock() - c_pace < 512u * (uint32_t)kb) {}
                        }
#pragma unroll
                        for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
                            umma_pair_n(d_tmem, a_desc + 2u * k, b_desc + 2u * k, idesc, (kb | k) != 0 ? 1u : 0u);
                        umma_commit_both(empty_bar(stage));
                    }
                    if (++stage == S_STAGES) { stage = 0; phase ^= 1u; }
                }
                if (__any_sync(0xFFFFFFFFu, bad != 0u)) break;
                if (lead_lane) umma_commit_both(tfull_bar(acc));
                if (stats) stat_b += (uint32_t)clock() - c_loop;   // operand waits and MMA issue of the item's k loop
            }
        }
    } else if (warp == 2) {
        if (lane == 0 && rank == SCHED_RANK) {
            // scheduler: claim the next item, wait until every reader is done with the slot's previous item, write
            // the item into both CTAs' rings, signal both.  The item past the end is published once: it ends every
            // role's loop.
            int pub_k = 0;                                         // k-steps of the items published so far
            for (int i = 0;; ++i) {
                // Claimed work stays CLAIM_LEAD k-steps ahead of this CTA's producer, no more: the claim itself takes a few
                // k-steps' time, and an item claimed by a cluster that is not ready for it is imbalance at the end of the
                // kernel (with few, long items per cluster - eight of 224 k-steps each in a Mixtral-shaped down
                // projection - one item claimed too early by the cluster that finishes last costs a whole item's time).
                if (pub_k - *prod_k >= CLAIM_LEAD) {
                    const unsigned long long t0 = global_ns();
                    uint32_t n = 0;
                    bool give_up = false;
                    while (pub_k - *prod_k >= CLAIM_LEAD) {
                        __nanosleep(256);            // a k-step lasts a third of a microsecond: poll gently, this SM has an epilogue to run
                        if ((++n & 63u) == 0u && (*abort_flag || global_ns() - t0 > WAIT_LIMIT_NS)) { give_up = true; break; }
                    }
                    if (give_up) { *abort_flag = 1; break; }
                }
                const unsigned int c = atomicAdd(p.counter, 1u);
                const int w = c < (unsigned)total_items ? (int)c : total_items;
                const int q = i & (SCHED_SLOTS - 1);
                if (!mbar_wait(sched_empty(q), (((uint32_t)i / SCHED_SLOTS) & 1u) ^ 1u, abort_flag)) break;
                int4 item = make_int4(0, 0, 0, 0);
                if (w < walker.total) {
                    walker.get(w, t);
                    item = make_int4(t.row0, t.valid, t.w_row, t.wb | (t.tail << 29));
                    pub_k += p.k_steps;
                } else if (w < total_items) {          // dense problem: (weight block, token tile) over one segment
                    // Chunks of token tiles, inside a chunk weight block first, the chunk sized so that all weight
                    // blocks of its tiles are in flight together (clusters / weight blocks tiles): a token tile is then
                    // read from HBM once, by the clusters that work on it at the same k, instead of once per weight block
                    // (a dense segment's activations need not fit in L2: four Qwen1.5-shaped shared experts' hidden
                    // activations are 185 MB, and weight-block-major order read them eight times).
                    const int local = w - walker.total;
                    const int chunk = max(1, (int)(gridDim.x >> 1) / p.dense_w_blocks);
                    const int ch = local / (chunk * p.dense_w_blocks), r = local - ch * chunk * p.dense_w_blocks;
                    const int in_chunk = min(chunk, dense_tiles - ch * chunk);
                    const int wb = r / in_chunk, row0 = (ch * chunk + r - wb * in_chunk) * TILE_ROWS;
                    item = make_int4(row0, min(TILE_ROWS, p.dense_rows - row0), wb * ROWS_PER_BLOCK,
                                     wb | ((row0 > 0 ? 1 : 0) << 29) | (1 << 30));
                    pub_k += p.dense_k_steps;
                }
                sched_item[q] = item;
                st_cluster_v4(map_to_cta(smem_u32(&sched_item[q]), 1u - SCHED_RANK), item);
                mbar_arrive(sched_full(q));
                mbar_arrive_cluster_release(map_to_cta(sched_full(q), 1u - SCHED_RANK));
                if (w >= total_items) break;
            }
        }
    } else {
        const int quad = warp & 3;                                 // TMEM lane quadrant this warp may read
        const int cgroup = EPI_GROUPS == 1 ? 0 : (warp - 3) >> 2;  // which of the 32-token chunks this warp takes
        constexpr int CSTEP = 32 * EPI_GROUPS;
        const int c_first = 32 * cgroup;
        uint16_t* const out_a = static_cast<uint16_t*>(p.out);
        uint16_t* const out_b = static_cast<uint16_t*>(p.dense_out);
        const int lane_row = quad * 32 + lane;                     // weight row of this thread inside the CTA's 128
        bool ok = true;
        for (int it = 0; ok; ++it) {
            if (!(ok = take_item(it, t))) break;
            __syncwarp();
            if (lane == 0) release_item(it);
            if (t.valid == 0) break;
            const int acc = it & 1;
            const uint32_t c_wait = stats ? (uint32_t)clock() : 0u;
            if (!(ok = mbar_wait(tfull_bar(acc), ((uint32_t)it >> 1) & 1u, abort_flag))) break;
            const uint32_t c_drain = stats ? (uint32_t)clock() : 0u;
            stat_a += c_drain - c_wait;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * TOKEN_TILE);
            uint16_t* const out = t.prob ? out_b : out_a;
            const int out_pitch = t.prob ? p.dense_out_pitch : p.out_pitch;
            if constexpr (MODE == 0) {
                // even lane: one of (gate, up) for feature f, odd lane: the other; column = token.
                // The two lanes of a pair split the tokens: the even lane finishes the even tokens, the odd lane
                // the odd ones.  One shuffle per token pair hands each lane the partner value it needs, so all
                // 32 lanes stay active and no branch separates the shuffles.
                const int f = t.wb * 128 + (int)rank * 64 + (lane_row >> 1);
                const bool odd = (lane & 1) != 0;
                const bool i_am_gate = (!odd) == ((t.prob ? p.dense_gate_first : p.gate_first) != 0);
                uint16_t* ocol = out + (size_t)(t.row0 + (odd ? 1 : 0)) * out_pitch + f;
                const size_t two_rows = 2 * (size_t)out_pitch;
#pragma unroll 1
                for (int c = c_first; c < t.n; c += CSTEP) {
                    uint32_t v[32];
                    tmem_ld32(taddr + c, v);
                    tmem_ld_wait();
                    uint16_t* ptr = ocol + (size_t)c * out_pitch;       // my token of pair m is row c + 2m (+1 if odd)
                    const int rem = t.valid - c - (odd ? 1 : 0);        // store pair m iff 2m < rem
#pragma unroll
                    for (int m = 0; m < 16; ++m) {
                        const float mine = __uint_as_float(odd ? v[2 * m + 1] : v[2 * m]);   // my value at my token
                        const float send = __uint_as_float(odd ? v[2 * m] : v[2 * m + 1]);   // my value at the partner's token
                        const float other = __shfl_xor_sync(0xFFFFFFFFu, send, 1);           // partner's value at my token
                        const float g = i_am_gate ? mine : other, u = i_am_gate ? other : mine;
                        const float h = __fdividef(g * u, 1.0f + __expf(-g));
                        if (2 * m < rem) *ptr = __bfloat16_as_ushort(__float2bfloat16_rn(h));
                        ptr += two_rows;
                    }
                }
            } else {
                const int h_col = t.wb * 256 + (int)rank * 128 + lane_row;
                if (COMBINE && !t.prob) {
                    // lane j of the warp fetches token and gating weight of the chunk's j-th row; every lane then adds
                    // its own feature of that row into the token's accumulator (32 lanes = 128 contiguous bytes)
                    float* const acc_y = static_cast<float*>(p.out) + h_col;
#pragma unroll 1
                    for (int c = c_first; c < t.n; c += CSTEP) {
                        uint32_t v[32];
                        tmem_ld32(taddr + c, v);
                        const int rem = t.valid - c;
                        const int row = t.row0 + c + lane;
                        const int tok = lane < rem ? __ldg(p.row_token + row) : 0;
                        const float wgt = lane < rem ? __ldg(p.row_weight + row) : 0.0f;
                        tmem_ld_wait();
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int tj = __shfl_sync(0xFFFFFFFFu, tok, j);
                            const float wj = __shfl_sync(0xFFFFFFFFu, wgt, j);
                            if (j < rem) atomicAdd(acc_y + (size_t)tj * out_pitch, wj * __uint_as_float(v[j]));
                        }
                    }
                } else {
                uint16_t* ocol = out + (size_t)t.row0 * out_pitch + h_col;
#pragma unroll 1
                for (int c = c_first; c < t.n; c += CSTEP) {
                    uint32_t v[32];
                    tmem_ld32(taddr + c, v);
                    tmem_ld_wait();
                    uint16_t* ptr = ocol + (size_t)c * out_pitch;
                    const int rem = t.valid - c;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (j < rem) *ptr = __bfloat16_as_ushort(__float2bfloat16_rn(__uint_as_float(v[j])));
                        ptr += out_pitch;
                    }
                }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));
            if (stats) stat_b += (uint32_t)clock() - c_drain;
            stat_c += 1;
        }
    }

    // A role that gave up (an expired wait) tells the peer CTA of the pair, whose roles poll their own flag inside
    // their waits: both CTAs then drain within microseconds and meet at the closing cluster barrier, instead of the
    // peer running out its own two seconds.  (The peer is still resident: it cannot pass that barrier without us.)
    if (*abort_flag)
        asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(map_to_cta(smem_u32(const_cast<const int*>(abort_flag)), 1u - rank)),
                     "r"(1) : "memory");
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (threadIdx.x == 0 && *abort_flag) director_set_status(p.status, DIRECTOR_ERR_TIMEOUT);
    if (stats && blockIdx.x < (unsigned)kGemmClockCtas) {
        unsigned long long* const rec = p.clock_out + (size_t)blockIdx.x * kGemmClockWords;
        if (threadIdx.x == 0) {
            rec[0] = (unsigned long long)clock64() - t_start[0];
            rec[1] = global_ns() - t_start[1];
            rec[9] = 0ull;
        }
        if (threadIdx.x == 32) {                            // the MMA-issuing thread (idle in the peer CTA: zeros)
            rec[2] = (unsigned long long)stat_a;
            rec[3] = (unsigned long long)stat_b;
            rec[4] = (unsigned long long)stat_c;
            rec[5] = (unsigned long long)stat_d;
        }
        if (threadIdx.x == 96) {                            // lane 0 of the first epilogue warp
            rec[6] = (unsigned long long)stat_a;
            rec[7] = (unsigned long long)stat_b;
            rec[8] = (unsigned long long)stat_c;
        }
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 [rows, cols] row-major, box 64 x box_rows, 128-byte swizzle
bool map_2d(director_ctx* ctx, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows = 128) {
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {BLOCK_K, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
               map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Two bf16 [rows, cols] matrices `first` and `first + delta` seen as one tensor {cols, 2, rows}; a box of
// {64, 2, 64} lands in shared memory as 128 rows alternating between the two matrices.
bool map_interleaved(director_ctx* ctx, CUtensorMap* map, const void* first, uint64_t delta_bytes, uint64_t rows,
                     uint64_t cols) {
    const cuuint64_t dims[3] = {cols, 2, rows};
    const cuuint64_t strides[2] = {delta_bytes, cols * 2};
    const cuuint32_t box[3] = {BLOCK_K, 2, 64};
    const cuuint32_t estr[3] = {1, 1, 1};
    return reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
               map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(first), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int MODE, int EPI_GROUPS, bool GATHER, int STAGES>
int launch_swap_n(director_ctx* ctx, const char* name, const CUtensorMap& w, const CUtensorMap& x, const CUtensorMap& w2,
                  const CUtensorMap& x2, const SwapParams& p, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * ctx->pair_clusters));
    cfg.blockDim = dim3(96 + 128 * EPI_GROUPS);
    cfg.dynamicSmemBytes = (size_t)swap_smem_bytes(STAGES, p.G, p.slot_order != nullptr);
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;    // see chain_prologue()
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = chain_allowed(st) ? 2 : 1;
    LaunchScope scope(ctx, st, name);
    return cuda_status(cudaLaunchKernelEx(&cfg, grouped_gemm_swap_kernel<MODE, EPI_GROUPS, GATHER, STAGES>, w, x, w2, x2, p));
}

// w2 / x2: the dense problem's maps (any valid map when the launch has none)
template <int MODE, int EPI_GROUPS, bool GATHER>
int launch_swap(director_ctx* ctx, const char* name, const CUtensorMap& w, const CUtensorMap& x, const CUtensorMap& w2,
                const CUtensorMap& x2, const SwapParams& p, bool small, cudaStream_t st) {
    if constexpr (!GATHER) {
        if (small) return launch_swap_n<MODE, EPI_GROUPS, GATHER, S_SMALL_STAGES>(ctx, name, w, x, w2, x2, p, st);
    }
    return swap_stages(p.G, p.slot_order != nullptr) == 7 ? launch_swap_n<MODE, EPI_GROUPS, GATHER, 7>(ctx, name, w, x, w2, x2, p, st)
                                 : launch_swap_n<MODE, EPI_GROUPS, GATHER, 6>(ctx, name, w, x, w2, x2, p, st);
}

template <int MODE, int EPI_GROUPS, bool GATHER>
bool swap_opt_in() {
    if constexpr (!GATHER) {
        if (cudaFuncSetAttribute(grouped_gemm_swap_kernel<MODE, EPI_GROUPS, GATHER, S_SMALL_STAGES>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 swap_smem_bytes(S_SMALL_STAGES, kMaxG, true)) != cudaSuccess)
            return false;
    }
    return cudaFuncSetAttribute(grouped_gemm_swap_kernel<MODE, EPI_GROUPS, GATHER, 6>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize, swap_smem_bytes(6, kMaxG, true)) == cudaSuccess &&
           cudaFuncSetAttribute(grouped_gemm_swap_kernel<MODE, EPI_GROUPS, GATHER, 7>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize, S_MAX_SMEM) == cudaSuccess;
}

}  // namespace

int ffn_swap_init(director_ctx*) {
    if (!swap_opt_in<0, EPI_GROUPS_GEMM1, false>() || !swap_opt_in<0, EPI_GROUPS_GEMM1, true>() ||
        !swap_opt_in<1, EPI_GROUPS_GEMM2, false>() || !swap_opt_in<1, EPI_GROUPS_GEMM2, true>())
        return DIRECTOR_ERR_CUDA;
    return DIRECTOR_OK;
}

// in [rows, H] -> hidden [rows, Fw] -> out [rows, H] over a segment table, weight-stationary pair kernels.
// With gather_rows != nullptr, `in` is the un-permuted layer input [in_rows, H] and row i of the segment table
// is in[gather_rows[i]].
// dense (optional, not with gather_rows): a second FFN over ONE segment of dense->rows rows of dense->in with a single
// weight set - the shared experts - whose work items ride in the same two launches.
// max_seg_rows: an upper bound on the length of any segment of the table (`rows` if nothing better is known); with a
// bound of at most 64 the launches use the small-batch ring (see S_SMALL_STAGES) - correct for any table, since that
// ring also tiles the tokens by 64.
// fc (optional, not with gather_rows): the down projection combines in its epilogue - `out` is not written; every
// element of a routed row goes, times the row's gating weight, into fc->y_acc at the row's token (see the kernel's ALT).
// Returns DIRECTOR_ERR_UNSUPPORTED if a pair of weight arrays cannot be described by one interleaving map.
int ffn_pass_swap(director_ctx* ctx, const void* in, uint64_t in_rows, const int32_t* gather_rows, uint64_t rows,
                  const int32_t* seg_offsets, const int32_t* slot_expert, int G, const void* w_gate, const void* w_up,
                  const void* w_down, uint64_t n_experts, int Fw, void* hidden, void* out,
                  unsigned int* counters /* 2 zeroed work-item counters */, const DenseFfn* dense, uint64_t max_seg_rows,
                  const FusedCombine* fc, cudaStream_t st) {
    const int H = ctx->shape.H;
    // small-batch ring (tiles of 64 tokens, ten stages): when no segment, routed or dense, can be longer than a tile
    const bool small = !gather_rows && !fc && max_seg_rows <= 2u * swap_tok_rows(S_SMALL_STAGES) &&
                       (!dense || dense->rows <= 2u * swap_tok_rows(S_SMALL_STAGES));
    const uint32_t tok_box = small ? swap_tok_rows(S_SMALL_STAGES) : 128;
    struct Interleave { bool ok; bool gate_first; const void* first; uint64_t delta; };
    auto interleave = [](const void* g, const void* u) {
        const uintptr_t pg = reinterpret_cast<uintptr_t>(g), pu = reinterpret_cast<uintptr_t>(u);
        Interleave r{false, pg < pu, pg < pu ? g : u, pg < pu ? pu - pg : pg - pu};
        r.ok = pg != pu && r.delta % 16 == 0 && r.delta < (1ull << 40);
        return r;
    };
    const Interleave ia = interleave(w_gate, w_up);
    if (!ia.ok) return DIRECTOR_ERR_UNSUPPORTED;
    if ((dense || fc) && gather_rows) return DIRECTOR_ERR_INVALID_ARG;
    CUtensorMap m_in, m_gu, m_h, m_d;
    if (!map_2d(ctx, &m_in, in, in_rows, H, gather_rows ? 1 : tok_box) || !map_2d(ctx, &m_h, hidden, rows, Fw, tok_box) ||
        !map_2d(ctx, &m_d, w_down, n_experts * H, Fw))
        return DIRECTOR_ERR_CUDA;
    if (!map_interleaved(ctx, &m_gu, ia.first, ia.delta, n_experts * Fw, H)) return DIRECTOR_ERR_UNSUPPORTED;
    // the dense problem's maps default to the grouped problem's (never used then)
    CUtensorMap d_in = m_in, d_gu = m_gu, d_h = m_h, d_d = m_d;
    Interleave id{true, true, nullptr, 0};
    if (dense) {
        id = interleave(dense->w_gate, dense->w_up);
        if (!id.ok) return DIRECTOR_ERR_UNSUPPORTED;
        if (!map_2d(ctx, &d_in, dense->in, dense->rows, H, tok_box) ||
            !map_2d(ctx, &d_h, dense->hidden, dense->rows, dense->Fw, tok_box) ||
            !map_2d(ctx, &d_d, dense->w_down, H, dense->Fw))
            return DIRECTOR_ERR_CUDA;
        if (!map_interleaved(ctx, &d_gu, id.first, id.delta, dense->Fw, H)) return DIRECTOR_ERR_UNSUPPORTED;
    }
    const int d_rows = dense ? (int)dense->rows : 0, d_Fw = dense ? dense->Fw : 0;
    // the context's own slot table comes with its expert order (stored behind it); any other table is walked as is
    const int32_t* order = (slot_expert == ctx->d_slot_expert && G == ctx->G && swap_can_order(G)) ? slot_expert + G : nullptr;
    unsigned long long* const clk = ctx->gemm_stats ? ctx->d_gemm_clock : nullptr;
    SwapParams p1{seg_offsets, slot_expert, order, G, Fw / 128, H / BLOCK_K, Fw, Fw, ia.gate_first ? 1 : 0, hidden, ctx->d_status,
                  counters, gather_rows, nullptr, d_rows, d_Fw / 128, H / BLOCK_K, d_Fw, id.gate_first ? 1 : 0,
                  dense ? dense->hidden : nullptr, clk};
    int rc = gather_rows ? launch_swap<0, EPI_GROUPS_GEMM1, true>(ctx, "grouped_gemm_swiglu_kernel", m_gu, m_in, d_gu, d_in, p1, false, st)
                         : launch_swap<0, EPI_GROUPS_GEMM1, false>(ctx, "grouped_gemm_swiglu_kernel", m_gu, m_in, d_gu, d_in, p1, small, st);
    if (rc != DIRECTOR_OK) return rc;
    // with fc the routed experts' output is not Yp but the fp32 accumulator of y (pitch H floats), see the kernel's ALT
    SwapParams p2{seg_offsets, slot_expert, order, G, H / 256, Fw / BLOCK_K, H, H, 1, fc ? static_cast<void*>(fc->y_acc) : out,
                  ctx->d_status, counters + 1, fc ? fc->row_token : nullptr, fc ? fc->row_weight : nullptr,
                  d_rows, H / 256, d_Fw / BLOCK_K, H, 1, dense ? dense->out : nullptr,
                  clk ? clk + (size_t)kGemmClockWords * kGemmClockCtas : nullptr};
    if (fc) return launch_swap<1, EPI_GROUPS_GEMM2, true>(ctx, "grouped_gemm_down_fused_kernel", m_d, m_h, d_d, d_h, p2, false, st);
    return launch_swap<1, EPI_GROUPS_GEMM2, false>(ctx, "grouped_gemm_down_kernel", m_d, m_h, d_d, d_h, p2, small, st);
}

}  // namespace director
