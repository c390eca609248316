// Internal definitions shared by the translation units of libdirector.so.
#pragma once

#include <cuda_runtime.h>
#include <cuda.h>
#include <stdint.h>

#include <cstring>
#include <string>
#include <vector>

#include "director.h"

namespace director {

constexpr int kTokenTile = 256;   // tokens per CTA in the count / index kernels (8 warps)
constexpr int kMaxE = 256;
constexpr int kMaxK = 8;
constexpr int kMaxR = 64;
constexpr int kMaxC = 16;
constexpr int kMaxG = kMaxR * kMaxC;
constexpr int kSmallFfnTokens = 4;      // batches of at most this many tokens take the weight-streaming FFN kernels
constexpr int kGemmClockCtas = 512;   // CTAs per GEMM launch whose records fit the clock buffer
constexpr int kGemmClockWords = 10;   // 64-bit words per CTA record, see director_gemm_counters

struct KernelEvent {
    const char* name;
    cudaEvent_t start, stop;
};

}  // namespace director

struct director_ctx {
    director_shape shape{};
    int device = 0;
    int sm_count = 0;
    int G = 0;            // R * C_max
    int n_tiles_max = 0;  // ceil(T_max / kTokenTile)

    // placement tables (device): replicas of expert e are rep_slot[rep_start[e] .. rep_start[e+1])
    bool placement_set = false;
    int32_t* d_rep_start = nullptr;    // [E+1]
    int32_t* d_rep_slot = nullptr;     // [E*R] slot id of each replica, replicas by ascending rank
    int32_t* d_slot_expert = nullptr;  // [G] expert of each slot or -1
    // Placement bank: table sets for several placements (one per layer of a model, say) that share this context's
    // workspace.  The d_* pointers above always alias the selected set; set 0 is allocated with the context.
    struct PlacementTables {
        int32_t* rep_start;
        int32_t* rep_slot;
        int32_t* slot_expert;
        unsigned long long* host_mask;
        int n_replicas;
        bool set;
    };
    std::vector<PlacementTables> bank;
    int active_placement = 0;
    unsigned long long* d_host_mask = nullptr;   // [E] bit j set iff rank j hosts the expert
    int n_replicas = 0;                // rep_start[E]: hosted (expert, rank) pairs of the current placement
    int replica_policy = 0;            // DIRECTOR_REPLICA_*: which replica an assignment uses

    // dispatch / cost workspace
    int32_t* d_tile_counts = nullptr;   // [n_tiles_max, E] per-tile expert counts -> exclusive prefix
    int32_t* d_tile_rep = nullptr;      // [n_tiles_max, G] per-tile replica counts (locality-first dispatch)
    int32_t* d_seg_offsets = nullptr;   // [G+1] internal copy (placement-cost path, host forward)
    unsigned int* d_ticket = nullptr;   // [4]: [0] last-CTA-done counter, [1..2] grid barrier of the one-launch index kernel; self-resetting
    int plan_max_tiles = 0;             // most 256-token tiles that kernel's cooperative launch can hold
    int32_t* d_status = nullptr;        // sticky device status word

    // expert FFN workspace
    void* d_hidden = nullptr;          // bf16 [T_max*K, F]   SwiGLU activations of the routed experts
    void* d_hidden_shared = nullptr;   // bf16 [T_max, S*F]
    unsigned int* d_sched = nullptr;   // [4] work-item counters of the GEMM launches of one expert_ffn call
    int32_t* d_one_seg = nullptr;      // [2] segment table {0, T} used for the shared experts
    int32_t* d_zero_expert = nullptr;  // [1] = {0}
    unsigned long long* d_gemm_clock = nullptr;   // [2][kGemmClockCtas][kGemmClockWords] per-CTA records of the last gate|up / down launch

    // buffers of the host-buffer entry points; inputs, y and the histograms exist twice so that the
    // copies of one batch overlap the kernels of its neighbours
    float* e_logits2[2] = {nullptr, nullptr};
    void* e_x2[2] = {nullptr, nullptr};
    void* e_y2[2] = {nullptr, nullptr};
    int64_t* e_cost2[2] = {nullptr, nullptr};   // workload [R,E] | rank_load [R] | dispatch_tokens [R,R] | bytes [R,R]
    cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
    cudaEvent_t ev_h2d_done[2] = {nullptr, nullptr}, ev_compute_done[2] = {nullptr, nullptr},
                ev_d2h_done[2] = {nullptr, nullptr};
    int64_t submitted = 0;
    int64_t waited[2] = {-1, -1};      // per buffer slot: newest ticket known to have reached host memory
    int32_t* e_topk_idx = nullptr;
    float* e_topk_w = nullptr;
    void* e_xp = nullptr;
    void* e_yp = nullptr;
    void* e_y_shared = nullptr;
    int32_t* e_row_token = nullptr;
    int32_t* e_inv_row = nullptr;
    int32_t* e_dest_rank = nullptr;

    int pair_clusters = 0;              // CTA pairs the device can hold at once (pair variant's grid)
    int ffn_variant = 2;                // tile scheme of the expert-FFN GEMMs, see director_set_ffn_variant
    bool ffn_small = true;              // decode-sized batches (T <= kSmallFfnTokens) use the weight-streaming kernels
    bool gemm_stats = true;             // the expert GEMMs record their own clock and per-role cycle counters
    void* encode_tiled = nullptr;       // cuTensorMapEncodeTiled, resolved through the runtime

    int64_t launches = 0;
    int profiling = 0;                  // 0 off, 1 events around every kernel, 2 events around every stage
    bool stage_open = false;            // a stage bracket is recording (stages do not nest)
    std::string profile_filter;         // when not empty, only kernels whose name contains it are timed
    std::vector<director::KernelEvent> events;
    std::vector<director::KernelEvent> free_events;
};

namespace director {

// Programmatic dependent launch.  A kernel launched through launch_chained() may be scheduled onto free SMs while the
// kernel before it in the stream is still running; chain_prologue(), the first statement of such a kernel, lets the
// kernel AFTER it do the same and then blocks until the kernel before it has completed and its writes are visible.
// Nothing of the kernel runs ahead of its predecessor: what overlaps is the launch itself (a few microseconds, which is
// a good part of what a decode-sized step consists of).  Launched the ordinary way, both instructions do nothing.
#ifdef __CUDACC__
__device__ __forceinline__ void chain_prologue() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
// Not while the stream is being captured into a CUDA graph: a replayed graph has no launch latency to hide, and its
// programmatic edges made the decode-sized steps 3-8 us slower (measured), so captured launches are ordinary ones.
inline bool chain_allowed(cudaStream_t st) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    return cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone;
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = chain_allowed(st) ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Brackets one kernel launch: counts it and, when profiling is on, records events around it.
struct LaunchScope {
    director_ctx* ctx;
    cudaStream_t stream;
    KernelEvent ev{};
    bool timed = false;
    LaunchScope(director_ctx* c, cudaStream_t s, const char* name) : ctx(c), stream(s) {
        ctx->launches++;
        if (ctx->profiling == 1 && (ctx->profile_filter.empty() || strstr(name, ctx->profile_filter.c_str()) != nullptr)) {
            if (!ctx->free_events.empty()) {
                ev = ctx->free_events.back();
                ctx->free_events.pop_back();
                timed = true;
            } else {
                timed = cudaEventCreate(&ev.start) == cudaSuccess && cudaEventCreate(&ev.stop) == cudaSuccess;
            }
            ev.name = name;
            if (timed) cudaEventRecord(ev.start, stream);
        }
    }
    ~LaunchScope() {
        if (timed) {
            cudaEventRecord(ev.stop, stream);
            ctx->events.push_back(ev);
        }
    }
};

// Brackets all launches (kernels and memsets) of one stage of the layer with ONE pair of events when stage profiling
// is on: the stage's time on an otherwise idle stream, launch gaps between its kernels included, the cost of the event
// pair paid once per stage instead of once per kernel.
struct StageScope {
    director_ctx* ctx;
    cudaStream_t stream;
    KernelEvent ev{};
    bool timed = false;
    StageScope(director_ctx* c, cudaStream_t s, const char* name) : ctx(c), stream(s) {
        if (ctx->profiling != 2 || ctx->stage_open) return;
        if (!ctx->free_events.empty()) {
            ev = ctx->free_events.back();
            ctx->free_events.pop_back();
            timed = true;
        } else {
            timed = cudaEventCreate(&ev.start) == cudaSuccess && cudaEventCreate(&ev.stop) == cudaSuccess;
        }
        ev.name = name;
        if (timed) {
            ctx->stage_open = true;
            cudaEventRecord(ev.start, stream);
        }
    }
    ~StageScope() {
        if (timed) {
            cudaEventRecord(ev.stop, stream);
            ctx->events.push_back(ev);
            ctx->stage_open = false;
        }
    }
};

inline int cuda_status(cudaError_t e) { return e == cudaSuccess ? DIRECTOR_OK : DIRECTOR_ERR_CUDA; }

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Stage launchers implemented in the individual translation units.  All validate nothing:
// the extern "C" wrappers in director_api.cu check arguments first.
int launch_route(director_ctx*, int T, const float* logits, int32_t* topk_idx, float* topk_w, cudaStream_t);
bool front_small_applies(const director_ctx*, int T);
int launch_front_small(director_ctx*, int T, const float* logits, int32_t* topk_idx, float* topk_w, int32_t* row_token,
                       int32_t* inv_row, int32_t* dest_rank, int32_t* seg_offsets, int64_t* workload, int64_t* rank_load,
                       int64_t* dispatch_tokens, uint64_t* dispatch_bytes, cudaStream_t);
int launch_dispatch(director_ctx*, int T, const void* x, const int32_t* topk_idx, const int32_t* src_rank, void* xp,
                    int32_t* row_token, int32_t* inv_row, int32_t* dest_rank, int32_t* seg_offsets, cudaStream_t);
int launch_scatter_rows(director_ctx*, int T, const void* x, const int32_t* inv_row, void* xp, cudaStream_t);
int dispatch_local_init(director_ctx*);
int dispatch_init(director_ctx*);
int launch_dispatch_local_first(director_ctx*, int T, const void* x, const int32_t* topk_idx, const int32_t* src_rank,
                                void* xp, int32_t* row_token, int32_t* inv_row, int32_t* dest_rank,
                                int32_t* seg_offsets, cudaStream_t);
int launch_cost_local_first(director_ctx*, int T, const int32_t* topk_idx, const int32_t* src_rank, int64_t* workload,
                            int64_t* rank_load, int64_t* dispatch_tokens, uint64_t* dispatch_bytes, cudaStream_t);
int launch_dedup_volume(director_ctx*, int T, const int32_t* dest_rank, const int32_t* src_rank, int64_t* dedup_tokens,
                        cudaStream_t);
int launch_cost(director_ctx*, int T, const int32_t* topk_idx, const int32_t* src_rank, int64_t* workload,
                int64_t* rank_load, int64_t* dispatch_tokens, uint64_t* dispatch_bytes, cudaStream_t);
int launch_cost_batch(director_ctx*, const int64_t* workload, int n, const uint8_t* X, int64_t* rank_load,
                      int64_t* dispatch_tokens, int64_t* summary, cudaStream_t);
// A dense SwiGLU FFN over one segment (the shared experts as one wide FFN), see ffn_pass_swap.
struct DenseFfn {
    const void* in;        // bf16 [rows, H]
    uint64_t rows;
    const void* w_gate;    // bf16 [Fw, H]
    const void* w_up;      // bf16 [Fw, H]
    const void* w_down;    // bf16 [H, Fw]
    int Fw;
    void* hidden;          // bf16 [rows, Fw]
    void* out;             // bf16 [rows, H]
};
// The combining form of the down projection (see grouped_gemm_swap_kernel, ALT): per permuted row its token and gating
// weight, and the fp32 [T, H] accumulator of y (zeroed by the caller).
struct FusedCombine {
    const int32_t* row_token;
    const float* row_weight;
    float* y_acc;
};
int launch_expert_ffn_combine(director_ctx*, int T, const void* xp, const int32_t* seg_offsets, const int32_t* row_token,
                              const int32_t* inv_row, const float* topk_w, const void* w_gate, const void* w_up,
                              const void* w_down, const void* x, const void* ws_gate, const void* ws_up,
                              const void* ws_down, float* y_acc, float* row_weight, void* y, cudaStream_t);
int launch_expert_ffn(director_ctx*, int T, const void* xp, const int32_t* row_token, const int32_t* seg_offsets,
                      const void* w_gate, const void* w_up, const void* w_down, void* yp, const void* x,
                      const void* ws_gate, const void* ws_up, const void* ws_down, void* y_shared, cudaStream_t);
bool ffn_streams_weights(const director_ctx*, int T);   // batch small enough for the weight-streaming FFN kernels
int launch_combine(director_ctx*, int T, const void* yp, const int32_t* inv_row, const float* topk_w,
                   const void* y_shared, void* y, cudaStream_t);

}  // namespace director

// Device-side sticky status: keep the first error.
__device__ __forceinline__ void director_set_status(int32_t* status, int32_t code) {
    atomicCAS(status, 0, code);
}
