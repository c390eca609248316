// C-ABI entry points of libdirector.so: argument checks, context life cycle, placement tables,
// the host-buffer convenience call and the per-kernel timing hooks.  The kernels live in the
// director_<stage>.cu files.
#include "director_common.cuh"

#include <algorithm>
#include <cstring>
#include <new>

using namespace director;

namespace director {
int ffn_init(director_ctx* ctx);   // director_ffn.cu: shared-memory opt-in for the GEMM kernels
}

namespace {

template <typename T>
bool dev_alloc(T** p, size_t count) {
    if (count == 0) count = 1;
    return cudaMalloc(reinterpret_cast<void**>(p), count * sizeof(T)) == cudaSuccess;
}

bool shape_supported(const director_shape& s) {
    if (s.T_max < 1 || s.H < 256 || s.F < 128 || s.E < 1 || s.K < 1 || s.S < 0 || s.R < 1 || s.C_max < 1) return false;
    if (s.K > kMaxK || s.K > s.E || s.E > kMaxE || s.R > kMaxR || s.C_max > kMaxC) return false;
    if ((long long)s.E > (long long)s.R * s.C_max) return false;
    if (s.H % 256 != 0 || s.F % 128 != 0) return false;
    if ((long long)s.T_max * s.K >= (1ll << 31)) return false;
    if ((long long)s.E * s.F >= (1ll << 31) || (long long)s.E * s.H >= (1ll << 31)) return false;
    return true;
}

void free_all(director_ctx* c) {
    if (c->bank.empty())        // creation failed before the bank took ownership of the first table set
        c->bank.push_back({c->d_rep_start, c->d_rep_slot, c->d_slot_expert, c->d_host_mask, 0, false});
    for (auto& t : c->bank) {
        void* tables[] = {t.rep_start, t.rep_slot, t.slot_expert, t.host_mask};
        for (void* p : tables)
            if (p) cudaFree(p);
    }
    void* ptrs[] = {c->d_tile_counts, c->d_seg_offsets, c->d_ticket, c->d_tile_rep,
                    c->d_status, c->d_hidden, c->d_hidden_shared, c->d_one_seg, c->d_sched, c->d_gemm_clock,
                    c->d_zero_expert, c->e_logits2[0], c->e_logits2[1], c->e_x2[0], c->e_x2[1], c->e_topk_idx,
                    c->e_topk_w, c->e_xp, c->e_yp, c->e_y2[0], c->e_y2[1], c->e_y_shared, c->e_row_token, c->e_inv_row,
                    c->e_dest_rank, c->e_cost2[0], c->e_cost2[1]};
    for (void* p : ptrs)
        if (p) cudaFree(p);
    for (int i = 0; i < 2; ++i) {
        if (c->ev_h2d_done[i]) cudaEventDestroy(c->ev_h2d_done[i]);
        if (c->ev_compute_done[i]) cudaEventDestroy(c->ev_compute_done[i]);
        if (c->ev_d2h_done[i]) cudaEventDestroy(c->ev_d2h_done[i]);
    }
    if (c->h2d_stream) cudaStreamDestroy(c->h2d_stream);
    if (c->d2h_stream) cudaStreamDestroy(c->d2h_stream);
    for (auto& ev : c->events) { cudaEventDestroy(ev.start); cudaEventDestroy(ev.stop); }
    for (auto& ev : c->free_events) { cudaEventDestroy(ev.start); cudaEventDestroy(ev.stop); }
}

inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }

#define REQUIRE_CTX(ctx)                              \
    do {                                              \
        if ((ctx) == nullptr) return DIRECTOR_ERR_INVALID_ARG; \
    } while (0)
#define REQUIRE_T(ctx, T)                                                   \
    do {                                                                    \
        if ((T) < 1 || (T) > (ctx)->shape.T_max) return DIRECTOR_ERR_INVALID_ARG; \
    } while (0)
#define REQUIRE_PTR(p)                                                      \
    do {                                                                    \
        if ((p) == nullptr || !aligned16(p)) return DIRECTOR_ERR_INVALID_ARG; \
    } while (0)
#define REQUIRE_PLACEMENT(ctx)                                   \
    do {                                                         \
        if (!(ctx)->placement_set) return DIRECTOR_ERR_PLACEMENT; \
    } while (0)

// a1 + a2 + a5 on device buffers: one fused launch for decode-sized batches, the separate kernels otherwise
int launch_front(director_ctx* ctx, int T, const float* logits, const void* x, int32_t* topk_idx, float* topk_w, void* xp,
                 int32_t* row_token, int32_t* inv_row, int32_t* dest_rank, int32_t* seg_offsets, int64_t* workload,
                 int64_t* rank_load, int64_t* dispatch_tokens, uint64_t* dispatch_bytes, cudaStream_t st) {
    if (front_small_applies(ctx, T)) {
        int rc = launch_front_small(ctx, T, logits, topk_idx, topk_w, row_token, inv_row, dest_rank, seg_offsets, workload,
                                    rank_load, dispatch_tokens, dispatch_bytes, st);
        if (rc == DIRECTOR_OK && xp != nullptr) rc = launch_scatter_rows(ctx, T, x, inv_row, xp, st);
        return rc;
    }
    int rc = launch_route(ctx, T, logits, topk_idx, topk_w, st);
    if (rc == DIRECTOR_OK)
        rc = launch_dispatch(ctx, T, x, topk_idx, nullptr, xp, row_token, inv_row, dest_rank, seg_offsets, st);
    if (rc == DIRECTOR_OK)
        rc = launch_cost(ctx, T, topk_idx, nullptr, workload, rank_load, dispatch_tokens, dispatch_bytes, st);
    return rc;
}

}  // namespace

extern "C" {

int director_create(const director_shape* shape, director_ctx** out) {
    if (shape == nullptr || out == nullptr) return DIRECTOR_ERR_INVALID_ARG;
    *out = nullptr;
    if (!shape_supported(*shape)) return DIRECTOR_ERR_UNSUPPORTED;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DIRECTOR_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return DIRECTOR_ERR_CUDA;
    if (prop.major != 10) return DIRECTOR_ERR_UNSUPPORTED;   // tcgen05 / TMEM kernels: sm_100 only

    director_ctx* c = new (std::nothrow) director_ctx();
    if (c == nullptr) return DIRECTOR_ERR_WORKSPACE;
    c->shape = *shape;
    c->device = dev;
    c->sm_count = prop.multiProcessorCount;
    c->G = shape->R * shape->C_max;
    c->n_tiles_max = (shape->T_max + kTokenTile - 1) / kTokenTile;
    const director_shape& s = c->shape;
    const size_t A = (size_t)s.T_max * s.K, T = (size_t)s.T_max;
    const size_t cost_words = (size_t)s.R * s.E + s.R + 2 * (size_t)s.R * s.R;

    bool ok = dev_alloc(&c->d_rep_start, s.E + 1) && dev_alloc(&c->d_rep_slot, (size_t)s.E * s.R) &&
              dev_alloc(&c->d_slot_expert, 2 * (size_t)c->G) && dev_alloc(&c->d_tile_counts, (size_t)c->n_tiles_max * s.E) &&
              dev_alloc(&c->d_seg_offsets, c->G + 1) && dev_alloc(&c->d_ticket, 4) && dev_alloc(&c->d_status, 1) &&
              dev_alloc(&c->d_host_mask, s.E) && dev_alloc(&c->d_tile_rep, (size_t)c->n_tiles_max * c->G) &&
              dev_alloc(&c->d_one_seg, 2) && dev_alloc(&c->d_sched, 4) &&
              dev_alloc(&c->d_zero_expert, 1) &&
              dev_alloc(&c->d_gemm_clock, 2 * (size_t)kGemmClockWords * kGemmClockCtas) &&
              dev_alloc(reinterpret_cast<uint16_t**>(&c->d_hidden), A * s.F) &&
              dev_alloc(reinterpret_cast<uint16_t**>(&c->d_hidden_shared), T * s.S * s.F) &&
              dev_alloc(&c->e_logits2[0], T * s.E) && dev_alloc(&c->e_logits2[1], T * s.E) &&
              dev_alloc(reinterpret_cast<uint16_t**>(&c->e_x2[0]), T * s.H) &&
              dev_alloc(reinterpret_cast<uint16_t**>(&c->e_x2[1]), T * s.H) &&
              dev_alloc(&c->e_topk_idx, A) && dev_alloc(&c->e_topk_w, A) &&
              dev_alloc(reinterpret_cast<uint16_t**>(&c->e_xp), A * s.H) &&
              dev_alloc(reinterpret_cast<uint16_t**>(&c->e_yp), A * s.H) &&
              dev_alloc(reinterpret_cast<uint16_t**>(&c->e_y2[0]), T * s.H) &&
              dev_alloc(reinterpret_cast<uint16_t**>(&c->e_y2[1]), T * s.H) &&
              dev_alloc(reinterpret_cast<uint16_t**>(&c->e_y_shared), s.S > 0 ? T * s.H : 0) &&
              dev_alloc(&c->e_row_token, A) && dev_alloc(&c->e_inv_row, A) && dev_alloc(&c->e_dest_rank, A) &&
              dev_alloc(&c->e_cost2[0], cost_words) && dev_alloc(&c->e_cost2[1], cost_words);
    if (!ok) {
        cudaGetLastError();
        free_all(c);
        delete c;
        return DIRECTOR_ERR_WORKSPACE;
    }
    c->bank.push_back({c->d_rep_start, c->d_rep_slot, c->d_slot_expert, c->d_host_mask, 0, false});
    ok = cudaMemset(c->d_ticket, 0, 4 * sizeof(unsigned int)) == cudaSuccess &&
         cudaMemset(c->d_status, 0, sizeof(int32_t)) == cudaSuccess &&
         cudaMemset(c->d_zero_expert, 0, sizeof(int32_t)) == cudaSuccess &&
         cudaMemset(c->d_gemm_clock, 0, sizeof(unsigned long long) * 2 * kGemmClockWords * kGemmClockCtas) == cudaSuccess;

    cudaDriverEntryPointQueryResult qres;
    if (ok) {
        ok = cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &c->encode_tiled, 12000, cudaEnableDefault,
                                              &qres) == cudaSuccess &&
             qres == cudaDriverEntryPointSuccess && c->encode_tiled != nullptr;
    }
    if (ok) ok = ffn_init(c) == DIRECTOR_OK && dispatch_local_init(c) == DIRECTOR_OK && dispatch_init(c) == DIRECTOR_OK;
    if (ok) {
        ok = cudaStreamCreateWithFlags(&c->h2d_stream, cudaStreamNonBlocking) == cudaSuccess &&
             cudaStreamCreateWithFlags(&c->d2h_stream, cudaStreamNonBlocking) == cudaSuccess;
        for (int i = 0; i < 2 && ok; ++i)
            ok = cudaEventCreateWithFlags(&c->ev_h2d_done[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&c->ev_compute_done[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&c->ev_d2h_done[i], cudaEventDisableTiming) == cudaSuccess;
    }
    if (!ok) {
        cudaGetLastError();
        free_all(c);
        delete c;
        return DIRECTOR_ERR_CUDA;
    }
    *out = c;
    return DIRECTOR_OK;
}

int director_destroy(director_ctx* ctx) {
    REQUIRE_CTX(ctx);
    cudaSetDevice(ctx->device);
    cudaDeviceSynchronize();
    free_all(ctx);
    delete ctx;
    return DIRECTOR_OK;
}

int director_set_placement(director_ctx* ctx, const uint8_t* X, void* stream) {
    REQUIRE_CTX(ctx);
    if (X == nullptr) return DIRECTOR_ERR_INVALID_ARG;
    const director_shape& s = ctx->shape;
    const int E = s.E, R = s.R, C = s.C_max;
    // slot_expert [G] is followed by slot_order [G]: the slots sorted by (expert, slot), unused slots last
    std::vector<int32_t> rep_start(E + 1, 0), rep_slot, slot_expert(2 * (size_t)R * C, -1), slot_of((size_t)E * R, -1);
    // hosted(j): experts on rank j in ascending id -> slots j*C + 0,1,...   (capacity: sum_i x_ij <= C_max)
    for (int j = 0; j < R; ++j) {
        int p = 0;
        for (int e = 0; e < E; ++e) {
            const uint8_t v = X[(size_t)e * R + j];
            if (v > 1) return DIRECTOR_ERR_PLACEMENT;
            if (v == 1) {
                if (p >= C) return DIRECTOR_ERR_PLACEMENT;
                slot_expert[(size_t)j * C + p] = e;
                slot_of[(size_t)e * R + j] = j * C + p;
                ++p;
            }
        }
    }
    // reps(e): hosting ranks in ascending order                          (assignment: sum_j x_ij >= 1)
    for (int e = 0; e < E; ++e) {
        rep_start[e] = (int32_t)rep_slot.size();
        for (int j = 0; j < R; ++j)
            if (slot_of[(size_t)e * R + j] >= 0) rep_slot.push_back(slot_of[(size_t)e * R + j]);
        if ((int32_t)rep_slot.size() == rep_start[e]) return DIRECTOR_ERR_PLACEMENT;
    }
    rep_start[E] = (int32_t)rep_slot.size();
    {
        const size_t Gs = (size_t)R * C;
        size_t n = 0;
        for (int32_t v : rep_slot) slot_expert[Gs + n++] = v;          // replicas are listed by (expert, rank): that order
        for (size_t g = 0; g < Gs; ++g)
            if (slot_expert[g] < 0) slot_expert[Gs + n++] = (int32_t)g;   // the unused slots close the list
    }
    std::vector<unsigned long long> host_mask(E, 0ull);
    for (int e = 0; e < E; ++e)
        for (int j = 0; j < R; ++j)
            if (slot_of[(size_t)e * R + j] >= 0) host_mask[e] |= 1ull << j;
    cudaStream_t st = as_stream(stream);
    // pageable sources: the runtime stages them before returning, so the vectors may die here
    if (cudaMemcpyAsync(ctx->d_rep_start, rep_start.data(), rep_start.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(ctx->d_rep_slot, rep_slot.data(), rep_slot.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(ctx->d_slot_expert, slot_expert.data(), slot_expert.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(ctx->d_host_mask, host_mask.data(), host_mask.size() * 8, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    ctx->n_replicas = rep_start[E];
    ctx->placement_set = true;
    ctx->bank[ctx->active_placement].n_replicas = ctx->n_replicas;
    ctx->bank[ctx->active_placement].set = true;
    return DIRECTOR_OK;
}

int director_reserve_placements(director_ctx* ctx, int32_t n) {
    REQUIRE_CTX(ctx);
    if (n < 1 || n > 65536) return DIRECTOR_ERR_INVALID_ARG;
    if (cudaSetDevice(ctx->device) != cudaSuccess) return DIRECTOR_ERR_CUDA;
    const director_shape& s = ctx->shape;
    while ((int)ctx->bank.size() < n) {
        director_ctx::PlacementTables t{nullptr, nullptr, nullptr, nullptr, 0, false};
        const bool ok = dev_alloc(&t.rep_start, s.E + 1) && dev_alloc(&t.rep_slot, (size_t)s.E * s.R) &&
                        dev_alloc(&t.slot_expert, 2 * (size_t)ctx->G) && dev_alloc(&t.host_mask, s.E);
        if (!ok) {
            cudaGetLastError();
            void* tables[] = {t.rep_start, t.rep_slot, t.slot_expert, t.host_mask};
            for (void* p : tables)
                if (p) cudaFree(p);
            return DIRECTOR_ERR_WORKSPACE;
        }
        ctx->bank.push_back(t);
    }
    return DIRECTOR_OK;
}

int director_select_placement(director_ctx* ctx, int32_t slot) {
    REQUIRE_CTX(ctx);
    if (slot < 0 || slot >= (int)ctx->bank.size()) return DIRECTOR_ERR_INVALID_ARG;
    const auto& t = ctx->bank[slot];
    ctx->d_rep_start = t.rep_start;
    ctx->d_rep_slot = t.rep_slot;
    ctx->d_slot_expert = t.slot_expert;
    ctx->d_host_mask = t.host_mask;
    ctx->n_replicas = t.n_replicas;
    ctx->placement_set = t.set;
    ctx->active_placement = slot;
    return DIRECTOR_OK;
}

int director_route(director_ctx* ctx, int32_t T, const float* logits, int32_t* topk_idx, float* topk_w, void* stream) {
    REQUIRE_CTX(ctx);
    REQUIRE_T(ctx, T);
    REQUIRE_PTR(logits);
    REQUIRE_PTR(topk_idx);
    REQUIRE_PTR(topk_w);
    return launch_route(ctx, T, logits, topk_idx, topk_w, as_stream(stream));
}

int director_dispatch(director_ctx* ctx, int32_t T, const void* x, const int32_t* topk_idx, void* xp, int32_t* row_token,
                      int32_t* inv_row, int32_t* dest_rank, int32_t* seg_offsets, void* stream) {
    REQUIRE_CTX(ctx);
    REQUIRE_T(ctx, T);
    REQUIRE_PLACEMENT(ctx);
    REQUIRE_PTR(topk_idx);
    if (xp != nullptr) {      // xp == NULL: indices only
        REQUIRE_PTR(x);
        REQUIRE_PTR(xp);
    }
    REQUIRE_PTR(row_token);
    REQUIRE_PTR(inv_row);
    REQUIRE_PTR(dest_rank);
    REQUIRE_PTR(seg_offsets);
    return launch_dispatch(ctx, T, x, topk_idx, nullptr, xp, row_token, inv_row, dest_rank, seg_offsets, as_stream(stream));
}

int director_dispatch_src(director_ctx* ctx, int32_t T, const void* x, const int32_t* topk_idx,
                          const int32_t* token_src_rank, void* xp, int32_t* row_token, int32_t* inv_row,
                          int32_t* dest_rank, int32_t* seg_offsets, void* stream) {
    REQUIRE_CTX(ctx);
    REQUIRE_T(ctx, T);
    REQUIRE_PLACEMENT(ctx);
    REQUIRE_PTR(topk_idx);
    if (token_src_rank != nullptr && (reinterpret_cast<uintptr_t>(token_src_rank) & 3u)) return DIRECTOR_ERR_INVALID_ARG;
    if (xp != nullptr) {
        REQUIRE_PTR(x);
        REQUIRE_PTR(xp);
    }
    REQUIRE_PTR(row_token);
    REQUIRE_PTR(inv_row);
    REQUIRE_PTR(dest_rank);
    REQUIRE_PTR(seg_offsets);
    return launch_dispatch(ctx, T, x, topk_idx, token_src_rank, xp, row_token, inv_row, dest_rank, seg_offsets,
                           as_stream(stream));
}

int director_route_dispatch_cost(director_ctx* ctx, int32_t T, const float* logits, const void* x, int32_t* topk_idx,
                                 float* topk_w, void* xp, int32_t* row_token, int32_t* inv_row, int32_t* dest_rank,
                                 int32_t* seg_offsets, int64_t* workload, int64_t* rank_load, int64_t* dispatch_tokens,
                                 uint64_t* dispatch_bytes, void* stream) {
    REQUIRE_CTX(ctx);
    REQUIRE_T(ctx, T);
    REQUIRE_PLACEMENT(ctx);
    REQUIRE_PTR(logits);
    REQUIRE_PTR(topk_idx);
    REQUIRE_PTR(topk_w);
    if (xp != nullptr) {
        REQUIRE_PTR(x);
        REQUIRE_PTR(xp);
    }
    REQUIRE_PTR(row_token);
    REQUIRE_PTR(inv_row);
    REQUIRE_PTR(dest_rank);
    REQUIRE_PTR(seg_offsets);
    if (!workload || !rank_load || !dispatch_tokens || !dispatch_bytes) return DIRECTOR_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workload) | reinterpret_cast<uintptr_t>(rank_load) |
         reinterpret_cast<uintptr_t>(dispatch_tokens) | reinterpret_cast<uintptr_t>(dispatch_bytes)) & 7u)
        return DIRECTOR_ERR_INVALID_ARG;
    return launch_front(ctx, T, logits, x, topk_idx, topk_w, xp, row_token, inv_row, dest_rank, seg_offsets, workload,
                        rank_load, dispatch_tokens, dispatch_bytes, as_stream(stream));
}

int director_set_replica_policy(director_ctx* ctx, int32_t policy) {
    REQUIRE_CTX(ctx);
    if (policy != DIRECTOR_REPLICA_ROUND_ROBIN && policy != DIRECTOR_REPLICA_LOCAL_FIRST) return DIRECTOR_ERR_INVALID_ARG;
    ctx->replica_policy = policy;
    return DIRECTOR_OK;
}

int director_dedup_dispatch_tokens(director_ctx* ctx, int32_t T, const int32_t* dest_rank,
                                   const int32_t* token_src_rank, int64_t* dedup_tokens, void* stream) {
    REQUIRE_CTX(ctx);
    REQUIRE_T(ctx, T);
    if (dest_rank == nullptr || (reinterpret_cast<uintptr_t>(dest_rank) & 3u)) return DIRECTOR_ERR_INVALID_ARG;
    if (token_src_rank != nullptr && (reinterpret_cast<uintptr_t>(token_src_rank) & 3u)) return DIRECTOR_ERR_INVALID_ARG;
    if (dedup_tokens == nullptr || (reinterpret_cast<uintptr_t>(dedup_tokens) & 7u)) return DIRECTOR_ERR_INVALID_ARG;
    return launch_dedup_volume(ctx, T, dest_rank, token_src_rank, dedup_tokens, as_stream(stream));
}

int director_expert_ffn(director_ctx* ctx, int32_t T, const void* xp, const int32_t* seg_offsets, const void* w_gate,
                        const void* w_up, const void* w_down, void* yp, const void* x, const void* ws_gate,
                        const void* ws_up, const void* ws_down, void* y_shared, void* stream) {
    REQUIRE_CTX(ctx);
    REQUIRE_T(ctx, T);
    REQUIRE_PLACEMENT(ctx);
    REQUIRE_PTR(xp);
    REQUIRE_PTR(seg_offsets);
    REQUIRE_PTR(w_gate);
    REQUIRE_PTR(w_up);
    REQUIRE_PTR(w_down);
    REQUIRE_PTR(yp);
    if (ctx->shape.S > 0 && x != nullptr) {
        REQUIRE_PTR(x);
        REQUIRE_PTR(ws_gate);
        REQUIRE_PTR(ws_up);
        REQUIRE_PTR(ws_down);
        REQUIRE_PTR(y_shared);
    }
    return launch_expert_ffn(ctx, T, xp, nullptr, seg_offsets, w_gate, w_up, w_down, yp, x, ws_gate, ws_up, ws_down,
                             y_shared, as_stream(stream));
}

int director_expert_ffn_gather(director_ctx* ctx, int32_t T, const void* x, const int32_t* row_token,
                               const int32_t* seg_offsets, const void* w_gate, const void* w_up, const void* w_down,
                               void* yp, const void* ws_gate, const void* ws_up, const void* ws_down, void* y_shared,
                               void* stream) {
    REQUIRE_CTX(ctx);
    REQUIRE_T(ctx, T);
    REQUIRE_PLACEMENT(ctx);
    REQUIRE_PTR(x);
    REQUIRE_PTR(row_token);
    REQUIRE_PTR(seg_offsets);
    REQUIRE_PTR(w_gate);
    REQUIRE_PTR(w_up);
    REQUIRE_PTR(w_down);
    REQUIRE_PTR(yp);
    const bool shared = ctx->shape.S > 0 && y_shared != nullptr;
    if (shared) {
        REQUIRE_PTR(ws_gate);
        REQUIRE_PTR(ws_up);
        REQUIRE_PTR(ws_down);
        REQUIRE_PTR(y_shared);
    }
    if (ctx->ffn_variant != 2) return DIRECTOR_ERR_UNSUPPORTED;
    return launch_expert_ffn(ctx, T, nullptr, row_token, seg_offsets, w_gate, w_up, w_down, yp, x, ws_gate, ws_up, ws_down,
                             shared ? y_shared : nullptr, as_stream(stream));
}

int director_expert_ffn_combine(director_ctx* ctx, int32_t T, const void* xp, const int32_t* seg_offsets,
                                const int32_t* row_token, const int32_t* inv_row, const float* topk_w,
                                const void* w_gate, const void* w_up, const void* w_down, const void* x,
                                const void* ws_gate, const void* ws_up, const void* ws_down, float* y_acc,
                                float* row_weight, void* y, void* stream) {
    REQUIRE_CTX(ctx);
    REQUIRE_T(ctx, T);
    REQUIRE_PLACEMENT(ctx);
    REQUIRE_PTR(xp);
    REQUIRE_PTR(seg_offsets);
    REQUIRE_PTR(row_token);
    REQUIRE_PTR(inv_row);
    REQUIRE_PTR(topk_w);
    REQUIRE_PTR(w_gate);
    REQUIRE_PTR(w_up);
    REQUIRE_PTR(w_down);
    REQUIRE_PTR(y_acc);
    REQUIRE_PTR(row_weight);
    REQUIRE_PTR(y);
    const bool shared = ctx->shape.S > 0 && x != nullptr;
    if (shared) {
        REQUIRE_PTR(ws_gate);
        REQUIRE_PTR(ws_up);
        REQUIRE_PTR(ws_down);
    }
    if (ctx->ffn_variant != 2) return DIRECTOR_ERR_UNSUPPORTED;
    return launch_expert_ffn_combine(ctx, T, xp, seg_offsets, row_token, inv_row, topk_w, w_gate, w_up, w_down,
                                     shared ? x : nullptr, ws_gate, ws_up, ws_down, y_acc, row_weight, y,
                                     as_stream(stream));
}

int director_combine(director_ctx* ctx, int32_t T, const void* yp, const int32_t* inv_row, const float* topk_w,
                     const void* y_shared, void* y, void* stream) {
    REQUIRE_CTX(ctx);
    REQUIRE_T(ctx, T);
    REQUIRE_PTR(yp);
    REQUIRE_PTR(inv_row);
    REQUIRE_PTR(topk_w);
    REQUIRE_PTR(y);
    if (y_shared != nullptr && !aligned16(y_shared)) return DIRECTOR_ERR_INVALID_ARG;
    return launch_combine(ctx, T, yp, inv_row, topk_w, y_shared, y, as_stream(stream));
}

int director_placement_cost(director_ctx* ctx, int32_t T, const int32_t* topk_idx, const int32_t* token_src_rank,
                            int64_t* workload, int64_t* rank_load, int64_t* dispatch_tokens, uint64_t* dispatch_bytes,
                            void* stream) {
    REQUIRE_CTX(ctx);
    REQUIRE_T(ctx, T);
    REQUIRE_PLACEMENT(ctx);
    REQUIRE_PTR(topk_idx);
    if (token_src_rank != nullptr && (reinterpret_cast<uintptr_t>(token_src_rank) & 3u)) return DIRECTOR_ERR_INVALID_ARG;
    if (!workload || !rank_load || !dispatch_tokens || !dispatch_bytes) return DIRECTOR_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workload) | reinterpret_cast<uintptr_t>(rank_load) |
         reinterpret_cast<uintptr_t>(dispatch_tokens) | reinterpret_cast<uintptr_t>(dispatch_bytes)) & 7u)
        return DIRECTOR_ERR_INVALID_ARG;
    return launch_cost(ctx, T, topk_idx, token_src_rank, workload, rank_load, dispatch_tokens, dispatch_bytes,
                       as_stream(stream));
}

int director_placement_cost_batch(director_ctx* ctx, const int64_t* workload, int32_t n_candidates, const uint8_t* X,
                                  int64_t* rank_load, int64_t* dispatch_tokens, int64_t* summary, void* stream) {
    REQUIRE_CTX(ctx);
    if (n_candidates < 1 || n_candidates > 65535) return DIRECTOR_ERR_INVALID_ARG;
    if (!workload || !X || !rank_load || !dispatch_tokens || !summary) return DIRECTOR_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workload) | reinterpret_cast<uintptr_t>(rank_load) |
         reinterpret_cast<uintptr_t>(dispatch_tokens) | reinterpret_cast<uintptr_t>(summary)) & 7u)
        return DIRECTOR_ERR_INVALID_ARG;
    return launch_cost_batch(ctx, workload, n_candidates, X, rank_load, dispatch_tokens, summary, as_stream(stream));
}

int director_layer_submit_host(director_ctx* ctx, int32_t T, const float* logits, const void* x, const void* w_gate,
                               const void* w_up, const void* w_down, const void* ws_gate, const void* ws_up,
                               const void* ws_down, void* y, int64_t* rank_load, uint64_t* dispatch_bytes, void* stream,
                               int64_t* ticket) {
    REQUIRE_CTX(ctx);
    REQUIRE_T(ctx, T);
    REQUIRE_PLACEMENT(ctx);
    if (!logits || !x || !y || !ticket) return DIRECTOR_ERR_INVALID_ARG;
    REQUIRE_PTR(w_gate);
    REQUIRE_PTR(w_up);
    REQUIRE_PTR(w_down);
    const director_shape& s = ctx->shape;
    const bool shared = s.S > 0;
    if (shared) {
        REQUIRE_PTR(ws_gate);
        REQUIRE_PTR(ws_up);
        REQUIRE_PTR(ws_down);
    }
    cudaStream_t st = as_stream(stream);
    const int slot = (int)(ctx->submitted & 1);
    float* d_logits = ctx->e_logits2[slot];
    void* d_x = ctx->e_x2[slot];
    void* d_y = ctx->e_y2[slot];
    int64_t* c_w = ctx->e_cost2[slot];
    int64_t* c_load = c_w + (size_t)s.R * s.E;
    int64_t* c_tok = c_load + s.R;
    uint64_t* c_bytes = reinterpret_cast<uint64_t*>(c_tok + (size_t)s.R * s.R);

    // This slot's previous batch (two submissions ago) must have reached the host before its buffers are reused.  A
    // caller that keeps at most two batches in flight has already waited for it; one that has not is held here, on the
    // host, until that batch's copies have landed - so a ticket never reads as complete before its data is.
    const int64_t prev = ctx->submitted - 2;
    if (prev >= 0 && ctx->waited[slot] < prev) {
        if (cudaEventSynchronize(ctx->ev_d2h_done[slot]) != cudaSuccess) return DIRECTOR_ERR_CUDA;
        ctx->waited[slot] = prev;
    }
    // inputs: wait until the kernels of the batch that used this slot two submissions ago are done with it
    if (cudaStreamWaitEvent(ctx->h2d_stream, ctx->ev_compute_done[slot], 0) != cudaSuccess ||
        cudaMemcpyAsync(d_logits, logits, sizeof(float) * (size_t)T * s.E, cudaMemcpyHostToDevice, ctx->h2d_stream) != cudaSuccess ||
        cudaMemcpyAsync(d_x, x, 2 * (size_t)T * s.H, cudaMemcpyHostToDevice, ctx->h2d_stream) != cudaSuccess ||
        cudaEventRecord(ctx->ev_h2d_done[slot], ctx->h2d_stream) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    // kernels: need this batch's inputs, and the outputs of this slot must have left for the host
    if (cudaStreamWaitEvent(st, ctx->ev_h2d_done[slot], 0) != cudaSuccess ||
        cudaStreamWaitEvent(st, ctx->ev_d2h_done[slot], 0) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    // the permuted rows are materialised once: the weight-stationary GEMM reads every token tile once per weight
    // block, so gathering inside it (director_expert_ffn_gather) repeats the gather 2F/256 times and measured slower
    // (the weight-streaming kernels of a tiny batch stage their few rows from x themselves: no row copies then)
    const bool stream_w = ffn_streams_weights(ctx, T);
    int rc = launch_front(ctx, T, d_logits, d_x, ctx->e_topk_idx, ctx->e_topk_w, stream_w ? nullptr : ctx->e_xp,
                          ctx->e_row_token, ctx->e_inv_row, ctx->e_dest_rank, ctx->d_seg_offsets, c_w, c_load, c_tok,
                          c_bytes, st);
    if (rc == DIRECTOR_OK)
        rc = launch_expert_ffn(ctx, T, stream_w ? nullptr : ctx->e_xp, stream_w ? ctx->e_row_token : nullptr,
                               ctx->d_seg_offsets, w_gate, w_up, w_down, ctx->e_yp, (shared || stream_w) ? d_x : nullptr,
                               ws_gate, ws_up, ws_down, shared ? ctx->e_y_shared : nullptr, st);
    if (rc == DIRECTOR_OK)
        rc = launch_combine(ctx, T, ctx->e_yp, ctx->e_inv_row, ctx->e_topk_w, shared ? ctx->e_y_shared : nullptr, d_y, st);
    if (rc != DIRECTOR_OK) return rc;
    if (cudaEventRecord(ctx->ev_compute_done[slot], st) != cudaSuccess) return DIRECTOR_ERR_CUDA;
    // outputs
    if (cudaStreamWaitEvent(ctx->d2h_stream, ctx->ev_compute_done[slot], 0) != cudaSuccess ||
        cudaMemcpyAsync(y, d_y, 2 * (size_t)T * s.H, cudaMemcpyDeviceToHost, ctx->d2h_stream) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    if (rank_load &&
        cudaMemcpyAsync(rank_load, c_load, sizeof(int64_t) * s.R, cudaMemcpyDeviceToHost, ctx->d2h_stream) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    if (dispatch_bytes && cudaMemcpyAsync(dispatch_bytes, c_bytes, sizeof(uint64_t) * s.R * s.R, cudaMemcpyDeviceToHost,
                                          ctx->d2h_stream) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    if (cudaEventRecord(ctx->ev_d2h_done[slot], ctx->d2h_stream) != cudaSuccess) return DIRECTOR_ERR_CUDA;
    *ticket = ctx->submitted++;
    return DIRECTOR_OK;
}

int director_layer_wait_host(director_ctx* ctx, int64_t ticket) {
    REQUIRE_CTX(ctx);
    if (ticket < 0 || ticket >= ctx->submitted) return DIRECTOR_ERR_INVALID_ARG;
    const int slot = (int)(ticket & 1);
    if (ctx->waited[slot] >= ticket) return DIRECTOR_OK;   // already delivered (waited for, or its slot was reused since)
    if (cudaEventSynchronize(ctx->ev_d2h_done[slot]) != cudaSuccess) return DIRECTOR_ERR_CUDA;
    // the event now belongs to the newest batch of this slot, so every ticket of the slot up to that one is in host memory
    ctx->waited[slot] = ((ctx->submitted - 1) & 1) == slot ? ctx->submitted - 1 : ctx->submitted - 2;
    return DIRECTOR_OK;
}

int director_layer_forward(director_ctx* ctx, int32_t T, const float* logits, const void* x, const void* w_gate,
                           const void* w_up, const void* w_down, const void* ws_gate, const void* ws_up,
                           const void* ws_down, void* y, int64_t* workload, int64_t* rank_load, int64_t* dispatch_tokens,
                           uint64_t* dispatch_bytes, void* stream) {
    REQUIRE_CTX(ctx);
    REQUIRE_T(ctx, T);
    REQUIRE_PLACEMENT(ctx);
    REQUIRE_PTR(logits);
    REQUIRE_PTR(x);
    REQUIRE_PTR(w_gate);
    REQUIRE_PTR(w_up);
    REQUIRE_PTR(w_down);
    REQUIRE_PTR(y);
    const director_shape& s = ctx->shape;
    const bool shared = s.S > 0;
    if (shared) {
        REQUIRE_PTR(ws_gate);
        REQUIRE_PTR(ws_up);
        REQUIRE_PTR(ws_down);
    }
    if (!workload || !rank_load || !dispatch_tokens || !dispatch_bytes) return DIRECTOR_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workload) | reinterpret_cast<uintptr_t>(rank_load) |
         reinterpret_cast<uintptr_t>(dispatch_tokens) | reinterpret_cast<uintptr_t>(dispatch_bytes)) & 7u)
        return DIRECTOR_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    // the weight-streaming kernels of a tiny batch stage their few rows from x themselves: no row copies then
    const bool stream_w = ffn_streams_weights(ctx, T);
    int rc = launch_front(ctx, T, logits, x, ctx->e_topk_idx, ctx->e_topk_w, stream_w ? nullptr : ctx->e_xp,
                          ctx->e_row_token, ctx->e_inv_row, ctx->e_dest_rank, ctx->d_seg_offsets, workload, rank_load,
                          dispatch_tokens, dispatch_bytes, st);
    if (rc == DIRECTOR_OK)
        rc = launch_expert_ffn(ctx, T, stream_w ? nullptr : ctx->e_xp, stream_w ? ctx->e_row_token : nullptr,
                               ctx->d_seg_offsets, w_gate, w_up, w_down, ctx->e_yp, (shared || stream_w) ? x : nullptr,
                               ws_gate, ws_up, ws_down, shared ? ctx->e_y_shared : nullptr, st);
    if (rc == DIRECTOR_OK)
        rc = launch_combine(ctx, T, ctx->e_yp, ctx->e_inv_row, ctx->e_topk_w, shared ? ctx->e_y_shared : nullptr, y, st);
    return rc;
}

int director_layer_forward_host(director_ctx* ctx, int32_t T, const float* logits, const void* x, const void* w_gate,
                                const void* w_up, const void* w_down, const void* ws_gate, const void* ws_up,
                                const void* ws_down, void* y, int64_t* rank_load, uint64_t* dispatch_bytes, void* stream) {
    int64_t ticket = -1;
    const int rc = director_layer_submit_host(ctx, T, logits, x, w_gate, w_up, w_down, ws_gate, ws_up, ws_down, y,
                                              rank_load, dispatch_bytes, stream, &ticket);
    if (rc != DIRECTOR_OK) return rc;
    return director_layer_wait_host(ctx, ticket);
}

int director_last_status(director_ctx* ctx, void* stream) {
    REQUIRE_CTX(ctx);
    cudaStream_t st = as_stream(stream);
    int32_t h = 0;
    if (cudaMemcpyAsync(&h, ctx->d_status, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return DIRECTOR_ERR_CUDA;
    if (cudaMemsetAsync(ctx->d_status, 0, sizeof(h), st) != cudaSuccess) return DIRECTOR_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return DIRECTOR_ERR_CUDA;
    return h;
}

int director_batch_streams_weights(director_ctx* ctx, int32_t T) {
    if (ctx == nullptr || T < 1 || T > ctx->shape.T_max) return -DIRECTOR_ERR_INVALID_ARG;   // 1 is an answer here
    return ffn_streams_weights(ctx, T) ? 1 : 0;
}

int director_set_ffn_variant(director_ctx* ctx, int32_t variant) {
    REQUIRE_CTX(ctx);
    if (variant < 0 || (variant > 2 && variant != 6)) return DIRECTOR_ERR_INVALID_ARG;
    // 6: scheme 2 with the tensor-core kernels for every batch size (no weight-streaming path for tiny batches)
    ctx->ffn_small = variant == 2;
    ctx->ffn_variant = variant > 2 ? 2 : variant;
    return DIRECTOR_OK;
}

int director_pair_clusters(const director_ctx* ctx) { return ctx ? ctx->pair_clusters : -1; }

int director_gemm_counters(director_ctx* ctx, int32_t which, int64_t* out) {
    if (ctx == nullptr || which < 0 || which > 1 || out == nullptr) return DIRECTOR_ERR_INVALID_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return DIRECTOR_ERR_CUDA;
    std::vector<unsigned long long> h((size_t)kGemmClockWords * kGemmClockCtas);
    if (cudaMemcpy(h.data(), ctx->d_gemm_clock + (size_t)which * kGemmClockWords * kGemmClockCtas,
                   h.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess)
        return DIRECTOR_ERR_CUDA;
    const int ctas = std::min(2 * ctx->pair_clusters, (int)kGemmClockCtas);
    for (int k = 0; k < DIRECTOR_GEMM_COUNTERS; ++k) out[k] = 0;
    for (int i = 0; i < ctas; ++i) {
        const unsigned long long* r = h.data() + (size_t)i * kGemmClockWords;
        for (int k = 0; k < kGemmClockWords; ++k) out[k] += (int64_t)r[k];
        out[kGemmClockWords] = std::max<int64_t>(out[kGemmClockWords], (int64_t)r[1]);   // longest CTA, ns
    }
    out[kGemmClockWords + 1] = ctas;
    return DIRECTOR_OK;
}

double director_gemm_sm_mhz(director_ctx* ctx, int32_t which, double* busy_us) {
    int64_t c[DIRECTOR_GEMM_COUNTERS];
    if (director_gemm_counters(ctx, which, c) != DIRECTOR_OK) return -1.0;
    if (busy_us) *busy_us = (double)c[kGemmClockWords] * 1e-3;
    return c[1] > 0 ? (double)c[0] / (double)c[1] * 1e3 : 0.0;
}

int64_t director_launch_count(const director_ctx* ctx) { return ctx ? ctx->launches : -1; }

int director_set_profiling(director_ctx* ctx, int32_t enabled) {
    REQUIRE_CTX(ctx);
    if (cudaDeviceSynchronize() != cudaSuccess) return DIRECTOR_ERR_CUDA;
    for (auto& ev : ctx->events) ctx->free_events.push_back(ev);
    ctx->events.clear();
    ctx->profiling = enabled == 2 ? 2 : (enabled != 0 ? 1 : 0);
    return DIRECTOR_OK;
}

int director_set_profiling_filter(director_ctx* ctx, const char* name_substr) {
    REQUIRE_CTX(ctx);
    ctx->profile_filter = name_substr ? name_substr : "";
    return DIRECTOR_OK;
}

double director_kernel_time(director_ctx* ctx, const char* name_substr, int64_t* launches) {
    if (ctx == nullptr || name_substr == nullptr) return -1.0;
    if (cudaDeviceSynchronize() != cudaSuccess) return -1.0;
    double total = 0.0;
    int64_t n = 0;
    for (const auto& ev : ctx->events) {
        if (std::strstr(ev.name, name_substr) == nullptr) continue;
        float ms = 0.0f;
        if (cudaEventElapsedTime(&ms, ev.start, ev.stop) != cudaSuccess) return -1.0;
        total += ms;
        ++n;
    }
    if (launches) *launches = n;
    return total;
}

const char* director_status_string(int status) {
    switch (status) {
        case DIRECTOR_OK: return "ok";
        case DIRECTOR_ERR_INVALID_ARG: return "invalid argument";
        case DIRECTOR_ERR_PLACEMENT: return "invalid or missing expert placement";
        case DIRECTOR_ERR_WORKSPACE: return "workspace allocation failed";
        case DIRECTOR_ERR_CUDA: return "CUDA call failed";
        case DIRECTOR_ERR_UNSUPPORTED: return "unsupported shape or device";
        case DIRECTOR_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case DIRECTOR_ERR_BAD_INDEX: return "expert or rank index out of range on the device";
        case DIRECTOR_ERR_NONFINITE: return "non-finite router logit";
        case DIRECTOR_ERR_STATIC_LIMIT: return "problem exceeds the fixed scratch of an allocation-free call";
        default: return "unknown status";
    }
}

}  // extern "C"
