/*
 * director.h - C ABI of libdirector.so
 *
 * The expert-parallel Mixture-of-Experts layer forward under a given expert placement, on one
 * GPU, with the expert-parallel "ranks" as logical partitions of that GPU (no inter-GPU
 * traffic).  This is the computation whose latency the paper's proactive expert placement
 * reduces: gate -> all-to-all dispatch -> expert FFNs -> all-to-all aggregate (Section II-A,
 * Section II-B), together with the quantities its placement optimiser trades off (Section VI-A,
 * Eq. 1-4).
 *
 * Notation (paper, Section VI-A; indices are 0-based here, the paper counts from 1):
 *   T  tokens in the batch            H  hidden size            F  expert FFN width
 *   E  routed experts per layer       K  experts chosen per token (top-k)
 *   S  always-on shared experts       R  logical ranks (the GPU set G of the paper)
 *   C_max  expert slots per rank (the paper's per-GPU capacity C_max)
 *   X[E][R]  placement matrix, X[i][j] = 1 iff expert i is hosted on rank j (the variable
 *            x_{i,j} of Eq. 6: sum_j x_{i,j} >= 1, sum_i x_{i,j} <= C_max); an expert hosted on
 *            several ranks is replicated, all replicas use the same weight array.
 *   A = T*K  (token, choice) assignments;   G = R*C_max  slots.
 *   Slot g = j*C_max + p holds the p-th smallest expert id hosted on rank j (or nothing).
 *
 * Conventions
 *   - Every pointer marked "dev" is caller-owned device memory on the context's device,
 *     16-byte aligned, valid until the stream has reached the call.  "host" pointers are
 *     ordinary host memory.  The context owns only its internal workspace, sized at create
 *     time; no entry point allocates after director_create (except director_reserve_placements).
 *   - bf16 tensors are passed as void* (raw 16-bit patterns), row-major, innermost last.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Calls are asynchronous on `stream` and never synchronise unless stated.  Every function
 *     returns a director_status; nothing throws across the boundary.  Argument errors are
 *     detected on the host before anything is launched.  Faults only visible on the device
 *     (an expert id outside [0,E), a non-finite logit, a bounded wait that expired) set a
 *     sticky status word that director_last_status reads; the offending element is skipped,
 *     kernels never trap.
 *   - Supported ranges: 1 <= K <= 8, K <= E <= 256, 1 <= R <= 64, 1 <= C_max <= 16,
 *     E <= R*C_max, H % 256 == 0, F % 128 == 0, S >= 0, T_max*K < 2^31.
 */
#ifndef DIRECTOR_H
#define DIRECTOR_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct director_ctx director_ctx;

typedef enum {
    DIRECTOR_OK = 0,
    DIRECTOR_ERR_INVALID_ARG = 1,   /* NULL / misaligned pointer, size out of range            */
    DIRECTOR_ERR_PLACEMENT = 2,     /* an expert has no host, or a rank exceeds C_max, or unset */
    DIRECTOR_ERR_WORKSPACE = 3,     /* device allocation failed at create time                  */
    DIRECTOR_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed                        */
    DIRECTOR_ERR_UNSUPPORTED = 5,   /* shape outside the supported ranges, or not an sm_100 GPU */
    DIRECTOR_ERR_TIMEOUT = 6,       /* device: a bounded wait inside a kernel expired           */
    DIRECTOR_ERR_BAD_INDEX = 7,     /* device: expert id outside [0,E) met (element skipped)    */
    DIRECTOR_ERR_NONFINITE = 8,     /* device: NaN/Inf router logit met                         */
    DIRECTOR_ERR_STATIC_LIMIT = 9   /* problem larger than the fixed scratch of a *_static call */
} director_status;

typedef struct {
    int32_t T_max;   /* largest batch any call will pass */
    int32_t H, F, E, K, S, R, C_max;
} director_shape;

/* Life cycle.  director_create allocates the workspace on the current device (it is the only
 * call that allocates) and binds the context to that device. */
int director_create(const director_shape* shape, director_ctx** out);
int director_destroy(director_ctx* ctx);

/* Expert placement (Section VI-A placement map; Eq. 6 assignment and capacity constraints).
 * X_host: host, uint8 [E][R] row-major, entries 0/1.  Validates that every expert has at
 * least one host and no rank hosts more than C_max experts (DIRECTOR_ERR_PLACEMENT
 * otherwise, previous placement kept), builds the slot tables and uploads them on `stream`.
 * X_host may be reused as soon as the call returns. */
int director_set_placement(director_ctx* ctx, const uint8_t* X_host, void* stream);

/* Several placements on one context (the placement map P(l, i) of Section VI-A has one placement per layer l;
 * a model's layers can share one context's workspace and differ only in their tables).
 * director_reserve_placements makes room for n table sets (slots 0..n-1; slot 0 exists from creation; this is the
 * one call besides director_create that allocates).  director_select_placement makes a slot the current one: a
 * host-side switch, no copy, no stream work; kernels already launched keep the tables they were launched with.
 * director_set_placement fills the current slot; every entry point uses the current slot.  Selecting a slot that
 * was never filled leaves the context without a placement (DIRECTOR_ERR_PLACEMENT from the calls that need one). */
int director_reserve_placements(director_ctx* ctx, int32_t n);
int director_select_placement(director_ctx* ctx, int32_t slot);

/* (a1) Gating (Section II-A: relevance scores, top-k selection, scores used as weights).
 * logits: dev fp32 [T,E].  topk_idx: dev int32 [T,K], the K experts with the largest logits in
 * descending order, ties to the lower expert id.  topk_w: dev fp32 [T,K], softmax scores of
 * the chosen experts renormalised to sum to one. */
int director_route(director_ctx* ctx, int32_t T, const float* logits,
                   int32_t* topk_idx, float* topk_w, void* stream);

/* (a2) Dispatch (Section II-B: the first all-to-all moves every token to the ranks that host its experts;
 * here an on-device permutation, the bytes that would cross ranks are counted by
 * director_placement_cost).  Under the default replica policy (see director_set_replica_policy) the n-th
 * assignment of expert e in ascending token order goes to
 * replica n mod r_e of e (replicas ordered by rank) and becomes row n div r_e of that replica's
 * segment; segments lie in slot order.
 * x: dev bf16 [T,H].  topk_idx: dev int32 [T,K].
 * xp: dev bf16 [T*K,H] permuted copies of the rows of x.   row_token: dev int32 [T*K], token of
 * each row.  inv_row: dev int32 [T,K], row of each assignment.  dest_rank: dev int32 [T,K].
 * seg_offsets: dev int32 [R*C_max+1], first row of each slot's segment, last entry T*K.
 * xp may be NULL: only the indices are produced (x is then not read), for use with director_expert_ffn_gather. */
int director_dispatch(director_ctx* ctx, int32_t T, const void* x, const int32_t* topk_idx,
                      void* xp, int32_t* row_token, int32_t* inv_row, int32_t* dest_rank,
                      int32_t* seg_offsets, void* stream);

/* (a1) + (a2) + (a5) in one call: the front end of the layer.  Same arguments, same results (bit for bit) as
 * director_route, director_dispatch and director_placement_cost (token_src_rank = NULL) called in that order.
 * For batches of at most 256 tokens under the ROUND_ROBIN replica policy - the decode steps of serving, where
 * each of those stages moves a few KB - the gate, the counting sort and the histograms run in a single launch
 * (plus the row copies if xp != NULL); larger batches run the separate kernels. */
int director_route_dispatch_cost(director_ctx* ctx, int32_t T, const float* logits, const void* x,
                                 int32_t* topk_idx, float* topk_w, void* xp, int32_t* row_token,
                                 int32_t* inv_row, int32_t* dest_rank, int32_t* seg_offsets, int64_t* workload,
                                 int64_t* rank_load, int64_t* dispatch_tokens, uint64_t* dispatch_bytes,
                                 void* stream);

/* Which replica of a replicated expert an assignment uses.  The paper replicates hot experts to shrink the
 * dispatch volume of Eq. 3 (Section III) without fixing this choice; both rules below are this library's.
 *   ROUND_ROBIN (default)  the n-th assignment of expert e (ascending token id) uses replica n mod r_e.
 *   LOCAL_FIRST            an assignment whose token lives on a rank hosting e stays there; the others are
 *                          numbered m = 0,1,... in ascending token id and use replica m mod r_e.
 * In both, a segment holds its assignments in ascending token id.  The policy applies to director_dispatch,
 * director_dispatch_src, director_placement_cost, director_placement_cost_batch and the host entry points. */
enum { DIRECTOR_REPLICA_ROUND_ROBIN = 0, DIRECTOR_REPLICA_LOCAL_FIRST = 1 };
int director_set_replica_policy(director_ctx* ctx, int32_t policy);

/* director_dispatch with an explicit home rank per token.  token_src_rank: dev int32 [T] with values in [0,R),
 * or NULL for the block partition src(t) = floor(t*R/T) that director_dispatch uses.  Only LOCAL_FIRST looks at
 * it; a value out of range sets DIRECTOR_ERR_BAD_INDEX in the device status and the token is treated as having
 * no home (all its assignments travel). */
int director_dispatch_src(director_ctx* ctx, int32_t T, const void* x, const int32_t* topk_idx,
                          const int32_t* token_src_rank, void* xp, int32_t* row_token, int32_t* inv_row,
                          int32_t* dest_rank, int32_t* seg_offsets, void* stream);

/* De-duplicated dispatch volume (a variant of Eq. 3's count): dedup_tokens[j*R+k] = number of tokens on rank j with
 * at least one assignment executed on rank k, i.e. what the first all-to-all of Section II-B moves when a token
 * whose several experts share a rank is sent there once.  dest_rank: dev int32 [T,K] as written by
 * director_dispatch (entries < 0 are skipped).  token_src_rank: dev int32 [T] or NULL (block partition).
 * dedup_tokens: dev int64 [R,R], overwritten. */
int director_dedup_dispatch_tokens(director_ctx* ctx, int32_t T, const int32_t* dest_rank,
                                   const int32_t* token_src_rank, int64_t* dedup_tokens, void* stream);

/* (a3) Expert FFNs (Section II-A: each expert is an FFN sub-network), SwiGLU, bf16 operands,
 * fp32 accumulation on the tensor cores:  for every row i of the segment of slot g (expert e)
 *   yp[i,:] = ( silu(xp[i,:] . w_gate[e]^T) * (xp[i,:] . w_up[e]^T) ) . w_down[e]^T
 * xp: dev bf16 [T*K,H].  seg_offsets: dev int32 [R*C_max+1] as written by director_dispatch under
 * the current placement.  w_gate, w_up: dev bf16 [E,F,H].  w_down: dev bf16 [E,H,F].
 * yp: dev bf16 [T*K,H].
 * Shared experts (only if the context has S > 0 and x != NULL): the S always-on FFNs applied
 * to every token's own row, summed: x: dev bf16 [T,H]; ws_gate, ws_up: dev bf16 [S*F,H] (the S
 * experts stacked); ws_down: dev bf16 [H,S*F] (the S experts side by side);
 * y_shared: dev bf16 [T,H].
 * Batches of more than 4 tokens run as two grouped GEMMs on the tensor cores (tcgen05, accumulators in tensor
 * memory, operands by TMA).  A batch of at most 4 tokens is a stream of the touched experts' weights through a few
 * dot products, bound by HBM bandwidth: it runs as two weight-streaming kernels (one warp per pair of output
 * features, fp32 accumulation in a fixed order), which use every SM whatever the number of segments.  Both paths
 * round Hg to bf16 between the projections; their results agree within the layer's tolerance, not bit for bit. */
int director_expert_ffn(director_ctx* ctx, int32_t T, const void* xp, const int32_t* seg_offsets,
                        const void* w_gate, const void* w_up, const void* w_down, void* yp,
                        const void* x, const void* ws_gate, const void* ws_up, const void* ws_down,
                        void* y_shared, void* stream);

/* (a3) fused with the row movement of (a2): the routed experts read row i of the permuted order directly as
 * x[row_token[i]], so no permuted copy xp exists (the single-GPU analogue of hiding the dispatch cost the paper
 * attributes to the first all-to-all, Section I).  x: dev bf16 [T,H].  row_token, seg_offsets: as written by
 * director_dispatch (which may be called with xp = NULL).  Other arguments as for director_expert_ffn; the
 * shared experts run iff the context has S > 0 and y_shared != NULL.  Results are bit-identical to
 * director_dispatch + director_expert_ffn.  Needs the default tile scheme (director_set_ffn_variant 2), otherwise
 * DIRECTOR_ERR_UNSUPPORTED.
 * Cost: the weight-stationary GEMM reads each token tile once per 256-row weight block, so the gather is repeated
 * 2F/256 times per token row and runs as one-row TMA boxes; it saves memory (no xp), not time - the layer's
 * default path materialises xp once.  The exception is a batch small enough for the weight-streaming kernels
 * (director_batch_streams_weights): those stage a segment's few rows in shared memory once per CTA, from xp or
 * from x alike, so there the gathering form is the cheaper one (no row copies) and the one-call entry points use it. */
int director_expert_ffn_gather(director_ctx* ctx, int32_t T, const void* x, const int32_t* row_token,
                               const int32_t* seg_offsets, const void* w_gate, const void* w_up,
                               const void* w_down, void* yp, const void* ws_gate, const void* ws_up,
                               const void* ws_down, void* y_shared, void* stream);

/* (a3) and (a4) fused, the second half of the survey's "next-2" row: both projections run on the tensor-core
 * kernels and the down projection combines in its epilogue - every accumulator element, times its row's gating
 * weight, is added (fp32 atomic add) into an accumulator of y at its row's token, so that Yp is never written and
 * the combine step (Section II-A: y = sum of the chosen experts' outputs weighted by the gate) shrinks to one
 * rounding pass.  OPT-IN, for two reasons: the K contributions of a token arrive in no fixed order, so y is
 * reproducible only to fp32 rounding (the default path is bit-reproducible and placement-invariant); and it is
 * slower - the atomic traffic costs more than the separate combine kernel saves.
 * xp, seg_offsets, row_token, inv_row, topk_w: as written by director_dispatch / director_route.  x and ws_*: as for
 * director_expert_ffn (shared experts run iff the context has S > 0 and x != NULL).  y_acc: dev fp32 [T,H] scratch,
 * row_weight: dev fp32 [T*K] scratch (caller-owned, contents irrelevant on entry).  y: dev bf16 [T,H] out.
 * Needs the default tile scheme (director_set_ffn_variant 2), otherwise DIRECTOR_ERR_UNSUPPORTED. */
int director_expert_ffn_combine(director_ctx* ctx, int32_t T, const void* xp, const int32_t* seg_offsets,
                                const int32_t* row_token, const int32_t* inv_row, const float* topk_w,
                                const void* w_gate, const void* w_up, const void* w_down, const void* x,
                                const void* ws_gate, const void* ws_up, const void* ws_down, float* y_acc,
                                float* row_weight, void* y, void* stream);

/* (a4) Combine (Section II-A weighted summation; Section II-B second all-to-all):
 *   y[t,:] = bf16( sum_s topk_w[t,s] * yp[inv_row[t,s],:]  (+ y_shared[t,:]) ), fp32 accumulation
 * in slot order.  yp: dev bf16 [T*K,H].  inv_row: dev int32 [T,K].  topk_w: dev fp32 [T,K].
 * y_shared: dev bf16 [T,H] or NULL.  y: dev bf16 [T,H]. */
int director_combine(director_ctx* ctx, int32_t T, const void* yp, const int32_t* inv_row,
                     const float* topk_w, const void* y_shared, void* y, void* stream);

/* (a5) Placement cost (Section VI-A): workload matrix W, per-rank load of Eq. 1 and dispatch
 * volume of Eq. 3 for the current placement, counted per executed assignment.
 * topk_idx: dev int32 [T,K].  token_src_rank: dev int32 [T] home rank of each token, or NULL for
 * the block partition src(t) = floor(t*R/T).
 * workload: dev int64 [R,E], W[j][i] = tokens of rank j routed to expert i.
 * rank_load: dev int64 [R], assignments executed on rank j (lambda_j).
 * dispatch_tokens: dev int64 [R,R], [j][k] = assignments of tokens of rank j executed on rank k
 * (the diagonal is local traffic, which Eq. 4 leaves out).
 * dispatch_bytes: dev uint64 [R,R] = dispatch_tokens * d with d = 2*H bytes per token (Eq. 3). */
int director_placement_cost(director_ctx* ctx, int32_t T, const int32_t* topk_idx,
                            const int32_t* token_src_rank, int64_t* workload, int64_t* rank_load,
                            int64_t* dispatch_tokens, uint64_t* dispatch_bytes, void* stream);

/* Batched placement cost (Section VI-C: the placement search scores many candidate placements against the
 * same workload; Eq. 1 and Eq. 3 per candidate).  Needs no placement set on the context.
 * workload: dev int64 [R,E], the matrix W as written by director_placement_cost for the block partition of
 * tokens over source ranks (the closed form used here relies on each rank's tokens being contiguous).
 * X: dev uint8 [n,E,R], n candidate placement matrices (entries 0/1; replicas allowed, round-robin split as in
 * director_dispatch).  rank_load: dev int64 [n,R].  dispatch_tokens: dev int64 [n,R,R] (multiply by 2*H for
 * bytes).  summary: dev int64 [n,4] = {max_j rank_load[j]  (Eq. 2's straggler),  max_j sum_{k!=j} dispatch_tokens[j][k]
 * (Eq. 4's straggler, in tokens),  total cross-rank tokens,  1 if the candidate satisfies Eq. 6's assignment and
 * capacity constraints else 0}.  1 <= n <= 65535.  Results equal director_placement_cost's for every valid
 * candidate. */
int director_placement_cost_batch(director_ctx* ctx, const int64_t* workload, int32_t n_candidates,
                                  const uint8_t* X, int64_t* rank_load, int64_t* dispatch_tokens,
                                  int64_t* summary, void* stream);

/* Dispatch indices without a context and without any allocation.  (The paper has no counterpart:
 * this entry point exists for the library's users, not for the method.)
 *
 * director_create allocates its workspace, so it is closed to callers that must never call
 * cudaMalloc: code embedded in a host application that owns the device heap, latency-critical loops
 * that may not block on the allocator, processes running under a fixed memory reservation.  This
 * call computes the same permutation as director_dispatch (everything except the row copies) and
 * performs no cudaMalloc, cudaFree or other allocating call, on any invocation.  Its scratch (launch
 * ticket, status word, per-tile expert counts) is a fixed 1 MiB array inside the library image that
 * each device holds from library load to process exit.
 *
 * Inputs, all dev: topk_idx int32 [T,K]; the placement as replica tables: rep_start int32 [E+1]
 * (exclusive prefix of replica counts, rep_start[0] = 0) and rep_slot int32 [rep_start[E]], the slot
 * g = rank*C_max + p of each replica, an expert's replicas in ascending rank order (slot numbering as
 * in the header comment; the caller builds the tables: an expert that is routed to but has no replica, or a
 * slot outside [0, R*C_max), is skipped and reported as DIRECTOR_ERR_BAD_INDEX, the assignment's row is -1).
 * Outputs, all dev: row_token int32 [T*K], inv_row int32 [T,K], dest_rank int32 [T,K], seg_offsets
 * int32 [R*C_max+1], exactly as director_dispatch writes them.  device_status: dev int32 [1] that the
 * caller has zeroed, receives DIRECTOR_ERR_BAD_INDEX if an expert id outside [0,E) was skipped; may be
 * NULL (the flag is then kept in the scratch and lost).
 * Limits: ceil(T/256) * E <= 262080 (e.g. T <= 524032 at E = 128), otherwise DIRECTOR_ERR_STATIC_LIMIT
 * is returned and nothing is launched; K, E, R, C_max within the ranges of the header comment.
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress); make
 * that first call outside any stream capture.  All calls on a device share the one array and it
 * keeps the previous call's contents: the call clears what must start at zero itself, but two calls
 * whose kernels overlap on the GPU (different streams, no dependency) race on it - serialise them. */
int director_dispatch_index_static(int32_t T, int32_t K, int32_t E, int32_t R, int32_t C_max,
                                   const int32_t* topk_idx, const int32_t* rep_start, const int32_t* rep_slot,
                                   int32_t* row_token, int32_t* inv_row, int32_t* dest_rank,
                                   int32_t* seg_offsets, int32_t* device_status, void* stream);

/* The whole layer (a1)-(a5) in one call on device buffers: the gate, the permutation, the expert FFNs and the
 * combine run on the context's own workspace (the intermediates of the stage calls are not exposed), the layer
 * output and the placement-cost histograms go to the caller's buffers.  Same results, bit for bit, as the stage
 * calls in order.  logits: dev fp32 [T,E].  x: dev bf16 [T,H].  Weights as for director_expert_ffn (ws_* may be
 * NULL when S == 0).  y: dev bf16 [T,H].  workload: dev int64 [R,E].  rank_load: dev int64 [R].
 * dispatch_tokens: dev int64 [R,R].  dispatch_bytes: dev uint64 [R,R].  Shares the workspace with the host entry
 * points below: do not run both at the same time on one context. */
int director_layer_forward(director_ctx* ctx, int32_t T, const float* logits, const void* x,
                           const void* w_gate, const void* w_up, const void* w_down,
                           const void* ws_gate, const void* ws_up, const void* ws_down, void* y,
                           int64_t* workload, int64_t* rank_load, int64_t* dispatch_tokens,
                           uint64_t* dispatch_bytes, void* stream);

/* The whole layer for callers that hold their batch in host memory: copies logits and x to the
 * device, runs (a1)-(a5) on context-owned buffers and copies y and the histograms back; returns
 * when the results are in the host buffers (director_layer_submit_host + director_layer_wait_host).
 * logits: host fp32 [T,E].  x: host bf16 [T,H].  Weights: dev, as for director_expert_ffn
 * (ws_* may be NULL when S == 0).  y: host bf16 [T,H].  rank_load: host int64 [R] or NULL.
 * dispatch_bytes: host uint64 [R,R] or NULL.  Pinned host buffers make the copies asynchronous. */
int director_layer_forward_host(director_ctx* ctx, int32_t T, const float* logits, const void* x,
                                const void* w_gate, const void* w_up, const void* w_down,
                                const void* ws_gate, const void* ws_up, const void* ws_down,
                                void* y, int64_t* rank_load, uint64_t* dispatch_bytes, void* stream);

/* The same, split in two so that a stream of batches overlaps its transfers with its kernels (the
 * serving loop of Section IV feeds one batch after another): submit enqueues the host->device copies
 * on an internal copy stream, the kernels on `stream` and the device->host copies on a second internal
 * copy stream, chained by events, and returns at once with a ticket; wait blocks until that batch's
 * results are in its host buffers.  Inputs, y and the histograms are double-buffered on the device, so
 * the copies of batch i+1 and of batch i-1 run while the kernels of batch i do.  Two batches can be in
 * flight: wait for ticket i-1 (at the latest) before submitting batch i+1.  A submit issued while two
 * batches are still undelivered does not fail: it blocks on the host until the older of them has reached
 * its host buffers (so it degrades to a synchronous call), and a later wait for that ticket returns at
 * once.  wait never returns DIRECTOR_OK before the batch's y and histograms are in host memory.  The host
 * buffers of a batch (pinned, for real overlap) must stay valid and untouched until its wait returns or
 * until two later submits have returned.
 * Arguments as for director_layer_forward_host; ticket: host, receives the batch's sequence number. */
int director_layer_submit_host(director_ctx* ctx, int32_t T, const float* logits, const void* x,
                               const void* w_gate, const void* w_up, const void* w_down,
                               const void* ws_gate, const void* ws_up, const void* ws_down,
                               void* y, int64_t* rank_load, uint64_t* dispatch_bytes, void* stream,
                               int64_t* ticket);
int director_layer_wait_host(director_ctx* ctx, int64_t ticket);

/* Synchronises `stream`, returns the sticky device status word (DIRECTOR_OK if clean) and
 * clears it. */
int director_last_status(director_ctx* ctx, void* stream);

/* Self-test of the failure-detection path (not part of the layer).  Every wait inside the GEMM pipelines
 * is bounded: when a wait runs out, the waiting role raises its CTA's abort flag, every role leaves its
 * loop, and the kernel records DIRECTOR_ERR_TIMEOUT in the sticky status word instead of hanging the
 * GPU.  This call launches a one-warp kernel that waits, with that same helper, on an mbarrier nobody
 * arrives at, for at most limit_ns (1 us .. 100 ms) - so the wait expires by construction, harmlessly.
 * Afterwards director_last_status returns DIRECTOR_ERR_TIMEOUT once, then DIRECTOR_OK, and the context
 * is usable as before.  waited_ns: dev uint64 [1] or NULL, receives the nanoseconds the wait lasted.
 * Returns DIRECTOR_ERR_INVALID_ARG for a limit outside the range. */
int director_selftest_bounded_wait(director_ctx* ctx, uint64_t limit_ns, uint64_t* waited_ns, void* stream);

/* Tile scheme of the expert-FFN GEMMs (results are bit-identical across the tensor-core schemes):
 *   2 (default) weight-stationary CTA pairs: 256 weight rows x up to 256 tokens per tile, the token count
 *               of a tile is a runtime operand in steps of 32, so ragged segment tails cost almost nothing;
 *               batches of at most 4 tokens take the weight-streaming kernels instead (see director_expert_ffn);
 *   1           token-stationary CTA pairs: 256 tokens x 256 weight rows per tile;
 *   0           token-stationary single CTAs: 128 tokens x 256 weight rows per tile;
 *   6           scheme 2 with the tensor-core kernels for every batch size.
 * Scheme 2 falls back to scheme 0 when w_gate and w_up cannot be described by one strided tensor map
 * (their addresses differ by 2^40 bytes or more). */
int director_set_ffn_variant(director_ctx* ctx, int32_t variant);

/* 1 if a batch of T tokens takes the weight-streaming FFN kernels under the current tile scheme (T <= 4, scheme 2, and
 * the rows of a segment fit in shared memory), 0 if it takes the tensor-core kernels, -DIRECTOR_ERR_INVALID_ARG for a
 * NULL context or T outside [1, T_max].  A caller that drives the stages itself can then skip the row copies: xp = NULL in
 * director_dispatch / director_route_dispatch_cost, followed by director_expert_ffn_gather.  No paper counterpart
 * (an implementation detail of Section II-A's expert FFNs at decode-sized batches). */
int director_batch_streams_weights(director_ctx* ctx, int32_t T);

/* SM clock the expert GEMMs really ran at.  Every CTA of a grouped-GEMM launch reads the SM cycle counter and
 * the global nanosecond timer when it starts and when it ends; this call synchronises the device and returns
 * (sum of cycles) / (sum of nanoseconds) over the CTAs of the context's most recent launch, in MHz.
 * which: 0 = gate|up GEMM, 1 = down GEMM.  busy_us: host, or NULL; receives the longest CTA's time in
 * microseconds.  A host-side clock sampler has millisecond resolution and lags; this is the clock during
 * the kernel itself, the one a tensor-pipe roofline has to be read against.  Negative on error. */
double director_gemm_sm_mhz(director_ctx* ctx, int32_t which, double* busy_us);

/* What the expert GEMM kernels (default tile scheme) measured about themselves in their most recent launch, summed
 * over the CTAs; which: 0 = gate|up GEMM, 1 = down GEMM; out: host int64 [DIRECTOR_GEMM_COUNTERS].  Synchronises
 * the device.  All times are SM cycles of the reading thread unless noted:
 *   [0] cycles and [1] nanoseconds every CTA spent in the kernel (cycles / ns = SM clock);
 *   the MMA-issuing thread of every CTA pair: [2] cycles waiting for a free accumulator buffer (the epilogue of
 *   an earlier tile had not finished), [3] cycles from an item's first operand wait to the issue of its last MMA,
 *   [4] k-steps issued, [5] work items (so [3] / [4] = cycles per k-step as the issuing thread sees them);
 *   one epilogue warp of every CTA: [6] cycles waiting for a complete accumulator, [7] cycles draining
 *   accumulators (tensor memory -> registers -> bf16 -> global), [8] token tiles drained;
 *   [9] reserved;  [10] the longest CTA's nanoseconds;  [11] number of CTAs summed. */
#define DIRECTOR_GEMM_COUNTERS 12
int director_gemm_counters(director_ctx* ctx, int32_t which, int64_t* out);

/* Number of kernels this context has launched since it was created. */
int64_t director_launch_count(const director_ctx* ctx);

/* Device timing.  enabled = 1: every kernel launch is bracketed by CUDA events on its stream.  enabled = 2:
 * every STAGE (route, dispatch, expert FFN, combine, placement cost; all kernels and memsets of the stage) is
 * bracketed by one pair of events, recorded under the names "stage_route", "stage_dispatch", "stage_expert_ffn",
 * "stage_combine", "stage_placement_cost" ("stage_front_small" for the one-launch front end of decode batches) -
 * the stage's time on an otherwise idle stream with the event pair paid once.  enabled = 0: off.
 * director_kernel_time synchronises the device, then returns the summed duration in milliseconds and the
 * number of brackets whose name contains `name_substr` since profiling was last enabled; negative on error. */
int director_set_profiling(director_ctx* ctx, int32_t enabled);
/* Restricts the timing to kernels whose name contains `name_substr` (NULL or "" = all kernels): two event records
 * per launch are cheap but not free, and a measurement that wants one kernel's duration inside an otherwise
 * undisturbed run times only that kernel. */
int director_set_profiling_filter(director_ctx* ctx, const char* name_substr);
double director_kernel_time(director_ctx* ctx, const char* name_substr, int64_t* launches);

const char* director_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* DIRECTOR_H */
