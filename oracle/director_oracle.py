"""CPU oracle for the expert-parallel MoE layer forward under an expert placement.

THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, fp64 restatement of what
the layer computes, written from the paper's definitions so that it can be checked against
them by eye.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may use it;
it shares no code with the CUDA library and never calls it.

Notation follows the paper (Section VI-A): T tokens, E experts (0-based here, the paper counts
from 1), G = set of GPUs -> R logical ranks, C_max = expert slots per rank, placement variable
x_{i,j} -> matrix X[E, R] in {0,1} (expert i hosted on rank j; "sum_j x_{i,j} >= 1" allows
replicas, "sum_i x_{i,j} <= C_max" is the capacity), workload matrix W[j, i] = tokens on rank
j routed to expert i.

Where the paper fixes no detail, the reading taken is stated at the function.  Those readings
(tie-breaks, renormalised top-k softmax, round-robin and locality-first replica choice, the
de-duplicated dispatch volume, block partition of tokens over source ranks, shared experts,
SwiGLU) are **parity unpinned by the paper**: they are
pinned only by the invariants in the CPU tests (weights sum to one, identity round trip,
loads sum to T*K, capacity, brute-force counts, scalar-loop FFN, closed forms).
"""
from __future__ import annotations

import numpy as np


# ----------------------------------------------------------------------------------------------
# helpers (input decoding only)
# ----------------------------------------------------------------------------------------------

def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact value of bf16 bit patterns (uint16) as fp64.  Arrays that are already fp64 pass through,
    so callers may decode their weights once and keep them resident in the compute precision."""
    bits = np.asarray(bits)
    if bits.dtype == np.float64:
        return bits
    assert bits.dtype == np.uint16
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def f64_to_bf16_bits(v: np.ndarray) -> np.ndarray:
    """fp64 -> fp32 -> bf16 (round to nearest even) bit patterns; used to compare with bf16 outputs."""
    u = np.asarray(v, dtype=np.float64).astype(np.float32).view(np.uint32)
    u = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (u >> np.uint32(16)).astype(np.uint16)


# ----------------------------------------------------------------------------------------------
# (a1) gating: Section II-A (the gate scores the experts per token, keeps the k best, their scores weight the sum)
# ----------------------------------------------------------------------------------------------

def route(logits: np.ndarray, K: int):
    """Top-k softmax gating.

    Scores are the softmax over all E experts of the fp32 router logits (computed in fp64).
    The K experts are chosen on the raw logits in the order (logit descending, expert id
    ascending); the K scores are renormalised to sum to one.

    Returns (topk_idx int32 [T,K], topk_w float32 [T,K], topk_w64 float64 [T,K]).
    """
    l = np.asarray(logits, dtype=np.float32)
    T, E = l.shape
    assert 1 <= K <= E
    l64 = l.astype(np.float64)
    m = l64.max(axis=1, keepdims=True) if T else l64
    p = np.exp(l64 - m)
    p /= p.sum(axis=1, keepdims=True)
    # stable sort of the negated logits: equal logits keep ascending expert id
    order = np.argsort(-l, axis=1, kind="stable")
    idx = order[:, :K].astype(np.int32)
    pk = np.take_along_axis(p, idx.astype(np.int64), axis=1)
    w64 = pk / pk.sum(axis=1, keepdims=True)
    return idx, w64.astype(np.float32), w64


# ----------------------------------------------------------------------------------------------
# source ranks: Section VI-A (every token lives on one GPU; W counts tokens per GPU and expert)
# ----------------------------------------------------------------------------------------------

def source_ranks(T: int, R: int) -> np.ndarray:
    """Default home rank of each token: contiguous balanced blocks, src(t) = floor(t*R/T)."""
    t = np.arange(T, dtype=np.int64)
    return ((t * R) // max(T, 1)).astype(np.int32)


# ----------------------------------------------------------------------------------------------
# placement structures: Section VI-A placement map, Eq. 6 assignment and capacity constraints
# ----------------------------------------------------------------------------------------------

class PlacementError(ValueError):
    pass


def placement_tables(X: np.ndarray, C_max: int):
    """From X[E,R]: reps[e] = ascending ranks hosting e; hosted[j] = ascending experts on rank j;
    slot_expert[j*C_max + p] = hosted[j][p] (or -1 for an unused slot).

    Raises PlacementError when an expert has no host (violates sum_j x_{i,j} >= 1) or a rank
    holds more than C_max experts (violates sum_i x_{i,j} <= C_max).
    """
    X = np.asarray(X)
    E, R = X.shape
    if not np.isin(X, (0, 1)).all():
        raise PlacementError("placement entries must be 0 or 1")
    reps = [np.flatnonzero(X[e]).astype(np.int64) for e in range(E)]
    hosted = [np.flatnonzero(X[:, j]).astype(np.int64) for j in range(R)]
    for e in range(E):
        if len(reps[e]) < 1:
            raise PlacementError(f"expert {e} has no host")
    for j in range(R):
        if len(hosted[j]) > C_max:
            raise PlacementError(f"rank {j} hosts {len(hosted[j])} > C_max={C_max} experts")
    slot_expert = np.full(R * C_max, -1, dtype=np.int32)
    for j in range(R):
        slot_expert[j * C_max: j * C_max + len(hosted[j])] = hosted[j]
    return reps, hosted, slot_expert


def _slot_of(hosted, C_max: int, rank: int, e: int) -> int:
    return rank * C_max + int(np.searchsorted(hosted[rank], e))


# ----------------------------------------------------------------------------------------------
# (a2) dispatch: Section II-B (first all-to-all: every token travels to the GPUs that host its chosen experts)
# ----------------------------------------------------------------------------------------------

def dispatch(topk_idx: np.ndarray, X: np.ndarray, C_max: int, x_bits: np.ndarray | None = None,
             policy: str = "round_robin", src: np.ndarray | None = None):
    """Placement-aware permutation of the T*K (token, choice) assignments.

    policy "local_first" is handled by dispatch_local_first (below); the text here is the default
    round-robin rule.

    For expert e take its assignments in ascending token id, n = 0,1,... being the position in
    that list.  With r_e replicas on ranks reps[e][0] < reps[e][1] < ..., assignment n goes to
    replica q = n mod r_e (round-robin) and is the (n div r_e)-th row of that replica's
    segment.  Segments are laid out in slot order (rank ascending, expert id ascending inside a
    rank); seg_offsets is the exclusive prefix sum of segment lengths.

    Returns dict: row_token int32 [A], inv_row int32 [T,K], dest_rank int32 [T,K],
    seg_offsets int32 [R*C_max+1], slot_expert int32 [R*C_max], xp (uint16 [A,H] or None).
    """
    if policy == "local_first":
        return dispatch_local_first(topk_idx, X, C_max, x_bits, src)
    if policy != "round_robin":
        raise ValueError(policy)
    idx = np.asarray(topk_idx)
    T, K = idx.shape
    E, R = np.asarray(X).shape
    A = T * K
    reps, hosted, slot_expert = placement_tables(X, C_max)
    G = R * C_max

    seg_len = np.zeros(G, dtype=np.int64)
    per_expert = []
    for e in range(E):
        tt, ss = np.nonzero(idx == e)          # row-major scan => ascending token id
        per_expert.append((tt, ss))
        r_e = len(reps[e])
        for q in range(r_e):
            n_e = len(tt)
            cnt = 0 if n_e <= q else -(-(n_e - q) // r_e)
            seg_len[_slot_of(hosted, C_max, int(reps[e][q]), e)] = cnt
    seg_offsets = np.zeros(G + 1, dtype=np.int64)
    seg_offsets[1:] = np.cumsum(seg_len)
    assert seg_offsets[G] == A

    inv_row = np.full((T, K), -1, dtype=np.int32)
    dest_rank = np.full((T, K), -1, dtype=np.int32)
    row_token = np.full(A, -1, dtype=np.int32)
    for e in range(E):
        tt, ss = per_expert[e]
        r_e = len(reps[e])
        slots_e = np.array([_slot_of(hosted, C_max, int(j), e) for j in reps[e]], dtype=np.int64)
        n = np.arange(len(tt), dtype=np.int64)
        q = n % r_e
        row = seg_offsets[slots_e[q]] + n // r_e
        inv_row[tt, ss] = row
        dest_rank[tt, ss] = reps[e][q]
        row_token[row] = tt
    xp = None
    if x_bits is not None:
        xp = np.asarray(x_bits)[row_token]       # exact row copies
    return dict(row_token=row_token, inv_row=inv_row, dest_rank=dest_rank,
                seg_offsets=seg_offsets.astype(np.int32), slot_expert=slot_expert, xp=xp)


def dispatch_local_first(topk_idx: np.ndarray, X: np.ndarray, C_max: int, x_bits: np.ndarray | None = None,
                         src: np.ndarray | None = None):
    """Locality-first replica choice (a reading of this build: the paper replicates experts to cut
    the dispatch volume of Eq. 3 but does not say which replica a token uses).

    Token t lives on rank src(t) (default: source_ranks).  Its assignment to expert e
      * stays on rank src(t) when that rank hosts a replica of e (x_{e,src(t)} = 1);
      * otherwise it is the m-th such "travelling" assignment of e in ascending token id
        (m = 0,1,...) and goes to replica reps[e][m mod r_e].
    A segment (rank, expert) holds the assignments that chose it in ascending token id; segments
    are laid out in slot order exactly as in the round-robin rule.  Same outputs as dispatch().
    """
    idx = np.asarray(topk_idx)
    T, K = idx.shape
    Xa = np.asarray(X)
    E, R = Xa.shape
    A = T * K
    reps, hosted, slot_expert = placement_tables(Xa, C_max)
    G = R * C_max
    src = source_ranks(T, R) if src is None else np.asarray(src)

    dest_rank = np.full((T, K), -1, dtype=np.int32)
    travelling = np.zeros(E, dtype=np.int64)            # m counter per expert
    for t in range(T):                                  # ascending token id
        for s in range(K):
            e = int(idx[t, s])
            j = int(src[t])
            if Xa[e, j]:
                dest_rank[t, s] = j
            else:
                dest_rank[t, s] = reps[e][travelling[e] % len(reps[e])]
                travelling[e] += 1

    slot = np.empty((T, K), dtype=np.int64)
    for t in range(T):
        for s in range(K):
            slot[t, s] = _slot_of(hosted, C_max, int(dest_rank[t, s]), int(idx[t, s]))
    seg_len = np.bincount(slot.reshape(-1), minlength=G)
    seg_offsets = np.zeros(G + 1, dtype=np.int64)
    seg_offsets[1:] = np.cumsum(seg_len)
    assert seg_offsets[G] == A

    inv_row = np.full((T, K), -1, dtype=np.int32)
    row_token = np.full(A, -1, dtype=np.int32)
    fill = seg_offsets[:-1].copy()
    for t in range(T):                                  # ascending token id inside every segment
        for s in range(K):
            g = slot[t, s]
            inv_row[t, s] = fill[g]
            row_token[fill[g]] = t
            fill[g] += 1
    xp = None
    if x_bits is not None:
        xp = np.asarray(x_bits)[row_token]
    return dict(row_token=row_token, inv_row=inv_row, dest_rank=dest_rank,
                seg_offsets=seg_offsets.astype(np.int32), slot_expert=slot_expert, xp=xp)


def dedup_dispatch_tokens(dest_rank: np.ndarray, src: np.ndarray, R: int) -> np.ndarray:
    """Dispatch volume in tokens when a token whose several experts sit on one rank is sent there once:
    U[j,k] = number of distinct tokens on rank j with at least one assignment executed on rank k.
    (Eq. 3 counts every assignment; this is the volume a de-duplicating all-to-all would move.)"""
    dest = np.asarray(dest_rank)
    U = np.zeros((R, R), dtype=np.int64)
    for t in range(dest.shape[0]):
        for k in set(int(v) for v in dest[t] if v >= 0):
            U[int(src[t]), k] += 1
    return U


# ----------------------------------------------------------------------------------------------
# (a3) expert FFN: Section II-A (an expert is a feed-forward sub-network; here SwiGLU, no bias)
# ----------------------------------------------------------------------------------------------

def swiglu_ffn_rows(rows_f64: np.ndarray, wg_bits, wu_bits, wd_bits) -> np.ndarray:
    """One expert on a block of rows, fp64 throughout, no intermediate rounding:
    g = rows . Wg^T, u = rows . Wu^T, a = g/(1+exp(-g)) * u, out = a . Wd^T.
    wg, wu: [F,H]; wd: [H,F]; bf16 bits or already-decoded fp64."""
    wg, wu, wd = bf16_to_f64(wg_bits), bf16_to_f64(wu_bits), bf16_to_f64(wd_bits)
    g = rows_f64 @ wg.T
    u = rows_f64 @ wu.T
    a = g / (1.0 + np.exp(-g)) * u
    return a @ wd.T


def expert_ffn(xp_bits: np.ndarray, seg_offsets: np.ndarray, slot_expert: np.ndarray,
               w_gate, w_up, w_down, rows: np.ndarray | None = None) -> np.ndarray:
    """Grouped FFN over the permuted rows: every row of segment g runs expert slot_expert[g].
    If ``rows`` (sorted global row ids) is given only those rows are computed and returned in
    that order; otherwise all A rows."""
    A, H = xp_bits.shape
    sel = np.arange(A, dtype=np.int64) if rows is None else np.asarray(rows, dtype=np.int64)
    out = np.zeros((len(sel), H), dtype=np.float64)
    for g in range(len(slot_expert)):
        lo, hi = int(seg_offsets[g]), int(seg_offsets[g + 1])
        if hi <= lo:
            continue
        m = (sel >= lo) & (sel < hi)
        if not m.any():
            continue
        e = int(slot_expert[g])
        out[m] = swiglu_ffn_rows(bf16_to_f64(xp_bits[sel[m]]), w_gate[e], w_up[e], w_down[e])
    return out


def shared_ffn(x_bits: np.ndarray, ws_gate, ws_up, ws_down, tokens: np.ndarray | None = None) -> np.ndarray:
    """Always-on shared experts: every token's own row goes through each of the S shared FFNs
    and the S outputs are added (weight 1, no gate).  ws_gate, ws_up: [S,F,H]; ws_down: [S,H,F]."""
    sel = np.arange(x_bits.shape[0]) if tokens is None else np.asarray(tokens)
    rows = bf16_to_f64(x_bits[sel])
    out = np.zeros((len(sel), x_bits.shape[1]), dtype=np.float64)
    for s in range(ws_gate.shape[0]):
        out += swiglu_ffn_rows(rows, ws_gate[s], ws_up[s], ws_down[s])
    return out


# ----------------------------------------------------------------------------------------------
# (a4) combine: Section II-A weighted summation; Section II-B second all-to-all
# ----------------------------------------------------------------------------------------------

def combine(yp: np.ndarray, inv_row: np.ndarray, topk_w: np.ndarray, y_shared: np.ndarray | None = None) -> np.ndarray:
    """y[t] = sum_s w[t,s] * yp[inv_row[t,s]] (+ y_shared[t]); fp64."""
    T, K = inv_row.shape
    y = np.zeros((T, yp.shape[1]), dtype=np.float64)
    w = np.asarray(topk_w, dtype=np.float64)
    for s in range(K):
        y += w[:, s:s + 1] * yp[inv_row[:, s]]
    if y_shared is not None:
        y += y_shared
    return y


# ----------------------------------------------------------------------------------------------
# (a5) placement cost: Section VI-A workload matrix W, Eq. 1 (load), Eq. 3 (dispatch volume)
# ----------------------------------------------------------------------------------------------

def placement_cost(topk_idx: np.ndarray, X: np.ndarray, C_max: int, H: int, src: np.ndarray | None = None,
                   policy: str = "round_robin"):
    """Per executed assignment (token t on rank src(t), expert e, destination replica rank k):
    W[src, e] += 1;  rank_load[k] += 1 (Eq. 1 counted per executed assignment);
    dispatch_tokens[src, k] += 1;  dispatch_bytes = dispatch_tokens * d with d = 2*H bytes
    (one bf16 hidden state, Eq. 3).  The diagonal of the dispatch matrices is local traffic
    (Eq. 4 sums k != j only).  Shared experts add nothing."""
    idx = np.asarray(topk_idx)
    T, K = idx.shape
    E, R = np.asarray(X).shape
    if src is None:
        src = source_ranks(T, R)
    dest = dispatch(idx, X, C_max, policy=policy, src=src)["dest_rank"]
    W = np.zeros((R, E), dtype=np.int64)
    lam = np.zeros(R, dtype=np.int64)
    D = np.zeros((R, R), dtype=np.int64)
    src_a = np.repeat(np.asarray(src, dtype=np.int64), K)
    np.add.at(W, (src_a, idx.reshape(-1).astype(np.int64)), 1)
    np.add.at(lam, dest.reshape(-1).astype(np.int64), 1)
    np.add.at(D, (src_a, dest.reshape(-1).astype(np.int64)), 1)
    return dict(workload=W, rank_load=lam, dispatch_tokens=D,
                dispatch_bytes=(D * (2 * H)).astype(np.uint64))


def cost_summary(cost: dict) -> dict:
    """Host-side reductions the optimiser's objective is built from: the straggler load of
    Eq. 2 (max_j lambda_j) and the straggler send volume of Eq. 4 (max_j sum_{k != j} D[j,k])."""
    D = cost["dispatch_bytes"].astype(np.int64)
    off = D.sum(axis=1) - np.diag(D)
    return dict(max_rank_load=int(cost["rank_load"].max()), cross_rank_bytes=int(off.sum()),
                max_send_bytes=int(off.max()), send_bytes=off)


# ----------------------------------------------------------------------------------------------
# load-balanced placement used as an *input* by some workloads (greedy; not the paper's LP)
# ----------------------------------------------------------------------------------------------

def _replica_count(n_e: int, q: int, r_e: int) -> int:
    return 0 if n_e <= q else -(-(n_e - q) // r_e)


def balanced_placement(N: np.ndarray, R: int, C_max: int, primary: np.ndarray | None = None) -> np.ndarray:
    """Greedy replica-and-pack placement from per-expert token counts N[e].

    Phase A: hand the R*C_max - E spare slots one at a time to the expert with the largest
    N_e / r_e (ties -> lower id), never beyond R copies, never to an expert with no tokens.
    Phase B: copies are packed largest-first (count desc, expert asc, copy asc) onto the least
    loaded rank that has a free slot and does not host that expert yet (ties -> lower rank);
    a copy that fits nowhere is dropped.  If ``primary`` (rank per expert) is given, copy 0 of
    every expert is pinned there first.  Integer arithmetic only.  Returns X uint8 [E,R].
    """
    N = [int(v) for v in N]
    E = len(N)
    r = [1] * E
    spare = R * C_max - E
    assert spare >= 0
    while spare > 0:
        best = -1
        for e in range(E):
            if r[e] >= R or N[e] <= 0:
                continue
            # N[e]/r[e] > N[best]/r[best]  <=>  N[e]*r[best] > N[best]*r[e]
            if best < 0 or N[e] * r[best] > N[best] * r[e]:
                best = e
        if best < 0:
            break
        r[best] += 1
        spare -= 1
    X = np.zeros((E, R), dtype=np.uint8)
    load = [0] * R
    used = [0] * R
    copies = []
    for e in range(E):
        q0 = 0
        if primary is not None:
            j = int(primary[e])
            X[e, j] = 1
            used[j] += 1
            load[j] += _replica_count(N[e], 0, r[e])
            q0 = 1
        for q in range(q0, r[e]):
            copies.append((-_replica_count(N[e], q, r[e]), e, q))
    copies.sort()
    for negc, e, q in copies:
        best = -1
        for j in range(R):
            if used[j] >= C_max or X[e, j]:
                continue
            if best < 0 or load[j] < load[best]:
                best = j
        if best < 0:
            continue
        X[e, best] = 1
        used[best] += 1
        load[best] += -negc
    return X


def replicate_hottest(N: np.ndarray, X: np.ndarray, n_hot: int = 2) -> np.ndarray:
    """Add one replica of each of the n_hot experts with the most tokens (ties -> lower id) on the
    currently least-loaded rank that does not host it yet (ties -> lower rank); loads are those
    of the given single-copy placement X (Eq. 1) and are not updated between the additions,
    but a rank is used for at most one new replica."""
    N = np.asarray(N, dtype=np.int64)
    X = np.array(X, dtype=np.uint8)
    E, R = X.shape
    lam = np.array([int(N[X[:, j] == 1].sum()) for j in range(R)], dtype=np.int64)
    hot = sorted(range(E), key=lambda e: (-int(N[e]), e))[:n_hot]
    taken = set()
    for e in hot:
        cands = [j for j in range(R) if not X[e, j] and j not in taken]
        j = min(cands, key=lambda j: (int(lam[j]), j))
        X[e, j] = 1
        taken.add(j)
    return X
