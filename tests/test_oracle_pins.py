"""Pins for the CPU oracle: each check ties one oracle function to something other than the
oracle itself - a closed form, an invariant the method guarantees, a textbook/library routine
the function must reduce to in a special case, or brute force on tiny inputs.  (The paper
prints no worked numeric example for this path.)"""
import itertools
import math

import numpy as np
import pytest
import scipy.special

from oracle import director_oracle as orc
from paper_2607_08782_b200 import synth


def _rng(seed):
    return np.random.default_rng(seed)


def _random_placement(rng, E, R, C_max, extra=0):
    """Random valid placement: every expert once, then `extra` replicas where room remains."""
    while True:
        X = np.zeros((E, R), dtype=np.uint8)
        slots = [j for j in range(R) for _ in range(C_max)]
        rng.shuffle(slots)
        for e in range(E):
            X[e, slots[e]] = 1
        ok = True
        for _ in range(extra):
            free = [(e, j) for e in range(E) for j in range(R) if not X[e, j] and X[:, j].sum() < C_max]
            if not free:
                ok = False
                break
            e, j = free[rng.integers(len(free))]
            X[e, j] = 1
        if ok:
            return X


# ------------------------------------------------------------------------------- route (a1)

def test_route_hand_example_closed_form():
    # logits ln(1..4): softmax = (.1,.2,.3,.4); top-2 = experts 3,2 with weights 4/7, 3/7
    l = np.log(np.array([[1.0, 2.0, 3.0, 4.0]])).astype(np.float32)
    idx, w, w64 = orc.route(l, 2)
    assert idx.tolist() == [[3, 2]]
    assert np.allclose(w64, [[4 / 7, 3 / 7]], atol=1e-7)
    assert w.dtype == np.float32 and idx.dtype == np.int32


def test_route_weights_sum_to_one_and_descend():
    l = synth.make_logits(synth.shape_for("c1_tiny"))
    idx, w, w64 = orc.route(l, 2)
    assert np.allclose(w64.sum(axis=1), 1.0, atol=1e-12)
    assert np.all(np.abs(w.astype(np.float64).sum(axis=1) - 1.0) <= 1e-6)
    assert np.all(w64[:, 0] >= w64[:, 1])
    # the chosen experts are distinct
    assert np.all(idx[:, 0] != idx[:, 1])


def test_route_all_equal_logits_tie_break_and_uniform_weights():
    l = np.full((5, 8), 0.25, dtype=np.float32)
    idx, w, _ = orc.route(l, 3)
    assert np.array_equal(idx, np.tile(np.arange(3, dtype=np.int32), (5, 1)))
    assert np.allclose(w, 1.0 / 3.0, atol=1e-7)


def test_route_signed_zero_is_a_tie():
    l = np.array([[-0.0, 0.0, -1.0, 0.0]], dtype=np.float32)
    idx, _, _ = orc.route(l, 3)
    assert idx.tolist() == [[0, 1, 3]]


def test_route_k_equals_e_is_the_library_softmax():
    l = _rng(0).normal(size=(17, 6)).astype(np.float32)
    idx, _, w64 = orc.route(l, 6)
    full = scipy.special.softmax(l.astype(np.float64), axis=1)
    assert np.allclose(np.take_along_axis(full, idx.astype(np.int64), 1), w64, atol=1e-14)
    assert np.array_equal(np.sort(idx, axis=1), np.tile(np.arange(6), (17, 1)))


def test_route_shift_invariance_and_softmax_over_winners():
    l = _rng(1).normal(size=(33, 10)).astype(np.float32)
    idx, _, w64 = orc.route(l, 4)
    idx2, _, w64b = orc.route((l.astype(np.float64) + 2.0).astype(np.float32), 4)
    # +2.0 is exact for these magnitudes only up to rounding: compare selection where unaffected
    assert np.mean(idx == idx2) > 0.99
    # renormalised top-k of the full softmax == softmax over the K winning logits
    lk = np.take_along_axis(l.astype(np.float64), idx.astype(np.int64), 1)
    assert np.allclose(scipy.special.softmax(lk, axis=1), w64, atol=1e-14)


def test_route_selection_brute_force():
    rng = _rng(2)
    l = rng.integers(-3, 4, size=(40, 7)).astype(np.float32)   # many ties
    idx, _, _ = orc.route(l, 3)
    for t in range(l.shape[0]):
        taken = []
        for _ in range(3):
            best = None
            for e in range(l.shape[1]):
                if e in taken:
                    continue
                if best is None or l[t, e] > l[t, best]:
                    best = e
            taken.append(best)
        assert idx[t].tolist() == taken


# ------------------------------------------------------------------------------ dispatch (a2)

def _brute_dispatch(idx, X, C_max):
    """Sort-based simulation: walk tokens in order, give each expert's n-th assignment to replica
    n mod r_e, then order all assignments by (destination rank, expert id, token id)."""
    T, K = idx.shape
    E, R = X.shape
    reps = [[j for j in range(R) if X[e, j]] for e in range(E)]
    seen = [0] * E
    items = []
    for t in range(T):
        for s in range(K):
            e = int(idx[t, s])
            items.append((reps[e][seen[e] % len(reps[e])], e, t, s))
            seen[e] += 1
    items.sort()
    inv_row = np.zeros((T, K), dtype=np.int32)
    dest = np.zeros((T, K), dtype=np.int32)
    row_token = np.zeros(T * K, dtype=np.int32)
    for row, (j, e, t, s) in enumerate(items):
        inv_row[t, s], dest[t, s], row_token[row] = row, j, t
    seg = np.zeros(R * C_max + 1, dtype=np.int64)
    for j in range(R):
        hosted = [e for e in range(E) if X[e, j]]
        for p, e in enumerate(hosted):
            seg[j * C_max + p + 1] = sum(1 for it in items if it[0] == j and it[1] == e)
    return inv_row, dest, row_token, np.cumsum(seg).astype(np.int32)


@pytest.mark.parametrize("seed,E,K,R,C,extra", [(0, 8, 2, 4, 2, 0), (1, 8, 2, 4, 3, 4), (2, 6, 3, 3, 4, 5),
                                                 (3, 5, 5, 2, 5, 3), (4, 4, 1, 4, 1, 0)])
def test_dispatch_equals_sort_based_brute_force(seed, E, K, R, C, extra):
    rng = _rng(seed)
    T = 37
    l = rng.normal(size=(T, E)).astype(np.float32) - np.arange(E, dtype=np.float32)
    idx, _, _ = orc.route(l, K)
    X = _random_placement(rng, E, R, C, extra)
    d = orc.dispatch(idx, X, C)
    inv_row, dest, row_token, seg = _brute_dispatch(idx, X, C)
    assert np.array_equal(d["inv_row"], inv_row)
    assert np.array_equal(d["dest_rank"], dest)
    assert np.array_equal(d["row_token"], row_token)
    assert np.array_equal(d["seg_offsets"], seg)


def test_dispatch_structure_invariants_on_c1():
    wl = synth.make_workload("c1_tiny")
    s = wl.shape
    idx, _, _ = orc.route(wl.logits, s.K)
    N = np.bincount(idx.ravel(), minlength=s.E)
    for X in (wl.X_primary, orc.balanced_placement(N, s.R, 3), ):
        C = 3 if X.sum() > s.E else s.C_max
        d = orc.dispatch(idx, X, C, wl.x)
        A = s.T * s.K
        assert sorted(d["inv_row"].ravel().tolist()) == list(range(A))            # bijection
        t_of = np.repeat(np.arange(s.T), s.K).reshape(s.T, s.K)
        assert np.array_equal(d["row_token"][d["inv_row"]], t_of)
        so = d["seg_offsets"]
        assert so[0] == 0 and so[-1] == A and np.all(np.diff(so) >= 0)
        for g in range(s.R * C):
            rows = d["row_token"][so[g]:so[g + 1]]
            assert np.all(np.diff(rows) > 0)                                       # ascending tokens
            if len(rows):
                e = d["slot_expert"][g]
                assert e >= 0 and X[e, g // C] == 1
                # every row of the segment really chose expert e
                assert all(e in idx[t] for t in rows)
        # replica segment lengths of one expert differ by at most one and sum to N_e
        for e in range(s.E):
            lens = [so[g + 1] - so[g] for g in range(s.R * C) if d["slot_expert"][g] == e]
            assert sum(lens) == N[e] and max(lens) - min(lens) <= 1
        assert np.array_equal(d["xp"], wl.x[d["row_token"]])


def test_dispatch_single_copy_is_stable_sort_by_rank_then_expert():
    rng = _rng(7)
    T, E, K, R, C = 200, 12, 3, 4, 3
    idx, _, _ = orc.route(rng.normal(size=(T, E)).astype(np.float32), K)
    ranks = np.repeat(np.arange(R), C)[rng.permutation(E)]
    X = synth.placement_from_ranks(ranks, R)
    d = orc.dispatch(idx, X, C)
    flat_e = idx.ravel()
    flat_t = np.repeat(np.arange(T), K)
    order = np.lexsort((flat_t, flat_e, ranks[flat_e]))       # library sort: last key is primary
    assert np.array_equal(d["row_token"], flat_t[order])
    assert np.array_equal(d["dest_rank"].ravel(), ranks[flat_e])


def test_placement_validation():
    X = np.zeros((4, 2), dtype=np.uint8)
    X[[0, 1, 2], [0, 0, 1]] = 1
    with pytest.raises(orc.PlacementError):        # expert 3 unhosted: violates sum_j x_ij >= 1
        orc.placement_tables(X, 2)
    X[3, 0] = 1
    with pytest.raises(orc.PlacementError):        # rank 0 hosts 3 > C_max
        orc.placement_tables(X, 2)
    orc.placement_tables(X, 3)


# ------------------------------------------------------------- identity round trip (a2 + a4)

def test_dispatch_then_combine_with_identity_experts_reproduces_input():
    wl = synth.make_workload("c1_tiny")
    s = wl.shape
    idx, w, w64 = orc.route(wl.logits, s.K)
    d = orc.dispatch(idx, wl.X_primary, s.C_max, wl.x)
    yp = orc.bf16_to_f64(d["xp"])
    y = orc.combine(yp, d["inv_row"], w64)
    assert np.allclose(y, orc.bf16_to_f64(wl.x), rtol=0, atol=1e-14)
    # with the fp32-rounded weights the result still rounds back to the same bf16 values
    y32 = orc.combine(yp, d["inv_row"], w)
    assert np.array_equal(orc.f64_to_bf16_bits(y32), wl.x)
    # one-hot weights: exact in any precision
    onehot = np.zeros_like(w64)
    onehot[:, 0] = 1.0
    assert np.array_equal(orc.combine(yp, d["inv_row"], onehot), orc.bf16_to_f64(wl.x))


def test_combine_is_the_weighted_sum_by_loops():
    rng = _rng(3)
    T, K, H = 5, 3, 4
    yp = rng.normal(size=(T * K, H))
    inv = rng.permutation(T * K).reshape(T, K).astype(np.int32)
    w = rng.random(size=(T, K))
    ysh = rng.normal(size=(T, H))
    got = orc.combine(yp, inv, w, ysh)
    for t in range(T):
        for h in range(H):
            want = sum(w[t, s] * yp[inv[t, s], h] for s in range(K)) + ysh[t, h]
            assert abs(got[t, h] - want) < 1e-14


# -------------------------------------------------------------------------------- FFN (a3)

def _scalar_ffn(x, wg, wu, wd):
    """Scalar triple loop of the SwiGLU FFN with math.exp: independent of any matmul routine."""
    H, F = len(x), len(wg)
    a = []
    for f in range(F):
        g = sum(x[h] * wg[f][h] for h in range(H))
        u = sum(x[h] * wu[f][h] for h in range(H))
        a.append(g / (1.0 + math.exp(-g)) * u)
    return [sum(a[f] * wd[h][f] for f in range(F)) for h in range(H)]


def test_ffn_matches_scalar_loops_on_tiny_grouped_problem():
    T, H, F, E, K, R, C = 6, 8, 16, 3, 2, 2, 2
    sd = 77
    x = synth.normal_bf16(sd, 2, (T, H), 0.5)
    wg = synth.normal_bf16(sd, 3, (E, F, H), 0.3)
    wu = synth.normal_bf16(sd, 4, (E, F, H), 0.3)
    wd = synth.normal_bf16(sd, 5, (E, H, F), 0.3)
    l = synth.normal_f64(sd, 0, 0, T * E).reshape(T, E).astype(np.float32)
    idx, w, w64 = orc.route(l, K)
    X = np.array([[1, 0], [0, 1], [1, 1]], dtype=np.uint8)
    d = orc.dispatch(idx, X, C, x)
    yp = orc.expert_ffn(d["xp"], d["seg_offsets"], d["slot_expert"], wg, wu, wd)
    y = orc.combine(yp, d["inv_row"], w64)
    xf, wgf, wuf, wdf = (orc.bf16_to_f64(a).tolist() for a in (x, wg, wu, wd))
    for t in range(T):
        want = [0.0] * H
        for s in range(K):
            e = int(idx[t, s])
            out = _scalar_ffn(xf[t], wgf[e], wuf[e], wdf[e])
            want = [want[h] + float(w64[t, s]) * out[h] for h in range(H)]
        assert np.allclose(y[t], want, rtol=1e-12, atol=1e-14)


def test_ffn_closed_form_with_identity_like_weights():
    # W_gate = c*I, W_up = I, W_down = I (H == F): out[h] = silu(c*x[h]) * x[h]
    H = 8
    c = 2.0
    eye = np.eye(H, dtype=np.float32)
    bits = lambda a: orc.f64_to_bf16_bits(a)
    x = synth.normal_bf16(5, 2, (3, H), 0.5)
    out = orc.swiglu_ffn_rows(orc.bf16_to_f64(x), bits(c * eye), bits(eye), bits(eye))
    xv = orc.bf16_to_f64(x)
    want = (c * xv) / (1.0 + np.exp(-c * xv)) * xv
    assert np.allclose(out, want, rtol=1e-14, atol=0)


def test_ffn_zero_and_doubled_down_projection():
    wl = synth.make_workload("c1_tiny")
    s, w = wl.shape, wl.weights
    rows = orc.bf16_to_f64(wl.x[:4])
    base = orc.swiglu_ffn_rows(rows, w.w_gate[0], w.w_up[0], w.w_down[0])
    zero = orc.swiglu_ffn_rows(rows, w.w_gate[0], w.w_up[0], np.zeros_like(w.w_down[0]))
    assert np.all(zero == 0.0)
    wd2 = orc.f64_to_bf16_bits(2.0 * orc.bf16_to_f64(w.w_down[0]))      # exact in bf16
    dbl = orc.swiglu_ffn_rows(rows, w.w_gate[0], w.w_up[0], wd2)
    assert np.array_equal(dbl, 2.0 * base)


def test_layer_output_is_invariant_to_placement_and_token_order():
    wl = synth.make_workload("c1_tiny")
    s, w = wl.shape, wl.weights
    idx, _, w64 = orc.route(wl.logits, s.K)

    def layer(X, C, logits=wl.logits, x=wl.x):
        i, _, ww = orc.route(logits, s.K)
        d = orc.dispatch(i, X, C, x)
        yp = orc.expert_ffn(d["xp"], d["seg_offsets"], d["slot_expert"], w.w_gate, w.w_up, w.w_down)
        return orc.combine(yp, d["inv_row"], ww)

    y0 = layer(wl.X_primary, s.C_max)
    rng = _rng(9)
    for extra in (0, 3, 6):
        X = _random_placement(rng, s.E, s.R, 4, extra)
        assert np.allclose(layer(X, 4), y0, rtol=1e-12, atol=1e-15)
    perm = rng.permutation(s.T)
    assert np.allclose(layer(wl.X_primary, s.C_max, wl.logits[perm], wl.x[perm]), y0[perm], rtol=1e-12, atol=1e-15)


def test_shared_experts_equal_one_wide_ffn():
    # S separate FFNs summed == one FFN of width S*F with concatenated weights
    S, F, H, T = 3, 8, 4, 5
    x = synth.normal_bf16(1, 2, (T, H), 0.5)
    sg = synth.normal_bf16(1, 6, (S, F, H), 0.3)
    su = synth.normal_bf16(1, 7, (S, F, H), 0.3)
    sdn = synth.normal_bf16(1, 8, (S, H, F), 0.3)
    got = orc.shared_ffn(x, sg, su, sdn)
    wide = orc.swiglu_ffn_rows(orc.bf16_to_f64(x), sg.reshape(S * F, H), su.reshape(S * F, H),
                               synth.concat_shared_down(sdn))
    assert np.allclose(got, wide, rtol=1e-12, atol=1e-15)
    xf = orc.bf16_to_f64(x).tolist()
    want0 = [0.0] * H
    for s_ in range(S):
        o = _scalar_ffn(xf[0], orc.bf16_to_f64(sg[s_]).tolist(), orc.bf16_to_f64(su[s_]).tolist(),
                        orc.bf16_to_f64(sdn[s_]).tolist())
        want0 = [a + b for a, b in zip(want0, o)]
    assert np.allclose(got[0], want0, rtol=1e-12, atol=1e-15)


# ------------------------------------------------------------------------ placement cost (a5)

def test_cost_equals_brute_force_triple_loop_with_replicas():
    rng = _rng(11)
    T, E, K, R, C, H = 41, 6, 2, 3, 4, 256
    idx, _, _ = orc.route(rng.normal(size=(T, E)).astype(np.float32), K)
    X = _random_placement(rng, E, R, C, 4)
    src = rng.integers(0, R, size=T).astype(np.int32)
    c = orc.placement_cost(idx, X, C, H, src)
    reps = [[j for j in range(R) if X[e, j]] for e in range(E)]
    seen = [0] * E
    W = [[0] * E for _ in range(R)]
    lam = [0] * R
    D = [[0] * R for _ in range(R)]
    for t in range(T):
        for s in range(K):
            e = int(idx[t, s])
            k = reps[e][seen[e] % len(reps[e])]
            seen[e] += 1
            W[src[t]][e] += 1
            lam[k] += 1
            D[src[t]][k] += 1
    assert c["workload"].tolist() == W
    assert c["rank_load"].tolist() == lam
    assert c["dispatch_tokens"].tolist() == D
    assert c["dispatch_bytes"].tolist() == [[v * 2 * H for v in row] for row in D]
    assert c["dispatch_bytes"].dtype == np.uint64


def test_cost_single_copy_matches_eq1_and_eq3_matrix_forms():
    wl = synth.make_workload("c1_tiny", with_weights=False)
    s = wl.shape
    idx, _, _ = orc.route(wl.logits, s.K)
    c = orc.placement_cost(idx, wl.X_primary, s.C_max, s.H)
    W = c["workload"]
    P = synth.primary_ranks(s)
    N = W.sum(axis=0)
    d = 2 * s.H
    for j in range(s.R):
        assert c["rank_load"][j] == sum(N[i] for i in range(s.E) if P[i] == j)          # Eq. 1
        for k in range(s.R):
            assert c["dispatch_bytes"][j, k] == d * sum(W[j, i] for i in range(s.E) if P[i] == k)   # Eq. 3
    # conservation laws
    assert c["rank_load"].sum() == s.T * s.K
    assert np.array_equal(N, np.bincount(idx.ravel(), minlength=s.E))
    Tj = np.bincount(orc.source_ranks(s.T, s.R), minlength=s.R)
    assert np.array_equal(W.sum(axis=1), s.K * Tj)
    assert np.array_equal(c["dispatch_tokens"].sum(axis=1), s.K * Tj)
    assert np.array_equal(c["dispatch_tokens"].sum(axis=0), c["rank_load"])


def test_cost_one_rank_is_all_local_and_source_partition():
    rng = _rng(5)
    idx, _, _ = orc.route(rng.normal(size=(10, 4)).astype(np.float32), 2)
    X = np.ones((4, 1), dtype=np.uint8)
    c = orc.placement_cost(idx, X, 4, 64)
    assert c["dispatch_tokens"].tolist() == [[20]] and c["rank_load"].tolist() == [20]
    assert orc.cost_summary(c)["cross_rank_bytes"] == 0
    assert orc.source_ranks(1, 16).tolist() == [0]
    assert orc.source_ranks(8, 4).tolist() == [0, 0, 1, 1, 2, 2, 3, 3]
    assert np.bincount(orc.source_ranks(10, 4)).tolist() == [3, 2, 3, 2]


def test_cost_summary_reductions_against_hand_written_numbers():
    """Eq. 2's straggler load and Eq. 4's send volumes on a 3-rank example worked by hand.  Row sums,
    column sums, diagonal, maximum and total all differ, so `sum` for `max`, rows for columns, or a
    diagonal left in would each fail."""
    #   tokens sent j -> k            off-diagonal of row j     column sums (= lambda_k, Eq. 1)
    D_tokens = np.array([[5, 2, 1],   # 2 + 1 = 3               5 + 0 + 3 = 8
                         [0, 7, 4],   # 0 + 4 = 4               2 + 7 + 3 = 12
                         [3, 3, 0]],  # 3 + 3 = 6               1 + 4 + 0 = 5
                        dtype=np.int64)
    d = 8                             # bytes per token: H = 4 hidden values of 2 bytes
    cost = dict(rank_load=D_tokens.sum(axis=0), dispatch_tokens=D_tokens,
                dispatch_bytes=(D_tokens * d).astype(np.uint64))
    s = orc.cost_summary(cost)
    assert s["max_rank_load"] == 12                       # Eq. 2: the straggler executes 12 assignments
    assert s["send_bytes"].tolist() == [24, 32, 48]       # Eq. 4: sum over k != j of D[j,k], in bytes
    assert s["max_send_bytes"] == 48                      # the straggler sender (rank 2), not the total
    assert s["cross_rank_bytes"] == 104                   # 24 + 32 + 48; the diagonal (5, 7, 0) is local
    # the same quantities through placement_cost on an assignment list that realises this D exactly:
    # K = 1, single-copy placement expert k -> rank k, so D[j,k] = tokens of rank j that chose expert k
    src, idx = [], []
    for j in range(3):
        for k in range(3):
            src += [j] * int(D_tokens[j, k])
            idx += [k] * int(D_tokens[j, k])
    c = orc.placement_cost(np.array(idx, dtype=np.int32)[:, None], np.eye(3, dtype=np.uint8), 1, 4,
                           np.array(src, dtype=np.int32))
    assert np.array_equal(c["dispatch_tokens"], D_tokens) and c["rank_load"].tolist() == [8, 12, 5]
    s2 = orc.cost_summary(c)
    assert (s2["max_rank_load"], s2["max_send_bytes"], s2["cross_rank_bytes"]) == (12, 48, 104)
    assert s2["send_bytes"].tolist() == [24, 32, 48]


# ------------------------------------------------------------------- balanced placement input

def test_balanced_placement_is_valid_and_near_brute_force_optimum_on_c1():
    wl = synth.make_workload("c1_tiny", with_weights=False)
    s = wl.shape
    idx, _, _ = orc.route(wl.logits, s.K)
    N = np.bincount(idx.ravel(), minlength=s.E)
    X = orc.balanced_placement(N, s.R, s.C_max)
    orc.placement_tables(X, s.C_max)                       # valid: raises otherwise
    assert X.sum() == s.E                                   # no spare slots -> single copy
    lam = np.array([N[X[:, j] == 1].sum() for j in range(s.R)])
    # brute force over all single-copy placements with <= C_max experts per rank
    best = None
    for assign in itertools.product(range(s.R), repeat=s.E):
        cnt = np.bincount(assign, minlength=s.R)
        if cnt.max() > s.C_max:
            continue
        m = max(sum(int(N[e]) for e in range(s.E) if assign[e] == j) for j in range(s.R))
        best = m if best is None else min(best, m)
    assert lam.max() >= best
    assert lam.max() * 3 <= best * 4


def test_balanced_placement_with_fixed_primaries_and_replicas():
    N = np.array([100, 1, 1, 1, 50, 0, 0, 2])
    primary = np.array([0, 0, 1, 1, 2, 2, 3, 3])
    X = orc.balanced_placement(N, 4, 3, primary)
    assert np.all(X[np.arange(8), primary] == 1)
    assert X.sum(axis=0).max() <= 3
    assert X[0].sum() >= 2                                  # the hottest expert gets replicas
    assert X[5].sum() == 1 and X[6].sum() == 1              # experts without tokens get none
    idx = np.repeat(np.arange(8), N).reshape(-1, 1).astype(np.int32)
    c0 = orc.placement_cost(idx, synth.placement_from_ranks(primary, 4), 3, 64)
    c1 = orc.placement_cost(idx, X, 3, 64)
    assert c1["rank_load"].max() < c0["rank_load"].max()


def test_replicate_hottest():
    N = np.array([5, 90, 7, 60])
    X = synth.placement_from_ranks(np.arange(4), 4)
    Y = orc.replicate_hottest(N, X, 2)
    assert Y.sum() == 6 and Y[1].sum() == 2 and Y[3].sum() == 2
    assert Y[1, 0] == 1          # hottest expert -> least loaded rank (0, load 5)
    assert Y[3, 2] == 1          # second hottest -> next least loaded rank (2, load 7)


# ------------------------------------------------------- locality-first replica choice, de-duplicated volume

def _sorted_local_first(idx, X, C_max, src):
    """Definition by lists and sorting (no running counters): per expert, the travelling assignments are those
    whose home rank does not host it, numbered by sorting them on token id; then one global sort."""
    T, K = idx.shape
    E, R = X.shape
    reps = [[j for j in range(R) if X[e, j]] for e in range(E)]
    dest = {}
    for e in range(E):
        mine = sorted((t, s) for t in range(T) for s in range(K) if idx[t, s] == e)
        away = [ts for ts in mine if not X[e, src[ts[0]]]]
        for ts in mine:
            dest[ts] = int(src[ts[0]]) if X[e, src[ts[0]]] else reps[e][away.index(ts) % len(reps[e])]
    order = sorted((dest[(t, s)], int(idx[t, s]), t, s) for t in range(T) for s in range(K))
    inv_row = np.zeros((T, K), dtype=np.int32)
    dr = np.zeros((T, K), dtype=np.int32)
    row_token = np.zeros(T * K, dtype=np.int32)
    for row, (j, e, t, s) in enumerate(order):
        inv_row[t, s], dr[t, s], row_token[row] = row, j, t
    seg = [0]
    for j in range(R):
        hosted = [e for e in range(E) if X[e, j]]
        for p in range(C_max):
            seg.append(seg[-1] + (sum(1 for o in order if o[0] == j and o[1] == hosted[p]) if p < len(hosted) else 0))
    return inv_row, dr, row_token, np.array(seg, dtype=np.int32)


@pytest.mark.parametrize("seed,E,K,R,C,extra,custom_src", [(0, 8, 2, 4, 3, 4, False), (1, 8, 2, 4, 3, 4, True),
                                                            (2, 6, 3, 3, 4, 5, True), (3, 5, 5, 2, 5, 3, False),
                                                            (4, 4, 1, 4, 1, 0, True), (5, 8, 2, 4, 2, 0, False)])
def test_local_first_dispatch_equals_sort_based_definition(seed, E, K, R, C, extra, custom_src):
    rng = _rng(100 + seed)
    T = 43
    idx, _, _ = orc.route(rng.normal(size=(T, E)).astype(np.float32) - 0.5 * np.arange(E, dtype=np.float32), K)
    X = _random_placement(rng, E, R, C, extra)
    src = rng.integers(0, R, size=T).astype(np.int32) if custom_src else orc.source_ranks(T, R)
    d = orc.dispatch(idx, X, C, policy="local_first", src=src if custom_src else None)
    inv_row, dest, row_token, seg = _sorted_local_first(idx, X, C, src)
    assert np.array_equal(d["inv_row"], inv_row)
    assert np.array_equal(d["dest_rank"], dest)
    assert np.array_equal(d["row_token"], row_token)
    assert np.array_equal(d["seg_offsets"], seg)


def test_local_first_without_replicas_is_the_round_robin_dispatch():
    rng = _rng(120)
    T, E, K, R, C = 61, 8, 2, 4, 2
    idx, _, _ = orc.route(rng.normal(size=(T, E)).astype(np.float32), K)
    X = _random_placement(rng, E, R, C, 0)
    src = rng.integers(0, R, size=T).astype(np.int32)
    a, b = orc.dispatch(idx, X, C), orc.dispatch(idx, X, C, policy="local_first", src=src)
    for k in ("row_token", "inv_row", "dest_rank", "seg_offsets", "slot_expert"):
        assert np.array_equal(a[k], b[k]), k


def test_local_first_with_every_expert_everywhere_moves_nothing():
    rng = _rng(121)
    T, E, K, R, H = 50, 4, 2, 3, 64
    idx, _, _ = orc.route(rng.normal(size=(T, E)).astype(np.float32), K)
    X = np.ones((E, R), dtype=np.uint8)
    src = orc.source_ranks(T, R)
    d = orc.dispatch(idx, X, E, policy="local_first")
    assert np.array_equal(d["dest_rank"], np.repeat(src[:, None], K, axis=1))
    c = orc.placement_cost(idx, X, E, H, policy="local_first")
    D = c["dispatch_tokens"]
    assert np.array_equal(D, np.diag(np.bincount(src, minlength=R) * K))
    assert orc.cost_summary(c)["cross_rank_bytes"] == 0
    assert c["rank_load"].tolist() == (np.bincount(src, minlength=R) * K).tolist()


def test_local_first_invariants_and_never_more_cross_traffic_than_round_robin():
    for seed in range(6):
        rng = _rng(130 + seed)
        T, E, K, R, C, H = 97, 12, 3, 4, 5, 128
        idx, _, _ = orc.route(rng.normal(size=(T, E)).astype(np.float32) - 0.3 * np.arange(E, dtype=np.float32), K)
        X = _random_placement(rng, E, R, C, 6)
        src = rng.integers(0, R, size=T).astype(np.int32)
        d = orc.dispatch(idx, X, C, policy="local_first", src=src)
        dest, inv_row, row_token, seg = d["dest_rank"], d["inv_row"], d["row_token"], d["seg_offsets"]
        # a hosted expert is used at home; a travelling assignment lands on some replica
        for t in range(T):
            for s in range(K):
                e = idx[t, s]
                assert X[e, dest[t, s]] == 1
                if X[e, src[t]]:
                    assert dest[t, s] == src[t]
        # travelling assignments of an expert are dealt round-robin: replica counts differ by at most one,
        # earlier replicas hold the extras
        for e in range(E):
            tt, ss = np.nonzero(idx == e)
            away = [dest[t, s] for t, s in zip(tt, ss) if not X[e, src[t]]]
            reps = np.flatnonzero(X[e])
            counts = [away.count(j) for j in reps]
            assert max(counts) - min(counts) <= 1 and counts == sorted(counts, reverse=True)
        # permutation structure
        assert sorted(inv_row.reshape(-1).tolist()) == list(range(T * K))
        assert np.array_equal(row_token[inv_row], np.repeat(np.arange(T)[:, None], K, axis=1))
        for g in range(R * C):
            rows = row_token[seg[g]:seg[g + 1]]
            assert np.all(np.diff(rows) > 0)                       # ascending token id, no token twice
            if len(rows):
                e = d["slot_expert"][g]
                assert e >= 0 and all(e in idx[t] for t in rows)
        # Eq. 3 volume off the diagonal can only shrink
        lf = orc.cost_summary(orc.placement_cost(idx, X, C, H, src, policy="local_first"))
        rr = orc.cost_summary(orc.placement_cost(idx, X, C, H, src))
        assert lf["cross_rank_bytes"] <= rr["cross_rank_bytes"]
        cl = orc.placement_cost(idx, X, C, H, src, policy="local_first")
        assert cl["rank_load"].sum() == T * K and np.array_equal(cl["workload"], orc.placement_cost(idx, X, C, H, src)["workload"])


def test_layer_output_does_not_depend_on_the_replica_policy():
    wl = synth.make_workload("c1_tiny")
    s, w = wl.shape, wl.weights
    idx, _, ww = orc.route(wl.logits, s.K)
    X = _random_placement(_rng(150), s.E, s.R, 4, 6)
    ys = []
    for policy in ("round_robin", "local_first"):
        d = orc.dispatch(idx, X, 4, wl.x, policy=policy)
        yp = orc.expert_ffn(d["xp"], d["seg_offsets"], d["slot_expert"], w.w_gate, w.w_up, w.w_down)
        ys.append(orc.combine(yp, d["inv_row"], ww))
    assert np.allclose(ys[0], ys[1], rtol=1e-12, atol=1e-15)      # same rows, other segment shapes: fp64 rounding order only


def test_dedup_volume_properties():
    rng = _rng(140)
    T, E, R, C = 83, 10, 4, 4
    X = _random_placement(rng, E, R, C, 5)
    src = rng.integers(0, R, size=T).astype(np.int32)
    for K in (1, 3):
        idx, _, _ = orc.route(rng.normal(size=(T, E)).astype(np.float32), K)
        for policy in ("round_robin", "local_first"):
            dest = orc.dispatch(idx, X, C, policy=policy, src=src)["dest_rank"]
            U = orc.dedup_dispatch_tokens(dest, src, R)
            D = orc.placement_cost(idx, X, C, 64, src, policy=policy)["dispatch_tokens"]
            assert np.all(U <= D)
            if K == 1:
                assert np.array_equal(U, D)
            # distinct (token, destination) pairs, counted with a library routine
            pairs = np.unique(np.stack([np.repeat(np.arange(T), K), dest.reshape(-1)], axis=1), axis=0)
            want = np.zeros((R, R), dtype=np.int64)
            np.add.at(want, (src[pairs[:, 0]], pairs[:, 1]), 1)
            assert np.array_equal(U, want)
            assert np.all(U.sum(axis=1) >= np.bincount(src, minlength=R))      # every token goes somewhere
    # all experts on one rank: every token is sent there exactly once whatever K
    X1 = np.zeros((E, R), dtype=np.uint8)
    X1[:, 2] = 1
    idx, _, _ = orc.route(rng.normal(size=(T, E)).astype(np.float32), 3)
    U = orc.dedup_dispatch_tokens(orc.dispatch(idx, X1, E)["dest_rank"], src, R)
    assert np.array_equal(U[:, 2], np.bincount(src, minlength=R)) and U.sum() == T
