"""GPU parity of the locality-first replica rule and of the de-duplicated dispatch volume: every index, segment
offset and histogram bit-exact against the oracle, the layer output bitwise independent of the rule."""
import numpy as np
import pytest

from oracle import director_oracle as orc
from paper_2607_08782_b200 import synth

from gpu_harness import GpuCase
from test_gpu_parity import _check_outputs, _custom, _random_placement

pytestmark = pytest.mark.gpu

LOCAL_FIRST = 1


def _oracle_local_first(shape, logits, x_bits, X, C_max, src):
    idx, w, w64 = orc.route(logits, shape.K)
    d = orc.dispatch(idx, X, C_max, x_bits, policy="local_first", src=src)
    c = orc.placement_cost(idx, X, C_max, shape.H, src, policy="local_first")
    return idx, w, w64, d, c


@pytest.mark.parametrize("seed,T,H,E,K,F,S,R,C,extra", [
    (21, 777, 256, 12, 3, 384, 0, 4, 4, 4),      # several 256-token tiles and a ragged tail, replicas
    (22, 1000, 512, 60, 4, 256, 2, 8, 8, 4),     # E not a multiple of 32, shared experts
    (23, 300, 256, 5, 5, 128, 0, 2, 5, 5),       # every expert on every rank: nothing travels
    (24, 1, 256, 8, 2, 128, 1, 4, 2, 0),         # a single token, no replicas
    (25, 513, 768, 128, 8, 256, 0, 16, 9, 16),   # Qwen3-like routing sizes, many empty segments
    (26, 260, 256, 256, 8, 128, 0, 64, 4, 0),    # the largest supported E and R
    (27, 2100, 256, 16, 4, 128, 0, 8, 16, 100),  # heavy replication, the largest C_max
])
def test_local_first_small_cases_full_tensor_parity(seed, T, H, E, K, F, S, R, C, extra):
    shape, logits, x, weights = _custom(seed, T, H, E, K, F, S, R, C)
    X = _random_placement(seed, E, R, C, extra)
    src = (synth.raw_u64(seed, 50, 0, T) % np.uint64(R)).astype(np.int32) if seed % 2 else None
    case = GpuCase(shape, logits, x, weights)
    g = case.run(X, src=src, policy=LOCAL_FIRST)
    src_o = orc.source_ranks(T, R) if src is None else src
    idx, w, w64, d, c = _oracle_local_first(shape, logits, x, X, C, src)
    _check_outputs(shape, g, x, weights, idx, w, w64, d, c, np.arange(T), f"local-first{seed}")
    assert np.array_equal(g.dedup_tokens, orc.dedup_dispatch_tokens(d["dest_rank"], src_o, R))
    # the rule changes where rows sit, not what a token computes
    g_rr = case.run(X, src=src)
    assert np.array_equal(g.y, g_rr.y)
    d_rr = orc.dispatch(idx, X, C)
    assert np.array_equal(g_rr.dest_rank, d_rr["dest_rank"]) and np.array_equal(g_rr.inv_row, d_rr["inv_row"])
    assert np.array_equal(g_rr.dedup_tokens, orc.dedup_dispatch_tokens(d_rr["dest_rank"], src_o, R))
    off = lambda D: int(D.sum() - np.trace(D))
    assert off(g.dispatch_tokens) <= off(g_rr.dispatch_tokens)
    if extra == 0:
        assert np.array_equal(g.inv_row, g_rr.inv_row) and np.array_equal(g.seg_offsets, g_rr.seg_offsets)


@pytest.mark.parametrize("name,T", [("c3_dsv2lite", None), ("c5_qwen3", 32768), ("c5_qwen3", 64)])
def test_local_first_on_paper_shaped_routing(name, T):
    """Indices and histograms at full size (the expert GEMMs are covered by the other full-size tests)."""
    wl = synth.make_workload(name, T)
    s = wl.shape
    case = GpuCase(s, wl.logits, wl.x, wl.weights)
    idx, _, _ = orc.route(wl.logits, s.K)
    N = np.bincount(idx.ravel(), minlength=s.E)
    X = orc.balanced_placement(N, s.R, s.C_max, synth.primary_ranks(s))
    g = case.run(X, policy=LOCAL_FIRST, stages="front")
    d = orc.dispatch(idx, X, s.C_max, wl.x, policy="local_first")
    c = orc.placement_cost(idx, X, s.C_max, s.H, policy="local_first")
    assert g.status == 0
    for k in ("row_token", "inv_row", "dest_rank", "seg_offsets"):
        assert np.array_equal(getattr(g, k), d[k]), k
    assert np.array_equal(g.xp, d["xp"])
    for k in ("workload", "rank_load", "dispatch_tokens", "dispatch_bytes"):
        assert np.array_equal(getattr(g, k), c[k]), k
    assert np.array_equal(g.dedup_tokens, orc.dedup_dispatch_tokens(d["dest_rank"], orc.source_ranks(s.T, s.R), s.R))
    rr = orc.cost_summary(orc.placement_cost(idx, X, s.C_max, s.H))
    lf = orc.cost_summary(c)
    U = g.dedup_tokens
    print(f"{name}/T={s.T}: cross-rank bytes round-robin {rr['cross_rank_bytes']:.4g} -> locality-first "
          f"{lf['cross_rank_bytes']:.4g}; de-duplicated {int(U.sum() - np.trace(U)) * 2 * s.H:.4g}")
    assert lf["cross_rank_bytes"] <= rr["cross_rank_bytes"]


def test_batched_candidate_scores_follow_the_policy():
    import torch
    shape, logits, x, weights = _custom(31, 1500, 256, 24, 4, 128, 0, 6, 6, 0)
    case = GpuCase(shape, logits, x, weights)
    L = case.layer
    idx, _, _ = orc.route(logits, shape.K)
    cands = [_random_placement(300 + i, shape.E, shape.R, shape.C_max, 3 * i) for i in range(5)]
    L.set_placement(cands[0])
    L.route(shape.T, case.logits)
    L.placement_cost(shape.T)                                  # fills L.workload
    n = len(cands)
    Xd = torch.from_numpy(np.stack(cands)).cuda()
    load = torch.empty((n, shape.R), dtype=torch.int64, device="cuda")
    disp = torch.empty((n, shape.R, shape.R), dtype=torch.int64, device="cuda")
    summ = torch.empty((n, 4), dtype=torch.int64, device="cuda")
    for policy, pname in ((1, "local_first"), (0, "round_robin")):
        L.set_replica_policy(policy)
        try:
            L.d.placement_cost_batch(L.workload, n, Xd, load, disp, summ)
            torch.cuda.synchronize()
        finally:
            L.set_replica_policy(0)
        for i, X in enumerate(cands):
            c = orc.placement_cost(idx, X, shape.C_max, shape.H, policy=pname)
            cs = orc.cost_summary(c)
            assert np.array_equal(load[i].cpu().numpy(), c["rank_load"]), (pname, i)
            assert np.array_equal(disp[i].cpu().numpy(), c["dispatch_tokens"]), (pname, i)
            assert summ[i].tolist() == [cs["max_rank_load"], cs["max_send_bytes"] // (2 * shape.H),
                                        cs["cross_rank_bytes"] // (2 * shape.H), 1]


def test_policy_argument_is_checked():
    from paper_2607_08782_b200.binding import DirectorError
    shape, logits, x, weights = _custom(32, 64, 256, 8, 2, 128, 0, 4, 2, 0)
    case = GpuCase(shape, logits, x, weights)
    with pytest.raises(DirectorError):
        case.layer.set_replica_policy(2)
    case.layer.set_replica_policy(1)
    case.layer.set_replica_policy(0)


def test_front_end_call_honours_the_policy_for_small_and_large_batches():
    """director_route_dispatch_cost under LOCAL_FIRST: decode-sized batches may not take the fused round-robin kernel."""
    import torch
    for seed, T in ((41, 100), (42, 700)):
        shape, logits, x, weights = _custom(seed, T, 256, 20, 3, 128, 0, 5, 6, 1.2)
        X = _random_placement(seed, 20, 5, 6, 8)
        case = GpuCase(shape, logits, x, weights)
        L = case.layer
        L.set_placement(X)
        L.set_replica_policy(LOCAL_FIRST)
        try:
            L.d.route_dispatch_cost(T, case.logits, case.x, L.topk_idx, L.topk_w, L.xp, L.row_token, L.inv_row,
                                    L.dest_rank, L.seg_offsets, L.workload, L.rank_load, L.dispatch_tokens,
                                    L.dispatch_bytes)
            torch.cuda.synchronize()
        finally:
            L.set_replica_policy(0)
        idx, _, _ = orc.route(logits, shape.K)
        d = orc.dispatch(idx, X, 6, x, policy="local_first")
        c = orc.placement_cost(idx, X, 6, shape.H, policy="local_first")
        assert np.array_equal(L.inv_row[:T].cpu().numpy(), d["inv_row"])
        assert np.array_equal(L.dest_rank[:T].cpu().numpy(), d["dest_rank"])
        assert np.array_equal(L.seg_offsets.cpu().numpy(), d["seg_offsets"])
        assert np.array_equal(L.dispatch_tokens.cpu().numpy(), c["dispatch_tokens"])
        assert np.array_equal(L.rank_load.cpu().numpy(), c["rank_load"])
