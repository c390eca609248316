"""GPU: the batched placement-cost kernel against the oracle (bit-exact), and the placement search scored on the GPU."""
import numpy as np
import pytest

from oracle import director_oracle as orc
from paper_2607_08782_b200 import optimizer as opt
from paper_2607_08782_b200 import synth

pytestmark = pytest.mark.gpu


def _setup(shape, C_max=None):
    import torch
    from paper_2607_08782_b200.binding import Director
    s = shape
    C = C_max or s.C_max
    logits = synth.make_logits(s)
    idx, _, _ = orc.route(logits, s.K)
    d = Director(s.T, s.H, s.F, s.E, s.K, s.S, s.R, C)
    X0 = synth.placement_from_ranks(np.arange(s.E) % s.R, s.R)
    W_o = orc.placement_cost(idx, X0, max(C, -(-s.E // s.R)), s.H)["workload"]
    W = torch.from_numpy(W_o).cuda()
    return d, idx, W, W_o, C


def _oracle_summary(idx, X, C, H):
    try:
        c = orc.placement_cost(idx, X, C, H)
    except orc.PlacementError:
        return None
    D = c["dispatch_tokens"]
    send = D.sum(axis=1) - np.diag(D)
    return c["rank_load"], D, np.array([c["rank_load"].max(), send.max(), send.sum(), 1], dtype=np.int64)


def test_batch_cost_matches_the_oracle_on_random_candidates_with_replicas():
    import torch
    shape = synth.Shape("opt", 3001, 256, 24, 4, 128, 0, 6, 6, 1.2, 81)
    d, idx, W, W_o, C = _setup(shape)
    rng = np.random.default_rng(5)
    cands = []
    for n in range(40):
        X = np.zeros((shape.E, shape.R), dtype=np.uint8)
        X[np.arange(shape.E), rng.integers(0, shape.R, size=shape.E)] = 1
        for _ in range(int(rng.integers(0, 8))):
            X[rng.integers(shape.E), rng.integers(shape.R)] = 1
        if n == 7:
            X[3, :] = 0                                   # unhosted expert -> invalid
        cands.append(X)
    Xb = np.stack(cands)
    load = torch.empty((len(Xb), shape.R), dtype=torch.int64, device="cuda")
    disp = torch.empty((len(Xb), shape.R, shape.R), dtype=torch.int64, device="cuda")
    summ = torch.empty((len(Xb), 4), dtype=torch.int64, device="cuda")
    d.placement_cost_batch(W, len(Xb), torch.from_numpy(Xb).cuda(), load, disp, summ)
    torch.cuda.synchronize()
    load, disp, summ = load.cpu().numpy(), disp.cpu().numpy(), summ.cpu().numpy()
    n_valid = 0
    for n, X in enumerate(Xb):
        o = _oracle_summary(idx, X, C, shape.H)
        if o is None:
            assert summ[n, 3] == 0, f"candidate {n} should be flagged invalid"
            continue
        n_valid += 1
        assert np.array_equal(load[n], o[0]) and np.array_equal(disp[n], o[1]) and np.array_equal(summ[n], o[2]), n
    assert n_valid >= 10 and n_valid < len(Xb)
    assert d.last_status() == 0


def test_all_2520_placements_of_the_tiny_workload_in_one_batch_and_the_search_finds_the_optimum():
    import torch
    s = synth.shape_for("c1_tiny")
    d, idx, W, W_o, C = _setup(s)
    ev = opt.GpuPlacementEvaluator(d, W)
    allX = opt.enumerate_single_copy(s.E, s.R, s.C_max)
    S = ev(allX)
    assert (S[:, 3] == 1).all()
    for n in (0, 1, 77, 1234, 2519):                      # spot-check against the oracle, candidate by candidate
        assert np.array_equal(S[n], _oracle_summary(idx, allX[n], C, s.H)[2])
    model = opt.LatencyModel(1.0, 0.0, 0.5 / (2 * s.H), 2 * s.H)
    brute = float(model.latency(S[:, 0], S[:, 1]).min())
    res = opt.optimize_placement(W_o, s.C_max, model, ev)
    assert brute - 1e-9 <= res["latency"] <= brute * 1.10
    assert res["lp_bound"] <= brute * (1 + 2e-3)
    assert ev.evaluated > 2520                            # the search really ran its batches through the GPU


def test_search_improves_the_default_placement_of_a_skewed_workload():
    s = synth.shape_for("c3_dsv2lite")
    small = synth.Shape("opt3", 2048, s.H, s.E, s.K, s.F, 0, s.R, s.C_max, s.zipf_s, 83)
    d, idx, W, W_o, C = _setup(small)
    ev = opt.GpuPlacementEvaluator(d, W)
    model = opt.LatencyModel(1.0, 0.0, 0.2 / (2 * s.H), 2 * s.H)
    X0 = synth.placement_from_ranks(synth.primary_ranks(s), s.R)
    s0 = ev(X0[None])[0]
    base = float(model.latency(s0[0], s0[1]))
    res = opt.optimize_placement(W_o, C, model, ev, allow_replicas=True)
    o = _oracle_summary(idx, res["X"], C, s.H)
    assert o is not None                                  # valid under Eq. 6's constraints
    assert abs(float(model.latency(o[2][0], o[2][1])) - res["latency"]) < 1e-6     # GPU score == oracle score
    assert res["latency"] < base * 0.9
    assert res["lp_bound"] <= res["latency"] * (1 + 1e-6) or res["X"].sum() > s.E   # LP bounds single-copy placements
