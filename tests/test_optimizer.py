"""Host logic of the placement search (Section VI: cost model, LP relaxation of Eq. 6, Algorithm 1's binary
search), scored here with the CPU oracle so that it runs without a GPU."""
import numpy as np
import pytest

from oracle import director_oracle as orc
from paper_2607_08782_b200 import optimizer as opt
from paper_2607_08782_b200 import synth


def oracle_evaluator(idx, C_max, H):
    """summary rows (max load, max send tokens, cross tokens, valid) computed by the oracle, one candidate at a time."""
    def ev(Xb):
        out = np.zeros((len(Xb), 4), dtype=np.int64)
        for n, X in enumerate(Xb):
            try:
                c = orc.placement_cost(idx, X, C_max, H)
            except orc.PlacementError:
                continue
            D = c["dispatch_tokens"]
            send = D.sum(axis=1) - np.diag(D)
            out[n] = (c["rank_load"].max(), send.max(), send.sum(), 1)
        return out
    return ev


@pytest.fixture(scope="module")
def c1():
    wl = synth.make_workload("c1_tiny", with_weights=False)
    s = wl.shape
    idx, _, _ = orc.route(wl.logits, s.K)
    W = orc.placement_cost(idx, wl.X_primary, s.C_max, s.H)["workload"]
    return wl, s, idx, W


def test_enumeration_counts_every_single_copy_placement():
    assert len(opt.enumerate_single_copy(8, 4, 2)) == 2520          # 8! / (2!)^4
    assert len(opt.enumerate_single_copy(3, 2, 2)) == 6               # 2^3 minus the two all-on-one-rank


def test_lp_is_a_lower_bound_and_bisection_finds_its_optimum(c1):
    wl, s, idx, W = c1
    model = opt.LatencyModel(comp_per_token=1.0, comm_per_byte=0.25 / (2 * s.H), bytes_per_token=2 * s.H)
    ev = oracle_evaluator(idx, s.C_max, s.H)
    allX = opt.enumerate_single_copy(s.E, s.R, s.C_max)
    S = ev(allX)
    brute = float(model.latency(S[:, 0], S[:, 1]).min())
    x_bar, lp_val = opt.lp_minimum(W, s.C_max, model)
    assert lp_val <= brute + 1e-9                                     # relaxation of the integer problem
    assert np.allclose(x_bar.sum(axis=1), 1.0, atol=1e-6) and x_bar.sum(axis=0).max() <= s.C_max + 1e-6
    x_b, beta = opt.binary_search_budget(W, s.C_max, model, beta_high=brute * 2)
    assert abs(beta - lp_val) <= 2e-3 * beta                          # Algorithm 1's bisection reaches the LP optimum
    assert opt.lp_feasible(W, s.C_max, model, lp_val * 0.98) is None  # and nothing below it is feasible


def test_optimizer_reaches_the_brute_force_optimum_on_the_tiny_workload(c1):
    wl, s, idx, W = c1
    ev = oracle_evaluator(idx, s.C_max, s.H)
    allX = opt.enumerate_single_copy(s.E, s.R, s.C_max)
    S = ev(allX)
    for model in (opt.LatencyModel(1.0, 0.0, 0.0, 2 * s.H),                       # computation only (Eq. 2)
                  opt.LatencyModel(1.0, 0.0, 0.5 / (2 * s.H), 2 * s.H),           # both terms
                  opt.LatencyModel(0.0, 0.0, 1.0 / (2 * s.H), 2 * s.H)):          # communication only (Eq. 4)
        brute = float(model.latency(S[:, 0], S[:, 1]).min())
        res = opt.optimize_placement(W, s.C_max, model, ev)
        orc.placement_tables(res["X"], s.C_max)                                   # valid placement
        assert res["lp_bound"] <= brute * (1 + 2e-3)
        assert brute - 1e-9 <= res["latency"] <= brute * 1.10, (res["latency"], brute)


def test_local_search_never_gets_worse_and_respects_capacity(c1):
    wl, s, idx, W = c1
    ev = oracle_evaluator(idx, 3, s.H)
    model = opt.LatencyModel(1.0, 0.0, 0.1 / (2 * s.H), 2 * s.H)
    X0 = synth.placement_from_ranks(np.arange(s.E) // 2, s.R)
    lat0 = float(model.latency(*ev(X0[None])[0][:2]))
    X, lat, rounds = opt.local_search(ev, X0, 3, model, allow_replicas=True)
    assert lat <= lat0 and X.sum(axis=0).max() <= 3 and (X.sum(axis=1) >= 1).all()


def test_rounding_gives_one_copy_per_expert_within_capacity():
    rng = np.random.default_rng(0)
    x_bar = rng.dirichlet(np.ones(4), size=10)
    X = opt.round_placement(x_bar, rng.integers(1, 100, size=10), 3)
    assert (X.sum(axis=1) == 1).all() and X.sum(axis=0).max() <= 3
