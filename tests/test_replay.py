"""Replay of a shifting workload under static / reactive / proactive placement (Section III's motivation),
policy logic scored with the CPU oracle here and through the CUDA library in the GPU test."""
import numpy as np
import pytest

from oracle import director_oracle as orc
from paper_2607_08782_b200 import optimizer as opt
from paper_2607_08782_b200 import replay, synth


def _oracle_workloads(cfg):
    idxs, workloads = [], []
    X_any = synth.placement_from_ranks(np.arange(cfg.E) % cfg.R, cfg.R)
    for layer in range(cfg.layers):
        logits = synth.make_logits(replay.layer_shape(cfg, layer))
        li, lw = [], []
        for b in range(cfg.batches):
            idx, _, _ = orc.route(logits[b * cfg.tokens_per_batch:(b + 1) * cfg.tokens_per_batch], cfg.K)
            li.append(idx)
            lw.append(orc.placement_cost(idx, X_any, -(-cfg.E // cfg.R), cfg.H)["workload"])
        idxs.append(li)
        workloads.append(lw)
    return idxs, workloads


def _oracle_score(idxs, cfg):
    def score(layer, b, X):
        c = orc.placement_cost(idxs[layer][b], X, cfg.C_max, cfg.H)
        D = c["dispatch_tokens"]
        return c["rank_load"].max(), (D.sum(axis=1) - np.diag(D)).max()
    return score


def test_proactive_beats_reactive_beats_nothing_on_a_shifting_stream():
    cfg = replay.ReplayConfig(layers=2, batches=6, tokens_per_batch=512, E=16, K=2, R=4, C_max=5, seed=7100)
    model = opt.LatencyModel(1.0, 0.0, 0.0, 2 * cfg.H)                      # computation term only: the straggler load
    idxs, workloads = _oracle_workloads(cfg)
    lat, placements = replay.run_policies(workloads, cfg, model, _oracle_score(idxs, cfg))
    out = replay.summarize(lat, cfg)
    assert out["mean_latency"]["proactive"] <= out["mean_latency"]["reactive"]
    assert out["mean_latency"]["proactive"] <= out["mean_latency"]["static"]
    assert 0.0 < out["proactive_vs_reactive_gain"] < 1.0
    # the reactive policy runs batch b under the proactive placement of batch b-1
    for layer in range(cfg.layers):
        for b in range(1, cfg.batches):
            assert np.array_equal(placements["reactive"][layer][b], placements["proactive"][layer][b - 1])
        assert all(np.array_equal(placements["static"][layer][b], placements["static"][layer][0]) for b in range(cfg.batches))
    # every placement the policies produce satisfies the assignment and capacity constraints
    for p in placements.values():
        for row in p:
            for X in row:
                orc.placement_tables(X, cfg.C_max)
    # a lower bound no placement can beat: the mean load per rank
    for layer in range(cfg.layers):
        for b in range(cfg.batches):
            assert lat["proactive"][layer, b] >= cfg.tokens_per_batch * cfg.K / cfg.R


@pytest.mark.gpu
def test_replay_through_the_cuda_library_matches_the_oracle_scores():
    cfg = replay.ReplayConfig(layers=2, batches=5, tokens_per_batch=768, E=24, K=3, R=4, C_max=7, seed=7200)
    model = opt.LatencyModel(1.0, 0.0, 0.3 / (2 * cfg.H), 2 * cfg.H)
    out = replay.replay_on_gpu(cfg, model)
    idxs, workloads = _oracle_workloads(cfg)
    for layer in range(cfg.layers):
        for b in range(cfg.batches):
            assert np.array_equal(out["workloads"][layer][b], workloads[layer][b])          # W bit-exact
    score = _oracle_score(idxs, cfg)
    lat_o, _ = replay.run_policies(workloads, cfg, model, score)
    want = replay.summarize(lat_o, cfg)
    for p in ("static", "reactive", "proactive"):
        assert np.allclose(out["per_batch"][p], want["per_batch"][p], rtol=0, atol=1e-9)
    assert out["proactive_vs_reactive_gain"] > 0.0


@pytest.mark.gpu
def test_replay_with_the_gpu_scored_search_as_chooser():
    cfg = replay.ReplayConfig(layers=1, batches=4, tokens_per_batch=512, E=12, K=2, R=3, C_max=5, seed=7300,
                              chooser="search")
    out = replay.replay_on_gpu(cfg)
    assert out["mean_latency"]["proactive"] <= out["mean_latency"]["reactive"] * (1 + 1e-9)
