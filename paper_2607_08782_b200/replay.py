"""Multi-layer replay of a stream of batches whose expert popularity shifts over time.

The paper's motivation (Section III): request patterns shift, so the placement that was best for the last batch
is not the best for the next one; a placement chosen *before* a batch runs from (a prediction of) that batch's own
routing - proactive - beats one chosen from the previous batch's routing - reactive - and both beat a placement
fixed offline.  This module replays such a stream through the library on one GPU: for every layer and batch it
routes the tokens (`director_route`), builds the workload matrix (`director_placement_cost`), lets a policy pick the
placement, and scores that placement with the cost model of Section VI-A (Eq. 1-4, affine latency stand-ins).
No weights move: on one GPU a placement change is a new placement matrix.

Policies
  static     one placement per layer, chosen from the sum of the first `warmup` batches' workload matrices
  reactive   batch b runs under the placement chosen from batch b-1's workload (batch 0: the static one)
  proactive  batch b runs under the placement chosen from its own workload (ground-truth routing, the paper's
             upper bound for any predictor)
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import optimizer as opt
from . import placement as greedy
from . import synth


@dataclass
class ReplayConfig:
    layers: int = 2
    batches: int = 8
    tokens_per_batch: int = 1024
    H: int = 256
    E: int = 32
    K: int = 4
    R: int = 4
    C_max: int = 9
    zipf_s_range: tuple = (0.8, 1.6)
    seed: int = 7000
    warmup: int = 2
    chooser: str = "greedy"          # "greedy": placement.greedy_balanced; "search": optimizer.optimize_placement


def layer_shape(cfg: ReplayConfig, layer: int) -> synth.Shape:
    """All batches of one layer as one token stream whose popularity law is redrawn every batch."""
    return synth.Shape(f"replay_l{layer}", cfg.batches * cfg.tokens_per_batch, cfg.H, cfg.E, cfg.K, 128, 0, cfg.R,
                       cfg.C_max, 1.2, cfg.seed + 101 * layer, segment_tokens=cfg.tokens_per_batch,
                       zipf_s_range=cfg.zipf_s_range)


def choose_placement(W: np.ndarray, cfg: ReplayConfig, model: opt.LatencyModel, evaluate=None) -> np.ndarray:
    """A placement for workload matrix W [R,E] under the configured chooser."""
    if cfg.chooser == "greedy":
        return greedy.greedy_balanced(greedy.expert_counts(W), cfg.R, cfg.C_max)
    if cfg.chooser == "search":
        return opt.optimize_placement(W, cfg.C_max, model, evaluate, allow_replicas=True)["X"]
    raise ValueError(cfg.chooser)


def run_policies(workloads, cfg: ReplayConfig, model: opt.LatencyModel, score, evaluator_for=None):
    """workloads[layer][batch] = W [R,E] (numpy int64).  score(layer, batch, X) -> (max_load, max_send_tokens) of
    running that batch under placement X.  Returns per-policy latency arrays [layers, batches] and the placements."""
    L, B = cfg.layers, cfg.batches
    lat = {p: np.zeros((L, B)) for p in ("static", "reactive", "proactive")}
    placements = {p: [[None] * B for _ in range(L)] for p in lat}
    for layer in range(L):
        ev = evaluator_for(layer) if evaluator_for else None
        W_warm = sum(workloads[layer][b] for b in range(min(cfg.warmup, B)))
        X_static = choose_placement(W_warm, cfg, model, ev(W_warm) if ev else None)
        X_prev = X_static
        for b in range(B):
            W = workloads[layer][b]
            X_pro = choose_placement(W, cfg, model, ev(W) if ev else None)
            for name, X in (("static", X_static), ("reactive", X_prev), ("proactive", X_pro)):
                max_load, max_send = score(layer, b, X)
                lat[name][layer, b] = float(model.latency(max_load, max_send))
                placements[name][layer][b] = X
            X_prev = X_pro                      # what a reactive system knows when batch b+1 arrives
    return lat, placements


def summarize(lat: dict, cfg: ReplayConfig) -> dict:
    """Model latency per batch summed over layers (Eq. 2 + Eq. 4 sum over l), averaged over the batches after warm-up."""
    sl = slice(min(cfg.warmup, cfg.batches - 1), None)
    per = {p: v.sum(axis=0)[sl] for p, v in lat.items()}
    mean = {p: float(v.mean()) for p, v in per.items()}
    return {
        "mean_latency": mean,
        "proactive_vs_reactive_gain": 1.0 - mean["proactive"] / mean["reactive"],
        "proactive_vs_static_gain": 1.0 - mean["proactive"] / mean["static"],
        "per_batch": {p: [float(x) for x in v] for p, v in per.items()},
    }


def replay_on_gpu(cfg: ReplayConfig, model: opt.LatencyModel | None = None, device: str = "cuda") -> dict:
    """The whole replay through the CUDA library: routing, workload matrices and every score come from
    director_route / director_placement_cost / director_placement_cost_batch."""
    import torch
    from .binding import Director

    model = model or opt.LatencyModel(1.0, 0.0, 0.2 / (2 * cfg.H), 2 * cfg.H)
    T = cfg.tokens_per_batch
    d = Director(T, cfg.H, 128, cfg.E, cfg.K, 0, cfg.R, cfg.C_max)
    i64 = dict(dtype=torch.int64, device=device)
    idx = torch.empty((T, cfg.K), dtype=torch.int32, device=device)
    wts = torch.empty((T, cfg.K), dtype=torch.float32, device=device)
    Wd, load, dt, db = (torch.empty(s, **i64) for s in ((cfg.R, cfg.E), (cfg.R,), (cfg.R, cfg.R), (cfg.R, cfg.R)))
    X_any = np.zeros((cfg.E, cfg.R), dtype=np.uint8)
    X_any[np.arange(cfg.E), np.arange(cfg.E) % cfg.R] = 1
    d.set_placement(X_any)

    workloads, W_dev = [], []
    for layer in range(cfg.layers):
        logits = torch.from_numpy(synth.make_logits(layer_shape(cfg, layer))).to(device)
        ws, wd = [], []
        for b in range(cfg.batches):
            d.route(T, logits[b * T:(b + 1) * T], idx, wts)
            d.placement_cost(T, idx, None, Wd, load, dt, db)          # W does not depend on the placement
            wd.append(Wd.clone())
            ws.append(Wd.cpu().numpy().copy())
        workloads.append(ws)
        W_dev.append(wd)
    d.check_device_status()

    evaluators = {}

    def evaluator(layer, b):
        key = (layer, b)
        if key not in evaluators:
            evaluators[key] = opt.GpuPlacementEvaluator(d, W_dev[layer][b], chunk=4096)
        return evaluators[key]

    def score(layer, b, X):
        s = evaluator(layer, b)(X[None])[0]
        assert s[3] == 1, "policy produced an invalid placement"
        return s[0], s[1]

    def evaluator_for(layer):
        def for_workload(W):                       # an evaluator bound to an arbitrary (possibly summed) workload matrix
            return opt.GpuPlacementEvaluator(d, torch.from_numpy(np.ascontiguousarray(W)).to(device), chunk=4096)
        return for_workload

    lat, placements = run_policies(workloads, cfg, model, score, evaluator_for if cfg.chooser == "search" else None)
    out = summarize(lat, cfg)
    out["config"] = cfg.__dict__ | {"zipf_s_range": list(cfg.zipf_s_range)}
    out["workloads"] = workloads
    out["placements"] = placements
    return out


if __name__ == "__main__":
    import json
    res = replay_on_gpu(ReplayConfig())
    print(json.dumps({k: res[k] for k in ("mean_latency", "proactive_vs_reactive_gain", "proactive_vs_static_gain")}))
