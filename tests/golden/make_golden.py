"""Writes tests/golden/c1_tiny_oracle.json: outputs of the CPU oracle on the tiny workload (config 1).

The paper prints no worked numeric example for this path, so these are not paper values: they freeze the
oracle's own results (and, through them, the seeded input generator) so that an accidental change to either
shows up as a diff.  This script calls only the input generator and `oracle/`; nothing here comes from the CUDA
path.  Run from the repository root:  python tests/golden/make_golden.py
"""
import hashlib
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import director_oracle as orc           # noqa: E402
from paper_2607_08782_b200 import synth            # noqa: E402


def sha(a: np.ndarray) -> str:
    return hashlib.sha256(np.ascontiguousarray(a).tobytes()).hexdigest()


def compute() -> dict:
    wl = synth.make_workload("c1_tiny")
    s, w = wl.shape, wl.weights
    idx, wt, w64 = orc.route(wl.logits, s.K)
    d = orc.dispatch(idx, wl.X_primary, s.C_max, wl.x)
    c = orc.placement_cost(idx, wl.X_primary, s.C_max, s.H)
    yp = orc.expert_ffn(d["xp"], d["seg_offsets"], d["slot_expert"], w.w_gate, w.w_up, w.w_down)
    y = orc.combine(yp, d["inv_row"], w64)
    # the same routing under a placement with replicas (one more slot per rank), both replica rules
    N = np.bincount(idx.ravel(), minlength=s.E)
    Xr = orc.replicate_hottest(N, wl.X_primary, 3)
    src = orc.source_ranks(s.T, s.R)
    rr = orc.dispatch(idx, Xr, s.C_max + 1)
    lf = orc.dispatch(idx, Xr, s.C_max + 1, policy="local_first")
    replicated = {
        "placement": Xr.tolist(),
        "round_robin": {"seg_offsets": rr["seg_offsets"].tolist(), "inv_row_sha256": sha(rr["inv_row"]),
                        "dispatch_tokens": orc.placement_cost(idx, Xr, s.C_max + 1, s.H)["dispatch_tokens"].tolist(),
                        "dedup_tokens": orc.dedup_dispatch_tokens(rr["dest_rank"], src, s.R).tolist()},
        "local_first": {"seg_offsets": lf["seg_offsets"].tolist(), "inv_row_sha256": sha(lf["inv_row"]),
                        "dispatch_tokens": orc.placement_cost(idx, Xr, s.C_max + 1, s.H,
                                                              policy="local_first")["dispatch_tokens"].tolist(),
                        "dedup_tokens": orc.dedup_dispatch_tokens(lf["dest_rank"], src, s.R).tolist()},
    }
    return {
        "replicated": replicated,
        "inputs": {"logits_sha256": sha(wl.logits), "x_sha256": sha(wl.x), "w_gate_sha256": sha(w.w_gate),
                   "w_down_sha256": sha(w.w_down), "placement": wl.X_primary.tolist()},
        "topk_idx_first4": idx[:4].tolist(),
        "topk_w_first4": [[round(float(v), 9) for v in r] for r in w64[:4]],
        "topk_idx_sha256": sha(idx),
        "seg_offsets": d["seg_offsets"].tolist(),
        "slot_expert": d["slot_expert"].tolist(),
        "inv_row_sha256": sha(d["inv_row"]),
        "rank_load": c["rank_load"].tolist(),
        "dispatch_tokens": c["dispatch_tokens"].tolist(),
        "workload_row_sums": c["workload"].sum(axis=1).tolist(),
        "y_l2_norm": round(float(np.linalg.norm(y)), 9),
        "y_first_row_first4": [round(float(v), 12) for v in y[0, :4]],
        "y_bf16_sha256": sha(orc.f64_to_bf16_bits(y)),
    }


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_tiny_oracle.json")
    with open(path, "w") as f:
        json.dump(compute(), f, indent=1)
    print("wrote", path)
