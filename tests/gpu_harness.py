"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI on a seeded workload and
hand back every output as numpy, and the oracle-side counterparts."""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from oracle import director_oracle as orc
from paper_2607_08782_b200 import synth


@dataclass
class GpuResult:
    topk_idx: np.ndarray
    topk_w: np.ndarray
    xp: np.ndarray           # bf16 bits
    yp: np.ndarray           # bf16 bits
    row_token: np.ndarray
    inv_row: np.ndarray
    dest_rank: np.ndarray
    seg_offsets: np.ndarray
    y: np.ndarray            # bf16 bits
    y_shared: np.ndarray | None
    workload: np.ndarray
    rank_load: np.ndarray
    dispatch_tokens: np.ndarray
    dispatch_bytes: np.ndarray
    status: int
    launches: int
    dedup_tokens: np.ndarray | None = None


class GpuCase:
    """Uploads a workload once; `run(X)` executes the five stages under placement X."""

    def __init__(self, shape: synth.Shape, logits, x_bits, weights: synth.Weights, C_max=None, T_max=None):
        import torch
        from paper_2607_08782_b200.layer import MoELayer, bf16_bits_to_tensor
        self.torch = torch
        self.shape = shape
        s = shape
        self.C_max = C_max or s.C_max
        dev = "cuda"
        self.logits = torch.from_numpy(np.ascontiguousarray(logits)).to(dev)
        self.x = bf16_bits_to_tensor(x_bits, dev)
        w = weights
        wg, wu, wd = (bf16_bits_to_tensor(a, dev) for a in (w.w_gate, w.w_up, w.w_down))
        sg = su = sd = None
        if s.S > 0:
            sg = bf16_bits_to_tensor(w.ws_gate.reshape(s.S * s.F, s.H), dev)
            su = bf16_bits_to_tensor(w.ws_up.reshape(s.S * s.F, s.H), dev)
            sd = bf16_bits_to_tensor(synth.concat_shared_down(w.ws_down), dev)
        self.layer = MoELayer(T_max or s.T, s.H, s.F, s.E, s.K, s.S, s.R, self.C_max, wg, wu, wd, sg, su, sd, dev)

    def run(self, X, T=None, src=None, stages="all", policy=0) -> GpuResult:
        from paper_2607_08782_b200.layer import tensor_to_bf16_bits
        torch, L, s = self.torch, self.layer, self.shape
        T = T or s.T
        L.set_placement(X)
        n0 = L.d.launch_count()
        src_t = None if src is None else torch.from_numpy(np.ascontiguousarray(src, dtype=np.int32)).cuda()
        L.set_replica_policy(policy)
        try:
            L.route(T, self.logits)
            L.dispatch(T, self.x, token_src_rank=src_t)       # the home ranks matter to the locality-first rule only
            if stages == "all":
                L.expert_ffn(T, self.x)
                L.combine(T)
            L.placement_cost(T, src_t)
            dedup = L.dedup_dispatch_tokens(T, src_t).cpu().numpy()
        finally:
            L.set_replica_policy(0)
        torch.cuda.synchronize()
        status = L.d.last_status()
        A = T * s.K
        return GpuResult(
            topk_idx=L.topk_idx[:T].cpu().numpy(), topk_w=L.topk_w[:T].cpu().numpy(),
            xp=tensor_to_bf16_bits(L.xp[:A]), yp=tensor_to_bf16_bits(L.yp[:A]),
            row_token=L.row_token[:A].cpu().numpy(), inv_row=L.inv_row[:T].cpu().numpy(),
            dest_rank=L.dest_rank[:T].cpu().numpy(), seg_offsets=L.seg_offsets.cpu().numpy(),
            y=tensor_to_bf16_bits(L.y[:T]),
            y_shared=None if L.y_shared is None else tensor_to_bf16_bits(L.y_shared[:T]),
            workload=L.workload.cpu().numpy(), rank_load=L.rank_load.cpu().numpy(),
            dispatch_tokens=L.dispatch_tokens.cpu().numpy(),
            dispatch_bytes=L.dispatch_bytes.cpu().numpy().view(np.uint64),
            status=status, launches=L.d.launch_count() - n0, dedup_tokens=dedup)


def rel_l2(a: np.ndarray, b: np.ndarray) -> float:
    den = float(np.sqrt(np.sum(b.astype(np.float64) ** 2)))
    return float(np.sqrt(np.sum((a.astype(np.float64) - b) ** 2))) / max(den, 1e-300)


def max_abs(a: np.ndarray, b: np.ndarray) -> float:
    return float(np.max(np.abs(a.astype(np.float64) - b))) if a.size else 0.0


def check_integer_parity(g: GpuResult, idx_o, d_o, c_o, label=""):
    """Bit-exact comparison of everything integer against the oracle."""
    assert np.array_equal(g.topk_idx, idx_o), f"{label}: topk_idx differs"
    for name in ("row_token", "inv_row", "dest_rank", "seg_offsets"):
        assert np.array_equal(getattr(g, name), d_o[name]), f"{label}: {name} differs"
    for name in ("workload", "rank_load", "dispatch_tokens", "dispatch_bytes"):
        assert np.array_equal(getattr(g, name), c_o[name]), f"{label}: {name} differs"


def oracle_layer_tokens(wl_shape, x_bits, weights, idx_o, w64_o, d_o, tokens):
    """Oracle y (fp64) and the yp rows of the given tokens (all K assignments and the shared experts)."""
    s = wl_shape
    tokens = np.asarray(tokens, dtype=np.int64)
    rows = np.unique(d_o["inv_row"][tokens].ravel())
    yp_rows = orc.expert_ffn(d_o["xp"], d_o["seg_offsets"], d_o["slot_expert"], weights.w_gate, weights.w_up,
                             weights.w_down, rows=rows)
    # the oracle's own combine, on row ids renumbered into the sampled row list
    inv_local = np.searchsorted(rows, d_o["inv_row"][tokens]).astype(np.int32)
    ysh = None
    if s.S > 0:
        ysh = orc.shared_ffn(x_bits, weights.ws_gate, weights.ws_up, weights.ws_down, tokens)
    y = orc.combine(yp_rows, inv_local, w64_o[tokens], ysh)
    return y, rows, yp_rows, ysh


def sample_tokens(d_o, T, n_random, seed):
    """First and last row's token of every non-empty segment plus n_random seeded tokens."""
    so = d_o["seg_offsets"]
    edge = []
    for g in range(len(so) - 1):
        if so[g + 1] > so[g]:
            edge += [int(d_o["row_token"][so[g]]), int(d_o["row_token"][so[g + 1] - 1])]
    rnd = synth.raw_u64(seed, 99, 0, n_random) % np.uint64(T)
    return np.unique(np.array(edge + [int(v) for v in rnd], dtype=np.int64))
