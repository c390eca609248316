"""Device-tensor convenience around the C entry points: owns the output tensors of one MoE layer
and calls the five stages in order on the current stream.  Allocation and marshalling only."""
from __future__ import annotations

import numpy as np
import torch

from .binding import Director


def bf16_bits_to_tensor(bits: np.ndarray, device="cuda") -> torch.Tensor:
    """uint16 bf16 bit patterns (numpy) -> torch.bfloat16 tensor on `device` (bit-exact)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)


def tensor_to_bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class MoELayer:
    """Routed experts w_gate/w_up [E,F,H], w_down [E,H,F]; optional shared experts ws_gate/ws_up [S*F,H],
    ws_down [H,S*F] (all torch.bfloat16 CUDA tensors, kept by reference)."""

    def __init__(self, T_max, H, F, E, K, S, R, C_max, w_gate, w_up, w_down, ws_gate=None, ws_up=None,
                 ws_down=None, device="cuda"):
        self.dims = dict(T_max=T_max, H=H, F=F, E=E, K=K, S=S, R=R, C_max=C_max)
        self.d = Director(T_max, H, F, E, K, S, R, C_max)
        self.ffn_variant = 2
        self.w = (w_gate, w_up, w_down)
        self.ws = (ws_gate, ws_up, ws_down)
        A, G = T_max * K, R * C_max
        i32 = dict(dtype=torch.int32, device=device)
        self.topk_idx = torch.empty((T_max, K), **i32)
        self.topk_w = torch.empty((T_max, K), dtype=torch.float32, device=device)
        self.xp = torch.empty((A, H), dtype=torch.bfloat16, device=device)
        self.yp = torch.empty((A, H), dtype=torch.bfloat16, device=device)
        self.row_token = torch.empty((A,), **i32)
        self.inv_row = torch.empty((T_max, K), **i32)
        self.dest_rank = torch.empty((T_max, K), **i32)
        self.seg_offsets = torch.empty((G + 1,), **i32)
        self.y = torch.empty((T_max, H), dtype=torch.bfloat16, device=device)
        self.y_shared = torch.empty((T_max, H), dtype=torch.bfloat16, device=device) if S > 0 else None
        i64 = dict(dtype=torch.int64, device=device)
        self.workload = torch.empty((R, E), **i64)
        self.rank_load = torch.empty((R,), **i64)
        self.dispatch_tokens = torch.empty((R, R), **i64)
        self.dispatch_bytes = torch.empty((R, R), **i64)     # bit pattern of uint64

    def set_placement(self, X: np.ndarray):
        self.d.set_placement(X)

    def set_ffn_variant(self, variant: int):
        """Tile scheme of the expert GEMMs (see director_set_ffn_variant); only scheme 2 can gather from x."""
        self.d.set_ffn_variant(variant)
        self.ffn_variant = variant

    def route(self, T, logits):
        self.d.route(T, logits, self.topk_idx, self.topk_w)

    def set_replica_policy(self, policy: int):
        """0: round-robin over an expert's replicas; 1: locality first (see director_set_replica_policy)."""
        self.d.set_replica_policy(policy)

    def dispatch(self, T, x, indices_only=False, token_src_rank=None):
        xp = None if indices_only else self.xp
        if token_src_rank is None:
            self.d.dispatch(T, x, self.topk_idx, xp, self.row_token, self.inv_row, self.dest_rank, self.seg_offsets)
        else:
            self.d.dispatch_src(T, x, self.topk_idx, token_src_rank, xp, self.row_token, self.inv_row,
                                self.dest_rank, self.seg_offsets)

    def dedup_dispatch_tokens(self, T, token_src_rank=None):
        """[R,R] int64: tokens each rank sends to each rank when a token goes to a rank once (after dispatch)."""
        R = self.dims["R"]
        if getattr(self, "dedup_tokens", None) is None:
            self.dedup_tokens = torch.empty((R, R), dtype=torch.int64, device=self.topk_idx.device)
        self.d.dedup_dispatch_tokens(T, self.dest_rank, token_src_rank, self.dedup_tokens)
        return self.dedup_tokens

    def expert_ffn_gather(self, T, x):
        """The routed experts read their rows from x through row_token (no permuted copy)."""
        S = self.dims["S"]
        self.d.expert_ffn_gather(T, x, self.row_token, self.seg_offsets, *self.w, self.yp,
                                 *(self.ws if S > 0 else (None, None, None)), self.y_shared if S > 0 else None)

    def expert_ffn(self, T, x=None):
        S = self.dims["S"]
        self.d.expert_ffn(T, self.xp, self.seg_offsets, *self.w, self.yp,
                          x if S > 0 else None, *(self.ws if S > 0 else (None, None, None)),
                          self.y_shared if S > 0 else None)

    def combine(self, T):
        self.d.combine(T, self.yp, self.inv_row, self.topk_w, self.y_shared, self.y)

    def expert_ffn_combine(self, T, x=None):
        """Expert FFN with the combine fused into the down projection's epilogue (fp32 atomic adds into an accumulator
        of y: not bit-reproducible, and slower than the two separate steps - see director_expert_ffn_combine)."""
        d = self.dims
        if getattr(self, "y_acc", None) is None:
            dev = self.y.device
            self.y_acc = torch.empty((d["T_max"], d["H"]), dtype=torch.float32, device=dev)
            self.row_weight = torch.empty((d["T_max"] * d["K"],), dtype=torch.float32, device=dev)
        S = d["S"]
        self.d.expert_ffn_combine(T, self.xp, self.seg_offsets, self.row_token, self.inv_row, self.topk_w, *self.w,
                                  x if S > 0 else None, *(self.ws if S > 0 else (None, None, None)), self.y_acc,
                                  self.row_weight, self.y)

    def placement_cost(self, T, token_src_rank=None):
        self.d.placement_cost(T, self.topk_idx, token_src_rank, self.workload, self.rank_load,
                              self.dispatch_tokens, self.dispatch_bytes)

    def forward(self, T, logits, x, with_cost=True, fused=False, fused_combine=False):
        """One pass of the whole layer on device tensors; returns y[:T] (a view of the owned buffer).
        fused: dispatch produces indices only and the expert GEMM gathers its rows from x.  Off by default: the
        weight-stationary GEMM re-reads a token tile once per weight block, so the gather is repeated 2F/256 times
        and costs more than the single row copy it saves."""
        # a batch small enough for the weight-streaming FFN kernels needs no permuted copy either: they stage a
        # segment's few rows from x themselves
        gather = (fused and self.ffn_variant == 2) or (self.d.batch_streams_weights(T) and not fused_combine)
        if with_cost:          # front end in one call (a single launch for decode-sized batches)
            self.d.route_dispatch_cost(T, logits, x, self.topk_idx, self.topk_w, None if gather else self.xp,
                                       self.row_token, self.inv_row, self.dest_rank, self.seg_offsets, self.workload,
                                       self.rank_load, self.dispatch_tokens, self.dispatch_bytes)
        else:
            self.route(T, logits)
            self.dispatch(T, x, indices_only=gather)
        if fused_combine and not gather:          # combine inside the down projection (opt-in, see expert_ffn_combine)
            self.expert_ffn_combine(T, x)
            return self.y[:T]
        if gather:
            self.expert_ffn_gather(T, x)
        else:
            self.expert_ffn(T, x)
        self.combine(T)
        return self.y[:T]

    def capture(self, T, logits, x, with_cost=True, fused=False, fused_combine=False):
        """Records one pass of the layer (fixed T, fixed input and output buffers) into a CUDA graph and returns it;
        `graph.replay()` re-runs the pass with a single launch, which matters for decode-sized batches where the
        handful of kernel launches cost more than the kernels.  Per-kernel profiling must be off while capturing."""
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):                      # first pass outside the capture: lazy module loading
            self.forward(T, logits, x, with_cost, fused, fused_combine)
        torch.cuda.current_stream().wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.forward(T, logits, x, with_cost, fused, fused_combine)
        return graph
