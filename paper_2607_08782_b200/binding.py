"""Thin ctypes binding of ``libdirector.so`` (see ``include/director.h``).

Argument marshalling only: torch tensors supply device memory and the current CUDA stream; every
step of the layer runs in the library's own kernels.  There is no fallback: if the library is
missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
from ctypes import POINTER, c_char_p, c_double, c_float, c_int, c_int32, c_int64, c_uint8, c_uint64, c_void_p

from . import build as _build

STATUS_NAMES = {
    0: "DIRECTOR_OK", 1: "DIRECTOR_ERR_INVALID_ARG", 2: "DIRECTOR_ERR_PLACEMENT", 3: "DIRECTOR_ERR_WORKSPACE",
    4: "DIRECTOR_ERR_CUDA", 5: "DIRECTOR_ERR_UNSUPPORTED", 6: "DIRECTOR_ERR_TIMEOUT", 7: "DIRECTOR_ERR_BAD_INDEX",
    8: "DIRECTOR_ERR_NONFINITE", 9: "DIRECTOR_ERR_STATIC_LIMIT",
}

# every symbol include/director.h declares
EXPORTED = (
    "director_create", "director_destroy", "director_set_placement", "director_route", "director_dispatch",
    "director_expert_ffn", "director_combine", "director_placement_cost", "director_layer_forward_host",
    "director_last_status", "director_launch_count", "director_set_profiling", "director_kernel_time",
    "director_status_string", "director_dispatch_index_static", "director_layer_submit_host",
    "director_layer_wait_host", "director_set_ffn_variant", "director_batch_streams_weights", "director_expert_ffn_combine", "director_placement_cost_batch",
    "director_expert_ffn_gather", "director_set_replica_policy", "director_dispatch_src",
    "director_dedup_dispatch_tokens", "director_route_dispatch_cost", "director_layer_forward",
    "director_reserve_placements", "director_select_placement", "director_set_profiling_filter",
    "director_selftest_bounded_wait", "director_gemm_sm_mhz", "director_gemm_counters",
)

REPLICA_ROUND_ROBIN, REPLICA_LOCAL_FIRST = 0, 1


class DirectorShape(ctypes.Structure):
    _fields_ = [(n, c_int32) for n in ("T_max", "H", "F", "E", "K", "S", "R", "C_max")]


class DirectorError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


_lib = None


def load_library(rebuild_if_stale: bool = True) -> ctypes.CDLL:
    """Loads libdirector.so from the package directory (building it first if the sources are newer).
    Raises if it cannot be built or loaded - there is no other implementation to fall back to."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build_director() if rebuild_if_stale else _build.DIRECTOR_LIB
    lib = ctypes.CDLL(str(path))
    vp = c_void_p
    lib.director_create.argtypes = [POINTER(DirectorShape), POINTER(vp)]
    lib.director_destroy.argtypes = [vp]
    lib.director_set_placement.argtypes = [vp, vp, vp]
    lib.director_route.argtypes = [vp, c_int32, vp, vp, vp, vp]
    lib.director_dispatch.argtypes = [vp, c_int32, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.director_expert_ffn.argtypes = [vp, c_int32] + [vp] * 12
    lib.director_expert_ffn_gather.argtypes = [vp, c_int32] + [vp] * 12
    lib.director_combine.argtypes = [vp, c_int32, vp, vp, vp, vp, vp, vp]
    lib.director_expert_ffn_combine.argtypes = [vp, c_int32] + [vp] * 16
    lib.director_placement_cost.argtypes = [vp, c_int32, vp, vp, vp, vp, vp, vp, vp]
    lib.director_layer_forward_host.argtypes = [vp, c_int32] + [vp] * 12
    lib.director_layer_forward.argtypes = [vp, c_int32] + [vp] * 14
    lib.director_placement_cost_batch.argtypes = [vp, vp, c_int32, vp, vp, vp, vp, vp]
    lib.director_layer_submit_host.argtypes = [vp, c_int32] + [vp] * 13
    lib.director_layer_wait_host.argtypes = [vp, c_int64]
    lib.director_dispatch_index_static.argtypes = [c_int32] * 5 + [vp] * 9
    lib.director_last_status.argtypes = [vp, vp]
    lib.director_launch_count.argtypes = [vp]
    lib.director_launch_count.restype = c_int64
    lib.director_set_profiling.argtypes = [vp, c_int32]
    lib.director_set_profiling_filter.argtypes = [vp, c_char_p]
    lib.director_set_ffn_variant.argtypes = [vp, c_int32]
    lib.director_batch_streams_weights.argtypes = [vp, c_int32]
    lib.director_set_replica_policy.argtypes = [vp, c_int32]
    lib.director_reserve_placements.argtypes = [vp, c_int32]
    lib.director_select_placement.argtypes = [vp, c_int32]
    lib.director_route_dispatch_cost.argtypes = [vp, c_int32] + [vp] * 14
    lib.director_dispatch_src.argtypes = [vp, c_int32] + [vp] * 9
    lib.director_dedup_dispatch_tokens.argtypes = [vp, c_int32, vp, vp, vp, vp]
    lib.director_selftest_bounded_wait.argtypes = [vp, c_uint64, vp, vp]
    lib.director_gemm_sm_mhz.argtypes = [vp, c_int32, POINTER(c_double)]
    lib.director_gemm_sm_mhz.restype = c_double
    lib.director_gemm_counters.argtypes = [vp, c_int32, POINTER(c_int64)]
    lib.director_kernel_time.argtypes = [vp, c_char_p, POINTER(c_int64)]
    lib.director_kernel_time.restype = c_double
    lib.director_status_string.argtypes = [c_int]
    lib.director_status_string.restype = c_char_p
    for name in EXPORTED:
        if name not in ("director_launch_count", "director_kernel_time", "director_status_string", "director_gemm_sm_mhz"):
            getattr(lib, name).restype = c_int
    _lib = lib
    return lib


def _ptr(t):
    """Device (or host) address of a torch tensor / numpy array / None."""
    if t is None:
        return None
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def _stream():
    import torch
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, where: str):
    if status != 0:
        raise DirectorError(status, where)


class Director:
    """One MoE layer context: shape, placement and workspace.  Methods mirror the C entry points and
    take torch CUDA tensors (bf16 tensors as torch.bfloat16).  One context serves one stream at a time."""

    def __init__(self, T_max: int, H: int, F: int, E: int, K: int, S: int, R: int, C_max: int):
        self.lib = load_library()
        self.shape = DirectorShape(T_max, H, F, E, K, S, R, C_max)
        self._ctx = c_void_p()
        _check(self.lib.director_create(ctypes.byref(self.shape), ctypes.byref(self._ctx)), "director_create")

    def close(self):
        if getattr(self, "_ctx", None) is not None and self._ctx.value:
            self.lib.director_destroy(self._ctx)
            self._ctx = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- placement -----------------------------------------------------------------------------
    def set_placement(self, X):
        """X: numpy uint8 [E, R] (C-contiguous)."""
        import numpy as np
        X = np.ascontiguousarray(X, dtype=np.uint8)
        assert X.shape == (self.shape.E, self.shape.R)
        _check(self.lib.director_set_placement(self._ctx, X.ctypes.data, _stream()), "director_set_placement")

    # -- stages --------------------------------------------------------------------------------
    def route(self, T, logits, topk_idx, topk_w):
        _check(self.lib.director_route(self._ctx, T, _ptr(logits), _ptr(topk_idx), _ptr(topk_w), _stream()),
               "director_route")

    def dispatch(self, T, x, topk_idx, xp, row_token, inv_row, dest_rank, seg_offsets):
        _check(self.lib.director_dispatch(self._ctx, T, _ptr(x), _ptr(topk_idx), _ptr(xp), _ptr(row_token),
                                          _ptr(inv_row), _ptr(dest_rank), _ptr(seg_offsets), _stream()),
               "director_dispatch")

    def route_dispatch_cost(self, T, logits, x, topk_idx, topk_w, xp, row_token, inv_row, dest_rank, seg_offsets,
                            workload, rank_load, dispatch_tokens, dispatch_bytes):
        _check(self.lib.director_route_dispatch_cost(
            self._ctx, T, _ptr(logits), _ptr(x), _ptr(topk_idx), _ptr(topk_w), _ptr(xp), _ptr(row_token), _ptr(inv_row),
            _ptr(dest_rank), _ptr(seg_offsets), _ptr(workload), _ptr(rank_load), _ptr(dispatch_tokens),
            _ptr(dispatch_bytes), _stream()), "director_route_dispatch_cost")

    def dispatch_src(self, T, x, topk_idx, token_src_rank, xp, row_token, inv_row, dest_rank, seg_offsets):
        _check(self.lib.director_dispatch_src(self._ctx, T, _ptr(x), _ptr(topk_idx), _ptr(token_src_rank), _ptr(xp),
                                              _ptr(row_token), _ptr(inv_row), _ptr(dest_rank), _ptr(seg_offsets),
                                              _stream()), "director_dispatch_src")

    def reserve_placements(self, n: int):
        _check(self.lib.director_reserve_placements(self._ctx, n), "director_reserve_placements")

    def select_placement(self, slot: int):
        _check(self.lib.director_select_placement(self._ctx, slot), "director_select_placement")

    def set_replica_policy(self, policy: int):
        _check(self.lib.director_set_replica_policy(self._ctx, policy), "director_set_replica_policy")

    def dedup_dispatch_tokens(self, T, dest_rank, token_src_rank, dedup_tokens):
        _check(self.lib.director_dedup_dispatch_tokens(self._ctx, T, _ptr(dest_rank), _ptr(token_src_rank),
                                                       _ptr(dedup_tokens), _stream()),
               "director_dedup_dispatch_tokens")

    def expert_ffn(self, T, xp, seg_offsets, w_gate, w_up, w_down, yp, x=None, ws_gate=None, ws_up=None,
                   ws_down=None, y_shared=None):
        _check(self.lib.director_expert_ffn(self._ctx, T, _ptr(xp), _ptr(seg_offsets), _ptr(w_gate), _ptr(w_up),
                                            _ptr(w_down), _ptr(yp), _ptr(x), _ptr(ws_gate), _ptr(ws_up),
                                            _ptr(ws_down), _ptr(y_shared), _stream()), "director_expert_ffn")

    def expert_ffn_gather(self, T, x, row_token, seg_offsets, w_gate, w_up, w_down, yp, ws_gate=None, ws_up=None,
                          ws_down=None, y_shared=None):
        _check(self.lib.director_expert_ffn_gather(self._ctx, T, _ptr(x), _ptr(row_token), _ptr(seg_offsets),
                                                   _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(yp), _ptr(ws_gate),
                                                   _ptr(ws_up), _ptr(ws_down), _ptr(y_shared), _stream()),
               "director_expert_ffn_gather")

    def expert_ffn_combine(self, T, xp, seg_offsets, row_token, inv_row, topk_w, w_gate, w_up, w_down, x, ws_gate, ws_up,
                           ws_down, y_acc, row_weight, y):
        _check(self.lib.director_expert_ffn_combine(self._ctx, T, _ptr(xp), _ptr(seg_offsets), _ptr(row_token),
                                                    _ptr(inv_row), _ptr(topk_w), _ptr(w_gate), _ptr(w_up), _ptr(w_down),
                                                    _ptr(x), _ptr(ws_gate), _ptr(ws_up), _ptr(ws_down), _ptr(y_acc),
                                                    _ptr(row_weight), _ptr(y), _stream()), "director_expert_ffn_combine")

    def combine(self, T, yp, inv_row, topk_w, y_shared, y):
        _check(self.lib.director_combine(self._ctx, T, _ptr(yp), _ptr(inv_row), _ptr(topk_w), _ptr(y_shared),
                                         _ptr(y), _stream()), "director_combine")

    def placement_cost(self, T, topk_idx, token_src_rank, workload, rank_load, dispatch_tokens, dispatch_bytes):
        _check(self.lib.director_placement_cost(self._ctx, T, _ptr(topk_idx), _ptr(token_src_rank), _ptr(workload),
                                                _ptr(rank_load), _ptr(dispatch_tokens), _ptr(dispatch_bytes),
                                                _stream()), "director_placement_cost")

    def placement_cost_batch(self, workload, n, X, rank_load, dispatch_tokens, summary):
        """n candidate placements X (CUDA uint8 [n,E,R]) against one workload matrix (CUDA int64 [R,E])."""
        _check(self.lib.director_placement_cost_batch(self._ctx, _ptr(workload), n, _ptr(X), _ptr(rank_load),
                                                      _ptr(dispatch_tokens), _ptr(summary), _stream()),
               "director_placement_cost_batch")

    def layer_forward(self, T, logits, x, w_gate, w_up, w_down, ws_gate, ws_up, ws_down, y, workload, rank_load,
                      dispatch_tokens, dispatch_bytes):
        """The whole layer on device tensors in one call (intermediates stay in the context's workspace)."""
        _check(self.lib.director_layer_forward(self._ctx, T, _ptr(logits), _ptr(x), _ptr(w_gate), _ptr(w_up),
                                               _ptr(w_down), _ptr(ws_gate), _ptr(ws_up), _ptr(ws_down), _ptr(y),
                                               _ptr(workload), _ptr(rank_load), _ptr(dispatch_tokens),
                                               _ptr(dispatch_bytes), _stream()), "director_layer_forward")

    def layer_forward_host(self, T, logits, x, w_gate, w_up, w_down, ws_gate, ws_up, ws_down, y,
                           rank_load=None, dispatch_bytes=None):
        """logits, x, y, rank_load, dispatch_bytes: host (pinned torch CPU tensors or numpy); weights: device."""
        _check(self.lib.director_layer_forward_host(self._ctx, T, _ptr(logits), _ptr(x), _ptr(w_gate), _ptr(w_up),
                                                    _ptr(w_down), _ptr(ws_gate), _ptr(ws_up), _ptr(ws_down), _ptr(y),
                                                    _ptr(rank_load), _ptr(dispatch_bytes), _stream()),
               "director_layer_forward_host")

    def layer_submit_host(self, T, logits, x, w_gate, w_up, w_down, ws_gate, ws_up, ws_down, y,
                          rank_load=None, dispatch_bytes=None) -> int:
        """Enqueues one batch (host buffers as for layer_forward_host) and returns its ticket; at most two
        batches may be in flight."""
        ticket = c_int64(-1)
        _check(self.lib.director_layer_submit_host(self._ctx, T, _ptr(logits), _ptr(x), _ptr(w_gate), _ptr(w_up),
                                                   _ptr(w_down), _ptr(ws_gate), _ptr(ws_up), _ptr(ws_down), _ptr(y),
                                                   _ptr(rank_load), _ptr(dispatch_bytes), _stream(),
                                                   ctypes.byref(ticket)), "director_layer_submit_host")
        return int(ticket.value)

    def layer_wait_host(self, ticket: int):
        _check(self.lib.director_layer_wait_host(self._ctx, ticket), "director_layer_wait_host")

    # -- status / instrumentation --------------------------------------------------------------
    def last_status(self) -> int:
        return int(self.lib.director_last_status(self._ctx, _stream()))

    def check_device_status(self):
        _check(self.last_status(), "device status")

    def selftest_bounded_wait(self, limit_ns: int, waited_ns=None):
        """Launches the kernel whose bounded wait expires by construction (see director_selftest_bounded_wait)."""
        _check(self.lib.director_selftest_bounded_wait(self._ctx, int(limit_ns), _ptr(waited_ns), _stream()),
               "director_selftest_bounded_wait")

    def set_ffn_variant(self, variant: int):
        _check(self.lib.director_set_ffn_variant(self._ctx, variant), "director_set_ffn_variant")

    def batch_streams_weights(self, T: int) -> bool:
        """True if a batch of T tokens takes the weight-streaming FFN kernels (which need no permuted copy of x)."""
        rc = int(self.lib.director_batch_streams_weights(self._ctx, T))
        if rc < 0:
            raise DirectorError(-rc, "director_batch_streams_weights")
        return rc == 1

    def gemm_sm_mhz(self, which: int = 0):
        """(SM MHz, longest CTA's microseconds) of the most recent gate|up (0) or down (1) GEMM launch, measured
        by the kernel itself (cycle counter against the global timer)."""
        busy = c_double(0.0)
        mhz = float(self.lib.director_gemm_sm_mhz(self._ctx, which, ctypes.byref(busy)))
        if mhz < 0:
            raise DirectorError(4, "director_gemm_sm_mhz")
        return mhz, float(busy.value)

    def gemm_counters(self, which: int = 0) -> dict:
        """What the most recent gate|up (0) or down (1) GEMM launch measured about itself (see
        director_gemm_counters), as derived figures."""
        raw = (c_int64 * 12)()
        _check(self.lib.director_gemm_counters(self._ctx, which, raw), "director_gemm_counters")
        c = [int(v) for v in raw]
        pairs = max(c[11] // 2, 1)
        return {
            "sm_mhz": c[0] / c[1] * 1e3 if c[1] else 0.0,
            "cycles_per_cta": c[0] / max(c[11], 1),
            "k_steps_per_pair": c[4] / pairs, "items_per_pair": c[5] / pairs,
            "cycles_per_k_step": c[3] / c[4] if c[4] else 0.0,
            "issuer_wait_for_accumulator_frac": c[2] / (c[0] / 2) if c[0] else 0.0,
            "issuer_k_loop_frac": c[3] / (c[0] / 2) if c[0] else 0.0,
            "epilogue_drain_cycles_per_tile": c[7] / c[8] if c[8] else 0.0,
            "epilogue_wait_cycles_per_tile": c[6] / c[8] if c[8] else 0.0,
            "longest_cta_us": c[10] * 1e-3,
        }

    def launch_count(self) -> int:
        return int(self.lib.director_launch_count(self._ctx))

    def set_profiling(self, enabled, only: str | None = None):
        """Device timing: True / 1 = events around every kernel, 2 = one pair of events around every stage, False /
        0 = off; `only`: time just the kernels whose name contains this string (per-kernel mode)."""
        _check(self.lib.director_set_profiling_filter(self._ctx, only.encode() if only else None),
               "director_set_profiling_filter")
        _check(self.lib.director_set_profiling(self._ctx, int(enabled)), "director_set_profiling")

    def kernel_time(self, name_substr: str):
        """(total milliseconds, launches) of kernels whose name contains name_substr since profiling was enabled."""
        n = c_int64(0)
        ms = float(self.lib.director_kernel_time(self._ctx, name_substr.encode(), ctypes.byref(n)))
        if ms < 0:
            raise DirectorError(4, "director_kernel_time")
        return ms, int(n.value)


def status_string(status: int) -> str:
    return load_library().director_status_string(status).decode()


def dispatch_index_static(T, K, E, R, C_max, topk_idx, rep_start, rep_slot, row_token, inv_row, dest_rank,
                          seg_offsets, device_status=None):
    """Context-free, allocation-free dispatch indices (director_dispatch_index_static): for callers
    that may not allocate device memory.  All tensor arguments are caller-owned CUDA int32 tensors."""
    st = load_library().director_dispatch_index_static(
        T, K, E, R, C_max, _ptr(topk_idx), _ptr(rep_start), _ptr(rep_slot), _ptr(row_token), _ptr(inv_row),
        _ptr(dest_rank), _ptr(seg_offsets), _ptr(device_status), _stream())
    _check(st, "director_dispatch_index_static")
