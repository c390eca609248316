"""Seeded synthetic workloads shaped like the paper's MoE models (Table 1: experts / top-k).

This module holds none of the MoE layer's arithmetic.  It produces the *inputs* that both
the CUDA library and the CPU oracle consume: router logits, hidden states, expert weights
and the fixed ("primary") part of each expert placement.  The real prompts and trained
weights of the paper's evaluation are not available, so only shapes and routing skew are
reproduced:

* hidden states      x      ~ N(0, 0.5^2)   rounded to bf16
* expert weights     W      ~ N(0, 0.02^2)  rounded to bf16
* router logits      l[t,e] = fp32(N(0,1) + b_e),  b_e = -s * ln(1 + pi(e))
  where pi is a seeded permutation of the experts: a rank-frequency (Zipf-like, exponent s)
  popularity law over the experts.

All numbers come from a counter-based generator (see ``csrc/synth_gen.c``); bf16 tensors
are returned as ``uint16`` bit patterns so that neither consumer depends on the other's
conversion code.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass, field

import numpy as np

from . import build as _build

# stream ids of the counter-based generator
ST_LOGIT, ST_BIAS_PERM, ST_X = 0, 1, 2
ST_WG, ST_WU, ST_WD = 3, 4, 5
ST_SG, ST_SU, ST_SD = 6, 7, 8
ST_PLACEMENT, ST_SEG_S = 9, 10

_lib = None


def _synth():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(_build.build_synth()))
        u64, i64, dbl, ptr = ctypes.c_uint64, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.synth_u64.argtypes = [u64, u64, u64, i64, ptr]
        lib.synth_uniform_f64.argtypes = [u64, u64, u64, i64, ptr]
        lib.synth_normal_f64.argtypes = [u64, u64, u64, i64, dbl, ptr]
        lib.synth_normal_bf16.argtypes = [u64, u64, u64, i64, dbl, ptr]
        for f in (lib.synth_u64, lib.synth_uniform_f64, lib.synth_normal_f64, lib.synth_normal_bf16):
            f.restype = None
        _lib = lib
    return _lib


def raw_u64(seed: int, stream: int, offset: int, n: int) -> np.ndarray:
    out = np.empty(n, dtype=np.uint64)
    _synth().synth_u64(seed, stream, offset, n, out.ctypes.data)
    return out


def uniform_f64(seed: int, stream: int, offset: int, n: int) -> np.ndarray:
    out = np.empty(n, dtype=np.float64)
    _synth().synth_uniform_f64(seed, stream, offset, n, out.ctypes.data)
    return out


def normal_f64(seed: int, stream: int, offset: int, n: int, scale: float = 1.0) -> np.ndarray:
    out = np.empty(n, dtype=np.float64)
    _synth().synth_normal_f64(seed, stream, offset, n, scale, out.ctypes.data)
    return out


def normal_bf16(seed: int, stream: int, shape, scale: float, offset: int = 0) -> np.ndarray:
    """bf16 bit patterns (uint16) of ``scale * N(0,1)``, flat row-major counter = element index."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    _synth().synth_normal_bf16(seed, stream, offset, n, scale, out.ctypes.data)
    return out.reshape(shape)


def permutation(seed: int, stream: int, n: int, offset: int = 0) -> np.ndarray:
    """Fisher-Yates shuffle of 0..n-1 driven by the counter-based generator."""
    a = np.arange(n, dtype=np.int64)
    r = raw_u64(seed, stream, offset, n)
    for i in range(n - 1, 0, -1):
        j = int(r[i] % np.uint64(i + 1))
        a[i], a[j] = a[j], a[i]
    return a


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ----------------------------------------------------------------------------------------------
# workload definitions
# ----------------------------------------------------------------------------------------------

@dataclass(frozen=True)
class Shape:
    """Problem dimensions: T tokens, H hidden, E routed experts, K top-k, F expert FFN dim,
    S shared experts, R logical ranks, C_max expert slots per rank."""
    name: str
    T: int
    H: int
    E: int
    K: int
    F: int
    S: int
    R: int
    C_max: int
    zipf_s: float
    seed: int
    segment_tokens: int = 0          # >0: the popularity law is redrawn every this many tokens
    zipf_s_range: tuple = (0.0, 0.0)


SHAPES = {
    # tiny layer: everything the oracle can brute-force
    "c1_tiny": Shape("c1_tiny", 64, 256, 8, 2, 512, 0, 4, 2, 1.2, 1000),
    # Mixtral-8x7B-shaped (8 experts, top-2)
    "c2_mixtral": Shape("c2_mixtral", 4096, 4096, 8, 2, 14336, 0, 8, 2, 1.0, 2000),
    # DeepSeek-V2-Lite-shaped (64 routed top-6, 2 shared)
    "c3_dsv2lite": Shape("c3_dsv2lite", 8192, 2048, 64, 6, 1408, 2, 8, 9, 1.2, 3000),
    # Qwen1.5-MoE-A2.7B-shaped (60 routed top-4, 4 shared), shifting popularity every 512 tokens
    "c4_qwen15": Shape("c4_qwen15", 16384, 2048, 60, 4, 1408, 4, 8, 8, 1.2, 4000,
                       segment_tokens=512, zipf_s_range=(0.8, 1.6)),
    # Qwen3-30B-A3B-shaped (128 experts top-8); T is swept over 1 / 64 / 1024 / 32768
    "c5_qwen3": Shape("c5_qwen3", 32768, 2048, 128, 8, 768, 0, 16, 9, 1.4, 5000),
}
C5_SWEEP = (1, 64, 1024, 32768)


def shape_for(name: str, T: int | None = None, E: int | None = None) -> Shape:
    """The named workload's shape; T overrides the batch size (config 5's sweep), E the number of routed experts
    (a cut-down copy of a workload with the same tile shapes and a smaller device footprint, for profiler captures)."""
    s = SHAPES[name]
    if (T is None or T == s.T) and (E is None or E == s.E):
        return s
    T = s.T if T is None else T
    E = s.E if E is None else E
    if not (s.K <= E <= s.E):
        raise ValueError(f"{name}: experts must be in [{s.K}, {s.E}]")
    seed = s.seed + (C5_SWEEP.index(T) if (name == "c5_qwen3" and T in C5_SWEEP) else 0)
    return Shape(s.name, T, s.H, E, s.K, s.F, s.S, s.R, s.C_max, s.zipf_s, seed,
                 s.segment_tokens, s.zipf_s_range)


def expert_bias(shape: Shape) -> np.ndarray:
    """b[g, e] (fp64): popularity bias of expert e for token segment g."""
    if shape.segment_tokens <= 0:
        pi = permutation(shape.seed, ST_BIAS_PERM, shape.E)
        return (-shape.zipf_s * np.log1p(pi.astype(np.float64)))[None, :]
    n_seg = -(-shape.T // shape.segment_tokens)
    lo, hi = shape.zipf_s_range
    s_g = lo + (hi - lo) * uniform_f64(shape.seed, ST_SEG_S, 0, n_seg)
    out = np.empty((n_seg, shape.E), dtype=np.float64)
    for g in range(n_seg):
        pi = permutation(shape.seed, ST_BIAS_PERM, shape.E, offset=g * shape.E)
        out[g] = -s_g[g] * np.log1p(pi.astype(np.float64))
    return out


def make_logits(shape: Shape) -> np.ndarray:
    """fp32 router logits [T, E]."""
    noise = normal_f64(shape.seed, ST_LOGIT, 0, shape.T * shape.E).reshape(shape.T, shape.E)
    b = expert_bias(shape)
    if b.shape[0] == 1:
        noise += b
    else:
        seg = np.arange(shape.T) // shape.segment_tokens
        noise += b[seg]
    return noise.astype(np.float32)


def make_x(shape: Shape) -> np.ndarray:
    """bf16 bit patterns [T, H] of hidden states ~ N(0, 0.5^2)."""
    return normal_bf16(shape.seed, ST_X, (shape.T, shape.H), 0.5)


@dataclass
class Weights:
    """bf16 bit patterns. w_gate, w_up: [E, F, H]; w_down: [E, H, F];
    shared experts (S > 0) ws_gate, ws_up: [S, F, H]; ws_down: [S, H, F]."""
    w_gate: np.ndarray
    w_up: np.ndarray
    w_down: np.ndarray
    ws_gate: np.ndarray | None = None
    ws_up: np.ndarray | None = None
    ws_down: np.ndarray | None = None


def make_weights(shape: Shape) -> Weights:
    E, F, H, S, sd = shape.E, shape.F, shape.H, shape.S, shape.seed
    w = Weights(
        w_gate=normal_bf16(sd, ST_WG, (E, F, H), 0.02),
        w_up=normal_bf16(sd, ST_WU, (E, F, H), 0.02),
        w_down=normal_bf16(sd, ST_WD, (E, H, F), 0.02),
    )
    if S > 0:
        w.ws_gate = normal_bf16(sd, ST_SG, (S, F, H), 0.02)
        w.ws_up = normal_bf16(sd, ST_SU, (S, F, H), 0.02)
        w.ws_down = normal_bf16(sd, ST_SD, (S, H, F), 0.02)
    return w


def concat_shared_down(ws_down: np.ndarray) -> np.ndarray:
    """[S, H, F] -> [H, S*F]: the S shared experts seen as one FFN of width S*F (pure re-layout)."""
    S, H, F = ws_down.shape
    return np.ascontiguousarray(ws_down.transpose(1, 0, 2).reshape(H, S * F))


def primary_ranks(shape: Shape) -> np.ndarray:
    """Rank of the single fixed copy of each expert (int64 [E]) for each named workload."""
    E, R = shape.E, shape.R
    e = np.arange(E, dtype=np.int64)
    if shape.name == "c1_tiny":
        perm = permutation(shape.seed, ST_PLACEMENT, E)
        ranks = np.empty(E, dtype=np.int64)
        ranks[perm] = np.arange(E) // 2
        return ranks
    if shape.name == "c2_mixtral":
        return e.copy()
    if shape.name == "c3_dsv2lite":
        return e // 8
    if shape.name == "c4_qwen15":
        return (e * 8) // max(E, 60)
    if shape.name == "c5_qwen3":
        return e % R
    raise KeyError(shape.name)


def placement_from_ranks(ranks: np.ndarray, R: int) -> np.ndarray:
    """Single-copy placement matrix X[E, R] (uint8) from a rank per expert."""
    X = np.zeros((len(ranks), R), dtype=np.uint8)
    X[np.arange(len(ranks)), ranks] = 1
    return X


@dataclass
class Workload:
    shape: Shape
    logits: np.ndarray
    x: np.ndarray
    weights: Weights | None
    X_primary: np.ndarray = field(default=None)


def make_workload(name: str, T: int | None = None, with_weights: bool = True, E: int | None = None) -> Workload:
    shape = shape_for(name, T, E)
    return Workload(
        shape=shape,
        logits=make_logits(shape),
        x=make_x(shape),
        weights=make_weights(shape) if with_weights else None,
        X_primary=placement_from_ranks(primary_ranks(shape), shape.R),
    )
