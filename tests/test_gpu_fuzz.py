"""Seeded random sweep over the supported shape ranges: whole-layer parity (integers bit-exact, bf16 outputs within
tolerance on every token) under both replica rules, with and without caller-supplied home ranks."""
import numpy as np
import pytest

from oracle import director_oracle as orc
from paper_2607_08782_b200 import synth

from gpu_harness import GpuCase
from test_gpu_parity import _check_outputs, _custom, _random_placement

pytestmark = pytest.mark.gpu


def _draw(seed):
    rng = np.random.default_rng(7700 + seed)
    E = int(rng.choice([1, 2, 3, 7, 8, 13, 32, 60, 64, 100, 128, 200, 256]))
    K = int(rng.integers(1, min(8, E) + 1))
    R = int(rng.choice([1, 2, 3, 4, 8, 16, 33, 64]))
    C_min = -(-E // R)
    if C_min > 16:
        R = 64
        C_min = -(-E // R)
    C = int(rng.integers(C_min, min(16, C_min + 6) + 1))
    T = int(rng.choice([1, 2, 31, 32, 33, 255, 256, 257, 500, 1023, 1400]))
    H = int(rng.choice([256, 512, 768]))
    F = int(rng.choice([128, 256, 384]))
    S = int(rng.choice([0, 0, 1, 2]))
    extra = int(rng.integers(0, max(1, R * C - E) + 1))
    policy = int(rng.integers(0, 2))
    with_src = bool(rng.integers(0, 2))
    return T, H, E, K, F, S, R, C, extra, policy, with_src


@pytest.mark.parametrize("seed", range(24))
def test_random_shapes_match_the_oracle(seed):
    T, H, E, K, F, S, R, C, extra, policy, with_src = _draw(seed)
    shape, logits, x, weights = _custom(8800 + seed, T, H, E, K, F, S, R, C)
    X = _random_placement(8800 + seed, E, R, C, extra)
    src = (synth.raw_u64(8800 + seed, 51, 0, T) % np.uint64(R)).astype(np.int32) if with_src else None
    case = GpuCase(shape, logits, x, weights)
    g = case.run(X, src=src, policy=policy)
    pname = "local_first" if policy else "round_robin"
    idx, w, w64 = orc.route(logits, K)
    d = orc.dispatch(idx, X, C, x, policy=pname, src=src)
    c = orc.placement_cost(idx, X, C, H, src, policy=pname)
    label = f"fuzz{seed} T={T} H={H} E={E} K={K} F={F} S={S} R={R} C={C} extra={extra} {pname} src={with_src}"
    _check_outputs(shape, g, x, weights, idx, w, w64, d, c, np.arange(T), label)
    src_o = orc.source_ranks(T, R) if src is None else src
    assert np.array_equal(g.dedup_tokens, orc.dedup_dispatch_tokens(d["dest_rank"], src_o, R)), label
