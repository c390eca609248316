"""The seeded input generator: the C implementation equals a NumPy restatement of the same
counter-based recipe, and the workloads have the shapes and skew they are meant to have."""
import numpy as np

from paper_2607_08782_b200 import synth

M64 = (1 << 64) - 1


def _mix64(z):
    z = (z + 0x9E3779B97F4A7C15) & M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & M64
    return z ^ (z >> 31)


def _rnd(seed, stream, i):
    return _mix64((_mix64((seed + stream * 0xD1B54A32D192ED03) & M64) + i) & M64)


def test_raw_stream_matches_python_restatement():
    got = synth.raw_u64(1234, 7, 5, 64)
    want = [_rnd(1234, 7, 5 + k) for k in range(64)]
    assert [int(v) for v in got] == want


def test_uniform_and_normal_match_restatement():
    n = 32
    u = synth.uniform_f64(99, 2, 0, n)
    want_u = np.array([(_rnd(99, 2, k) >> 11) * 2.0 ** -53 for k in range(n)])
    assert np.array_equal(u, want_u)
    z = synth.normal_f64(99, 2, 0, n)
    r = np.sqrt(-2.0 * np.log(1.0 - want_u[0::2]))
    a = 2.0 * np.pi * want_u[1::2]
    want = np.empty(n)
    want[0::2], want[1::2] = r * np.cos(a), r * np.sin(a)
    assert np.allclose(z, want, rtol=0, atol=1e-12)


def test_offset_is_a_pure_counter_shift():
    a = synth.normal_f64(5, 3, 0, 100)
    b = synth.normal_f64(5, 3, 40, 60)
    assert np.array_equal(a[40:], b)


def test_bf16_rounding_is_nearest_even():
    bits = synth.normal_bf16(11, 4, (4096,), 0.02)
    exact = synth.normal_f64(11, 4, 0, 4096, 0.02).astype(np.float32)
    back = synth.bf16_bits_to_f32(bits)
    # nearest: error at most half a bf16 ulp (2^-9 relative)
    assert np.all(np.abs(back - exact) <= np.abs(exact) * 2.0 ** -8)
    # and the rounded value is one of the two neighbours chosen correctly: re-rounding is idempotent
    u = back.view(np.uint32)
    assert np.all((u & 0xFFFF) == 0)


def test_normal_moments():
    z = synth.normal_f64(1, 0, 0, 200_000)
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1.0) < 0.01


def test_permutation_is_a_permutation():
    p = synth.permutation(3, 1, 60)
    assert sorted(p.tolist()) == list(range(60))


def test_workload_shapes_and_skew():
    wl = synth.make_workload("c1_tiny")
    s = wl.shape
    assert wl.logits.shape == (s.T, s.E) and wl.logits.dtype == np.float32
    assert wl.x.shape == (s.T, s.H) and wl.x.dtype == np.uint16
    assert wl.weights.w_gate.shape == (s.E, s.F, s.H)
    assert wl.weights.w_down.shape == (s.E, s.H, s.F)
    assert wl.X_primary.sum(axis=1).tolist() == [1] * s.E
    assert wl.X_primary.sum(axis=0).max() <= s.C_max
    x = synth.bf16_bits_to_f32(wl.x)
    assert abs(x.std() - 0.5) < 0.02
    w = synth.bf16_bits_to_f32(wl.weights.w_up)
    assert abs(w.std() - 0.02) < 0.001
    # the popularity bias makes the mean logit of the favourite expert larger than the least favourite
    m = wl.logits.mean(axis=0)
    assert m.max() - m.min() > 1.0


def test_c4_bias_shifts_between_segments():
    shape = synth.shape_for("c4_qwen15")
    b = synth.expert_bias(shape)
    assert b.shape == (32, 60)
    assert not np.array_equal(np.argsort(b[0]), np.argsort(b[1]))


def test_primaries_respect_capacity():
    for name in synth.SHAPES:
        s = synth.shape_for(name)
        X = synth.placement_from_ranks(synth.primary_ranks(s), s.R)
        assert X.sum(axis=0).max() <= s.C_max, name
        assert (X.sum(axis=1) == 1).all()
