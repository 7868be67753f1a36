"""The seeded input generator: determinism, ranges, moments, bf16 rounding."""
import numpy as np

from paper_2605_13319_b200 import synth


def test_counter_based_and_deterministic():
    a = synth.uniform_f32(1000, 7, 5)
    b = synth.uniform_f32(1000, 7, 5)
    c = synth.uniform_f32(500, 7, 5)
    assert np.array_equal(a, b)
    assert np.array_equal(a[:500], c)            # element i does not depend on n
    assert not np.array_equal(a, synth.uniform_f32(1000, 8, 5))
    assert not np.array_equal(a, synth.uniform_f32(1000, 7, 6))


def test_uniform_range_and_grid():
    u = synth.uniform_f32(200000, 1, 2)
    assert u.min() >= 0.0 and u.max() < 1.0
    m = u.astype(np.float64) * 2 ** 24
    assert np.array_equal(m, np.round(m))         # multiples of 2^-24
    assert abs(u.mean() - 0.5) < 5e-3
    assert abs(u.var() - 1 / 12) < 2e-3


def test_normal_moments_and_bf16():
    z = synth.normal_f32(400001, 3, 9)
    assert abs(z.mean()) < 1e-2 and abs(z.std() - 1.0) < 1e-2
    assert abs(np.mean(z.astype(np.float64) ** 4) - 3.0) < 0.1
    w = synth.normal_bf16((300, 333), 3, 9, 0.02)
    wf = synth.bf16_to_f32(w)
    assert abs(wf.std() - 0.02) < 5e-4
    # bf16 rounding is round-to-nearest-even of the fp32 value
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -9, -2.5, 3.140625], np.float32)
    r = synth.bf16_to_f32(synth.f32_to_bf16(x))
    assert np.array_equal(r, np.array([1.0, 1.0, 1.0 + 2 ** -6, 1.0, -2.5, 3.140625], np.float32))


def test_tokens_and_ints():
    t = synth.tokens_i32(100000, 0, 3, 1024)
    assert t.min() >= 0 and t.max() < 1024
    assert len(np.unique(t)) == 1024
    k = synth.ints_i32(5000, 0, 9, 1, 16)
    assert k.min() == 1 and k.max() == 16


def test_weights_shapes():
    w = synth.make_weights(synth.TINY, 0)
    s = synth.TINY
    assert w["tok_emb"].shape == (s.vocab, s.d_model) and w["tok_emb"].dtype == np.uint16
    assert len(w["layers"]) == s.n_layers
    assert w["layers"][0]["wd"].shape == (s.d_model, s.d_ffn)
    assert np.all(w["layers"][1]["attn_norm"] == 1.0)
    assert not np.array_equal(w["layers"][0]["wq"], w["layers"][1]["wq"])
    n = sum(v.size for l in w["layers"] for k, v in l.items() if v.dtype == np.uint16) \
        + w["tok_emb"].size + w["lm_head"].size
    assert n == s.weight_elems()
