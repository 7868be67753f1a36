"""Pins for the CPU checker's building blocks: closed forms, invariants, a library matrix product.

None of these re-type the checker's own loops; each compares it with something fixed by the
mathematics (paper Sec. 2.2 only fixes WHAT the verify pass returns; the Llama-style blocks are
the workload's definition)."""
import math

import numpy as np
import pytest

import oracle
from paper_2605_13319_b200 import synth


def test_linear_matches_library_matmul():
    rng = np.random.default_rng(0)
    for (M, N, K) in [(1, 7, 5), (3, 16, 33), (9, 40, 64), (37, 12, 50)]:
        W = synth.normal_bf16((N, K), 1, 77, 0.5)
        x = rng.standard_normal((M, K))
        want = x @ synth.bf16_to_f32(W).astype(np.float64).T
        got = oracle.linear(W, x)
        assert np.allclose(got, want, rtol=0, atol=1e-12)


def test_linear_special_cases():
    # identity picks the input; a one-hot row picks one input element (catches a transposed operand)
    K = 6
    eye = synth.f32_to_bf16(np.eye(K, dtype=np.float32))
    x = np.arange(12, dtype=np.float64).reshape(2, K)
    assert np.array_equal(oracle.linear(eye, x), x)
    W = np.zeros((4, K), np.float32)
    W[2, 5] = 2.0
    y = oracle.linear(synth.f32_to_bf16(W), x)
    assert y.shape == (2, 4)
    assert np.array_equal(y[:, 2], 2.0 * x[:, 5]) and np.count_nonzero(y) == 2


def test_rmsnorm_closed_form_and_invariants():
    g = np.ones(2, np.float32)
    y = oracle.rmsnorm([3.0, 4.0], g, 0.0)
    r = math.sqrt(12.5)
    assert np.allclose(y, [3 / r, 4 / r], atol=1e-15)
    x = np.random.default_rng(1).standard_normal(257)
    g = np.ones(257, np.float32)
    y = oracle.rmsnorm(x, g, 0.0)
    assert abs(np.sqrt(np.mean(y ** 2)) - 1.0) < 1e-14
    assert np.allclose(oracle.rmsnorm(1000.0 * x, g, 0.0), y, atol=1e-13)      # scale invariance
    # eps enters under the square root, next to the mean of squares
    y2 = oracle.rmsnorm([2.0, 2.0], np.ones(2, np.float32), 5.0)
    assert np.allclose(y2, [2 / 3, 2 / 3], atol=1e-15)
    # gain multiplies element-wise
    y3 = oracle.rmsnorm([1.0, 1.0], np.array([2.0, -3.0], np.float32), 0.0)
    assert np.allclose(y3, [2.0, -3.0], atol=1e-15)


def test_rope_closed_form_and_invariants():
    # hd=2: one pair, theta_0 = 1, so position p rotates (x0,x1) by p radians
    v = oracle.rope([1.0, 0.0], 1, 10000.0)
    assert np.allclose(v, [math.cos(1), math.sin(1)], atol=1e-15)
    # hd=4: pairs are (0,2) and (1,3); theta_1 = base^(-1/2)
    v = oracle.rope([1.0, 1.0, 0.0, 0.0], 3, 100.0)
    assert np.allclose(v, [math.cos(3), math.cos(0.3), math.sin(3), math.sin(0.3)], atol=1e-15)
    rng = np.random.default_rng(2)
    q, k = rng.standard_normal(64), rng.standard_normal(64)
    assert np.array_equal(oracle.rope(q, 0, 1e4), q)                        # position 0 is the identity
    assert abs(np.linalg.norm(oracle.rope(q, 1234, 1e4)) - np.linalg.norm(q)) < 1e-12
    # scores depend on the position difference only
    a = oracle.rope(q, 17, 1e4) @ oracle.rope(k, 5, 1e4)
    b = oracle.rope(q, 17 + 4000, 1e4) @ oracle.rope(k, 5 + 4000, 1e4)
    assert abs(a - b) < 1e-9
    c = oracle.rope(q, 18, 1e4) @ oracle.rope(k, 5, 1e4)
    assert abs(a - c) > 1e-3


def test_softmax_closed_forms():
    assert np.allclose(oracle.softmax(np.full(8, 3.5)), 1 / 8, atol=1e-16)
    p = oracle.softmax([math.log(2.0), 0.0])
    assert np.allclose(p, [2 / 3, 1 / 3], atol=1e-15)
    l = np.random.default_rng(3).standard_normal(5000) * 4
    p = oracle.softmax(l)
    assert abs(p.sum() - 1.0) < 1e-12
    assert np.allclose(oracle.softmax(l + 1000.0), p, atol=1e-13)           # shift invariance, no overflow
    assert np.argmax(p) == np.argmax(l)


def test_attend_special_cases():
    rng = np.random.default_rng(4)
    hd, n = 16, 9
    q = rng.standard_normal(hd)
    kc = rng.standard_normal((n, hd)).astype(np.float32)
    const = rng.standard_normal(hd).astype(np.float32)
    out = oracle.attend(q, kc, np.tile(const, (n, 1)))
    assert np.allclose(out, const, atol=1e-14)                               # constant V
    vc = rng.standard_normal((n, hd)).astype(np.float32)
    assert np.allclose(oracle.attend(q, kc[:1], vc[:1]), vc[0], atol=1e-15)  # single key
    # two keys, closed form: weights softmax([q.k0, q.k1] / sqrt(hd))
    q2 = np.array([1.0, 0.0, 0.0, 0.0])
    k2 = np.array([[2.0, 5, 5, 5], [0.0, 7, 7, 7]], np.float32)
    v2 = np.array([[1.0, 0, 0, 0], [0.0, 1, 0, 0]], np.float32)
    w0 = 1 / (1 + math.exp(-(2.0 - 0.0) / 2.0))                              # sqrt(4) = 2
    assert np.allclose(oracle.attend(q2, k2, v2), [w0, 1 - w0, 0, 0], atol=1e-15)
    # identical keys -> plain average of V
    same = np.tile(kc[0], (n, 1))
    assert np.allclose(oracle.attend(q, same, vc), vc.astype(np.float64).mean(0), atol=1e-14)
