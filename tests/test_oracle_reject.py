"""Pins for the accept / correct rule (paper Sec. 2.2 prose; Sec. 1: the target's output
distribution is preserved exactly; App. B: an extra token when every draft is accepted).

The rule is piecewise constant in its uniforms, which live on the grid m * 2^-24, so the
probability of any outcome can be counted EXACTLY by bisection over m instead of by sampling."""
import math

import numpy as np
import pytest

import oracle

G = 1 << 24


def _count_true(pred):
    """pred(m) is true for m < c and false for m >= c (m integer in [0, G)); return c."""
    lo, hi = 0, G          # invariant: pred true below lo, false from hi on
    while lo < hi:
        mid = (lo + hi) // 2
        if pred(mid):
            lo = mid + 1
        else:
            hi = mid
    return lo


def _logits_of(p):
    with np.errstate(divide="ignore"):
        return np.log(np.asarray(p, np.float64))


def _accept_prob(logits, q, drafts, pos):
    """P_u(draft `pos` accepted | earlier drafts accepted), exact on the 2^-24 grid."""
    k = len(drafts)

    def pred(m):
        u = np.zeros(k + 1, np.float32)       # u=0 accepts every other position that can be accepted
        u[pos] = m / G
        n_acc, _, _ = oracle.reject(logits, q, drafts, u)
        return n_acc > pos
    return _count_true(pred) / G


def _draw_dist(logits, q, drafts, u_accept):
    """Distribution of the emitted token over the final uniform, acceptance uniforms fixed."""
    k = len(drafts)
    V = logits.shape[1]
    counts = []
    for t in range(V):
        def pred(m, t=t):
            u = np.concatenate([u_accept, [m / G]]).astype(np.float32)
            _, tok, _ = oracle.reject(logits, q, drafts, u)
            return tok <= t
        counts.append(_count_true(pred))
    c = np.array([0] + counts, np.float64)
    assert counts[-1] == G
    return np.diff(c) / G


P_CASES = [
    ([0.5, 0.25, 0.125, 0.125], [0.25, 0.25, 0.25, 0.25]),
    ([0.7, 0.1, 0.2], [0.1, 0.6, 0.3]),
    ([0.3, 0.3, 0.4, 0.0], [0.0, 0.5, 0.25, 0.25]),       # zeros on both sides
    ([0.05, 0.9, 0.05], [0.9, 0.05, 0.05]),
]


@pytest.mark.parametrize("p,q", P_CASES)
def test_single_position_output_distribution_is_p(p, q):
    """Enumerate the draft x ~ q and integrate the uniforms exactly: P(output = t) = p(t)."""
    p, q = np.array(p), np.array(q, np.float32)
    V = len(p)
    # row 0 scores the draft; row 1 (extra token) is irrelevant for the first output token
    logits = np.stack([_logits_of(p), np.zeros(V)])
    out = np.zeros(V)
    for x in range(V):
        if q[x] == 0:
            continue
        a = _accept_prob(logits, q[None, :], [x], 0)
        assert abs(a - min(1.0, p[x] / float(q[x]))) < 2 / G
        out[x] += float(q[x]) * a
        if a < 1.0:
            corr = _draw_dist(logits, q[None, :], [x], np.array([np.float32(1 - 1 / G)]))  # forces rejection
            resid = np.maximum(0, p - q.astype(np.float64))
            assert np.allclose(corr, resid / resid.sum(), atol=4 / G)
            out += float(q[x]) * (1 - a) * corr
    assert np.allclose(out, p, atol=1e-6)


def test_two_positions_joint_and_extra_token():
    """k=2, rows fixed: P(x1 accepted, x1=a) = min(q0(a),p0(a)); given that, the second output
    token is distributed as p1; given both accepted, the extra token is distributed as p2."""
    p0, q0 = np.array([0.6, 0.3, 0.1]), np.array([0.2, 0.5, 0.3], np.float32)
    p1, q1 = np.array([0.1, 0.2, 0.7]), np.array([0.3, 0.3, 0.4], np.float32)
    p2 = np.array([0.25, 0.5, 0.25])
    logits = np.stack([_logits_of(p0), _logits_of(p1), _logits_of(p2)])
    q = np.stack([q0, q1])
    V = 3
    second = np.zeros(V)
    for a in range(V):
        acc1 = _accept_prob(logits, q, [a, 0], 0)
        assert abs(float(q0[a]) * acc1 - min(float(q0[a]), p0[a])) < 1e-6
    a = 0                                                    # p0(0) > q0(0): always accepted
    for b in range(V):
        acc2 = _accept_prob(logits, q, [a, b], 1)
        second[b] += float(q1[b]) * acc2
        if acc2 < 1:
            corr = _draw_dist(logits, q, [a, b], np.array([0.0, 1 - 1 / G], np.float32))
            second += float(q1[b]) * (1 - acc2) * corr
    assert np.allclose(second, p1, atol=1e-6)
    bonus = _draw_dist(logits, q, [0, 2], np.array([0.0, 0.0], np.float32))   # both accepted (u=0)
    n_acc, _, _ = oracle.reject(logits, q, [0, 2], np.zeros(3, np.float32))
    assert n_acc == 2
    assert np.allclose(bonus, p2, atol=4 / G)


def test_p_equals_q_accepts_everything():
    rng = np.random.default_rng(0)
    V, k = 50, 6
    logits = rng.standard_normal((k + 1, V)) * 2
    q = np.stack([oracle.softmax(logits[i]) for i in range(k)]).astype(np.float64)
    # hand q over at full precision of p by making p exactly representable: use logits = log(q32)
    q32 = q.astype(np.float32)
    logits[:k] = np.log(q32.astype(np.float64))
    for trial in range(50):
        drafts = rng.integers(0, V, k)
        u = rng.integers(0, G, k + 1).astype(np.float64) / G
        u[:k] = np.minimum(u[:k], 1 - 2.0 ** -20)              # ratio is 1 up to ~1e-7 (q32 does not sum to 1 exactly)
        n_acc, tok, _ = oracle.reject(logits, q32, drafts, u.astype(np.float32))
        assert n_acc == k


def test_one_hot_q_on_impossible_token_always_rejected_and_residual_is_p():
    p = np.array([0.5, 0.5, 0.0, 0.0])
    q = np.array([[0.0, 0.0, 1.0, 0.0]], np.float32)
    logits = np.stack([_logits_of(p), np.zeros(4)])
    for m in (0, 1, G // 2, G - 1):
        n_acc, tok, _ = oracle.reject(logits, q, [2], np.array([m / G, 0.3], np.float32))
        assert n_acc == 0 and tok == 0
    dist = _draw_dist(logits, q, [2], np.array([0.0], np.float32))
    assert np.allclose(dist, p, atol=4 / G)


def test_zero_q_positive_p_accepts_and_strict_inequality():
    p = np.array([0.25, 0.75])
    logits = np.stack([_logits_of(p), np.zeros(2)])
    q = np.array([[0.0, 1.0]], np.float32)
    n_acc, _, _ = oracle.reject(logits, q, [0], np.array([1 - 1 / G, 0.0], np.float32))
    assert n_acc == 1                                                       # ratio = +inf
    # ratio exactly 0.75: u = 0.75 is rejected (strict <), the grid point below is accepted
    n_hi, _, _ = oracle.reject(logits, q, [1], np.array([0.75, 0.0], np.float32))
    n_lo, _, _ = oracle.reject(logits, q, [1], np.array([0.75 - 1 / G, 0.0], np.float32))
    assert (n_hi, n_lo) == (0, 1)


def test_greedy_is_longest_argmax_matching_prefix():
    rng = np.random.default_rng(5)
    V, k = 40, 8
    for trial in range(200):
        logits = rng.standard_normal((k + 1, V))
        am = logits.argmax(1)
        match_len = int(rng.integers(0, k + 1))
        drafts = am[:k].copy()
        if match_len < k:
            drafts[match_len] = (am[match_len] + 1 + rng.integers(0, V - 1)) % V
            drafts[match_len + 1:] = rng.integers(0, V, k - match_len - 1)
        n_acc, tok, _ = oracle.reject(logits, None, drafts, np.zeros(k + 1, np.float32), greedy=True)
        want = 0
        while want < k and drafts[want] == am[want]:
            want += 1
        assert n_acc == want == match_len
        assert tok == am[n_acc]
    # exact tie: lowest index wins
    logits = np.zeros((2, 5)); logits[0, [1, 3]] = 2.0
    n_acc, tok, _ = oracle.reject(logits, None, [3], np.zeros(2, np.float32), greedy=True)
    assert (n_acc, tok) == (0, 1)


def test_acceptance_rate_is_one_minus_tv():
    """Per position, P(accept) over x ~ q and u is sum_j min(p_j, q_j) = 1 - TV(p,q)."""
    rng = np.random.default_rng(6)
    V = 30
    l = rng.standard_normal(V) * 1.5
    p = oracle.softmax(l)
    q = oracle.softmax(l + rng.standard_normal(V)).astype(np.float32)
    resid, _ = oracle.final_cdf(l, q)
    tv = 0.5 * np.abs(p - q.astype(np.float64)).sum()
    _, S = oracle.final_cdf(l, q)
    assert abs(S - np.maximum(0, p - q).sum()) < 1e-15
    assert abs(S - tv) < 1e-7                                  # sum max(0,p-q) = TV up to q's fp32 rounding
    n = 40000
    xs = rng.choice(V, size=n, p=q.astype(np.float64) / q.astype(np.float64).sum())
    us = (rng.integers(0, G, n) / G).astype(np.float32)
    logits = np.stack([l, np.zeros(V)])
    acc = sum(oracle.reject(logits, q[None, :], [int(x)], np.array([u, 0.0], np.float32))[0]
              for x, u in zip(xs, us))
    rate = acc / n
    sd = math.sqrt(tv * (1 - tv) / n)
    assert abs(rate - (1 - tv)) < 4 * sd


def test_final_cdf_matches_reject_draw():
    rng = np.random.default_rng(7)
    V = 200
    l = rng.standard_normal((2, V)) * 2
    q = oracle.softmax(l[0] + rng.standard_normal(V)).astype(np.float32)[None, :]
    cdf, S = oracle.final_cdf(l[0], q[0])
    assert abs(cdf[-1] - 1) < 1e-12 and np.all(np.diff(cdf) >= 0)
    for m in rng.integers(0, G, 200):
        u = m / G
        _, tok, _ = oracle.reject(l, q, [int(np.argmax(q[0]))], np.array([1 - 1 / G, u], np.float32))
        lo = cdf[tok - 1] if tok > 0 else 0.0
        assert lo - 1e-12 <= u < cdf[tok] + 1e-12
