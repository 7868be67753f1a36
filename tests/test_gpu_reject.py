"""The fused softmax / ratio / residual-resample kernel alone, on supplied logits, against the checker."""
import numpy as np
import pytest

import oracle
from paper_2605_13319_b200 import synth
from harness import Tally

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctxs():
    from paper_2605_13319_b200 import binding
    out = {}
    for V in (1008, 1024, 32000, 50256, 128256):      # 1008 and 50256: multiples of 16 only (ragged last warp range)
        shape = synth.TINY.scaled(name=f"v{V}", vocab=V, n_layers=1, d_model=64, d_ffn=64, n_q_heads=1,
                                  n_kv_heads=1)
        w = synth.make_weights(shape, 0)
        out[V] = binding.Context(shape, w, n_pages=4, max_seq=64, max_draft=16)
    yield out
    for c in out.values():
        c.close()


@pytest.mark.parametrize("V,k,trials", [(1008, 3, 40), (1024, 4, 60), (32000, 8, 24), (50256, 5, 12), (128256, 16, 8)])
@pytest.mark.parametrize("sigma", [0.3, 1.0, 3.0])
def test_reject_matches_oracle(ctxs, V, k, trials, sigma):
    ctx = ctxs[V]
    tally = Tally()
    for t in range(trials):
        seed = 1000 * k + t
        logits = (synth.normal_f32((k + 1, V), seed, 1) * 1.3).astype(np.float32)
        noise = synth.normal_f32((k, V), seed, 2)
        q = np.stack([oracle.softmax(logits[i].astype(np.float64) + sigma * noise[i]) for i in range(k)]).astype(np.float32)
        du = synth.uniform_f32(k, seed, 3)
        drafts = np.array([min(int(np.searchsorted(np.cumsum(q[i].astype(np.float64)), du[i] * q[i].astype(np.float64).sum(), side="right")), V - 1)
                           for i in range(k)], np.int32)
        u = synth.uniform_f32(k + 1, seed, 4)
        n_r, t_r, margins = oracle.reject(logits.astype(np.float64), q, drafts, u)
        got = ctx.reject_from_logits(logits, q, drafts, u)
        tally.check(got, dict(n_accepted=n_r, next_token=t_r, margins=margins), logits, q, u, where=f"V={V} t={t}")
    print("\n" + tally.report())
    # identical fp32 logits on both sides: only fp64 summation order differs, flips must be very rare
    assert tally.len_flip == 0 and tally.tok_flip <= max(1, trials // 8)


def test_reject_greedy_and_special_cases(ctxs):
    from paper_2605_13319_b200 import binding
    V, k = 1024, 6
    ctx = ctxs[V]
    rng = np.random.default_rng(0)
    for t in range(40):
        logits = rng.standard_normal((k + 1, V)).astype(np.float32)
        am = logits.argmax(1)
        drafts = am[:k].astype(np.int32).copy()
        cut = t % (k + 1)
        if cut < k:
            drafts[cut] = (drafts[cut] + 5) % V
        got = ctx.reject_from_logits(logits, None, drafts, np.zeros(k + 1, np.float32), mode=binding.MODE_GREEDY)
        want = oracle.reject(logits.astype(np.float64), None, drafts, np.zeros(k + 1, np.float32), greedy=True)[:2]
        assert got == want == (cut, int(am[cut]))
    # p == q: everything accepted, extra token drawn from p_k
    logits = rng.standard_normal((k + 1, V)).astype(np.float32) * 2
    q = np.stack([oracle.softmax(logits[i].astype(np.float64)) for i in range(k)]).astype(np.float32)
    u = np.minimum(synth.uniform_f32(k + 1, 5, 4), np.float32(0.999))
    drafts = rng.integers(0, V, k).astype(np.int32)
    got = ctx.reject_from_logits(logits, q, drafts, u)
    want = oracle.reject(logits.astype(np.float64), q, drafts, u)[:2]
    assert got == want and got[0] == k
    # one-hot q on a token the target gives ~0 mass: rejected at row 0, residual == p
    logits[0, 7] = -80.0
    q1 = q.copy(); q1[0] = 0; q1[0, 7] = 1.0
    drafts[0] = 7
    got = ctx.reject_from_logits(logits, q1, drafts, u)
    want = oracle.reject(logits.astype(np.float64), q1, drafts, u)[:2]
    assert got == want and got[0] == 0
    # q zero on the drafted token, p positive: ratio = +inf, accepted
    q2 = q.copy(); q2[0, drafts[1]] = 0.0; drafts[0] = drafts[1]; q2[0, drafts[0]] = 0.0
    got = ctx.reject_from_logits(logits, q2, drafts, u)
    want = oracle.reject(logits.astype(np.float64), q2, drafts, u)[:2]
    assert got == want and got[0] >= 1
    # u at the top of the grid: the last token with mass
    u_top = u.copy(); u_top[:] = 1 - 2.0 ** -24
    got = ctx.reject_from_logits(logits, q, drafts, u_top)
    want = oracle.reject(logits.astype(np.float64), q, drafts, u_top)[:2]
    assert got[0] == want[0]
