"""Pins for the checker's whole forward / verify / rollback (paper Sec. 2.2, App. B).

A hand-worked two-token model in closed form, plus invariants that a dropped term, a wrong index
or a transposed operand would break: chunking invariance (one pass over k+1 rows == k+1 single
steps), causality, GQA == MHA with replicated KV heads, rollback == a cache that only ever held
the committed rows.  The numpy re-statement at the end is a cross-check, not a pin."""
import math

import numpy as np
import pytest

import oracle
from paper_2605_13319_b200 import synth


def _bf16(x):
    return synth.f32_to_bf16(np.asarray(x, np.float32))


def _bf16r(x):
    return float(synth.bf16_to_f32(_bf16([x]))[0])


def test_hand_worked_two_token_model():
    """L=1, d=hd=2, one head, F=1, V=3, eps=0, small integer weights (exact in bf16)."""
    shape = synth.ModelShape("hand", 1, 2, 1, 1, 2, 1, 3, rms_eps=0.0, rope_base=10000.0)
    I2 = [[1.0, 0.0], [0.0, 1.0]]
    w = {"tok_emb": _bf16([[1, 1], [1, -1], [2, 0]]), "lm_head": _bf16([[1, 0], [0, 1], [1, 1]]),
         "final_norm": np.ones(2, np.float32),
         "layers": [{"wq": _bf16(I2), "wk": _bf16(I2), "wv": _bf16([[1, 0], [0, -1]]), "wo": _bf16(I2),
                     "wg": _bf16([[1, 0]]), "wu": _bf16([[2, 0]]), "wd": _bf16([[1], [-1]]),
                     "attn_norm": np.ones(2, np.float32), "ffn_norm": np.ones(2, np.float32)}]}
    o = oracle.Oracle(shape, w, 8)
    logits = o.forward([0, 1])
    silu = lambda z: z / (1 + math.exp(-z))

    def tail(x1a, x1b):
        # from the post-attention residual (x1a, x1b) to the three logits
        r = math.sqrt((x1a ** 2 + x1b ** 2) / 2)
        h = x1a / r                                   # only the first coordinate feeds gate / up
        a = silu(h) * 2 * h
        y0, y1 = x1a + a, x1b - a                     # down projection is (+a, -a)
        rr = math.sqrt((y0 ** 2 + y1 ** 2) / 2)
        return [y0 / rr, y1 / rr, (y0 + y1) / rr]

    # token 0 at position 0: x=(1,1) has rms 1; RoPE at 0 is the identity; one key => attn = v = (1,-1)
    want0 = tail(1 + 1, 1 - 1)
    assert np.allclose(logits[0], want0, atol=1e-14)
    # token 1 at position 1: x=h=(1,-1); q=k=(1,-1) rotated by 1 rad; v = (1, 1)
    c, s = math.cos(1), math.sin(1)
    q1 = (c + s, s - c)                               # (x0 c - x1 s, x1 c + x0 s) with (x0,x1)=(1,-1)
    k1 = (_bf16r(q1[0]), _bf16r(q1[1]))               # cached keys are rounded to bf16
    s0 = (q1[0] * 1 + q1[1] * 1) / math.sqrt(2)       # key 0 is (1,1) unrotated
    s1 = (q1[0] * k1[0] + q1[1] * k1[1]) / math.sqrt(2)
    w1 = 1 / (1 + math.exp(s0 - s1)); w0 = 1 - w1
    att = (w0 * 1 + w1 * 1, w0 * -1 + w1 * 1)         # v0=(1,-1), v1=(1,1)
    want1 = tail(1 + att[0], -1 + att[1])
    assert np.allclose(logits[1], want1, atol=1e-14)
    kk, vv = o.get_kv(0, 1)
    assert np.allclose(kk, k1) and np.array_equal(vv, [1.0, 1.0])
    assert o.len == 2


@pytest.fixture(scope="module")
def tiny():
    shape = synth.TINY.scaled(name="tiny-gqa", n_kv_heads=2, vocab=96, d_ffn=80, d_model=64, head_dim=16)
    return shape, synth.make_weights(shape, 3, std=0.2)


def test_chunking_invariance_and_causality(tiny):
    shape, w = tiny
    toks = synth.tokens_i32(12, 1, 3, shape.vocab)
    a = oracle.Oracle(shape, w, 32)
    la = a.forward(toks)                                        # one pass over 12 rows
    b = oracle.Oracle(shape, w, 32)
    lb = np.concatenate([b.forward(toks[:5]), b.forward(toks[5:6]), b.forward(toks[6:])])
    assert np.allclose(la, lb, atol=1e-11)
    for pos in (0, 7, 11):
        assert np.array_equal(a.get_kv(1, pos)[0], b.get_kv(1, pos)[0])
    # causality: changing a later token leaves earlier rows untouched
    t2 = toks.copy(); t2[8] = (t2[8] + 1) % shape.vocab
    c = oracle.Oracle(shape, w, 32)
    lc = c.forward(t2)
    assert np.array_equal(lc[:8], la[:8]) and not np.allclose(lc[8:], la[8:])


def test_gqa_equals_mha_with_replicated_kv_heads(tiny):
    shape, w = tiny
    grp = shape.n_q_heads // shape.n_kv_heads
    hd, d = shape.head_dim, shape.d_model
    mha = shape.scaled(name="mha", n_kv_heads=shape.n_q_heads)
    w2 = dict(w); w2["layers"] = []
    for l in w["layers"]:
        l2 = dict(l)
        for n in ("wk", "wv"):
            l2[n] = np.ascontiguousarray(np.repeat(l[n].reshape(shape.n_kv_heads, hd, d), grp, axis=0).reshape(-1, d))
        w2["layers"].append(l2)
    toks = synth.tokens_i32(9, 2, 3, shape.vocab)
    la = oracle.Oracle(shape, w, 16).forward(toks)
    lb = oracle.Oracle(mha, w2, 16).forward(toks)
    assert np.allclose(la, lb, atol=1e-12)


def test_verify_rollback_equals_committed_only_cache(tiny):
    shape, w = tiny
    V = shape.vocab
    prefix = synth.tokens_i32(10, 5, 3, V)
    o = oracle.Oracle(shape, w, 64)
    o.prefill(prefix)
    k = 4
    toks, q, seq_logits = o.draft_round(7, k, 1.0, synth.normal_f32((k, V), 5, 7), synth.uniform_f32(k, 5, 6))
    assert o.len == 10
    u = synth.make_accept_uniforms(k, 5)
    r = o.verify(toks, q, u)
    assert np.allclose(r["logits"], seq_logits, atol=1e-11)     # one pass == token-by-token
    assert o.len == 10 + k + 1
    o.rollback(r["base_len"], r["n_accepted"])
    assert o.len == 11 + r["n_accepted"]
    committed = list(prefix) + list(toks[:1 + r["n_accepted"]])
    ref = oracle.Oracle(shape, w, 64)
    ref.prefill(np.array(committed, np.int32))
    nxt = [r["next_token"], 3, 4]
    assert np.allclose(o.forward(nxt), ref.forward(nxt), atol=1e-11)


def test_verify_greedy_and_all_accept(tiny):
    shape, w = tiny
    V = shape.vocab
    o = oracle.Oracle(shape, w, 64)
    o.prefill(synth.tokens_i32(6, 9, 3, V))
    # drafts = the target's own greedy continuation => all accepted, extra token = argmax of last row
    toks = [5]
    for _ in range(3):
        toks.append(int(np.argmax(o.forward([toks[-1]])[0])))
    last = o.forward([toks[-1]])[0]
    o.truncate(6)
    r = o.verify(np.array(toks, np.int32), None, np.zeros(4, np.float32), greedy=True)
    assert r["n_accepted"] == 3 and r["next_token"] == int(np.argmax(last))
    o.rollback(r["base_len"], 3)
    assert o.len == 6 + 4


def test_cache_load_and_read_back_round_trip_and_transplant(tiny):
    """orc_set_kv / orc_set_len / orc_get_kv: what the full-size parity tests and the timed CPU baseline load
    their prefix through.  (1) rows written at a non-zero layer and position come back bit for bit, widened from
    bf16 exactly, and leave their neighbours alone; (2) a hand-sized cache (one key, V set by hand) gives the
    closed-form attention result, so the loaded values are the ones the forward reads; (3) a cache built by a
    prefill, copied row by row into a fresh instance, yields identical logits on the next forward."""
    shape, w = tiny
    wd = shape.n_kv_heads * shape.head_dim
    o = oracle.Oracle(shape, w, 32)
    # (1) bit-exact round trip, layer 1, positions 5..7; every bf16 exponent and sign pattern that is finite
    bits_k = synth.tokens_i32(3 * wd, 11, 1, 0x7f00).astype(np.uint16).reshape(3, wd)
    bits_v = (synth.tokens_i32(3 * wd, 11, 2, 0x7f00).astype(np.uint16) | np.uint16(0x8000)).reshape(3, wd)
    o.set_synthetic_kv(1, bits_k, bits_v, pos0=5)
    for p in range(3):
        kk, vv = o.get_kv(1, 5 + p)
        assert np.array_equal(kk.view(np.uint32), bits_k[p].astype(np.uint32) << 16)
        assert np.array_equal(vv.view(np.uint32), bits_v[p].astype(np.uint32) << 16)
    for layer, pos in ((0, 5), (1, 4), (1, 8)):          # neighbours in both directions stay zero
        kk, vv = o.get_kv(layer, pos)
        assert not kk.any() and not vv.any()
    assert o.len == 0                                     # set_kv does not move the length
    o.set_len(8)
    assert o.len == 8
    # (3) transplant: prefill -> get_kv -> set_kv + set_len into a fresh instance -> same logits, exactly
    a = oracle.Oracle(shape, w, 32)
    prefix = synth.tokens_i32(9, 12, 0, shape.vocab)
    a.prefill(prefix)
    b = oracle.Oracle(shape, w, 32)
    for l in range(shape.n_layers):
        rows = [a.get_kv(l, p) for p in range(9)]
        kb = synth.f32_to_bf16(np.stack([r[0] for r in rows]))
        vb = synth.f32_to_bf16(np.stack([r[1] for r in rows]))
        b.set_synthetic_kv(l, kb, vb)
    b.set_len(9)
    nxt = synth.tokens_i32(4, 12, 1, shape.vocab)
    assert np.array_equal(a.forward(nxt), b.forward(nxt))
    # a row loaded one position off, or into the wrong layer, changes the result
    c = oracle.Oracle(shape, w, 32)
    for l in range(shape.n_layers):
        rows = [a.get_kv(l, p) for p in range(9)]
        kb = synth.f32_to_bf16(np.stack([r[0] for r in rows]))
        vb = synth.f32_to_bf16(np.stack([r[1] for r in rows]))
        c.set_synthetic_kv(shape.n_layers - 1 - l, kb, vb)
    c.set_len(9)
    a.truncate(9)
    assert not np.array_equal(a.forward(nxt), c.forward(nxt))


def test_loaded_cache_is_what_attention_reads():
    """Closed form on the hand-sized model: with the prefix K rows all zero every cached score is 0, so a query row
    attends uniformly over the loaded V rows and itself; the loaded V values (exact small integers) appear in the
    logits through the known tail of that model."""
    shape = synth.ModelShape("hand", 1, 2, 1, 1, 2, 1, 3, rms_eps=0.0, rope_base=10000.0)
    I2 = [[1.0, 0.0], [0.0, 1.0]]
    Z2 = [[0.0, 0.0], [0.0, 0.0]]
    w = {"tok_emb": _bf16([[1, 1], [1, -1], [2, 0]]), "lm_head": _bf16([[1, 0], [0, 1], [1, 1]]),
         "final_norm": np.ones(2, np.float32),
         "layers": [{"wq": _bf16(I2), "wk": _bf16(Z2), "wv": _bf16(Z2), "wo": _bf16(I2),
                     "wg": _bf16([[0, 0]]), "wu": _bf16([[0, 0]]), "wd": _bf16([[0], [0]]),
                     "attn_norm": np.ones(2, np.float32), "ffn_norm": np.ones(2, np.float32)}]}
    o = oracle.Oracle(shape, w, 8)
    # three loaded positions: K = 0, V = (3, -6), (6, 0), (-3, 9); the new row's own K and V are 0 (zero matrices)
    o.set_synthetic_kv(0, _bf16([[0, 0]] * 3), _bf16([[3, -6], [6, 0], [-3, 9]]))
    o.set_len(3)
    logits = o.forward([0])[0]                 # x = (1, 1); attention = mean of the 4 V rows = (1.5, 0.75)
    x0, x1 = 1 + 6 / 4, 1 + 3 / 4
    r = math.sqrt((x0 ** 2 + x1 ** 2) / 2)
    assert np.allclose(logits, [x0 / r, x1 / r, (x0 + x1) / r], atol=1e-14)
    assert o.len == 4


def test_chained_rounds_equal_two_separate_rounds_by_enumeration():
    """App. B, cloud side of proactive transmission, enumerated on a small vocabulary: for EVERY candidate first
    buffered token b_1 and a grid of uniforms, the buffered tokens are kept exactly when all drafts were accepted
    and the extra token equals b_1; when kept, the second round's outcome and logits equal those of an instance
    that never chained (prefilled directly with the committed sequence, then verified); when discarded, the cache
    holds the first round's commit only and behaves like an instance that was never offered the buffered tokens."""
    shape = synth.TINY.scaled(name="chain", vocab=16, n_layers=1, d_model=32, n_q_heads=2, n_kv_heads=1, head_dim=16,
                              d_ffn=48)
    w = synth.make_weights(shape, 9)
    V, P, k, m = shape.vocab, 5, 2, 3
    prefix = synth.tokens_i32(P, 9, 0, V)
    kept = dropped = 0
    for trial in range(6):
        a = oracle.Oracle(shape, w, 32)
        a.prefill(prefix)
        pending = int(synth.tokens_i32(1, 9, 100 + trial, V)[0])
        # drafts from q = p (sigma 0) half of the time so that full acceptance is common, else noisy
        sigma = 0.0 if trial % 2 == 0 else 1.5
        toks, q, _ = a.draft_round(pending, k, sigma, synth.normal_f32((k, V), 9, 200 + trial),
                                   synth.uniform_f32(k, 9, 300 + trial))
        u = synth.uniform_f32(k + 1, 9, 400 + trial)
        rest = synth.tokens_i32(m - 1, 9, 500 + trial, V)
        q_buf = np.stack([oracle.softmax(synth.normal_f32(V, 9, 600 + trial + 50 * j).astype(np.float64))
                          for j in range(m - 1)]).astype(np.float32)
        u_buf = synth.uniform_f32(m, 9, 700 + trial)
        for b1 in range(V):
            buffered = np.concatenate([[b1], rest]).astype(np.int32)
            c = oracle.Oracle(shape, w, 32)
            c.prefill(prefix)
            r1, r2 = c.verify_chain(toks, q, u, buffered, q_buf, u_buf)
            # the first round is an ordinary round
            s = oracle.Oracle(shape, w, 32)
            s.prefill(prefix)
            ref1 = s.verify(toks, q, u)
            assert (r1["n_accepted"], r1["next_token"]) == (ref1["n_accepted"], ref1["next_token"])
            assert np.array_equal(r1["logits"], ref1["logits"])
            keep = ref1["n_accepted"] == k and ref1["next_token"] == b1
            assert (r2 is not None) == keep
            committed = list(prefix) + list(toks[:1 + ref1["n_accepted"]])
            if keep:
                kept += 1
                f = oracle.Oracle(shape, w, 32)
                f.prefill(np.array(committed, np.int32))
                ref2 = f.verify(buffered, q_buf, u_buf)
                assert (r2["n_accepted"], r2["next_token"]) == (ref2["n_accepted"], ref2["next_token"])
                assert np.allclose(r2["logits"], ref2["logits"], atol=1e-12)    # same values; prefill chunks differ
                assert c.len == len(committed) + 1 + ref2["n_accepted"]
            else:
                dropped += 1
                assert c.len == len(committed)
                nxt = np.array([ref1["next_token"], 3, 7], np.int32)
                f = oracle.Oracle(shape, w, 32)
                f.prefill(np.array(committed, np.int32))
                assert np.allclose(c.forward(nxt), f.forward(nxt), atol=1e-12)
    assert kept >= 2 and dropped >= 2 * 15, (kept, dropped)


def test_numpy_restatement_cross_check(tiny):
    """Not a pin (it re-states the formulas): a compact fp64 numpy forward as a second opinion."""
    shape, w = tiny
    f = lambda a: synth.bf16_to_f32(a).astype(np.float64)
    toks = synth.tokens_i32(7, 4, 3, shape.vocab)
    hd, Hq, Hkv = shape.head_dim, shape.n_q_heads, shape.n_kv_heads
    n = len(toks)
    x = f(w["tok_emb"])[toks]
    norm = lambda z: z / np.sqrt((z ** 2).mean(-1, keepdims=True) + shape.rms_eps)
    th = shape.rope_base ** (-2.0 * np.arange(hd // 2) / hd)
    ang = np.arange(n)[:, None] * th[None, :]

    def rope(z):                                       # z: [n, H, hd]
        a, b = z[..., :hd // 2], z[..., hd // 2:]
        c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
        return np.concatenate([a * c - b * s, b * c + a * s], -1)

    for l in w["layers"]:
        h = norm(x)
        q = rope((h @ f(l["wq"]).T).reshape(n, Hq, hd))
        k = rope((h @ f(l["wk"]).T).reshape(n, Hkv, hd))
        v = (h @ f(l["wv"]).T).reshape(n, Hkv, hd)
        k = synth.bf16_to_f32(synth.f32_to_bf16(k.astype(np.float32))).astype(np.float64)
        v = synth.bf16_to_f32(synth.f32_to_bf16(v.astype(np.float32))).astype(np.float64)
        k = np.repeat(k, Hq // Hkv, 1); v = np.repeat(v, Hq // Hkv, 1)
        sc = np.einsum("ihe,jhe->hij", q, k) / math.sqrt(hd)
        sc = np.where(np.tril(np.ones((n, n), bool))[None], sc, -np.inf)
        p = np.exp(sc - sc.max(-1, keepdims=True)); p /= p.sum(-1, keepdims=True)
        att = np.einsum("hij,jhe->ihe", p, v).reshape(n, Hq * hd)
        x = x + att @ f(l["wo"]).T
        h = norm(x)
        g = h @ f(l["wg"]).T
        x = x + ((g / (1 + np.exp(-g))) * (h @ f(l["wu"]).T)) @ f(l["wd"]).T
    want = norm(x) @ f(w["lm_head"]).T
    got = oracle.Oracle(shape, w, 16).forward(toks)
    assert np.allclose(got, want, atol=1e-10)
