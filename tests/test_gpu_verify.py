"""End-to-end parity of prefill / verify / rollback through the C ABI against the CPU checker."""
import numpy as np
import pytest

import oracle
from paper_2605_13319_b200 import synth
from harness import LOGIT_TOL, Tally, decisions_from_logits, draft_inputs, logit_rel_err

pytestmark = pytest.mark.gpu


def _mk(shape, seed, P, n_pages=None, **kw):
    from paper_2605_13319_b200 import binding
    w = synth.make_weights(shape, seed)
    max_seq = kw.pop("max_seq", P + 256)
    n_pages = n_pages or (max_seq // 16 + 2) * kw.get("max_requests", 1)
    ctx = binding.Context(shape, w, n_pages=n_pages, max_seq=max_seq, poison=True, **kw)
    orc = oracle.Oracle(shape, w, max_seq)
    return w, ctx, orc


def test_tiny_config_many_seeds():
    """2 layers, d 256, 4 heads x 64, FFN 688, vocab 1024; P=64, k=4, sigma=1; stochastic and greedy."""
    from paper_2605_13319_b200 import binding
    shape, P, k = synth.TINY, 64, 4
    w, ctx, orc = _mk(shape, 0, P)
    tally, gt = Tally(), Tally()
    prefix = synth.make_prefix(shape, P, 0)
    orc.prefill(prefix)
    req = ctx.req_open()
    last = ctx.prefill(req, prefix, want_last_logits=True)
    assert ctx.req_len(req) == P
    # KV written by the GPU prefill equals the oracle's bf16-rounded rows up to a crossed rounding boundary
    for layer in (0, 1):
        kg, vg = ctx.debug_read_kv(req, layer, 0, P)
        ko = np.stack([orc.get_kv(layer, p)[0] for p in range(P)])
        vo = np.stack([orc.get_kv(layer, p)[1] for p in range(P)])
        for got_bits, want in ((kg, ko), (vg, vo)):
            diff = np.abs(synth.bf16_to_f32(got_bits) - want)
            # Layer 0 sees identical inputs: a value differs only where the fp32-vs-fp64 difference crosses a
            # bf16 rounding boundary (one ulp).  Those crossings are the noise later layers start from:
            # rms sqrt(2 * eps * ulp) ~ 1e-4 of the value scale for eps ~ 3e-6, whatever the kernels do.
            slack, l1 = (2e-5, 1e-4) if layer == 0 else (5e-4, 5e-4)
            assert np.all(diff <= 2.0 ** -7 * np.abs(want) + slack)
            assert diff.sum() / np.abs(want).sum() < l1
    ref_last = oracle.Oracle(shape, w, P + 8)
    ref_last_logits = ref_last.prefill(prefix, want_last_logits=True)
    assert logit_rel_err(last[None], ref_last_logits).max() < LOGIT_TOL
    for seed in range(40):
        toks, q, u, _ = draft_inputs(orc, shape, k, 1.0, seed)
        for greedy in (False, True):
            ref = orc.verify(toks, q, u, greedy=greedy)
            orc.truncate(P)
            item = dict(req=req, tokens=toks, q=None if greedy else q, u=u,
                        mode=binding.MODE_GREEDY if greedy else binding.MODE_STOCHASTIC)
            (got,) = ctx.verify([item], flags=binding.Q_HOST)
            logits = ctx.debug_get_logits(k + 1)
            err = logit_rel_err(logits, ref["logits"]).max()
            assert err < LOGIT_TOL
            t = gt if greedy else tally
            t.max_logit_err = max(t.max_logit_err, err)
            t.check(got, ref, ref["logits"], q, u, greedy=greedy, where=f"seed {seed}")
            ctx.kv_rollback([req], [0])
            # rollback to n_accepted=0 keeps the pending token's row: undo it for the next trial via a fresh request
            ctx.req_close(req)
            req = ctx.req_open()
            ctx.prefill(req, prefix)
    print("\nstochastic: " + tally.report() + "\ngreedy:     " + gt.report())
    assert tally.max_logit_err < 1e-3      # fp32 activations + split-bf16 operands: far below the 2e-2 bar
    ctx.close()


def test_multi_round_verify_rollback_lockstep():
    """Rounds of verify + rollback: the cache grows by n_accepted+1 and is truncated each round; the checker
    leads (its decision is committed on both sides) so a counted near-tie cannot desynchronise later rounds.
    Two query heads per KV head and k up to 8: 4 to 18 query rows per KV head (one or two 16-row column blocks)."""
    from paper_2605_13319_b200 import binding
    shape = synth.TINY.scaled(name="tiny-gqa", n_kv_heads=2)
    P, rounds = 37, 24                       # prefix not a multiple of the page size
    w, ctx, orc = _mk(shape, 1, P, max_seq=P + rounds * 9 + 16)
    prefix = synth.make_prefix(shape, P, 1)
    orc.prefill(prefix)
    req = ctx.req_open()
    ctx.prefill(req, prefix)
    tally = Tally()
    pending = synth.make_pending(shape, 1)
    for r in range(rounds):
        k = 1 + (r * 5) % 8
        sigma = (0.3, 1.0, 3.0)[r % 3]
        toks, q, u, _ = draft_inputs(orc, shape, k, sigma, 1, round_=r, pending=pending)
        ref = orc.verify(toks, q, u)
        (got,) = ctx.verify([dict(req=req, tokens=toks, q=q, u=u)], flags=binding.Q_HOST)
        err = logit_rel_err(ctx.debug_get_logits(k + 1), ref["logits"]).max()
        assert err < LOGIT_TOL
        tally.max_logit_err = max(tally.max_logit_err, err)
        tally.check(got, ref, ref["logits"], q, u, where=f"round {r}")
        orc.rollback(ref["base_len"], ref["n_accepted"])
        ctx.kv_rollback([req], [ref["n_accepted"]])
        assert ctx.req_len(req) == orc.len
        pending = ref["next_token"]
    print("\n" + tally.report())
    assert tally.max_logit_err < 1e-3
    ctx.close()


@pytest.mark.parametrize("n_kv_heads", [2, 4])
def test_batched_ragged_verify_and_batch_invariance(n_kv_heads):
    """Several requests with different prefix lengths and draft counts in ONE call == each alone == checker.
    Two query heads per KV head: up to 34 query rows per KV head, one row group; one (MHA): up to 17, which the
    batch runs as row groups of 16 + 1."""
    from paper_2605_13319_b200 import binding
    shape = synth.TINY.scaled(name=f"tiny-kv{n_kv_heads}", n_kv_heads=n_kv_heads)
    n_req = 6
    lens, ks, sig = synth.ragged_requests(3, n_req, 5, 150, 1, 16)
    if n_kv_heads == 4:
        ks[1] = 16          # a request of 17 rows: the batch's row groups are cut at 16
    w = synth.make_weights(shape, 2)
    ctx = binding.Context(shape, w, n_pages=(200 // 16 + 2) * n_req * 2, max_seq=200, max_requests=2 * n_req,
                          max_rows=max(33, int(ks.sum() + n_req)), max_draft=16, poison=True)
    assert int(ks.sum() + n_req) > 32
    tally = Tally()
    items, refs, solo = [], [], []
    for i in range(n_req):
        orc = oracle.Oracle(shape, w, 200)
        prefix = synth.make_prefix(shape, int(lens[i]), 3, request=i)
        orc.prefill(prefix)
        toks, q, u, _ = draft_inputs(orc, shape, int(ks[i]), float(sig[i]), 3, request=i)
        refs.append((orc.verify(toks, q, u), q, u))
        for bank in (items, solo):
            req = ctx.req_open()
            ctx.prefill(req, prefix)
            bank.append(dict(req=req, tokens=toks, q=q, u=u))
    got = ctx.verify(items, flags=binding.Q_HOST)
    logits = ctx.debug_get_logits(int(ks.sum() + n_req))
    inv = Tally()        # alone vs in the batch: equal decisions but for ties under the batch's own logits (counted)
    row = 0
    for i in range(n_req):
        ref, q, u = refs[i]
        k = int(ks[i])
        assert logit_rel_err(logits[row:row + k + 1], ref["logits"]).max() < LOGIT_TOL
        tally.check(got[i], ref, ref["logits"], q, u, where=f"request {i}")
        # alone, on the kernels the batch ran on (more than 32 rows: the dense ones), then on the small-pass kernels
        ctx.debug_force_dense(True)
        (alone,) = ctx.verify([solo[i]], flags=binding.Q_HOST)
        inv.check(alone, decisions_from_logits(logits[row:row + k + 1], items[i]), logits[row:row + k + 1], q, u,
                  where=f"request {i}: alone vs in the batch")
        assert logit_rel_err(ctx.debug_get_logits(k + 1), ref["logits"]).max() < LOGIT_TOL
        ctx.debug_force_dense(False)
        ctx.kv_rollback([solo[i]["req"]], [0])
        ctx.debug_set_len(solo[i]["req"], int(lens[i]))
        (small,) = ctx.verify([solo[i]], flags=binding.Q_HOST)
        assert logit_rel_err(ctx.debug_get_logits(k + 1), ref["logits"]).max() < LOGIT_TOL
        tally.check(small, ref, ref["logits"], q, u, where=f"request {i} alone")
        row += k + 1
    ctx.kv_rollback([it["req"] for it in items], [g[0] for g in got])
    for i in range(n_req):
        assert ctx.req_len(items[i]["req"]) == int(lens[i]) + 1 + got[i][0]
    print("\nalone vs in the batch: " + inv.report())
    print("\n" + tally.report())
    ctx.close()


def test_draft_lengths_across_token_tile_counts():
    """k = 1, 7, 8, 15, 16, 31 (the maximum): 2, 8, 9, 16, 17 and 32 rows per pass, i.e. one to four 8-token
    tiles in the GEMMs and one or two 16-row column blocks in attention.  Prefix lengths straddle page and 128-key
    tile boundaries."""
    from paper_2605_13319_b200 import binding
    shape = synth.TINY
    w = synth.make_weights(shape, 5)
    tally = Tally()
    for n, (k, P) in enumerate(((1, 1), (7, 63), (8, 127), (15, 128), (16, 129), (31, 130))):
        ctx = binding.Context(shape, w, n_pages=16, max_seq=200, max_draft=31, poison=True)
        orc = oracle.Oracle(shape, w, 200)
        prefix = synth.make_prefix(shape, P, 5, request=n)
        orc.prefill(prefix)
        req = ctx.req_open()
        ctx.prefill(req, prefix)
        for greedy in (False, True):
            toks, q, u, _ = draft_inputs(orc, shape, k, 0.7, 50 + n)
            ref = orc.verify(toks, q, u, greedy=greedy)
            item = dict(req=req, tokens=toks, q=None if greedy else q, u=u,
                        mode=binding.MODE_GREEDY if greedy else binding.MODE_STOCHASTIC)
            (got,) = ctx.verify([item], flags=binding.Q_HOST)
            err = logit_rel_err(ctx.debug_get_logits(k + 1), ref["logits"]).max()
            assert err < LOGIT_TOL, (k, P, err)
            tally.max_logit_err = max(tally.max_logit_err, err)
            tally.check(got, ref, ref["logits"], q, u, greedy=greedy, where=f"k={k} P={P}")
            orc.truncate(P)
            ctx.kv_rollback([req], [0])
            ctx.debug_set_len(req, P)
        ctx.close()
    print("\n" + tally.report())
    assert tally.max_logit_err < 1e-3


def test_page_sizes_other_than_16():
    """Pages of 8, 24, 32, 64, 128 and 256 positions: a 128-key attention tile then covers sixteen pages, straddles
    pages unevenly, covers four, two, one, or half of one; the appended rows land across page boundaries."""
    from paper_2605_13319_b200 import binding
    shape = synth.TINY
    w = synth.make_weights(shape, 6)
    tally = Tally()
    for n, (ps, P, k) in enumerate(((8, 150, 5), (24, 101, 8), (32, 193, 3), (64, 130, 8), (128, 200, 12), (256, 300, 7))):
        ctx = binding.Context(shape, w, n_pages=(P + 48) // ps + 3, max_seq=P + 40, max_draft=16, page_size=ps,
                              poison=True)
        orc = oracle.Oracle(shape, w, P + 40)
        prefix = synth.make_prefix(shape, P, 6, request=n)
        orc.prefill(prefix)
        req = ctx.req_open()
        ctx.prefill(req, prefix)
        pending = None
        for r in range(3):              # the cache grows across a page boundary and is truncated again
            toks, q, u, _ = draft_inputs(orc, shape, k, 0.8, 60 + n, round_=r, pending=pending)
            ref = orc.verify(toks, q, u)
            (got,) = ctx.verify([dict(req=req, tokens=toks, q=q, u=u)], flags=binding.Q_HOST)
            err = logit_rel_err(ctx.debug_get_logits(k + 1), ref["logits"]).max()
            assert err < LOGIT_TOL, (ps, P, r, err)
            tally.max_logit_err = max(tally.max_logit_err, err)
            tally.check(got, ref, ref["logits"], q, u, where=f"page_size={ps} round {r}")
            orc.rollback(ref["base_len"], ref["n_accepted"])
            ctx.kv_rollback([req], [ref["n_accepted"]])
            assert ctx.req_len(req) == orc.len
            pending = ref["next_token"]
        ctx.close()
    print("\n" + tally.report())
    assert tally.max_logit_err < 1e-3


def test_host_side_errors_and_page_accounting():
    from paper_2605_13319_b200 import binding
    shape = synth.TINY
    w = synth.make_weights(shape, 0)
    ctx = binding.Context(shape, w, n_pages=6, max_seq=80, max_requests=2, max_draft=4)
    r0 = ctx.req_open(); r1 = ctx.req_open()
    with pytest.raises(binding.PipesdError) as e:
        ctx.req_open()
    assert e.value.code == binding.E_FULL
    ctx.prefill(r0, synth.make_prefix(shape, 60, 0))                 # 4 pages
    with pytest.raises(binding.PipesdError) as e:
        ctx.prefill(r1, synth.make_prefix(shape, 40, 0))             # needs 3, only 2 left
    assert e.value.code == binding.E_OOM_PAGES and ctx.req_len(r1) == 0
    toks = np.array([1, 2, 3, 4, 5], np.int32)
    u = np.zeros(5, np.float32)
    with pytest.raises(binding.PipesdError) as e:
        ctx.kv_rollback([r0], [0])
    assert e.value.code == binding.E_STATE
    g = dict(req=r0, tokens=toks, u=u, mode=binding.MODE_GREEDY)
    ctx.verify([g])
    with pytest.raises(binding.PipesdError) as e:
        ctx.verify([g])
    assert e.value.code == binding.E_STATE
    with pytest.raises(binding.PipesdError) as e:
        ctx.kv_rollback([r0], [5])
    assert e.value.code == binding.E_RANGE
    with pytest.raises(binding.PipesdError) as e:     # a request listed twice would be committed twice
        ctx.kv_rollback([r0, r0], [1, 1])
    assert e.value.code == binding.E_INVALID and ctx.req_len(r0) == 60
    with pytest.raises(binding.PipesdError) as e:
        ctx.kv_rollback([r0], [1], [shape.vocab])
    assert e.value.code == binding.E_INVALID and ctx.req_len(r0) == 60
    ctx.kv_rollback([r0], [4])
    assert ctx.req_len(r0) == 65
    with pytest.raises(binding.PipesdError) as e:     # no pending token was recorded at that rollback
        ctx.verify([dict(req=r0, tokens=np.array([binding.TOKEN_PENDING, 2], np.int32), u=u[:2], mode=binding.MODE_GREEDY)])
    assert e.value.code == binding.E_STATE
    with pytest.raises(binding.PipesdError) as e:
        ctx.verify([dict(req=r0, tokens=np.array([1, 99999], np.int32), u=u[:2], mode=binding.MODE_GREEDY)])
    assert e.value.code == binding.E_INVALID
    with pytest.raises(binding.PipesdError) as e:
        ctx.prefill(r0, synth.make_prefix(shape, 30, 0))
    assert e.value.code == binding.E_RANGE                            # beyond max_seq
    ctx.req_close(r0)
    ctx.prefill(r1, synth.make_prefix(shape, 40, 0))                  # pages came back
    assert ctx.req_len(r1) == 40
    ctx.close()
