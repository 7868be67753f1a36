"""Commit on the device, the recorded pending token, chained verification of proactively sent drafts (paper App. B)
and the device-side error path, all through the C ABI against the CPU checker."""
import numpy as np
import pytest

import oracle
from paper_2605_13319_b200 import synth
from harness import LOGIT_TOL, Tally, draft_inputs, logit_rel_err

pytestmark = pytest.mark.gpu


def _ctx(shape, w, **kw):
    from paper_2605_13319_b200 import binding
    return binding.Context(shape, w, poison=True, **kw)


def test_commit_on_device_equals_verify_plus_rollback():
    """The same rounds twice: verify + pipesd_kv_rollback(next_token) with PIPESD_TOKEN_PENDING opening the next
    round, and verify with PIPESD_AUTOCOMMIT (no rollback call).  Decisions, committed lengths and the
    device-resident state must agree round by round, and both must agree with the checker."""
    from paper_2605_13319_b200 import binding
    shape, P, rounds = synth.TINY, 41, 10
    w = synth.make_weights(shape, 4)
    a = _ctx(shape, w, n_pages=16, max_seq=P + 120)
    b = _ctx(shape, w, n_pages=16, max_seq=P + 120)
    orc = oracle.Oracle(shape, w, P + 120)
    prefix = synth.make_prefix(shape, P, 4)
    orc.prefill(prefix)
    ra, rb = a.req_open(), b.req_open()
    a.prefill(ra, prefix)
    b.prefill(rb, prefix)
    tally = Tally()
    pending = synth.make_pending(shape, 4)
    for r in range(rounds):
        k = 1 + (3 * r) % 7
        toks, q, u, _ = draft_inputs(orc, shape, k, 0.5, 4, round_=r, pending=pending)
        ref = orc.verify(toks, q, u)
        ta = toks.copy()
        if r > 0:
            ta[0] = binding.TOKEN_PENDING          # the library recorded it at the last rollback
        (ga,) = a.verify([dict(req=ra, tokens=ta, q=q, u=u)], flags=binding.Q_HOST)
        (gb,) = b.verify([dict(req=rb, tokens=toks, q=q, u=u)], flags=binding.Q_HOST | binding.AUTOCOMMIT)
        assert ga == gb, f"round {r}: rollback path {ga}, commit-on-device path {gb}"
        tally.check(ga, ref, ref["logits"], q, u, where=f"round {r}")
        if ga != (ref["n_accepted"], ref["next_token"]):
            break                                  # a counted near-tie: the two sides have parted ways
        a.kv_rollback([ra], [ga[0]], [ga[1]])
        orc.rollback(ref["base_len"], ref["n_accepted"])
        assert a.req_len(ra) == b.req_len(rb) == orc.len
        assert b.debug_req_state(rb) == (orc.len, ref["next_token"], int(ref["n_accepted"] == k))
        pending = ref["next_token"]
    with pytest.raises(binding.PipesdError) as e:   # nothing to roll back after a commit on the device
        b.kv_rollback([rb], [0])
    assert e.value.code == binding.E_STATE
    print("\n" + tally.report())
    a.close(); b.close()


def test_chained_verify_of_buffered_drafts_against_checker():
    """App. B on the device: round 1 with PIPESD_AUTOCOMMIT and, enqueued behind it without a host round trip, the
    round over the buffered early drafts with PIPESD_CHAIN.  Kept exactly when the checker keeps them (all accepted
    and extra token == first buffered token); a kept round matches the checker's second round, a discarded one
    reports PIPESD_DISCARDED and leaves the first round's commit alone."""
    from paper_2605_13319_b200 import binding
    shape, P, k, m = synth.TINY, 50, 3, 4
    w = synth.make_weights(shape, 8)
    prefix = synth.make_prefix(shape, P, 8)
    ctx = _ctx(shape, w, n_pages=32, max_seq=P + 64, max_requests=2)
    tally = Tally()
    kept = dropped = 0
    for trial in range(12):
        orc = oracle.Oracle(shape, w, P + 64)
        orc.prefill(prefix)
        sigma = 0.05 if trial % 3 else 1.0             # nearly q = p: full acceptance is the common case
        toks, q, u, _ = draft_inputs(orc, shape, k, sigma, 80 + trial)
        probe = oracle.Oracle(shape, w, P + 64)
        probe.prefill(prefix)
        first = probe.verify(toks, q, u)
        # the edge's early tokens: a right guess of the extra token in two trials of three, else a wrong one
        if first["n_accepted"] == k and trial % 3 != 2:
            b1 = first["next_token"]
        else:
            b1 = (first["next_token"] + 1 + trial) % shape.vocab
        probe.rollback(first["base_len"], first["n_accepted"])
        btoks, bq, bu, _ = draft_inputs(probe, shape, m - 1, 0.5, 90 + trial, pending=b1)
        r1, r2 = orc.verify_chain(toks, q, u, btoks, bq, bu)
        req = ctx.req_open()
        ctx.prefill(req, prefix)
        res1 = ctx.verify([dict(req=req, tokens=toks, q=q, u=u)], flags=binding.Q_HOST | binding.AUTOCOMMIT, sync=False)
        res2 = ctx.verify([dict(req=req, tokens=btoks, q=bq, u=bu)], flags=binding.Q_HOST | binding.CHAIN, sync=False)
        ctx.ctx_sync()
        g1 = (res1[0].n_accepted, res1[0].next_token)
        tally.check(g1, r1, r1["logits"], q, u, where=f"trial {trial} round 1")
        if g1 != (r1["n_accepted"], r1["next_token"]):
            ctx.req_close(req)
            continue                                   # counted near-tie in round 1: the condition may differ too
        if r2 is None:
            dropped += 1
            assert res2[0].status == binding.DISCARDED
            assert ctx.req_len(req) == P + 1 + r1["n_accepted"] == orc.len
            assert ctx.debug_req_state(req)[:2] == (orc.len, r1["next_token"])
        else:
            kept += 1
            assert res2[0].status == binding.OK
            err = logit_rel_err(ctx.debug_get_logits(m), r2["logits"]).max()
            assert err < LOGIT_TOL
            tally.max_logit_err = max(tally.max_logit_err, err)
            g2 = (res2[0].n_accepted, res2[0].next_token)
            tally.check(g2, r2, r2["logits"], bq, bu, where=f"trial {trial} round 2")
            if g2 == (r2["n_accepted"], r2["next_token"]):
                assert ctx.req_len(req) == orc.len
                assert ctx.debug_req_state(req) == (orc.len, r2["next_token"], int(r2["n_accepted"] == m - 1))
        ctx.req_close(req)
    print(f"\nbuffered drafts kept {kept}, discarded {dropped}; " + tally.report())
    assert kept >= 3 and dropped >= 3
    # a chained call needs a commit-on-device call in flight for the request
    req = ctx.req_open()
    ctx.prefill(req, prefix)
    with pytest.raises(binding.PipesdError) as e:
        ctx.verify([dict(req=req, tokens=btoks, q=bq, u=bu)], flags=binding.Q_HOST | binding.CHAIN)
    assert e.value.code == binding.E_STATE
    ctx.close()


def test_device_side_wait_that_runs_out_is_reported_and_survived():
    """A bounded device-side wait that gives up (a flag nothing sets, one millisecond) sets the device error word:
    the next synchronisation reports PIPESD_E_CUDA, results in flight are void, and the context keeps working."""
    from paper_2605_13319_b200 import binding
    shape, P, k = synth.TINY, 64, 4
    w = synth.make_weights(shape, 0)
    ctx = _ctx(shape, w, n_pages=16, max_seq=P + 64)
    orc = oracle.Oracle(shape, w, P + 64)
    prefix = synth.make_prefix(shape, P, 0)
    orc.prefill(prefix)
    req = ctx.req_open()
    ctx.prefill(req, prefix)
    toks, q, u, _ = draft_inputs(orc, shape, k, 1.0, 0)
    item = dict(req=req, tokens=toks, q=q, u=u)
    (before,) = ctx.verify([item], flags=binding.Q_HOST)
    ctx.kv_rollback([req], [0]); ctx.debug_set_len(req, P)
    res = ctx.verify([item], flags=binding.Q_HOST, sync=False)       # in flight when the wait gives up
    ctx.debug_wait_timeout(1000)
    with pytest.raises(binding.PipesdError) as e:
        ctx.ctx_sync()
    assert e.value.code == binding.E_CUDA and "timed out" in str(e.value)
    assert res[0].status == binding.E_CUDA
    ctx.ctx_sync()                                                   # the word was cleared: no error any more
    ctx.kv_rollback([req], [0]); ctx.debug_set_len(req, P)
    (after,) = ctx.verify([item], flags=binding.Q_HOST)
    assert after == before
    ref = orc.verify(toks, q, u)
    Tally().check(after, ref, ref["logits"], q, u, where="after the timeout")
    ctx.close()
