"""Shared helpers for the GPU parity tests: seeded cases, the near-tie accounting rule."""
from __future__ import annotations

import numpy as np

import oracle
from paper_2605_13319_b200 import synth

LOGIT_TOL = 2e-2     # max |gpu - oracle| per row, relative to the row's max |logit| (bf16 weights, fp32 accumulate)
TIE_BAND = 1e-3      # a decision whose ratio (or CDF edge) lies this close to its uniform may flip; it is counted
TIGHT_BAND = 1e-5    # reported as well


def logit_rel_err(gpu_logits, ref_logits):
    ref = np.asarray(ref_logits, np.float64)
    return np.abs(np.asarray(gpu_logits, np.float64) - ref).max(1) / np.abs(ref).max(1)


class Tally:
    """Counts decisions, exact matches and flips inside the two bands; flips outside TIE_BAND fail."""

    def __init__(self):
        self.n = self.len_flip = self.tok_flip = self.len_flip_tight = self.tok_flip_tight = 0
        self.max_logit_err = 0.0

    def check(self, gpu, ref, logits_ref, q, u, greedy=False, where=""):
        """gpu = (n_acc, token); ref = dict from Oracle.verify / reject-style fields."""
        self.n += 1
        k = len(u) - 1
        n_g, t_g = gpu
        n_r, t_r = ref["n_accepted"], ref["next_token"]
        if n_g != n_r:
            pos = min(n_g, n_r)
            if greedy:
                row = np.sort(np.asarray(logits_ref[pos], np.float64))
                gap = (row[-1] - row[-2]) / np.abs(row).max()
            else:
                gap = abs(ref["margins"][pos])
            assert gap < TIE_BAND, f"{where}: accepted length {n_g} != {n_r}, margin {gap:.3e} outside the band"
            self.len_flip += 1
            self.len_flip_tight += gap < TIGHT_BAND
            return
        if t_g != t_r:
            if greedy:
                row = np.asarray(logits_ref[n_r], np.float64)
                gap = abs(row[t_g] - row[t_r]) / np.abs(row).max()
            else:
                cdf, _ = oracle.final_cdf(logits_ref[n_r], q[n_r] if n_r < k else None)
                lo = cdf[t_g - 1] if t_g > 0 else 0.0
                hi = cdf[t_g]
                uu = float(u[k])
                gap = 0.0 if lo <= uu < hi else min(abs(uu - lo), abs(uu - hi))
            assert gap < TIE_BAND, f"{where}: emitted token {t_g} != {t_r}, distance {gap:.3e} outside the band"
            self.tok_flip += 1
            self.tok_flip_tight += gap < TIGHT_BAND

    def report(self):
        return (f"{self.n} decisions: accepted-length flips {self.len_flip} (within {TIGHT_BAND:g}: {self.len_flip_tight}), "
                f"token flips {self.tok_flip} (within {TIGHT_BAND:g}: {self.tok_flip_tight}), "
                f"max rel logit err {self.max_logit_err:.2e}")


def decisions_from_logits(logits_rows, item):
    """The accept/correct rule (CPU checker) applied to given logits rows [k+1, V] of one request: what a second run
    of the same request must decide, up to decisions that sit inside the tie band."""
    n, t, margins = oracle.reject(np.asarray(logits_rows, np.float64), item["q"], item["tokens"][1:], item["u"])
    return dict(n_accepted=n, next_token=t, margins=margins)


def draft_inputs(orc, shape, k, sigma, seed, request=0, round_=0, pending=None):
    """One round's inputs from the oracle's own target logits (q = softmax(l + sigma*noise))."""
    if pending is None:
        pending = synth.make_pending(shape, seed, request, round_)
    noise = synth.normal_f32((k, shape.vocab), seed, synth.STREAM_NOISE + 100 * request + 7919 * round_)
    du = synth.uniform_f32(k, seed, synth.STREAM_DRAFT_U + 100 * request + 7919 * round_)
    toks, q, logits = orc.draft_round(pending, k, sigma, noise, du)
    u = synth.make_accept_uniforms(k, seed, request, round_)
    return toks, q, u, logits
