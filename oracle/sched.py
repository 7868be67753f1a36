"""CPU checker for the edge-side scheduling model of PipeSD: the pipeline timing model, the optimal token batching it
defines, and the dual-threshold verification trigger.

TEST INFRASTRUCTURE ONLY: the product path never imports this module (the library's own implementation is
``pipesd_sched_*`` behind the C ABI); only the tests do.

Where the method reaches a result that has a plain definition, this file is that definition written out:

* ``round_time`` evaluates the timing model term by term (Sec. 3.2, Eq. 1-6): batch k holds the draft tokens
  b_k .. b_{k+1}-1 (the last batch runs to N), takes gamma per token to generate and alpha + beta per token to
  send; a batch's generation starts when the previous batch's generation ends, its transmission starts when both
  its own generation and the previous transmission have ended; T is the end of the last transmission.
* ``optimal_batching`` is the optimum of Eq. 6 by exhaustive search over all 2^(N-1) boundary sequences -- the
  definition of "optimal", not the paper's dynamic programme (Algorithm 1), which the library implements and which
  Theorem 4.1 claims to reach the same value.
* ``trigger_sequence`` follows Sec. 3.3 step by step: C1* = C1 * P(D_n); verification is triggered when C1* <= R1
  or when P(D_n) <= R2; C1 is the product over the tokens generated since the last verification, so it restarts at 1
  after either kind of trigger.
"""
from __future__ import annotations

import itertools


def round_time(N, alpha, beta, gamma, boundaries):
    """T of Eq. 6 for the boundary sequence B = (b_1 = 1 < b_2 < ... < b_K <= N) (Eq. 1)."""
    B = list(boundaries)
    K = len(B)
    assert K >= 1 and B[0] == 1 and all(B[i] < B[i + 1] for i in range(K - 1)) and B[-1] <= N
    size = [(B[k + 1] - B[k]) if k < K - 1 else (N + 1 - B[k]) for k in range(K)]
    t_c = [alpha + beta * n for n in size]                      # Eq. 2
    t_ag = [gamma * n for n in size]                            # Eq. 3
    tau_ag = [0.0] * K                                          # Eq. 4
    for k in range(1, K):
        tau_ag[k] = tau_ag[k - 1] + t_ag[k - 1]
    tau_c = [0.0] * K                                           # Eq. 5
    tau_c[0] = tau_ag[0] + t_ag[0]
    for k in range(1, K):
        tau_c[k] = max(tau_c[k - 1] + t_c[k - 1], tau_ag[k] + t_ag[k])
    return tau_c[K - 1] + t_c[K - 1] - tau_ag[0]                # Eq. 6


def all_batchings(N):
    """Every boundary sequence of Eq. 1, in lexicographic order of the chosen boundaries."""
    for r in range(N):
        for rest in itertools.combinations(range(2, N + 1), r):
            yield (1,) + rest


def optimal_batching(N, alpha, beta, gamma):
    """(minimal T, list of all boundary sequences that attain it) by exhaustive search."""
    best, argbest = None, []
    for B in all_batchings(N):
        T = round_time(N, alpha, beta, gamma, B)
        if best is None or T < best:
            best, argbest = T, [B]
        elif T == best:
            argbest.append(B)
    return best, argbest


def trigger_sequence(confidences, R1, R2):
    """For each draft token's confidence P(D_n), in order: (triggered?, C1 after the step)."""
    C1 = 1.0
    out = []
    for p in confidences:
        c_star = C1 * p
        fire = c_star <= R1 or p <= R2
        C1 = 1.0 if fire else c_star
        out.append((fire, C1))
    return out
