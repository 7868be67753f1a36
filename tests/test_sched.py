"""The edge-side scheduling model: pins of the CPU checker (oracle/sched.py) against closed forms, and the library's
host code (pipesd_sched_*) against the checker -- the dynamic programme of Algorithm 1 against exhaustive search over
all 2^(N-1) batchings (Theorem 4.1), bit for bit on T and, where the optimum is unique, on the boundaries.

All parameters are small dyadic rationals, so every sum and product below is exact in fp64 and the comparisons are
exact comparisons."""
import itertools

import pytest

from oracle import sched as ref

# (alpha, beta) of the paper's Table A.2 (ms) and others; gamma is not printed there: a spread of values
PARAMS = [(a, b, g) for a in (20.0, 100.0, 200.0) for b in (48.0, 72.0) for g in (10.0, 40.0, 64.0, 150.0)] + \
         [(0.0, 1.0, 1.0), (5.0, 0.25, 8.0), (3.5, 2.0, 0.0), (0.0, 0.0, 7.0), (12.0, 3.0, 3.0)]


# ---- pins of the checker itself
def test_checker_round_time_closed_forms():
    a, b, g = 20.0, 48.0, 30.0
    # one batch: generate everything, then one transmission
    for N in (1, 2, 7):
        assert ref.round_time(N, a, b, g, (1,)) == g * N + a + b * N
    # every token its own batch, transmission slower than generation (a + b > g): the first token's generation, then
    # N transmissions back to back; generation slower (g > a + b): N generations, then the last transmission
    assert ref.round_time(5, a, b, g, (1, 2, 3, 4, 5)) == g + 5 * (a + b)
    assert ref.round_time(5, 1.0, 2.0, 10.0, (1, 2, 3, 4, 5)) == 5 * 10.0 + 3.0
    # a worked two-batch case: tokens {1,2} then {3}: generation ends at 60 and 90; the first transmission runs
    # 60..176, so the second starts at max(176, 90) and takes 68
    assert ref.round_time(3, a, b, g, (1, 3)) == 176.0 + 68.0
    # and one where the second batch waits for its own generation: alpha = beta = 1, gamma = 10
    assert ref.round_time(3, 1.0, 1.0, 10.0, (1, 2)) == 30.0 + 3.0
    with pytest.raises(AssertionError):
        ref.round_time(3, a, b, g, (1, 1))


def test_checker_enumerates_every_batching_once():
    for N in range(1, 9):
        seen = list(ref.all_batchings(N))
        assert len(seen) == len(set(seen)) == 2 ** (N - 1)
        assert all(B[0] == 1 and list(B) == sorted(set(B)) and B[-1] <= N for B in seen)


def test_checker_optimum_special_cases():
    # no start-up cost and generation much slower than the link: everything but the last token travels while later
    # tokens are generated, so the optimum is reached by exactly the batchings whose last batch is the last token
    T, arg = ref.optimal_batching(6, 0.0, 1.0, 8.0)
    assert T == 6 * 8.0 + 1.0 and set(arg) == {B for B in ref.all_batchings(6) if B[-1] == 6}
    # instantaneous generation: nothing to overlap, one batch saves every extra start-up
    T, arg = ref.optimal_batching(6, 3.5, 2.0, 0.0)
    assert T == 3.5 + 12.0 and arg == [(1,)]
    # never worse than the two fixed strategies, never better than the bounds of the model
    for a, b, g in PARAMS:
        for N in (1, 4, 9):
            T, arg = ref.optimal_batching(N, a, b, g)
            assert T <= ref.round_time(N, a, b, g, (1,))
            assert T <= ref.round_time(N, a, b, g, tuple(range(1, N + 1)))
            assert T >= g * N + a + b            # the last token must be generated, then sent
            assert T >= g + a + b * N            # every token crosses the link after the first exists
            assert all(ref.round_time(N, a, b, g, B) == T for B in arg)


def test_checker_trigger_steps():
    # cumulative threshold: 0.9 * 0.9 = 0.81 > 0.8, times 0.95 falls below: fires on the third token, then restarts
    steps = ref.trigger_sequence([0.9, 0.9, 0.95, 0.9], R1=0.8, R2=0.0)
    assert [f for f, _ in steps] == [False, False, True, False]
    assert [c for _, c in steps] == [0.9, 0.9 * 0.9, 1.0, 0.9]
    # single-token threshold alone, and a token that trips both
    assert [f for f, _ in ref.trigger_sequence([0.99, 0.4, 0.99], R1=0.0, R2=0.5)] == [False, True, False]
    assert ref.trigger_sequence([0.3], R1=0.5, R2=0.5) == [(True, 1.0)]
    # thresholds at zero never fire on positive confidences; the product keeps shrinking
    steps = ref.trigger_sequence([0.5] * 6, R1=0.0, R2=0.0)
    assert not any(f for f, _ in steps) and steps[-1][1] == 0.5 ** 6


# ---- the library's host code against the checker
def test_library_round_time_equals_checker_on_every_batching():
    from paper_2605_13319_b200 import binding
    for a, b, g in PARAMS[:8] + PARAMS[-5:]:
        for N in (1, 2, 5, 8):
            for B in ref.all_batchings(N):
                assert binding.sched_round_time(N, a, b, g, B) == ref.round_time(N, a, b, g, B)
    for bad in ((2,), (1, 1), (1, 3, 2), (1, 9)):
        with pytest.raises(binding.PipesdError):
            binding.sched_round_time(8, 1.0, 1.0, 1.0, bad)


def test_library_dynamic_programme_equals_exhaustive_search():
    """Theorem 4.1 checked by brute force: for every N up to 12 and every parameter set the dynamic programme's T is
    the minimum over all 2^(N-1) batchings, its boundaries attain it, and they are THE optimum where it is unique."""
    from paper_2605_13319_b200 import binding
    unique = 0
    for a, b, g in PARAMS:
        for N in range(1, 13):
            T_ref, arg = ref.optimal_batching(N, a, b, g)
            B, T = binding.sched_optimal_batching(N, a, b, g)
            assert T == T_ref, (N, a, b, g)
            assert B in arg, (N, a, b, g, B, arg)
            assert ref.round_time(N, a, b, g, B) == T_ref
            if len(arg) == 1:
                unique += 1
                assert B == arg[0]
    assert unique > 50
    # beyond the reach of exhaustive search: the result is a valid batching whose time the model confirms
    B, T = binding.sched_optimal_batching(200, 20.0, 48.0, 30.0)
    assert B[0] == 1 and list(B) == sorted(set(B)) and B[-1] <= 200
    assert binding.sched_round_time(200, 20.0, 48.0, 30.0, B) == T == ref.round_time(200, 20.0, 48.0, 30.0, B)


def test_library_trigger_equals_checker():
    from paper_2605_13319_b200 import binding, synth
    for seed, (R1, R2) in enumerate(((0.5, 0.25), (0.125, 0.5), (0.75, 0.0), (0.0, 0.0), (1.0, 1.0))):
        conf = [float(x) for x in synth.uniform_f32(200, seed, 77)]
        want = ref.trigger_sequence(conf, R1, R2)
        c1, got = 1.0, []
        for p in conf:
            fire, c1 = binding.sched_trigger_step(c1, R1, R2, p)
            got.append((fire, c1))
        assert got == want
    with pytest.raises(binding.PipesdError):
        binding.sched_trigger_step(1.0, 0.5, 0.5, 1.5)
