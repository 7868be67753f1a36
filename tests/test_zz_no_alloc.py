"""pipesd_gemm_run_static: the weight-streaming GEMM for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is not an option (a plugin that only gets its input and
output buffers, a latency-critical loop that must not touch the allocator, a process with a memory budget
fixed at start-up), so they cannot supply the scratch that pipesd_gemm_run needs for the activations'
split-bf16 fragments.  The static variant keeps that scratch in a fixed array inside the library.  This file
checks, through the C ABI, that it returns what pipesd_gemm_run returns -- twice in a row with different
inputs, because the array is shared by all calls and still holds the previous call's contents -- and that
it refuses problems that do not fit the array.  It is named to be collected last, and it must pass alone in a fresh process too."""
import numpy as np
import pytest

import oracle
from paper_2605_13319_b200 import synth

pytestmark = pytest.mark.gpu

# (M, N, K): several K slices, a ragged row block, a single-slice case, and the largest M that fits at K = 11008
CASES = [(9, 4096, 4096), (5, 688, 2048), (16, 4096, 11008), (3, 128, 256), (160, 256, 11008)]


@pytest.mark.parametrize("M,N,K", CASES)
def test_static_scratch_gemm_matches_regular_entry_point_twice(M, N, K):
    import torch
    from paper_2605_13319_b200 import binding
    dev = torch.device("cuda", 0)
    W_bits = synth.normal_bf16((N, K), 21, 5, 0.02)
    W = torch.from_numpy(W_bits.view(np.int16)).to(dev)
    packed = binding.gemm_pack(W)
    scratch = binding.gemm_scratch(M, N, K, dev)
    need = binding.lib().pipesd_gemm_scratch_bytes(M, N, K)
    assert need <= binding.STATIC_SCRATCH_BYTES
    scale = 0.02 * np.sqrt(K)
    for call, (seed, amp) in enumerate([(31, 1.0), (32, 5.0)]):          # second call: other values, larger
        x_host = synth.normal_f32((M, K), seed, 9, amp)
        x = torch.from_numpy(x_host).to(dev)
        want = torch.full((M, N), float("nan"), device=dev)
        got = torch.full((M, N), float("nan"), device=dev)
        binding.gemm_run(packed, x, want, scratch, N, K)
        before = torch.cuda.memory_allocated(dev), torch.cuda.memory_reserved(dev)
        binding.gemm_run_static(packed, x, got, N, K)
        torch.cuda.synchronize()
        # nothing went through torch's allocator (the library itself calls no allocation routine: its only device
        # memory here is the built-in array)
        assert (torch.cuda.memory_allocated(dev), torch.cuda.memory_reserved(dev)) == before
        g, w = got.cpu().numpy(), want.cpu().numpy()
        assert np.isfinite(g).all(), f"call {call}: non-finite output"
        # both entry points run the same kernels in the same order on the same split-bf16 fragments: same bits
        assert np.array_equal(g, w), f"call {call}: the two entry points differ"
        # and both are right: the CPU checker's matrix product, at the tolerance of the GEMM parity tests
        # (fp32 accumulation over K, split-bf16 activations)
        ref = oracle.linear(W_bits, x_host.astype(np.float64))
        assert np.abs(g - ref).max() < 3e-5 * scale * 4 * amp, f"call {call}"


def test_static_scratch_gemm_rejects_what_does_not_fit():
    import torch
    from paper_2605_13319_b200 import binding
    dev = torch.device("cuda", 0)
    # the boundary at K = 11008: token rows are padded to whole blocks of 32, so 160 rows fit 8 MiB and 161 do not
    assert binding.lib().pipesd_gemm_scratch_bytes(160, 256, 11008) <= binding.STATIC_SCRATCH_BYTES
    assert binding.lib().pipesd_gemm_scratch_bytes(161, 256, 11008) > binding.STATIC_SCRATCH_BYTES
    M, N, K = 161, 256, 11008
    # no weights are touched: the size check comes before any launch, so small stand-in buffers are enough
    stub = torch.zeros(1024, dtype=torch.uint8, device=dev)
    x = torch.zeros((M, K), device=dev)
    y = torch.zeros((M, N), device=dev)
    with pytest.raises(binding.PipesdError) as e:
        binding.gemm_run_static(stub, x, y, N, K)
    assert e.value.code == binding.E_TOO_LARGE
    assert b"built-in" in binding.lib().pipesd_strerror(binding.E_TOO_LARGE)
    assert binding.lib().pipesd_gemm_run_static(None, None, None, 1, 128, 128, None) == binding.E_INVALID
