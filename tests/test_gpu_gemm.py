"""Small-M weight-streaming GEMM through the C ABI against the CPU checker's matrix product."""
import numpy as np
import pytest

import oracle
from paper_2605_13319_b200 import synth

pytestmark = pytest.mark.gpu

SHAPES = [  # (M, N, K): ragged row blocks (N % 128 != 0), several K slices, every token-tile count
    (1, 128, 256), (4, 688, 256), (5, 256, 688), (9, 1024, 2048), (9, 4096, 4096), (17, 2064, 1024),
    (25, 512, 512), (32, 384, 4096), (33, 256, 256), (70, 272, 1040), (9, 12288, 4096), (17, 4096, 11008),
]


@pytest.mark.parametrize("M,N,K", SHAPES)
def test_gemm_matches_oracle(M, N, K):
    import torch
    from paper_2605_13319_b200 import binding
    dev = torch.device("cuda", 0)
    W = synth.normal_bf16((N, K), 11, 40 + M, 0.02)
    x = synth.normal_f32((M, K), 11, 80 + M, 1.0)
    want = oracle.linear(W, x.astype(np.float64))
    Wd = torch.from_numpy(W.view(np.int16)).to(dev)
    packed = binding.gemm_pack(Wd)
    xd = torch.from_numpy(x).to(dev)
    y = torch.full((M, N), float("nan"), device=dev)
    scratch = binding.gemm_scratch(M, N, K, dev)
    binding.gemm_run(packed, xd, y, scratch, N, K)
    torch.cuda.synchronize()
    got = y.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    # fp32 accumulation of K products of |w|~0.02, |x|~1, activations carried as bf16 hi+lo (2^-17)
    scale = 0.02 * np.sqrt(K)
    assert np.abs(got - want).max() < 3e-5 * scale * 4
    # second call with different activations reuses the packed weights and the scratch
    x2 = synth.normal_f32((M, K), 12, 81 + M, 3.0)
    binding.gemm_run(packed, torch.from_numpy(x2).to(dev), y, scratch, N, K)
    torch.cuda.synchronize()
    want2 = oracle.linear(W, x2.astype(np.float64))
    assert np.abs(y.cpu().numpy() - want2).max() < 3e-5 * scale * 12


def test_gemm_rejects_bad_shapes():
    from paper_2605_13319_b200 import binding
    L = binding.lib()
    assert L.pipesd_gemm_pack(None, None, 128, 128, None) == binding.E_INVALID
    assert L.pipesd_gemm_run(None, None, None, None, 1, 100, 128, None) == binding.E_INVALID
