"""The C-ABI library builds for sm_100a, loads without a GPU and exports every symbol the header declares."""
import ctypes
import re
from pathlib import Path

from paper_2605_13319_b200 import binding, build

ROOT = Path(__file__).resolve().parent.parent


def _declared():
    text = (ROOT / "include" / "pipesd.h").read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pipesd_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    build.build_cuda()
    L = ctypes.CDLL(str(binding.LIB_PATH))
    names = _declared()
    assert len(names) >= 18
    for n in names:
        assert hasattr(L, n), f"{n} declared in pipesd.h but not exported"
    assert set(names) == set(binding._SIGNATURES), "binding and header disagree"


def test_pure_host_entry_points():
    L = binding.lib()
    assert L.pipesd_strerror(0) == b"ok"
    assert b"page" in L.pipesd_strerror(binding.E_OOM_PAGES)
    cfg = binding.ModelCfg(32, 4096, 32, 32, 128, 11008, 32000, 1e-5, 10000.0, 16, 256, 1, 16, 32, 4096, 0)
    sz = binding.Sizes()
    assert L.pipesd_query_sizes(ctypes.byref(cfg), ctypes.byref(sz)) == 0
    n_w = 32 * (3 * 4096 * 4096 + 4096 * 4096 + 3 * 11008 * 4096) + 2 * 32000 * 4096
    assert n_w * 2 <= sz.weights_bytes < n_w * 2 + (1 << 21)
    assert sz.kv_bytes == 32 * 256 * 2 * 32 * 16 * 128 * 2
    assert sz.workspace_bytes > 0
    bad = binding.ModelCfg(32, 4096, 32, 32, 96, 11008, 32000, 1e-5, 10000.0, 16, 256, 1, 16, 32, 4096, 0)
    assert L.pipesd_query_sizes(ctypes.byref(bad), ctypes.byref(sz)) == binding.E_INVALID   # head_dim 96
    bad = binding.ModelCfg(32, 4096, 32, 5, 128, 11008, 32000, 1e-5, 10000.0, 16, 256, 1, 16, 32, 4096, 0)
    assert L.pipesd_query_sizes(ctypes.byref(bad), ctypes.byref(sz)) == binding.E_INVALID   # 32 % 5
    assert L.pipesd_gemm_packed_bytes(4096, 11008) == 4096 * 11008 * 2
    assert L.pipesd_gemm_scratch_bytes(9, 4096, 11008) >= 9 * 4096 * 4


def test_attention_key_split_plan():
    """The split of a request's keys over CTAs: a function of the request (and the device) alone."""
    b200 = (148, 296)              # resident CTAs without / with the cut-down third ring slot (head_dim 128, up to 16 rows)
    # 2057 keys, 32 KV heads: 9 splits fill the wave (296 / 32); 240 keys each are two 128-key tiles, the second short
    assert binding.debug_attn_split(2057, 16, b200, 32) == (9, 240, 1)
    # with only the whole-slot footprint resident: 4 splits of 528 keys are five tiles; 4 is the fewest splits with five
    assert binding.debug_attn_split(2057, 16, (148, 0), 32) == (4, 528, 0)
    # fewer splits when they leave the same number of tiles: 521 keys, 8 KV heads: at most 5 splits by keys, all of
    # them one or two tiles -> 112 keys (one tile) needs 5; 3 splits of 176 would be two
    assert binding.debug_attn_split(521, 16, b200, 8) == (5, 112, 1)
    # short requests: one split per 128 keys at most
    assert binding.debug_attn_split(9, 16, b200, 8) == (1, 16, 1)
    assert binding.debug_attn_split(100, 8, b200, 8) == (1, 104, 1)
    assert binding.debug_attn_split(300, 64, b200, 8) == (3, 128, 1)
    # long contexts, few heads: sixteen splits at most; 8209 keys: 16 splits of 528 keys are five tiles each, and so
    # are 13 splits of 640
    assert binding.debug_attn_split(8209, 16, (148, 148), 8) == (13, 640, 0)
    assert binding.debug_attn_split(40000, 16, (148, 148), 8) == (16, 2512, 0)
    # every key is covered, splits are page multiples, whatever the length
    for total in list(range(1, 300)) + [1023, 1024, 1025, 2047, 2048, 4095, 4097, 6143, 6144, 12345]:
        for ps in (8, 16, 24, 64):
            for units in (1, 8, 32):
                n, chunk, short = binding.debug_attn_split(total, ps, b200, units)
                assert 1 <= n <= 16 and chunk % ps == 0 and n * chunk >= total
                assert (n - 1) * chunk < total or n == 1          # no split is wholly empty
                assert short == (chunk <= 240)
                if n > 1:   # one split fewer would mean more tiles per CTA
                    c1 = -(-(-(-total // (n - 1))) // ps) * ps
                    assert -(-c1 // 128) > -(-chunk // 128)
    import pytest
    with pytest.raises(binding.PipesdError):
        binding.debug_attn_split(100, 12, b200, 8)
