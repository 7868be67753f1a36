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
    """The split of a request's keys over clusters and CTAs: a function of the request alone."""
    wide = (48, 45, 41)            # clusters of 8, 9, 10 the device keeps resident (a B200, one query row tile)
    # 2057 keys: 8 splits of 272 keys are three 128-key tiles per CTA, 9 splits of 240 are two, 10 no fewer
    assert binding.debug_attn_split(2057, 16, wide, 32) == (1, 9, 240)
    # the wider cluster must still hold the whole request in one wave
    assert binding.debug_attn_split(2057, 16, (48, 31, 31), 32) == (1, 8, 272)
    assert binding.debug_attn_split(2057, 16, (48, 0, 0), 32) == (1, 8, 272)          # widths unavailable
    assert binding.debug_attn_split(2057, 16, (48, 31, 41), 32) == (1, 10, 208)       # 9 does not fit, 10 does: two tiles
    # 1030 keys: 9 splits of 128 keys are one tile each, 8 splits of 144 are two; 521 keys: one tile either way
    assert binding.debug_attn_split(1030, 16, wide, 8) == (1, 9, 128)
    assert binding.debug_attn_split(521, 16, wide, 8) == (1, 8, 80)
    # short requests: nothing to gain, stay at eight; splits are whole pages
    assert binding.debug_attn_split(9, 16, wide, 8) == (1, 8, 16)
    assert binding.debug_attn_split(100, 8, wide, 8) == (1, 8, 16)
    assert binding.debug_attn_split(100, 64, wide, 8) == (1, 8, 64)
    # one more cluster per 2048 keys, up to four, eight splits each
    assert binding.debug_attn_split(4096, 16, wide, 32) == (2, 8, 256)
    assert binding.debug_attn_split(8209, 16, wide, 16) == (4, 8, 272)
    assert binding.debug_attn_split(40000, 16, wide, 16) == (4, 8, 1264)
    # every key is covered, splits are page multiples, whatever the length
    for total in list(range(1, 300)) + [1023, 1024, 1025, 2047, 2048, 4095, 4097, 6143, 6144, 12345]:
        for ps in (8, 16, 24, 64):
            ncl, w, chunk = binding.debug_attn_split(total, ps, wide, 8)
            assert 8 <= w <= 10 and 1 <= ncl <= 4 and chunk % ps == 0
            assert ncl * w * chunk >= total
            assert (w == 8) or ncl == 1
            if w > 8:   # widened only for fewer tiles per CTA
                c8 = -(-(-(-total // 8)) // ps) * ps
                assert -(-chunk // 128) < -(-c8 // 128)
    import pytest
    with pytest.raises(binding.PipesdError):
        binding.debug_attn_split(100, 12, wide, 8)
