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
