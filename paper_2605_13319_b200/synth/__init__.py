"""Seeded synthetic inputs: model shapes, bf16 weights, token ids, uniforms, noise.

This module only manufactures inputs.  It contains no transformer arithmetic and
no acceptance rule; the CUDA library's callers and the CPU checker both draw
their arrays from here so that they see bit-identical data.

The number generator lives in ``synth.c`` (counter based: element ``i`` of
stream ``s`` under seed ``z`` is a pure function of ``(z, s, i)``).  It is built
with gcc on first use into ``_synth.so`` next to this file.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, replace
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SO = _HERE / "_synth.so"
_SRC = _HERE / "synth.c"
_lib = None


def build(force: bool = False) -> Path:
    """Compile synth.c into _synth.so (gcc, OpenMP). No fast-math: results must not
    depend on reassociation."""
    if force or not _SO.exists() or _SO.stat().st_mtime < _SRC.stat().st_mtime:
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
               str(_SRC), "-o", str(_SO), "-lm"]
        subprocess.run(cmd, check=True)
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_SO))
        i64, u64, f64, i32 = ctypes.c_int64, ctypes.c_uint64, ctypes.c_double, ctypes.c_int32
        vp = ctypes.c_void_p
        lib.synth_normal_bf16.argtypes = [vp, i64, u64, u64, f64]
        lib.synth_normal_f32.argtypes = [vp, i64, u64, u64, f64]
        lib.synth_uniform_f32.argtypes = [vp, i64, u64, u64]
        lib.synth_tokens_i32.argtypes = [vp, i64, u64, u64, i32]
        lib.synth_ints_i32.argtypes = [vp, i64, u64, u64, i32, i32]
        lib.synth_bf16_to_f32.argtypes = [vp, vp, i64]
        lib.synth_f32_to_bf16.argtypes = [vp, vp, i64]
        for f in (lib.synth_normal_bf16, lib.synth_normal_f32, lib.synth_uniform_f32,
                  lib.synth_tokens_i32, lib.synth_ints_i32, lib.synth_bf16_to_f32,
                  lib.synth_f32_to_bf16):
            f.restype = None
        _lib = lib
    return _lib


# --------------------------------------------------------------------------- streams
# Stream ids keep every array independent of every other one under the same seed.
STREAM_TOK_EMB = 1
STREAM_LM_HEAD = 2
STREAM_PREFIX = 3
STREAM_PENDING = 4
STREAM_ACCEPT_U = 5       # the k+1 uniforms handed to verify
STREAM_DRAFT_U = 6        # uniforms used to sample drafts from q
STREAM_NOISE = 7          # Gaussian noise added to the target logits to make q
STREAM_REQ_LEN = 8
STREAM_REQ_K = 9
STREAM_REQ_SIGMA = 10
STREAM_KV = 11            # synthetic K/V prefix rows
STREAM_LAYER0 = 1000      # layer l, tensor t -> STREAM_LAYER0 + 16*l + t
_LAYER_TENSORS = ("wq", "wk", "wv", "wo", "wg", "wu", "wd")


def normal_bf16(shape, seed: int, stream: int, std: float) -> np.ndarray:
    """bf16 bit patterns (uint16) of std*N(0,1), rounded to nearest even."""
    out = np.empty(shape, dtype=np.uint16)
    _load().synth_normal_bf16(out.ctypes.data, out.size, seed, stream, std)
    return out


def normal_f32(shape, seed: int, stream: int, std: float = 1.0) -> np.ndarray:
    out = np.empty(shape, dtype=np.float32)
    _load().synth_normal_f32(out.ctypes.data, out.size, seed, stream, std)
    return out


def uniform_f32(shape, seed: int, stream: int) -> np.ndarray:
    """Uniforms on [0,1) of the form m * 2**-24 (exact in fp32)."""
    out = np.empty(shape, dtype=np.float32)
    _load().synth_uniform_f32(out.ctypes.data, out.size, seed, stream)
    return out


def tokens_i32(n: int, seed: int, stream: int, vocab: int) -> np.ndarray:
    out = np.empty(n, dtype=np.int32)
    _load().synth_tokens_i32(out.ctypes.data, out.size, seed, stream, vocab)
    return out


def ints_i32(n: int, seed: int, stream: int, lo: int, hi: int) -> np.ndarray:
    """Uniform integers on [lo, hi] inclusive."""
    out = np.empty(n, dtype=np.int32)
    _load().synth_ints_i32(out.ctypes.data, out.size, seed, stream, lo, hi)
    return out


def bf16_to_f32(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.uint16)
    out = np.empty(a.shape, dtype=np.float32)
    _load().synth_bf16_to_f32(a.ctypes.data, out.ctypes.data, a.size)
    return out


def f32_to_bf16(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    out = np.empty(a.shape, dtype=np.uint16)
    _load().synth_f32_to_bf16(a.ctypes.data, out.ctypes.data, a.size)
    return out


# --------------------------------------------------------------------------- shapes
@dataclass(frozen=True)
class ModelShape:
    """Llama-style decoder shape (no arithmetic here, only sizes)."""
    name: str
    n_layers: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float = 1e-5
    rope_base: float = 10000.0

    @property
    def q_dim(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def kv_dim(self) -> int:
        return self.n_kv_heads * self.head_dim

    def weight_elems(self) -> int:
        per_layer = (self.q_dim + 2 * self.kv_dim) * self.d_model + self.d_model * self.q_dim \
            + 3 * self.d_ffn * self.d_model
        return self.n_layers * per_layer + 2 * self.vocab * self.d_model

    def scaled(self, **kw) -> "ModelShape":
        return replace(self, **kw)


# The five workload shapes (synthetic stand-ins for the paper's target models:
# Llama-2-7B / DeepSeek-Coder-6.7B class targets verified against drafts of a 1B-class model).
TINY = ModelShape("tiny", 2, 256, 4, 4, 64, 688, 1024)
B1 = ModelShape("1b", 16, 2048, 32, 8, 64, 8192, 32000)
B7 = ModelShape("7b", 32, 4096, 32, 32, 128, 11008, 32000)
B8 = ModelShape("8b", 32, 4096, 32, 8, 128, 14336, 128256, rope_base=500000.0)
SHAPES = {s.name: s for s in (TINY, B1, B7, B8)}


# --------------------------------------------------------------------------- weights
def make_weights(shape: ModelShape, seed: int = 0, std: float = 0.02) -> dict:
    """Random-init weights: every linear / embedding matrix ~ N(0, std^2) rounded to bf16
    (uint16 bit patterns, row-major [out, in]); RMSNorm gains are exactly 1 (fp32)."""
    d, F, V = shape.d_model, shape.d_ffn, shape.vocab
    dims = {"wq": (shape.q_dim, d), "wk": (shape.kv_dim, d), "wv": (shape.kv_dim, d),
            "wo": (d, shape.q_dim), "wg": (F, d), "wu": (F, d), "wd": (d, F)}
    w = {"tok_emb": normal_bf16((V, d), seed, STREAM_TOK_EMB, std),
         "lm_head": normal_bf16((V, d), seed, STREAM_LM_HEAD, std),
         "final_norm": np.ones(d, dtype=np.float32),
         "layers": []}
    for l in range(shape.n_layers):
        lw = {}
        for t, name in enumerate(_LAYER_TENSORS):
            lw[name] = normal_bf16(dims[name], seed, STREAM_LAYER0 + 16 * l + t, std)
        lw["attn_norm"] = np.ones(d, dtype=np.float32)
        lw["ffn_norm"] = np.ones(d, dtype=np.float32)
        w["layers"].append(lw)
    return w


def make_prefix(shape: ModelShape, n: int, seed: int, request: int = 0) -> np.ndarray:
    """Uniform random prefix token ids."""
    return tokens_i32(n, seed, STREAM_PREFIX + 100 * request, shape.vocab)


def make_pending(shape: ModelShape, seed: int, request: int = 0, round_: int = 0) -> int:
    return int(tokens_i32(round_ + 1, seed, STREAM_PENDING + 100 * request, shape.vocab)[round_])


def make_accept_uniforms(k: int, seed: int, request: int = 0, round_: int = 0) -> np.ndarray:
    """k+1 uniforms: k acceptance tests followed by the final (residual / bonus) draw."""
    u = uniform_f32((round_ + 1) * 64, seed, STREAM_ACCEPT_U + 100 * request)
    return np.ascontiguousarray(u[round_ * 64: round_ * 64 + k + 1])


_KV_BASE = {}


def make_synthetic_kv(shape: ModelShape, n_pos: int, seed: int, layer: int, request: int = 0,
                      std_k: float = 1.0, std_v: float = 0.1):
    """Seeded stand-in K and V rows (bf16 bit patterns, [n_pos, n_kv_heads*head_dim] each) for full-size
    cases where a CPU prefill is out of reach.  One block of normals is drawn per (seed, request); layer l
    uses it rotated by 16*l columns and l rows (pure data movement), so that layers differ without
    drawing 2*n_layers*n_pos*width normals."""
    key = (shape.kv_dim, n_pos, seed, request, std_k, std_v)
    if key not in _KV_BASE:
        if len(_KV_BASE) > 2:
            _KV_BASE.clear()
        base = STREAM_KV + 100 * request
        _KV_BASE[key] = (normal_bf16((n_pos, shape.kv_dim), seed, base, std_k),
                         normal_bf16((n_pos, shape.kv_dim), seed, base + 1, std_v))
    k, v = _KV_BASE[key]
    sh = (16 * layer) % shape.kv_dim
    return (np.ascontiguousarray(np.roll(np.roll(k, sh, axis=1), layer, axis=0)),
            np.ascontiguousarray(np.roll(np.roll(v, sh, axis=1), layer, axis=0)))


def ragged_requests(seed: int, n_req: int = 32, len_lo: int = 256, len_hi: int = 4096,
                    k_lo: int = 1, k_hi: int = 16, sig_lo: float = 0.3, sig_hi: float = 2.0):
    """Prefix lengths ~U[len_lo,len_hi], draft lengths ~U{k_lo..k_hi}, noise sigma ~U[sig_lo,sig_hi]."""
    lens = ints_i32(n_req, seed, STREAM_REQ_LEN, len_lo, len_hi)
    ks = ints_i32(n_req, seed, STREAM_REQ_K, k_lo, k_hi)
    sig = sig_lo + (sig_hi - sig_lo) * uniform_f32(n_req, seed, STREAM_REQ_SIGMA).astype(np.float64)
    return lens, ks, sig
