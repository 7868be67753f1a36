"""ctypes binding of libpipesd.so (include/pipesd.h): argument marshalling only.

PyTorch is used for device memory and streams; every step of the verify pass runs in the CUDA
kernels behind the C ABI.  There is no CPU or library fallback: if the shared library is missing
or fails to load, importing a symbol from here raises.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
LIB_PATH = _HERE / "libpipesd.so"
_lib = None

OK, E_INVALID, E_FULL, E_OOM_PAGES, E_STATE, E_RANGE, E_CUDA, E_NOMEM = 0, -1, -2, -3, -4, -5, -6, -7
E_TOO_LARGE = -8
STATIC_SCRATCH_BYTES = 8 << 20
MODE_STOCHASTIC, MODE_GREEDY = 0, 1
Q_HOST, AUTOCOMMIT, CHAIN = 1, 2, 4
TOKEN_PENDING = -1
DISCARDED = 1

i32, u32, u64, f32, vp = ctypes.c_int32, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_float, ctypes.c_void_p


class ModelCfg(ctypes.Structure):
    _fields_ = [(n, i32) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab")] \
        + [("rms_eps", f32), ("rope_base", f32)] \
        + [(n, i32) for n in ("page_size", "n_pages", "max_requests", "max_draft", "max_rows", "max_seq", "device", "reserved")]


class LayerWeights(ctypes.Structure):
    _fields_ = [(n, vp) for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "attn_norm", "ffn_norm")]


class Weights(ctypes.Structure):
    _fields_ = [("tok_emb", vp), ("lm_head", vp), ("final_norm", vp), ("layers", ctypes.POINTER(LayerWeights))]


class Sizes(ctypes.Structure):
    _fields_ = [("weights_bytes", u64), ("kv_bytes", u64), ("workspace_bytes", u64)]


class Mem(ctypes.Structure):
    _fields_ = [("weights", vp), ("weights_bytes", u64), ("kv", vp), ("kv_bytes", u64),
                ("workspace", vp), ("workspace_bytes", u64)]


class VerifyItem(ctypes.Structure):
    _fields_ = [("req", i32), ("k", i32), ("mode", i32), ("reserved", i32),
                ("tokens", vp), ("q", vp), ("u", vp)]


class VerifyResult(ctypes.Structure):
    _fields_ = [("n_accepted", i32), ("next_token", i32), ("status", i32), ("reserved", i32)]


class ProfileInfo(ctypes.Structure):
    _fields_ = [("kernel_launches", ctypes.c_int64), ("gemm_launches", ctypes.c_int64),
                ("gemm_ms", ctypes.c_double), ("gemm_bytes", ctypes.c_double)]


# name -> (restype, argtypes); mirrors include/pipesd.h one to one
_SIGNATURES = {
    "pipesd_strerror": (ctypes.c_char_p, [i32]),
    "pipesd_last_error": (ctypes.c_char_p, [vp]),
    "pipesd_query_sizes": (i32, [ctypes.POINTER(ModelCfg), ctypes.POINTER(Sizes)]),
    "pipesd_ctx_create": (i32, [ctypes.POINTER(ModelCfg), ctypes.POINTER(Weights), ctypes.POINTER(Mem), vp,
                                ctypes.POINTER(vp)]),
    "pipesd_ctx_destroy": (i32, [vp]),
    "pipesd_ctx_sync": (i32, [vp]),
    "pipesd_req_open": (i32, [vp, ctypes.POINTER(i32)]),
    "pipesd_req_close": (i32, [vp, i32]),
    "pipesd_req_len": (i32, [vp, i32, ctypes.POINTER(i32)]),
    "pipesd_prefill": (i32, [vp, i32, vp, i32, vp]),
    "pipesd_verify": (i32, [vp, i32, ctypes.POINTER(VerifyItem), ctypes.POINTER(VerifyResult), u32]),
    "pipesd_kv_rollback": (i32, [vp, i32, vp, vp, vp]),
    "pipesd_debug_get_logits": (i32, [vp, vp, i32]),
    "pipesd_debug_read_kv": (i32, [vp, i32, i32, i32, i32, vp, vp]),
    "pipesd_debug_write_kv": (i32, [vp, i32, i32, i32, i32, vp, vp]),
    "pipesd_reject_from_logits": (i32, [vp, i32, i32, vp, vp, vp, vp, ctypes.POINTER(VerifyResult)]),
    "pipesd_debug_set_len": (i32, [vp, i32, i32]),
    "pipesd_profile_enable": (i32, [vp, i32]),
    "pipesd_profile_read": (i32, [vp, ctypes.POINTER(ProfileInfo)]),
    "pipesd_gemm_packed_bytes": (u64, [i32, i32]),
    "pipesd_gemm_scratch_bytes": (u64, [i32, i32, i32]),
    "pipesd_gemm_pack": (i32, [vp, vp, i32, i32, vp]),
    "pipesd_gemm_run": (i32, [vp, vp, vp, vp, i32, i32, i32, vp]),
    "pipesd_gemm_run_static": (i32, [vp, vp, vp, i32, i32, i32, vp]),
    "pipesd_sched_round_time": (i32, [i32, ctypes.c_double, ctypes.c_double, ctypes.c_double, vp, i32,
                                      ctypes.POINTER(ctypes.c_double)]),
    "pipesd_sched_optimal_batching": (i32, [i32, ctypes.c_double, ctypes.c_double, ctypes.c_double, vp,
                                            ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_double)]),
    "pipesd_sched_trigger_step": (i32, [ctypes.POINTER(ctypes.c_double), ctypes.c_double, ctypes.c_double,
                                        ctypes.c_double, ctypes.POINTER(i32)]),
    "pipesd_debug_force_dense": (i32, [vp, i32]),
    "pipesd_debug_attn_slots": (i32, [vp, i32, ctypes.POINTER(ctypes.c_int32)]),
    "pipesd_debug_attn_split": (i32, [i32, i32, ctypes.POINTER(ctypes.c_int32), i32, ctypes.POINTER(ctypes.c_int32)]),
    "pipesd_debug_req_state": (i32, [vp, i32, ctypes.POINTER(ctypes.c_int32)]),
    "pipesd_debug_wait_timeout": (i32, [vp, i32]),
}


def lib():
    """Load libpipesd.so (no fallback: a missing library is an error)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: build it with paper_2605_13319_b200.build.build_cuda(); "
                               "there is no CPU path")
        L = ctypes.CDLL(str(LIB_PATH))
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


class PipesdError(RuntimeError):
    def __init__(self, code, where, detail=""):
        self.code = code
        msg = lib().pipesd_strerror(code).decode()
        super().__init__(f"{where}: {msg} ({code}) {detail}")


def _np_ptr(a):
    return a.ctypes.data if a is not None else None


class Context:
    """One verification context: a Llama-style target model, its paged KV pool and workspace.

    Method names follow the C entry points (pipesd_<name>)."""

    def __init__(self, shape, weights: dict, *, n_pages: int, max_requests: int = 1, max_draft: int = 16,
                 max_rows: int | None = None, max_seq: int = 4096, page_size: int = 16, device: int = 0,
                 stream=None, poison: bool = False):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: the verify pass has no CPU path")
        self.torch = torch
        self.shape = shape
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        if max_rows is None:
            max_rows = max(max_draft + 1, 32)
        self.cfg = ModelCfg(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                            shape.d_ffn, shape.vocab, shape.rms_eps, shape.rope_base, page_size, n_pages,
                            max_requests, max_draft, max_rows, max_seq, device, 0)
        L = lib()
        sz = Sizes()
        rc = L.pipesd_query_sizes(ctypes.byref(self.cfg), ctypes.byref(sz))
        if rc != OK:
            raise PipesdError(rc, "pipesd_query_sizes")
        self.sizes = sz
        with torch.cuda.stream(self.stream):
            self._wbuf = torch.empty(sz.weights_bytes, dtype=torch.uint8, device=self.device)
            self._kvbuf = torch.empty(sz.kv_bytes, dtype=torch.uint8, device=self.device)
            self._wsbuf = torch.zeros(sz.workspace_bytes, dtype=torch.uint8, device=self.device)
            if poison:
                # Every byte 0xFF: NaN as bf16 and as fp32, -1 as an index.  A read of a K/V row or of a workspace
                # element that this library did not write first then shows up in the results instead of passing
                # silently (pipesd_ctx_create initialises what it relies on itself).
                self._kvbuf.fill_(0xFF)
                self._wsbuf.fill_(0xFF)
            # upload the caller's row-major bf16 tensors; they are released after the repack
            up = lambda a: torch.from_numpy(a).to(self.device, non_blocking=False)
            lw = (LayerWeights * shape.n_layers)()
            keep = []
            for i, l in enumerate(weights["layers"]):
                for name in ("wq", "wk", "wv", "wo", "wg", "wu", "wd"):
                    t = up(l[name].view(np.int16))
                    keep.append(t)
                    setattr(lw[i], name, t.data_ptr())
                for name in ("attn_norm", "ffn_norm"):
                    t = up(l[name])
                    keep.append(t)
                    setattr(lw[i], name, t.data_ptr())
            te, lh, fn = up(weights["tok_emb"].view(np.int16)), up(weights["lm_head"].view(np.int16)), \
                up(weights["final_norm"])
            w = Weights(te.data_ptr(), lh.data_ptr(), fn.data_ptr(), lw)
            mem = Mem(self._wbuf.data_ptr(), sz.weights_bytes, self._kvbuf.data_ptr(), sz.kv_bytes,
                      self._wsbuf.data_ptr(), sz.workspace_bytes)
            h = vp()
            rc = L.pipesd_ctx_create(ctypes.byref(self.cfg), ctypes.byref(w), ctypes.byref(mem),
                                     vp(self.stream.cuda_stream), ctypes.byref(h))
            if rc != OK:
                raise PipesdError(rc, "pipesd_ctx_create")
            self._h = h
            self.ctx_sync()
            del keep, te, lh, fn
        self._alive = []   # host arrays referenced by an in-flight verify

    # -- helpers
    def _check(self, rc, where):
        if rc != OK:
            raise PipesdError(rc, where, lib().pipesd_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None):
            lib().pipesd_ctx_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- C entry points
    def ctx_sync(self):
        self._check(lib().pipesd_ctx_sync(self._h), "pipesd_ctx_sync")
        self._alive = []

    def req_open(self) -> int:
        r = i32()
        self._check(lib().pipesd_req_open(self._h, ctypes.byref(r)), "pipesd_req_open")
        return r.value

    def req_close(self, req: int):
        self._check(lib().pipesd_req_close(self._h, req), "pipesd_req_close")

    def req_len(self, req: int) -> int:
        n = i32()
        self._check(lib().pipesd_req_len(self._h, req, ctypes.byref(n)), "pipesd_req_len")
        return n.value

    def prefill(self, req: int, tokens, want_last_logits: bool = False):
        t = np.ascontiguousarray(tokens, np.int32)
        out = np.empty(self.shape.vocab, np.float32) if want_last_logits else None
        self._check(lib().pipesd_prefill(self._h, req, _np_ptr(t), t.size, _np_ptr(out)), "pipesd_prefill")
        return out

    def verify(self, items, flags: int = 0, sync: bool = True):
        """items: list of dict(req, tokens[k+1], q (torch cuda tensor / numpy with Q_HOST / None), u[k+1], mode).
        Returns a list of (n_accepted, next_token) when sync, else the ctypes result array (filled by ctx_sync)."""
        n = len(items)
        arr = (VerifyItem * n)()
        res = (VerifyResult * n)()
        alive = [arr, res]
        for i, it in enumerate(items):
            tok = np.ascontiguousarray(it["tokens"], np.int32)
            k = tok.size - 1
            u = it.get("u")
            u = np.ascontiguousarray(u, np.float32) if u is not None else None
            q = it.get("q")
            if q is None:
                qp = None
            elif isinstance(q, np.ndarray):
                assert flags & Q_HOST, "numpy q needs the Q_HOST flag"
                q = np.ascontiguousarray(q, np.float32)
                assert q.shape == (k, self.shape.vocab)
                qp = q.ctypes.data
            else:
                assert q.is_cuda and q.dtype == self.torch.float32 and q.is_contiguous()
                assert tuple(q.shape) == (k, self.shape.vocab)
                qp = q.data_ptr()
            alive += [tok, u, q]
            arr[i] = VerifyItem(it["req"], k, it.get("mode", MODE_STOCHASTIC), 0, tok.ctypes.data, qp,
                                u.ctypes.data if u is not None else None)
        self._alive = self._alive + alive if (flags & CHAIN) else alive
        self._check(lib().pipesd_verify(self._h, n, arr, res, flags), "pipesd_verify")
        if not sync:
            return res
        self.ctx_sync()
        return [(r.n_accepted, r.next_token) for r in res]

    def kv_rollback(self, reqs, n_accepted, next_token=None):
        r = np.ascontiguousarray(reqs, np.int32)
        a = np.ascontiguousarray(n_accepted, np.int32)
        t = np.ascontiguousarray(next_token, np.int32) if next_token is not None else None
        self._check(lib().pipesd_kv_rollback(self._h, r.size, _np_ptr(r), _np_ptr(a), _np_ptr(t)), "pipesd_kv_rollback")

    def debug_req_state(self, req: int):
        out = (ctypes.c_int32 * 3)()
        self._check(lib().pipesd_debug_req_state(self._h, req, out), "pipesd_debug_req_state")
        return tuple(out)

    def debug_force_dense(self, on: bool):
        self._check(lib().pipesd_debug_force_dense(self._h, int(on)), "pipesd_debug_force_dense")

    def debug_attn_slots(self, rows_per_kv_head: int):
        out = (ctypes.c_int32 * 2)()
        self._check(lib().pipesd_debug_attn_slots(self._h, rows_per_kv_head, out), "pipesd_debug_attn_slots")
        return tuple(out)

    def debug_wait_timeout(self, limit_us: int):
        self._check(lib().pipesd_debug_wait_timeout(self._h, limit_us), "pipesd_debug_wait_timeout")

    def debug_get_logits(self, rows: int) -> np.ndarray:
        out = np.empty((rows, self.shape.vocab), np.float32)
        self._check(lib().pipesd_debug_get_logits(self._h, _np_ptr(out), rows), "pipesd_debug_get_logits")
        return out

    def debug_read_kv(self, req: int, layer: int, pos0: int, n_pos: int):
        w = self.shape.n_kv_heads * self.shape.head_dim
        k = np.empty((n_pos, w), np.uint16)
        v = np.empty((n_pos, w), np.uint16)
        self._check(lib().pipesd_debug_read_kv(self._h, req, layer, pos0, n_pos, _np_ptr(k), _np_ptr(v)),
                    "pipesd_debug_read_kv")
        return k, v

    def debug_write_kv(self, req: int, layer: int, pos0: int, k_bf16, v_bf16):
        k = np.ascontiguousarray(k_bf16, np.uint16)
        v = np.ascontiguousarray(v_bf16, np.uint16)
        self._check(lib().pipesd_debug_write_kv(self._h, req, layer, pos0, k.shape[0], _np_ptr(k), _np_ptr(v)),
                    "pipesd_debug_write_kv")

    def debug_set_len(self, req: int, new_len: int):
        self._check(lib().pipesd_debug_set_len(self._h, req, new_len), "pipesd_debug_set_len")

    def profile_enable(self, time_gemms: bool = False):
        self._check(lib().pipesd_profile_enable(self._h, int(time_gemms)), "pipesd_profile_enable")

    def profile_read(self) -> dict:
        info = ProfileInfo()
        self._check(lib().pipesd_profile_read(self._h, ctypes.byref(info)), "pipesd_profile_read")
        return dict(kernel_launches=info.kernel_launches, gemm_launches=info.gemm_launches,
                    gemm_ms=info.gemm_ms, gemm_bytes=info.gemm_bytes)

    def reject_from_logits(self, logits, q, drafts, u, mode: int = MODE_STOCHASTIC):
        logits = np.ascontiguousarray(logits, np.float32)
        k = logits.shape[0] - 1
        q = np.ascontiguousarray(q, np.float32) if q is not None else None
        drafts = np.ascontiguousarray(drafts, np.int32)
        u = np.ascontiguousarray(u, np.float32)
        res = VerifyResult()
        self._check(lib().pipesd_reject_from_logits(self._h, k, mode, _np_ptr(logits), _np_ptr(q), _np_ptr(drafts),
                                                    _np_ptr(u), ctypes.byref(res)), "pipesd_reject_from_logits")
        return res.n_accepted, res.next_token


# ---- stand-alone GEMM entry points
def gemm_pack(W, stream=None):
    """W: torch cuda int16/bfloat16 tensor [N,K] (bf16 bit patterns) -> packed torch uint8 tensor."""
    import torch
    N, K = W.shape
    packed = torch.empty(lib().pipesd_gemm_packed_bytes(N, K), dtype=torch.uint8, device=W.device)
    st = stream if stream is not None else torch.cuda.current_stream(W.device)
    rc = lib().pipesd_gemm_pack(W.data_ptr(), packed.data_ptr(), N, K, vp(st.cuda_stream))
    if rc != OK:
        raise PipesdError(rc, "pipesd_gemm_pack")
    return packed


def gemm_scratch(M, N, K, device):
    import torch
    return torch.empty(max(int(lib().pipesd_gemm_scratch_bytes(M, N, K)), 16), dtype=torch.uint8, device=device)


def gemm_run(packed, x, y, scratch, N, K, stream=None):
    import torch
    M = x.shape[0]
    assert x.dtype == torch.float32 and y.dtype == torch.float32 and x.is_contiguous() and y.is_contiguous()
    assert x.shape[1] == K and tuple(y.shape) == (M, N)
    st = stream if stream is not None else torch.cuda.current_stream(x.device)
    rc = lib().pipesd_gemm_run(packed.data_ptr(), x.data_ptr(), y.data_ptr(), scratch.data_ptr(), M, N, K,
                               vp(st.cuda_stream))
    if rc != OK:
        raise PipesdError(rc, "pipesd_gemm_run")


def gemm_run_static(packed, x, y, N, K, stream=None):
    """pipesd_gemm_run_static: the GEMM with its split-K scratch inside the library, for callers that may
    not allocate device memory.  Same arguments as gemm_run minus the scratch tensor; nothing is allocated
    here either (the tensors are the caller's).  Raises PipesdError(E_TOO_LARGE) beyond the built-in limit."""
    import torch
    M = x.shape[0]
    assert x.dtype == torch.float32 and y.dtype == torch.float32 and x.is_contiguous() and y.is_contiguous()
    assert x.shape[1] == K and tuple(y.shape) == (M, N)
    st = stream if stream is not None else torch.cuda.current_stream(x.device)
    rc = lib().pipesd_gemm_run_static(packed.data_ptr(), x.data_ptr(), y.data_ptr(), M, N, K, vp(st.cuda_stream))
    if rc != OK:
        raise PipesdError(rc, "pipesd_gemm_run_static")


def debug_attn_split(total_keys: int, page_size: int, resident_ctas, units: int):
    """(key splits, keys per split, cut-down ring?) of one request: host arithmetic only."""
    res = (ctypes.c_int32 * 2)(*[int(x) for x in resident_ctas])
    out = (ctypes.c_int32 * 3)()
    rc = lib().pipesd_debug_attn_split(total_keys, page_size, res, units, out)
    if rc != 0:
        raise PipesdError(rc, "pipesd_debug_attn_split")
    return tuple(out)


# ---- the edge-side scheduling model (host code of the library)
def sched_round_time(N: int, alpha: float, beta: float, gamma: float, boundaries) -> float:
    b = np.ascontiguousarray(boundaries, np.int32)
    T = ctypes.c_double()
    rc = lib().pipesd_sched_round_time(N, alpha, beta, gamma, _np_ptr(b), b.size, ctypes.byref(T))
    if rc != OK:
        raise PipesdError(rc, "pipesd_sched_round_time")
    return T.value


def sched_optimal_batching(N: int, alpha: float, beta: float, gamma: float):
    """(boundaries b_1..b_K as a tuple, minimal T)."""
    b = np.zeros(max(N, 1), np.int32)
    K = i32()
    T = ctypes.c_double()
    rc = lib().pipesd_sched_optimal_batching(N, alpha, beta, gamma, _np_ptr(b), ctypes.byref(K), ctypes.byref(T))
    if rc != OK:
        raise PipesdError(rc, "pipesd_sched_optimal_batching")
    return tuple(int(x) for x in b[:K.value]), T.value


def sched_trigger_step(c1: float, R1: float, R2: float, p: float):
    """(triggered?, C1 after the step)."""
    c = ctypes.c_double(c1)
    fire = i32()
    rc = lib().pipesd_sched_trigger_step(ctypes.byref(c), R1, R2, p, ctypes.byref(fire))
    if rc != OK:
        raise PipesdError(rc, "pipesd_sched_trigger_step")
    return bool(fire.value), c.value
