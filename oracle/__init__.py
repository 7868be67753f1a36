"""CPU checker for the NAV verify pass: ctypes front end of ``nav_oracle.c``.

TEST INFRASTRUCTURE ONLY: the product path never imports this package.  Only the tests, the
smoke check and the benchmark's CPU-baseline leg do.  It shares no code with the CUDA path; the
only thing both sides use is the seeded input generator (``paper_2605_13319_b200.synth``), which
holds no verification arithmetic.

The verify pass (paper Sec. 2.2, App. B): one target-model forward over the pending token plus the
k draft tokens against the cached prefix, then accept drafts up to the first failure, emit one
correction (or, when all k pass, one extra) token, and keep only the accepted rows in the cache.
"""
from __future__ import annotations

import ctypes
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "nav_oracle.c"
_SO = _HERE / "_nav_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile nav_oracle.c with gcc (OpenMP, no fast-math so that sums stay in index order)."""
    if force or not _SO.exists() or _SO.stat().st_mtime < _SRC.stat().st_mtime:
        subprocess.run(["gcc", "-O3", "-mavx2", "-mfma", "-fopenmp", "-fPIC", "-shared",
                        str(_SRC), "-o", str(_SO), "-lm"], check=True)
    return _SO


class _Cfg(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn", "vocab", "max_pos")] \
        + [("rms_eps", ctypes.c_double), ("rope_base", ctypes.c_double)]


class _LayerW(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in
                ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "attn_norm", "ffn_norm")]


def lib():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(str(_SO))
        vp, i32, i64, f64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_double
        L.orc_rmsnorm.argtypes = [vp, vp, i32, f64, vp]
        L.orc_rope.argtypes = [vp, i32, i64, f64]
        L.orc_linear.argtypes = [vp, i32, i32, vp, i32, vp]
        L.orc_softmax.argtypes = [vp, i32, vp]
        L.orc_attend.argtypes = [vp, vp, vp, i64, i32, i32, vp]
        L.orc_create.argtypes = [ctypes.POINTER(_Cfg), vp, vp, vp, ctypes.POINTER(_LayerW)]
        L.orc_create.restype = vp
        L.orc_destroy.argtypes = [vp]
        L.orc_len.argtypes = [vp]
        L.orc_len.restype = i32
        L.orc_truncate.argtypes = [vp, i32]
        L.orc_truncate.restype = i32
        L.orc_set_kv.argtypes = [vp, i32, i32, i32, vp, vp]
        L.orc_set_len.argtypes = [vp, i32]
        L.orc_get_kv.argtypes = [vp, i32, i32, vp, vp]
        L.orc_forward.argtypes = [vp, vp, i32, i32, vp]
        L.orc_forward.restype = i32
        L.orc_final_cdf.argtypes = [vp, vp, i32, vp]
        L.orc_final_cdf.restype = f64
        L.orc_reject.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp, vp, vp]
        for f in (L.orc_rmsnorm, L.orc_rope, L.orc_linear, L.orc_softmax, L.orc_attend, L.orc_destroy,
                  L.orc_set_kv, L.orc_set_len, L.orc_get_kv, L.orc_reject):
            f.restype = None
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data


# ------------------------------------------------------------------ building blocks (for the pins)
def rmsnorm(x, g, eps):
    x = np.ascontiguousarray(x, np.float64)
    g = np.ascontiguousarray(g, np.float32)
    y = np.empty_like(x)
    lib().orc_rmsnorm(_p(x), _p(g), x.size, eps, _p(y))
    return y


def rope(v, pos, base):
    v = np.array(v, dtype=np.float64, order="C")
    lib().orc_rope(_p(v), v.size, int(pos), float(base))
    return v


def linear(W_bf16, x):
    """W: uint16 bf16 bit patterns [N,K]; x: [M,K] -> [M,N] (fp64)."""
    W = np.ascontiguousarray(W_bf16, np.uint16)
    x = np.ascontiguousarray(x, np.float64)
    M, K = x.shape
    N = W.shape[0]
    assert W.shape[1] == K
    y = np.empty((M, N), np.float64)
    lib().orc_linear(_p(W), N, K, _p(x), M, _p(y))
    return y


def softmax(l):
    l = np.ascontiguousarray(l, np.float64)
    p = np.empty_like(l)
    lib().orc_softmax(_p(l), l.size, _p(p))
    return p


def attend(q, kc, vc):
    """q: [hd]; kc, vc: float32 [n_keys, hd] -> [hd] (fp64)."""
    q = np.ascontiguousarray(q, np.float64)
    kc = np.ascontiguousarray(kc, np.float32)
    vc = np.ascontiguousarray(vc, np.float32)
    out = np.empty(q.size, np.float64)
    lib().orc_attend(_p(q), _p(kc), _p(vc), kc.shape[1], kc.shape[0], q.size, _p(out))
    return out


def final_cdf(logits_row, q_row=None):
    """Normalised inclusive CDF (token-id order) of the distribution the emitted token is drawn from."""
    l = np.ascontiguousarray(logits_row, np.float64)
    cdf = np.empty_like(l)
    qp = None
    if q_row is not None:
        q_row = np.ascontiguousarray(q_row, np.float32)
        qp = _p(q_row)
    S = lib().orc_final_cdf(_p(l), qp, l.size, _p(cdf))
    return cdf, S


def reject(logits, q, drafts, u, greedy=False):
    """Accept/correct rule. logits [k+1,V] fp64, q [k,V] fp32, drafts [k], u [k+1].
    Returns (n_accepted, emitted_token, margins[k])."""
    logits = np.ascontiguousarray(logits, np.float64)
    k = logits.shape[0] - 1
    V = logits.shape[1]
    drafts = np.ascontiguousarray(drafts, np.int32)
    u = np.ascontiguousarray(u, np.float32)
    assert drafts.size == k and u.size == k + 1
    if q is None:
        assert greedy
        q = np.zeros((max(k, 1), 1), np.float32)
    else:
        q = np.ascontiguousarray(q, np.float32)
        assert q.shape == (k, V)
    n_acc = ctypes.c_int32()
    tok = ctypes.c_int32()
    margins = np.empty(max(k, 1), np.float64)
    lib().orc_reject(_p(logits), _p(q), _p(drafts), _p(u), k, V, int(bool(greedy)),
                     ctypes.addressof(n_acc), ctypes.addressof(tok), _p(margins))
    return n_acc.value, tok.value, margins[:k]


# ------------------------------------------------------------------ the model
class Oracle:
    """Target model with its own contiguous KV cache (values bf16-rounded at write)."""

    def __init__(self, shape, weights: dict, max_pos: int):
        self.shape = shape
        self.w = weights  # keep the arrays alive: the C side borrows their memory
        cfg = _Cfg(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                   shape.d_ffn, shape.vocab, max_pos, shape.rms_eps, shape.rope_base)
        lw = (_LayerW * shape.n_layers)()
        for i, l in enumerate(weights["layers"]):
            for name in ("wq", "wk", "wv", "wo", "wg", "wu", "wd"):
                assert l[name].dtype == np.uint16 and l[name].flags.c_contiguous
                setattr(lw[i], name, _p(l[name]))
            for name in ("attn_norm", "ffn_norm"):
                assert l[name].dtype == np.float32
                setattr(lw[i], name, _p(l[name]))
        self._h = lib().orc_create(ctypes.byref(cfg), _p(weights["tok_emb"]), _p(weights["lm_head"]),
                                   _p(weights["final_norm"]), lw)
        self.max_pos = max_pos

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_destroy(self._h)
            self._h = None

    @property
    def len(self) -> int:
        return lib().orc_len(self._h)

    def forward(self, tokens, logits_from=0):
        """Append `tokens` at positions len.. and return fp64 logits of rows >= logits_from."""
        t = np.ascontiguousarray(tokens, np.int32)
        n = t.size
        m = n - logits_from
        out = np.empty((max(m, 0), self.shape.vocab), np.float64)
        rc = lib().orc_forward(self._h, _p(t), n, logits_from, _p(out) if m > 0 else None)
        if rc != 0:
            raise RuntimeError(f"orc_forward failed: {rc}")
        return out

    def prefill(self, tokens, want_last_logits=False):
        n = len(tokens)
        return self.forward(tokens, logits_from=n - 1 if want_last_logits else n)

    def truncate(self, new_len: int):
        if lib().orc_truncate(self._h, new_len) != 0:
            raise ValueError("bad truncate length")

    def set_synthetic_kv(self, layer: int, k_bf16, v_bf16, pos0: int = 0):
        k_bf16 = np.ascontiguousarray(k_bf16, np.uint16)
        v_bf16 = np.ascontiguousarray(v_bf16, np.uint16)
        lib().orc_set_kv(self._h, layer, pos0, k_bf16.shape[0], _p(k_bf16), _p(v_bf16))

    def set_len(self, n: int):
        lib().orc_set_len(self._h, n)

    def get_kv(self, layer: int, pos: int):
        w = self.shape.n_kv_heads * self.shape.head_dim
        k = np.empty(w, np.float32)
        v = np.empty(w, np.float32)
        lib().orc_get_kv(self._h, layer, pos, _p(k), _p(v))
        return k, v

    def verify(self, tokens, q, u, greedy=False):
        """tokens = [pending, d_1..d_k]. Forward over the k+1 rows, apply the rule.  The cache is
        left holding all k+1 rows (tentative); call rollback(n_acc) to commit.
        Returns dict(n_accepted, next_token, logits, margins, base_len)."""
        tokens = np.ascontiguousarray(tokens, np.int32)
        base = self.len
        logits = self.forward(tokens, 0)
        n_acc, tok, margins = reject(logits, q, tokens[1:], u, greedy)
        return dict(n_accepted=n_acc, next_token=tok, logits=logits, margins=margins, base_len=base)

    def rollback(self, base_len: int, n_accepted: int):
        """Keep the pending token's row and the accepted drafts' rows; drop the rejected tail."""
        self.truncate(base_len + 1 + n_accepted)

    def verify_chain(self, tokens, q, u, buffered, q_buf, u_buf, greedy=False):
        """One round followed by the cloud's handling of proactively sent drafts (paper App. B).  While this round
        was being verified the edge kept drafting: `buffered` = [b_1..b_m] are those early tokens, where b_1 is the
        edge's own guess at this round's extra token and b_2..b_m continue from it (q_buf [m-1, V], u_buf [m] belong
        to them).  After the round the cloud checks (i) every draft accepted and (ii) extra token == b_1.  If both
        hold the buffered tokens stay valid: the round is committed in full and b_1 (now the pending token) with
        b_2..b_m as drafts is the next round, verified at once.  Otherwise they are discarded and only the first
        round is committed.  Either way the cache is left committed.
        Returns (first round's dict, second round's dict or None when the buffered tokens were discarded)."""
        tokens = np.ascontiguousarray(tokens, np.int32)
        buffered = np.ascontiguousarray(buffered, np.int32)
        k = tokens.size - 1
        r1 = self.verify(tokens, q, u, greedy)
        self.rollback(r1["base_len"], r1["n_accepted"])
        if not (r1["n_accepted"] == k and r1["next_token"] == int(buffered[0])):
            return r1, None
        r2 = self.verify(buffered, q_buf, u_buf, greedy)
        self.rollback(r2["base_len"], r2["n_accepted"])
        return r1, r2

    def draft_round(self, pending: int, k: int, sigma: float, noise, draft_u):
        """Make one round's inputs by running the target one token at a time:
        q_i = softmax(l_{i-1} + sigma * eps_i), d_i drawn from q_i by inverse CDF with draft_u[i-1].
        noise: [k, V] standard normals. Returns (tokens[k+1], q[k,V] fp32, logits[k+1,V] fp64).
        The cache is restored to its length at entry."""
        base = self.len
        V = self.shape.vocab
        toks = [int(pending)]
        q = np.empty((k, V), np.float32)
        rows = []
        l = self.forward([pending], 0)[0]
        rows.append(l)
        for i in range(k):
            qi = softmax(l + sigma * np.asarray(noise[i], np.float64))
            q[i] = qi.astype(np.float32)
            cdf = np.cumsum(q[i].astype(np.float64))
            d = int(np.searchsorted(cdf, float(draft_u[i]) * cdf[-1], side="right"))
            d = min(d, V - 1)
            toks.append(d)
            l = self.forward([d], 0)[0]
            rows.append(l)
        self.truncate(base)
        return np.array(toks, np.int32), q, np.stack(rows)
