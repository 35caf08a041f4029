"""ctypes binding of the C oracle (test infrastructure; never on the product path).

``build()`` compiles ``spechub_oracle.c`` with gcc into ``oracle/_build`` and is
called lazily on first use.  All arrays are numpy; nothing here touches CUDA.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spechub_oracle.c")
_LIB = os.path.join(_HERE, "_build", "libspechub_oracle.so")
_lock = threading.Lock()
_lib = None

STATUS_BITS = {
    "NONFINITE": 1,
    "TOKEN_RANGE": 2,
    "DEGENERATE_Q": 4,
    "ZERO_MASS_DRAFT": 8,
    "ZERO_RESIDUAL": 16,
}

# mirrors struct orc_node
NODE_DTYPE = np.dtype(
    [
        ("beta", np.float64, (2,)),
        ("rate", np.float64, (3,)),
        ("margin", np.float64, (3,)),
        ("cond", np.float64, (2,)),
        ("accept_idx", np.int32),
        ("token", np.int32),
        ("hub", np.int32),
        ("status", np.uint32),
    ],
    align=True,
)

_dp = ctypes.POINTER(ctypes.c_double)
_fp = ctypes.POINTER(ctypes.c_float)
_ip = ctypes.POINTER(ctypes.c_int32)
_up = ctypes.POINTER(ctypes.c_uint32)
_bp = ctypes.POINTER(ctypes.c_uint8)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math: fp64 semantics are the point)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            os.makedirs(os.path.dirname(_LIB), exist_ok=True)
            tmp = _LIB + ".%d.tmp" % os.getpid()
            subprocess.check_call(
                ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fno-fast-math",
                 "-ffp-contract=off", "-o", tmp, _SRC, "-lm"]
            )
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.orc_softmax.restype = ctypes.c_uint
        lib.orc_softmax.argtypes = [_fp, ctypes.c_int, ctypes.c_double, _dp]
        lib.orc_hub.restype = ctypes.c_int
        lib.orc_hub.argtypes = [_fp, ctypes.c_int]
        lib.orc_inv_cdf.restype = ctypes.c_int
        lib.orc_inv_cdf.argtypes = [_dp, ctypes.c_int, ctypes.c_double, _dp, _dp]
        lib.orc_cdf_interval.restype = ctypes.c_int
        lib.orc_cdf_interval.argtypes = [_dp, ctypes.c_int, ctypes.c_int, _dp, _dp]
        lib.orc_spechub_draft.restype = ctypes.c_uint
        lib.orc_spechub_draft.argtypes = [_dp, ctypes.c_int, ctypes.c_int, ctypes.c_double,
                                          ctypes.c_double, _ip, _dp, _dp]
        lib.orc_spechub_residual.restype = None
        lib.orc_spechub_residual.argtypes = [_dp, _dp, ctypes.c_int, ctypes.c_int, _dp]
        lib.orc_spechub_verify.restype = None
        lib.orc_spechub_verify.argtypes = [_dp, _dp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                           ctypes.c_int, ctypes.c_double, ctypes.c_double,
                                           ctypes.c_double, ctypes.c_void_p]
        lib.orc_rrs_draft.restype = ctypes.c_uint
        lib.orc_rrs_draft.argtypes = [_dp, ctypes.c_int, ctypes.c_int, ctypes.c_double,
                                      ctypes.c_double, _ip, _dp]
        lib.orc_rrs_residual.restype = None
        lib.orc_rrs_residual.argtypes = [_dp, _dp, ctypes.c_int, ctypes.c_int, ctypes.c_int, _dp]
        lib.orc_rrs_verify.restype = None
        lib.orc_rrs_verify.argtypes = [_dp, _dp, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                       ctypes.c_int, ctypes.c_void_p]
        lib.orc_draft_batch.restype = None
        lib.orc_draft_batch.argtypes = [ctypes.c_int, _fp, _fp, ctypes.c_int, ctypes.c_int,
                                        ctypes.c_int, _fp, _ip, _ip, _dp, _dp, _up]
        lib.orc_verify_batch.restype = None
        lib.orc_verify_batch.argtypes = [ctypes.c_int, _fp, _fp, _fp, ctypes.c_int, ctypes.c_int,
                                         ctypes.c_int, _bp, _ip, _fp, ctypes.c_void_p]
        lib.orc_walk.restype = None
        lib.orc_walk.argtypes = [_ip, _ip, ctypes.c_int, ctypes.c_int, _ip, _bp, ctypes.c_int,
                                 _ip, _ip, _ip, _ip]
        lib.orc_rrs_k_draft.restype = ctypes.c_uint
        lib.orc_rrs_k_draft.argtypes = [_dp, ctypes.c_int, ctypes.c_int, ctypes.c_int, _dp, _ip, _dp]
        lib.orc_rrs_k_verify.restype = None
        lib.orc_rrs_k_verify.argtypes = [_dp, _dp, ctypes.c_int, ctypes.c_int, _ip, _dp, ctypes.c_double,
                                         ctypes.c_int, _ip, _ip, _dp, _dp, _dp, _dp, _up]
        lib.orc_rrs_k_residual.restype = None
        lib.orc_rrs_k_residual.argtypes = [_dp, _dp, ctypes.c_int, ctypes.c_int, _ip, ctypes.c_int, _dp]
        lib.orc_rrs_k_draft_batch.restype = None
        lib.orc_rrs_k_draft_batch.argtypes = [ctypes.c_int, ctypes.c_int, _fp, _fp, ctypes.c_int, ctypes.c_int,
                                              ctypes.c_int, _fp, _ip, _dp, _up]
        lib.orc_rrs_k_verify_batch.restype = None
        lib.orc_rrs_k_verify_batch.argtypes = [ctypes.c_int, ctypes.c_int, _fp, _fp, _fp, ctypes.c_int,
                                               ctypes.c_int, ctypes.c_int, _bp, _ip, _fp, _ip, _ip, _dp, _dp,
                                               _dp, _dp, _up]
        lib.orc_walk_k.restype = None
        lib.orc_walk_k.argtypes = [ctypes.c_int, _ip, _ip, ctypes.c_int, ctypes.c_int, _ip, _bp, ctypes.c_int,
                                   _ip, _ip, _ip, _ip]
        lib.orc_node_size.restype = ctypes.c_size_t
        assert lib.orc_node_size() == NODE_DTYPE.itemsize, (lib.orc_node_size(), NODE_DTYPE.itemsize)
        _lib = lib
    return _lib


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _ptr(a, t):
    return a.ctypes.data_as(t)


METHODS = {"spechub": 0, "rrs": 1, "rrsw": 2}


def _method(m):
    return METHODS[m] if isinstance(m, str) else int(m)


# ---- row-level functions (probabilities in, fp64) ---------------------------------------------

def softmax(logits, T=1.0):
    """Distribution of a row of logits at temperature T; returns (prob, status)."""
    l = _f32(logits)
    out = np.empty(l.shape[0], np.float64)
    st = _load().orc_softmax(_ptr(l, _fp), l.shape[0], float(T), _ptr(out, _dp))
    return out, int(st)


def hub(draft_logits):
    l = _f32(draft_logits)
    return int(_load().orc_hub(_ptr(l, _fp), l.shape[0]))


def inv_cdf(w, u):
    """(token, W, margin) of the inverse-CDF draw from weights w with uniform u."""
    w = _f64(w)
    W = ctypes.c_double()
    m = ctypes.c_double()
    tok = _load().orc_inv_cdf(_ptr(w, _dp), w.shape[0], float(u), ctypes.byref(W), ctypes.byref(m))
    return int(tok), W.value, m.value


def cdf_interval(w, token):
    """[lo, hi) of `token` in the normalised CDF of w."""
    w = _f64(w)
    lo = ctypes.c_double()
    hi = ctypes.c_double()
    _load().orc_cdf_interval(_ptr(w, _dp), w.shape[0], int(token), ctypes.byref(lo), ctypes.byref(hi))
    return lo.value, hi.value


def spechub_draft(q, a, u1, u2):
    """Draw (x1, x2) ~ Q.  Returns (tokens[2], prob[2] = (q(a), Q(x1,x2)), margin[2], status)."""
    q = _f64(q)
    tk = np.empty(2, np.int32)
    pr = np.empty(2, np.float64)
    mg = np.empty(2, np.float64)
    st = _load().orc_spechub_draft(_ptr(q, _dp), q.shape[0], int(a), float(u1), float(u2),
                                   _ptr(tk, _ip), _ptr(pr, _dp), _ptr(mg, _dp))
    return tk, pr, mg, int(st)


def spechub_residual(p, q, a):
    p = _f64(p)
    q = _f64(q)
    w = np.empty_like(p)
    _load().orc_spechub_residual(_ptr(p, _dp), _ptr(q, _dp), p.shape[0], int(a), _ptr(w, _dp))
    return w


def spechub_verify(p, q, a, x1, x2, r1, r2, u_res):
    """Algorithm 3 on one node; returns a NODE_DTYPE scalar record."""
    p = _f64(p)
    q = _f64(q)
    out = np.zeros(1, NODE_DTYPE)
    _load().orc_spechub_verify(_ptr(p, _dp), _ptr(q, _dp), p.shape[0], int(a), int(x1), int(x2),
                               float(r1), float(r2), float(u_res), out.ctypes.data)
    return out[0]


def rrs_draft(q, without_replacement, u1, u2):
    q = _f64(q)
    tk = np.empty(2, np.int32)
    mg = np.empty(2, np.float64)
    st = _load().orc_rrs_draft(_ptr(q, _dp), q.shape[0], int(bool(without_replacement)), float(u1),
                               float(u2), _ptr(tk, _ip), _ptr(mg, _dp))
    return tk, mg, int(st)


def rrs_residual(p, q, x1, without_replacement):
    p = _f64(p)
    q = _f64(q)
    w = np.empty_like(p)
    _load().orc_rrs_residual(_ptr(p, _dp), _ptr(q, _dp), p.shape[0], int(x1),
                             int(bool(without_replacement)), _ptr(w, _dp))
    return w


def rrs_verify(p, q, x1, x2, r1, r2, u_res, without_replacement):
    """Algorithm 1 on one node; returns a NODE_DTYPE scalar record."""
    p = _f64(p)
    q = _f64(q)
    out = np.zeros(1, NODE_DTYPE)
    _load().orc_rrs_verify(_ptr(p, _dp), _ptr(q, _dp), p.shape[0], int(x1), int(x2), float(r1),
                           float(r2), float(u_res), int(bool(without_replacement)), out.ctypes.data)
    return out[0]


# ---- batch / tree level (logits in) ------------------------------------------------------------

def _temps(temperature, B):
    t = np.asarray(temperature, dtype=np.float32)
    if t.ndim == 0:
        t = np.full(B, float(t), np.float32)
    assert t.shape == (B,)
    return np.ascontiguousarray(t)


def draft_batch(method, draft_logits, temperature, uniforms):
    """Draft step for logits [B][N][V].  Returns dict(tokens, hub, prob, margin, status)."""
    lq = _f32(draft_logits)
    B, N, V = lq.shape
    un = _f32(uniforms)
    assert un.shape == (B, N, 5)
    t = _temps(temperature, B)
    tokens = np.empty((B, N, 2), np.int32)
    hubs = np.empty((B, N), np.int32)
    prob = np.empty((B, N, 2), np.float64)
    margin = np.empty((B, N, 2), np.float64)
    status = np.zeros((B, N), np.uint32)
    _load().orc_draft_batch(_method(method), _ptr(lq, _fp), _ptr(t, _fp), B, N, V, _ptr(un, _fp),
                            _ptr(tokens, _ip), _ptr(hubs, _ip), _ptr(prob, _dp), _ptr(margin, _dp),
                            _ptr(status, _up))
    return dict(tokens=tokens, hub=hubs, prob=prob, margin=margin, status=status)


def verify_batch(method, target_logits, draft_logits, temperature, draft_tokens, uniforms,
                 node_kind=None):
    """Verification of every node of logits [B][N][V]; returns a [B][N] NODE_DTYPE array."""
    lp = _f32(target_logits)
    lq = _f32(draft_logits)
    B, N, V = lp.shape
    assert lq.shape == lp.shape
    un = _f32(uniforms)
    tk = _i32(draft_tokens)
    assert un.shape == (B, N, 5) and tk.shape == (B, N, 2)
    t = _temps(temperature, B)
    nk = None
    if node_kind is not None:
        nk = np.ascontiguousarray(node_kind, dtype=np.uint8)
        assert nk.shape == (N,)
    out = np.zeros((B, N), NODE_DTYPE)
    _load().orc_verify_batch(_method(method), _ptr(lp, _fp), _ptr(lq, _fp), _ptr(t, _fp), B, N, V,
                             _ptr(nk, _bp) if nk is not None else None, _ptr(tk, _ip),
                             _ptr(un, _fp), out.ctypes.data)
    return out


def walk(accept_idx, token, levels, child=None, node_kind=None):
    """Tree walk (Figure 2).  Returns dict(n_accepted, n_emitted, path_nodes, path_tokens)."""
    ai = _i32(accept_idx)
    tk = _i32(token)
    B, N = ai.shape
    ch = None
    if child is not None:
        ch = _i32(child)
        assert ch.shape == (N, 2)
    nk = None
    if node_kind is not None:
        nk = np.ascontiguousarray(node_kind, dtype=np.uint8)
    na = np.empty(B, np.int32)
    ne = np.empty(B, np.int32)
    pn = np.empty((B, levels), np.int32)
    pt = np.empty((B, levels), np.int32)
    _load().orc_walk(_ptr(ai, _ip), _ptr(tk, _ip), B, N, _ptr(ch, _ip) if ch is not None else None,
                     _ptr(nk, _bp) if nk is not None else None, int(levels), _ptr(na, _ip),
                     _ptr(ne, _ip), _ptr(pn, _ip), _ptr(pt, _ip))
    return dict(n_accepted=na, n_emitted=ne, path_nodes=pn, path_tokens=pt)


# ---- Algorithm 1 for general k ------------------------------------------------------------------

def rrs_k_draft(q, k, without_replacement, u):
    """k drafts from q (independent, or without replacement).  Returns (tokens[k], margin[k], status)."""
    q = _f64(q)
    u = _f64(u)
    tk = np.empty(k, np.int32)
    mg = np.empty(k, np.float64)
    st = _load().orc_rrs_k_draft(_ptr(q, _dp), q.shape[0], int(k), int(bool(without_replacement)),
                                 _ptr(u, _dp), _ptr(tk, _ip), _ptr(mg, _dp))
    return tk, mg, int(st)


def rrs_k_verify(p, q, tokens, r, u_res, without_replacement):
    """Algorithm 1 on one node with k = len(tokens) drafts.  Returns a dict."""
    p, q, r = _f64(p), _f64(q), _f64(r)
    tk = _i32(tokens)
    k = tk.shape[0]
    ai, tok, st = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_uint32()
    beta, rate = np.empty(k), np.empty(k + 1)
    margin, cond = np.empty(k + 1), np.empty(k)
    _load().orc_rrs_k_verify(_ptr(p, _dp), _ptr(q, _dp), p.shape[0], k, _ptr(tk, _ip), _ptr(r, _dp),
                             float(u_res), int(bool(without_replacement)), ctypes.byref(ai),
                             ctypes.byref(tok), _ptr(beta, _dp), _ptr(rate, _dp), _ptr(margin, _dp),
                             _ptr(cond, _dp), ctypes.byref(st))
    return dict(accept_idx=ai.value, token=tok.value, beta=beta, rate=rate, margin=margin, cond=cond,
                status=st.value)


def rrs_k_residual(p, q, tokens, without_replacement):
    p, q = _f64(p), _f64(q)
    tk = _i32(tokens)
    w = np.empty_like(p)
    _load().orc_rrs_k_residual(_ptr(p, _dp), _ptr(q, _dp), p.shape[0], tk.shape[0], _ptr(tk, _ip),
                               int(bool(without_replacement)), _ptr(w, _dp))
    return w


def rrs_k_draft_batch(k, without_replacement, draft_logits, temperature, uniforms):
    lq = _f32(draft_logits)
    B, N, V = lq.shape
    un = _f32(uniforms)
    assert un.shape == (B, N, 2 * k + 1)
    t = _temps(temperature, B)
    tokens = np.empty((B, N, k), np.int32)
    margin = np.empty((B, N, k), np.float64)
    status = np.zeros((B, N), np.uint32)
    _load().orc_rrs_k_draft_batch(int(k), int(bool(without_replacement)), _ptr(lq, _fp), _ptr(t, _fp), B, N, V,
                                  _ptr(un, _fp), _ptr(tokens, _ip), _ptr(margin, _dp), _ptr(status, _up))
    return dict(tokens=tokens, margin=margin, status=status)


def rrs_k_verify_batch(k, without_replacement, target_logits, draft_logits, temperature, draft_tokens,
                       uniforms, node_kind=None):
    lp, lq = _f32(target_logits), _f32(draft_logits)
    B, N, V = lp.shape
    un, tk = _f32(uniforms), _i32(draft_tokens)
    assert un.shape == (B, N, 2 * k + 1) and tk.shape == (B, N, k)
    t = _temps(temperature, B)
    nk = None if node_kind is None else np.ascontiguousarray(node_kind, dtype=np.uint8)
    out = dict(accept_idx=np.empty((B, N), np.int32), token=np.empty((B, N), np.int32),
               beta=np.empty((B, N, k)), rate=np.empty((B, N, k + 1)), margin=np.empty((B, N, k + 1)),
               cond=np.empty((B, N, k)), status=np.zeros((B, N), np.uint32))
    _load().orc_rrs_k_verify_batch(int(k), int(bool(without_replacement)), _ptr(lp, _fp), _ptr(lq, _fp),
                                   _ptr(t, _fp), B, N, V, _ptr(nk, _bp) if nk is not None else None,
                                   _ptr(tk, _ip), _ptr(un, _fp), _ptr(out["accept_idx"], _ip),
                                   _ptr(out["token"], _ip), _ptr(out["beta"], _dp), _ptr(out["rate"], _dp),
                                   _ptr(out["margin"], _dp), _ptr(out["cond"], _dp), _ptr(out["status"], _up))
    return out


def walk_k(k, accept_idx, token, levels, child=None, node_kind=None):
    ai, tk = _i32(accept_idx), _i32(token)
    B, N = ai.shape
    ch = None if child is None else _i32(child)
    nk = None if node_kind is None else np.ascontiguousarray(node_kind, dtype=np.uint8)
    na, ne = np.empty(B, np.int32), np.empty(B, np.int32)
    pn, pt = np.empty((B, levels), np.int32), np.empty((B, levels), np.int32)
    _load().orc_walk_k(int(k), _ptr(ai, _ip), _ptr(tk, _ip), B, N, _ptr(ch, _ip) if ch is not None else None,
                       _ptr(nk, _bp) if nk is not None else None, int(levels), _ptr(na, _ip), _ptr(ne, _ip),
                       _ptr(pn, _ip), _ptr(pt, _ip))
    return dict(n_accepted=na, n_emitted=ne, path_nodes=pn, path_tokens=pt)
