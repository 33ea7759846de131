"""CPU oracle (test infrastructure only): ctypes front end of ``oracle.c``.

The oracle is the plain statement of what the FreeCache hot path computes.  It is used by
the tests, by the smoke check and by the CPU-baseline leg of the benchmark, never by the
product path, and it shares no code with the CUDA library.  Arguments are numpy arrays;
floating-point inputs are fp32 (bf16 values widened exactly by the caller).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_SO = os.path.join(_HERE, "liboracle.so")

ERR_CAPACITY = 1
ERR_INDEX = 2

_lib = None


def build(force: bool = False) -> str:
    """Compile ``oracle.c`` with gcc (OpenMP, no fast-math) if the shared object is stale."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _p(a, dtype):
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags["C_CONTIGUOUS"], (
        f"expected contiguous {dtype} array, got {type(a)} {getattr(a, 'dtype', None)}")
    return a.ctypes.data_as(ctypes.c_void_p)


def attn_step(cache_k, cache_v, cache_len, q, k_new, v_new, q_len=None, scale=None):
    """One layer's attention step.  Shapes: cache [B,Hkv,Lcap,D], q [B,Hq,q_cap,D],
    k_new/v_new [B,Hkv,q_cap,D] (all fp32), cache_len/q_len int32 [B].
    Returns (out fp32 [B,Hq,q_cap,D], lse fp32 [B,Hq,q_cap])."""
    B, Hkv, Lcap, D = cache_k.shape
    _, Hq, q_cap, _ = q.shape
    assert cache_v.shape == cache_k.shape and k_new.shape == (B, Hkv, q_cap, D) == v_new.shape
    if scale is None:
        scale = 1.0 / float(np.sqrt(D))
    out = np.empty((B, Hq, q_cap, D), np.float32)
    lse = np.empty((B, Hq, q_cap), np.float32)
    rc = _load().oracle_attn_step(
        B, Hq, Hkv, D, Lcap, q_cap, _p(cache_k, np.float32), _p(cache_v, np.float32),
        _p(cache_len, np.int32), _p(q_len, np.int32), _p(q, np.float32), _p(k_new, np.float32),
        _p(v_new, np.float32), ctypes.c_float(scale), _p(out, np.float32), _p(lse, np.float32))
    assert rc == 0, rc
    return out, lse


def kv_cache_commit(cache_k, cache_v, cache_len, k_new, v_new, src_idx=None, dst_pos=None,
                    n_rows=None, n_max=None, advance_len=False, layer_begin=0, layer_end=None, dst_mode=0):
    """In-place commit on uint16 bit patterns.  cache [NL,B,Hkv,Lcap,D], new
    [layer_end-layer_begin,B,Hkv,src_len,D].  Returns the error bit mask."""
    NL, B, Hkv, Lcap, D = cache_k.shape
    if layer_end is None:
        layer_end = NL
    nl, _, _, src_len, _ = k_new.shape
    assert nl == layer_end - layer_begin and k_new.shape == v_new.shape
    if n_max is None:
        n_max = src_idx.shape[1] if src_idx is not None else (
            dst_pos.shape[1] if dst_pos is not None else src_len)
    return int(_load().oracle_kv_cache_commit(
        NL, B, Hkv, Lcap, D, _p(cache_k, np.uint16), _p(cache_v, np.uint16),
        _p(cache_len, np.int32), _p(k_new, np.uint16), _p(v_new, np.uint16), src_len,
        _p(src_idx, np.int32), _p(dst_pos, np.int32), int(dst_mode), _p(n_rows, np.int32), n_max,
        int(bool(advance_len)), layer_begin, layer_end))


def unmask_select(logits, masked, tokens, k):
    """logits fp32 [B,Lblk,V]; masked uint8 [B,Lblk] and tokens int32 [B,Lblk] are updated
    in place when k > 0.  Returns (tok, conf, sel_idx, n_sel); the last two are None for k == 0."""
    B, Lblk, V = logits.shape
    tok = np.empty((B, Lblk), np.int32)
    conf = np.empty((B, Lblk), np.float32)
    sel_idx = np.full((B, max(k, 1)), -1, np.int32) if k > 0 else None
    n_sel = np.zeros((B,), np.int32) if k > 0 else None
    rc = _load().oracle_unmask_select(
        B, Lblk, V, _p(logits, np.float32), _p(masked, np.uint8), _p(tokens, np.int32), k,
        _p(tok, np.int32), _p(conf, np.float32), _p(sel_idx, np.int32), _p(n_sel, np.int32))
    assert rc == 0, rc
    return tok, conf, sel_idx, n_sel


def guided_accept(tok_dlm, tok_ar, masked, tokens, fallback_source=0):
    """int32 [B,Lblk] proposals; masked/tokens updated in place.
    Returns (accept uint8 [B,Lblk], acc_idx int32 [B,Lblk], n_acc int32 [B])."""
    B, Lblk = tok_dlm.shape
    accept = np.empty((B, Lblk), np.uint8)
    acc_idx = np.empty((B, Lblk), np.int32)
    n_acc = np.empty((B,), np.int32)
    rc = _load().oracle_guided_accept(
        B, Lblk, _p(tok_dlm, np.int32), _p(tok_ar, np.int32), _p(masked, np.uint8),
        _p(tokens, np.int32), int(fallback_source), _p(accept, np.uint8),
        _p(acc_idx, np.int32), _p(n_acc, np.int32))
    assert rc == 0, rc
    return accept, acc_idx, n_acc


def guided_accept_topk(tok_dlm, tok_ar_topk, masked, tokens, fallback_source=0):
    """Top-K match variant: tok_ar_topk int32 [B,Lblk,K] in rank order.  Returns (accept, acc_idx, n_acc)."""
    B, Lblk = tok_dlm.shape
    K = tok_ar_topk.shape[2]
    assert tok_ar_topk.shape == (B, Lblk, K)
    accept = np.empty((B, Lblk), np.uint8)
    acc_idx = np.empty((B, Lblk), np.int32)
    n_acc = np.empty((B,), np.int32)
    rc = _load().oracle_guided_accept_topk(
        B, Lblk, K, _p(tok_dlm, np.int32), _p(tok_ar_topk, np.int32), _p(masked, np.uint8),
        _p(tokens, np.int32), int(fallback_source), _p(accept, np.uint8),
        _p(acc_idx, np.int32), _p(n_acc, np.int32))
    assert rc == 0, rc
    return accept, acc_idx, n_acc


def unmask_scores(logits, masked):
    """Per-position statistics (see oracle.c): returns (tok, conf, zmax, neg_entropy, margin)."""
    B, Lblk, V = logits.shape
    tok = np.empty((B, Lblk), np.int32)
    outs = [np.empty((B, Lblk), np.float32) for _ in range(4)]
    rc = _load().oracle_unmask_scores(B, Lblk, V, _p(logits, np.float32), _p(masked, np.uint8), _p(tok, np.int32),
                                      *[_p(o, np.float32) for o in outs])
    assert rc == 0, rc
    return (tok, *outs)


SCORE_CONFIDENCE, SCORE_NEG_ENTROPY, SCORE_MARGIN, SCORE_LOG_CONF_PLUS_NOISE = 0, 1, 2, 3


def unmask_select_scored(logits, masked, tokens, k, kind, noise=None):
    """Top-k unmasking ranked by the chosen score.  Returns (tok, conf, score, zmax, sel_idx, n_sel)."""
    B, Lblk, V = logits.shape
    tok = np.empty((B, Lblk), np.int32)
    conf, score, zmax = (np.empty((B, Lblk), np.float32) for _ in range(3))
    sel_idx = np.full((B, max(k, 1)), -1, np.int32) if k > 0 else None
    n_sel = np.zeros((B,), np.int32) if k > 0 else None
    rc = _load().oracle_unmask_select_scored(
        B, Lblk, V, _p(logits, np.float32), _p(masked, np.uint8), _p(tokens, np.int32), k, int(kind),
        _p(noise, np.float32), _p(tok, np.int32), _p(conf, np.float32), _p(score, np.float32), _p(zmax, np.float32),
        _p(sel_idx, np.int32), _p(n_sel, np.int32))
    assert rc == 0, rc
    return tok, conf, score, zmax, sel_idx, n_sel


def guided_accept_threshold(tok_dlm, zmax_dlm, tok_ar_topk, logit_ar_topk, tau, masked, tokens, fallback_source=0):
    """Top-K match accept plus the confidence threshold of App. C.3.  Returns (accept, acc_idx, n_acc)."""
    B, Lblk = tok_dlm.shape
    K = tok_ar_topk.shape[2]
    assert tok_ar_topk.shape == (B, Lblk, K) == logit_ar_topk.shape and zmax_dlm.shape == (B, Lblk)
    accept = np.empty((B, Lblk), np.uint8)
    acc_idx = np.empty((B, Lblk), np.int32)
    n_acc = np.empty((B,), np.int32)
    rc = _load().oracle_guided_accept_threshold(
        B, Lblk, K, _p(tok_dlm, np.int32), _p(zmax_dlm, np.float32), _p(tok_ar_topk, np.int32),
        _p(logit_ar_topk, np.float32), ctypes.c_float(tau), _p(masked, np.uint8), _p(tokens, np.int32),
        int(fallback_source), _p(accept, np.uint8), _p(acc_idx, np.int32), _p(n_acc, np.int32))
    assert rc == 0, rc
    return accept, acc_idx, n_acc


def qkv_project(x, w, bias, Hq, Hkv, D):
    """x fp32 [B,q_cap,d_model], w fp32 [(Hq+2Hkv)*D, d_model], bias fp32 [(Hq+2Hkv)*D] or None.
    Returns (q [B,Hq,q_cap,D], k [B,Hkv,q_cap,D], v [B,Hkv,q_cap,D]) fp32."""
    B, q_cap, d_model = x.shape
    assert w.shape == ((Hq + 2 * Hkv) * D, d_model)
    q = np.empty((B, Hq, q_cap, D), np.float32)
    k = np.empty((B, Hkv, q_cap, D), np.float32)
    v = np.empty((B, Hkv, q_cap, D), np.float32)
    rc = _load().oracle_qkv_project(B, q_cap, d_model, Hq, Hkv, D, _p(x, np.float32), _p(w, np.float32),
                                    _p(bias, np.float32), _p(q, np.float32), _p(k, np.float32), _p(v, np.float32))
    assert rc == 0, rc
    return q, k, v


def qkv_project_rope(x, w, bias, rope_cos, rope_sin, Hq, Hkv, D):
    """qkv_project followed by the rotary embedding of the query and key heads (half-split pairs d, d + D/2);
    rope_cos, rope_sin fp32 [B,q_cap,D/2].  Returns (q, k, v) like qkv_project."""
    B, q_cap, d_model = x.shape
    assert w.shape == ((Hq + 2 * Hkv) * D, d_model) and rope_cos.shape == (B, q_cap, D // 2) == rope_sin.shape
    q = np.empty((B, Hq, q_cap, D), np.float32)
    k = np.empty((B, Hkv, q_cap, D), np.float32)
    v = np.empty((B, Hkv, q_cap, D), np.float32)
    rc = _load().oracle_qkv_project_rope(B, q_cap, d_model, Hq, Hkv, D, _p(x, np.float32), _p(w, np.float32),
                                         _p(bias, np.float32), _p(rope_cos, np.float32), _p(rope_sin, np.float32),
                                         _p(q, np.float32), _p(k, np.float32), _p(v, np.float32))
    assert rc == 0, rc
    return q, k, v


def out_project(o, wo, bias):
    """o fp32 [B,Hq,q_cap,D], wo fp32 [d_model, Hq*D], bias fp32 [d_model] or None.  Returns y fp32 [B,q_cap,d_model]."""
    B, Hq, q_cap, D = o.shape
    d_model = wo.shape[0]
    assert wo.shape == (d_model, Hq * D)
    y = np.empty((B, q_cap, d_model), np.float32)
    rc = _load().oracle_out_project(B, q_cap, d_model, Hq, D, _p(o, np.float32), _p(wo, np.float32), _p(bias, np.float32),
                                    _p(y, np.float32))
    assert rc == 0, rc
    return y
