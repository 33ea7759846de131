"""ctypes binding of libdlm.so: argument marshalling only.

Every function has the name and the argument order of its C counterpart in include/dlm.h.
Tensors are torch CUDA tensors (PyTorch is used for device memory and streams only); each
call passes raw device pointers and the current CUDA stream.  There is no fallback: if the
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

DLM_OK = 0
DLM_ERR_NULL, DLM_ERR_SHAPE, DLM_ERR_UNSUPPORTED, DLM_ERR_CAPACITY = -1, -2, -3, -4
DLM_ERR_WORKSPACE, DLM_ERR_CUDA, DLM_ERR_TIMEOUT, DLM_ERR_INDEX, DLM_ERR_DEVICE = -5, -6, -7, -8, -9
DLM_DST_APPEND, DLM_DST_WINDOW = 0, 1


class DlmError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: {dlm_strerror(code)} ({code})")


class dlm_kv_cache(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p), ("cache_len", ctypes.c_void_p),
                ("n_layers", ctypes.c_int32), ("batch", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
                ("capacity", ctypes.c_int32), ("head_dim", ctypes.c_int32)]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libdlm.so (in-tree).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: run `python -m paper_2505_21467_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    L = ctypes.CDLL(path)
    vp, i32, f32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
    L.dlm_create.argtypes = [ctypes.POINTER(vp), i32]
    L.dlm_destroy.argtypes = [vp]
    L.dlm_get_status.argtypes = [vp, vp]
    L.dlm_strerror.argtypes = [i32]
    L.dlm_strerror.restype = ctypes.c_char_p
    L.dlm_selftest_wait_timeout.argtypes = [vp, ctypes.c_uint64, vp]
    L.dlm_selftest_wait_timeout.restype = i32
    L.dlm_selftest_set_wait_limit.argtypes = [vp, ctypes.c_uint64]
    L.dlm_selftest_set_wait_limit.restype = i32
    L.dlm_selftest_set_attn_team_max.argtypes = [vp, ctypes.c_int, ctypes.c_int]
    L.dlm_selftest_set_attn_team_max.restype = i32
    L.dlm_launch_count.argtypes = [vp]
    L.dlm_launch_count.restype = ctypes.c_int64
    L.dlm_kv_cache_commit.argtypes = [vp, ctypes.POINTER(dlm_kv_cache), vp, vp, i32, vp, vp, i32, vp, i32, i32,
                                      i32, i32, vp]
    L.dlm_attn_workspace_bytes.argtypes = [vp, ctypes.POINTER(dlm_kv_cache), i32, i32, i32]
    L.dlm_attn_workspace_bytes.restype = sz
    ip = ctypes.POINTER(ctypes.c_int)
    L.dlm_selftest_attn_schedule.argtypes = [vp, ctypes.POINTER(dlm_kv_cache), i32, i32, i32, i32, ip, ip, ip, ip]
    L.dlm_selftest_attn_schedule.restype = i32
    L.dlm_freecache_attn_step.argtypes = [vp, ctypes.POINTER(dlm_kv_cache), i32, i32, vp, vp, vp, i32, i32,
                                          vp, f32, i32, vp, vp, vp, sz, vp]
    L.dlm_unmask_workspace_bytes.argtypes = [vp, i32, i32, i32]
    L.dlm_unmask_workspace_bytes.restype = sz
    L.dlm_unmask_select.argtypes = [vp, vp, i32, i32, i32, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp]
    L.dlm_unmask_select_static.argtypes = [vp, i32, i32, i32, vp, vp, i32, vp, vp, vp, vp, vp]
    L.dlm_guided_accept.argtypes = [vp, vp, vp, i32, i32, vp, vp, i32, vp, vp, vp, vp]
    L.dlm_guided_accept_topk.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, i32, vp, vp, vp, vp]
    L.dlm_unmask_scored_workspace_bytes.argtypes = [vp, i32, i32, i32]
    L.dlm_unmask_scored_workspace_bytes.restype = sz
    L.dlm_unmask_select_scored.argtypes = [vp, vp, i32, i32, i32, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.dlm_guided_accept_threshold.argtypes = [vp, vp, vp, vp, vp, i32, f32, i32, i32, vp, vp, i32, vp, vp, vp, vp]
    L.dlm_window_proj_workspace_bytes.argtypes = [vp, i32, i32, i32]
    L.dlm_window_proj_workspace_bytes.restype = sz
    L.dlm_window_qkv_project.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, sz, vp]
    L.dlm_window_qkv_project_rope.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp, sz, vp]
    L.dlm_window_qkv_project_stage.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp,
                                               ctypes.POINTER(dlm_kv_cache), i32, vp, sz, vp]
    L.dlm_window_qkv_project_stage.restype = i32
    L.dlm_window_out_project.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, sz, vp]
    for name in ("dlm_unmask_select_scored", "dlm_guided_accept_threshold", "dlm_window_qkv_project", "dlm_window_qkv_project_rope",
                 "dlm_window_out_project"):
        getattr(L, name).restype = i32
    for name in ("dlm_create", "dlm_destroy", "dlm_get_status", "dlm_kv_cache_commit",
                 "dlm_freecache_attn_step", "dlm_unmask_select", "dlm_unmask_select_static", "dlm_guided_accept", "dlm_guided_accept_topk"):
        getattr(L, name).restype = i32
    _lib = L
    return L


def dlm_strerror(code: int) -> str:
    return lib().dlm_strerror(int(code)).decode()


def _check(code, where):
    if code != DLM_OK:
        raise DlmError(code, where)


def _ptr(t, dtype=None):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
        raise TypeError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"expected dtype {dtype}, got {t.dtype}")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def dlm_create(device: int = 0) -> ctypes.c_void_p:
    ctx = ctypes.c_void_p()
    _check(lib().dlm_create(ctypes.byref(ctx), int(device)), "dlm_create")
    return ctx


def dlm_destroy(ctx) -> None:
    _check(lib().dlm_destroy(ctx), "dlm_destroy")


def dlm_get_status(ctx) -> int:
    """Synchronises the current stream; returns (and clears) the first device-side error code."""
    return int(lib().dlm_get_status(ctx, _stream()))


def dlm_launch_count(ctx) -> int:
    return int(lib().dlm_launch_count(ctx))


def make_kv_cache(k: torch.Tensor, v: torch.Tensor, cache_len: torch.Tensor) -> dlm_kv_cache:
    """View of caller-owned tensors: k, v bf16 [NL,B,Hkv,Lcap,D]; cache_len int32 [B]."""
    if k.dtype != torch.bfloat16 or k.shape != v.shape or k.dim() != 5:
        raise TypeError("k and v must be bf16 tensors of the same 5-d shape")
    NL, B, Hkv, Lcap, D = k.shape
    if cache_len.shape != (B,):
        raise TypeError("cache_len must have shape [batch]")
    c = dlm_kv_cache(_ptr(k).value, _ptr(v).value, _ptr(cache_len, torch.int32).value, NL, B, Hkv, Lcap, D)
    c._keepalive = (k, v, cache_len)
    return c


def dlm_kv_cache_commit(ctx, cache, k_new, v_new, src_len, src_idx, dst_pos, dst_mode, n_rows, n_max, advance_len,
                        layer_begin, layer_end) -> None:
    _check(lib().dlm_kv_cache_commit(
        ctx, ctypes.byref(cache), _ptr(k_new, torch.bfloat16), _ptr(v_new, torch.bfloat16), int(src_len),
        _ptr(src_idx, torch.int32), _ptr(dst_pos, torch.int32), int(dst_mode), _ptr(n_rows, torch.int32), int(n_max),
        int(bool(advance_len)), int(layer_begin), int(layer_end), _stream()), "dlm_kv_cache_commit")


def dlm_attn_workspace_bytes(ctx, cache, n_layers_in_call, n_q_heads, q_cap) -> int:
    return int(lib().dlm_attn_workspace_bytes(ctx, ctypes.byref(cache), int(n_layers_in_call), int(n_q_heads),
                                              int(q_cap)))


def dlm_selftest_attn_schedule(ctx, cache, n_layers_in_call, n_q_heads, q_cap, cache_len_hint=0) -> dict:
    g, c, w, r = ctypes.c_int(), ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    _check(lib().dlm_selftest_attn_schedule(ctx, ctypes.byref(cache), int(n_layers_in_call), int(n_q_heads), int(q_cap),
                                            int(cache_len_hint), ctypes.byref(g), ctypes.byref(c), ctypes.byref(w),
                                            ctypes.byref(r)), "dlm_selftest_attn_schedule")
    return {"grid": g.value, "team": c.value, "whole_units": w.value, "chunk_rows": r.value}


def dlm_freecache_attn_step(ctx, cache, layer_begin, layer_end, q, k_new, v_new, n_q_heads, q_cap, q_len,
                            softmax_scale, cache_len_hint, out, lse, workspace) -> None:
    _check(lib().dlm_freecache_attn_step(
        ctx, ctypes.byref(cache), int(layer_begin), int(layer_end), _ptr(q, torch.bfloat16),
        _ptr(k_new, torch.bfloat16), _ptr(v_new, torch.bfloat16), int(n_q_heads), int(q_cap),
        _ptr(q_len, torch.int32), float(softmax_scale), int(cache_len_hint), _ptr(out, torch.bfloat16),
        _ptr(lse, torch.float32), _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
        "dlm_freecache_attn_step")


def dlm_unmask_workspace_bytes(ctx, batch, block_len, vocab) -> int:
    return int(lib().dlm_unmask_workspace_bytes(ctx, int(batch), int(block_len), int(vocab)))


def dlm_unmask_select(ctx, logits, batch, block_len, vocab, masked, tokens, k, tok, conf, sel_idx, n_sel,
                      workspace) -> None:
    _check(lib().dlm_unmask_select(
        ctx, _ptr(logits, torch.float32), int(batch), int(block_len), int(vocab), _ptr(masked, torch.uint8),
        _ptr(tokens, torch.int32), int(k), _ptr(tok, torch.int32), _ptr(conf, torch.float32),
        _ptr(sel_idx, torch.int32), _ptr(n_sel, torch.int32), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _stream()), "dlm_unmask_select")


def dlm_unmask_select_static(logits, batch, block_len, vocab, masked, tokens, k, tok, conf, sel_idx, n_sel) -> None:
    """dlm_unmask_select without a context or a workspace (scratch is a fixed array inside the library)."""
    _check(lib().dlm_unmask_select_static(
        _ptr(logits, torch.float32), int(batch), int(block_len), int(vocab), _ptr(masked, torch.uint8),
        _ptr(tokens, torch.int32), int(k), _ptr(tok, torch.int32), _ptr(conf, torch.float32),
        _ptr(sel_idx, torch.int32), _ptr(n_sel, torch.int32), _stream()), "dlm_unmask_select_static")


def dlm_guided_accept(ctx, tok_dlm, tok_ar, batch, block_len, masked, tokens, fallback_source, accept,
                      acc_idx, n_acc) -> None:
    _check(lib().dlm_guided_accept(
        ctx, _ptr(tok_dlm, torch.int32), _ptr(tok_ar, torch.int32), int(batch), int(block_len),
        _ptr(masked, torch.uint8), _ptr(tokens, torch.int32), int(fallback_source), _ptr(accept, torch.uint8),
        _ptr(acc_idx, torch.int32), _ptr(n_acc, torch.int32), _stream()), "dlm_guided_accept")


def dlm_guided_accept_topk(ctx, tok_dlm, tok_ar_topk, top_k, batch, block_len, masked, tokens, fallback_source, accept,
                           acc_idx, n_acc) -> None:
    _check(lib().dlm_guided_accept_topk(
        ctx, _ptr(tok_dlm, torch.int32), _ptr(tok_ar_topk, torch.int32), int(top_k), int(batch), int(block_len),
        _ptr(masked, torch.uint8), _ptr(tokens, torch.int32), int(fallback_source), _ptr(accept, torch.uint8),
        _ptr(acc_idx, torch.int32), _ptr(n_acc, torch.int32), _stream()), "dlm_guided_accept_topk")


DLM_SCORE_CONFIDENCE, DLM_SCORE_NEG_ENTROPY, DLM_SCORE_MARGIN, DLM_SCORE_LOG_CONF_PLUS_NOISE = 0, 1, 2, 3


def dlm_unmask_scored_workspace_bytes(ctx, batch, block_len, vocab) -> int:
    return int(lib().dlm_unmask_scored_workspace_bytes(ctx, int(batch), int(block_len), int(vocab)))


def dlm_unmask_select_scored(ctx, logits, batch, block_len, vocab, masked, tokens, k, score_kind, noise, tok, conf, score,
                             zmax, sel_idx, n_sel, workspace) -> None:
    _check(lib().dlm_unmask_select_scored(
        ctx, _ptr(logits, torch.float32), int(batch), int(block_len), int(vocab), _ptr(masked, torch.uint8),
        _ptr(tokens, torch.int32), int(k), int(score_kind), _ptr(noise, torch.float32), _ptr(tok, torch.int32),
        _ptr(conf, torch.float32), _ptr(score, torch.float32), _ptr(zmax, torch.float32), _ptr(sel_idx, torch.int32),
        _ptr(n_sel, torch.int32), _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
        "dlm_unmask_select_scored")


def dlm_guided_accept_threshold(ctx, tok_dlm, zmax_dlm, tok_ar_topk, logit_ar_topk, top_k, tau, batch, block_len, masked,
                                tokens, fallback_source, accept, acc_idx, n_acc) -> None:
    _check(lib().dlm_guided_accept_threshold(
        ctx, _ptr(tok_dlm, torch.int32), _ptr(zmax_dlm, torch.float32), _ptr(tok_ar_topk, torch.int32),
        _ptr(logit_ar_topk, torch.float32), int(top_k), float(tau), int(batch), int(block_len), _ptr(masked, torch.uint8),
        _ptr(tokens, torch.int32), int(fallback_source), _ptr(accept, torch.uint8), _ptr(acc_idx, torch.int32),
        _ptr(n_acc, torch.int32), _stream()), "dlm_guided_accept_threshold")


def dlm_window_proj_workspace_bytes(ctx, rows, n_out, k_total) -> int:
    return int(lib().dlm_window_proj_workspace_bytes(ctx, int(rows), int(n_out), int(k_total)))


def dlm_window_qkv_project(ctx, x, w, bias, batch, q_cap, d_model, n_q_heads, n_kv_heads, head_dim, q_out, k_out, v_out,
                           workspace) -> None:
    _check(lib().dlm_window_qkv_project(
        ctx, _ptr(x, torch.bfloat16), _ptr(w, torch.bfloat16), _ptr(bias, torch.bfloat16), int(batch), int(q_cap), int(d_model),
        int(n_q_heads), int(n_kv_heads), int(head_dim), _ptr(q_out, torch.bfloat16), _ptr(k_out, torch.bfloat16),
        _ptr(v_out, torch.bfloat16), _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
        "dlm_window_qkv_project")


def dlm_window_qkv_project_rope(ctx, x, w, bias, rope_cos, rope_sin, batch, q_cap, d_model, n_q_heads, n_kv_heads, head_dim,
                                q_out, k_out, v_out, workspace) -> None:
    _check(lib().dlm_window_qkv_project_rope(
        ctx, _ptr(x, torch.bfloat16), _ptr(w, torch.bfloat16), _ptr(bias, torch.bfloat16), _ptr(rope_cos, torch.float32),
        _ptr(rope_sin, torch.float32), int(batch), int(q_cap), int(d_model), int(n_q_heads), int(n_kv_heads), int(head_dim),
        _ptr(q_out, torch.bfloat16), _ptr(k_out, torch.bfloat16), _ptr(v_out, torch.bfloat16), _ptr(workspace),
        workspace.numel() * workspace.element_size(), _stream()), "dlm_window_qkv_project_rope")


def dlm_window_qkv_project_stage(ctx, x, w, bias, rope_cos, rope_sin, batch, q_cap, d_model, n_q_heads, n_kv_heads, head_dim,
                                 q_len, q_out, k_out, v_out, cache, layer, workspace) -> None:
    _check(lib().dlm_window_qkv_project_stage(
        ctx, _ptr(x, torch.bfloat16), _ptr(w, torch.bfloat16), _ptr(bias, torch.bfloat16), _ptr(rope_cos, torch.float32),
        _ptr(rope_sin, torch.float32), int(batch), int(q_cap), int(d_model), int(n_q_heads), int(n_kv_heads), int(head_dim),
        _ptr(q_len, torch.int32), _ptr(q_out, torch.bfloat16), _ptr(k_out, torch.bfloat16), _ptr(v_out, torch.bfloat16),
        ctypes.byref(cache), int(layer), _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
        "dlm_window_qkv_project_stage")


def dlm_window_out_project(ctx, o, wo, bias, batch, q_cap, d_model, n_q_heads, head_dim, y, workspace) -> None:
    _check(lib().dlm_window_out_project(
        ctx, _ptr(o, torch.bfloat16), _ptr(wo, torch.bfloat16), _ptr(bias, torch.bfloat16), int(batch), int(q_cap), int(d_model),
        int(n_q_heads), int(head_dim), _ptr(y, torch.bfloat16), _ptr(workspace), workspace.numel() * workspace.element_size(),
        _stream()), "dlm_window_out_project")


def dlm_selftest_set_wait_limit(ctx, limit_ns: int) -> None:
    _check(lib().dlm_selftest_set_wait_limit(ctx, ctypes.c_uint64(int(limit_ns))), "dlm_selftest_set_wait_limit")


def dlm_selftest_set_attn_team_max(ctx, max_blocks: int, force: bool = False) -> None:
    _check(lib().dlm_selftest_set_attn_team_max(ctx, int(max_blocks), int(force)), "dlm_selftest_set_attn_team_max")


def dlm_selftest_wait_timeout(ctx, limit_ns: int) -> None:
    _check(lib().dlm_selftest_wait_timeout(ctx, ctypes.c_uint64(int(limit_ns)), _stream()), "dlm_selftest_wait_timeout")
