"""Thin ctypes binding of libspec.so: the same entry points as include/spec.h, taking torch
CUDA tensors.  It only marshals arguments (pointers, sizes, the current stream); every step of
the path runs in the library's kernels.  There is no fallback: a missing library raises."""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

from . import build as _build

SPEC_OK = 0
ERR_BAD_ARG, ERR_ALIGNMENT, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = -1, -2, -3, -4, -5, -6
REDUCE_SUM, REDUCE_MAX = 0, 1
POOL_MAX, POOL_AVG, POOL_AVG_THEN_MAX = 0, 1, 2

EXPORTS = ("spec_workspace_bytes", "spec_last_error", "spec_score", "spec_pool_topk", "spec_pool_topk_vert",
           "spec_compact_kv", "specpc_token_select", "spec_gather_tokens", "specpc_token_select_static")
STATIC_MAX_TOKENS = 262144


class SpecError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__("spec error %d: %s" % (code, message))
        self.code = code


class spec_problem(ctypes.Structure):
    _fields_ = [
        ("n_seq", ctypes.c_int32), ("cu_seqlens", ctypes.c_void_p), ("n_in", ctypes.c_int32),
        ("total_tokens", ctypes.c_int32), ("n_layers", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("n_lookahead", ctypes.c_int32),
        ("n_window", ctypes.c_int32), ("softmax_scale", ctypes.c_float),
        ("k_stride_layer", ctypes.c_int64), ("k_stride_head", ctypes.c_int64), ("k_stride_token", ctypes.c_int64),
        ("v_stride_layer", ctypes.c_int64), ("v_stride_head", ctypes.c_int64), ("v_stride_token", ctypes.c_int64),
    ]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libspec.so (built in-tree by build.py).  Raises if it is missing."""
    global _lib
    if _lib is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            raise RuntimeError("%s is missing: run `python -m paper_2506_08373_b200.build` (needs nvcc); "
                               "there is no fallback path" % path)
        L = ctypes.CDLL(path)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        pp = ctypes.POINTER(spec_problem)
        L.spec_workspace_bytes.restype = sz
        L.spec_workspace_bytes.argtypes = [pp]
        L.spec_last_error.restype = ctypes.c_char_p
        L.spec_last_error.argtypes = []
        L.spec_score.restype = i32
        L.spec_score.argtypes = [pp, vp, vp, vp, i32, i32, vp, vp, sz, vp, vp]
        L.spec_pool_topk.restype = i32
        L.spec_pool_topk.argtypes = [pp, vp, i32, i32, i32, i32, vp, vp, vp, sz, vp, vp]
        L.spec_pool_topk_vert.restype = i32
        L.spec_pool_topk_vert.argtypes = [pp, vp, i32, i32, i32, i32, vp, vp, i32, vp, vp, vp, sz, vp, vp]
        L.spec_compact_kv.restype = i32
        L.spec_compact_kv.argtypes = [pp, vp, vp, vp, i32, vp, vp, vp, i32, i32, vp, vp]
        L.specpc_token_select.restype = i32
        L.specpc_token_select.argtypes = [pp, vp, i32, i32, i32, i32, i32, i32, vp, i32, vp, vp, sz, vp, vp]
        L.spec_gather_tokens.restype = i32
        L.spec_gather_tokens.argtypes = [pp, vp, vp, vp, i32, vp, vp, vp, i32, vp, vp, vp]
        L.specpc_token_select_static.restype = i32
        L.specpc_token_select_static.argtypes = [pp, vp, i32, i32, i32, i32, i32, i32, vp, i32, vp, vp, vp]
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc: int):
    if rc != SPEC_OK:
        raise SpecError(rc, lib().spec_last_error().decode())


def make_problem(*, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, n_lookahead: int,
                 n_window: int, softmax_scale: float, total_tokens: int, n_in: int = 0, n_seq: int = 1,
                 cu_seqlens: Optional[torch.Tensor] = None, k: Optional[torch.Tensor] = None,
                 v: Optional[torch.Tensor] = None) -> spec_problem:
    """Fills a spec_problem.  k / v, when given, are [n_layers, n_kv_heads, T, head_dim] views (any
    strides with a contiguous last axis) from which the strides are taken."""
    p = spec_problem()
    p.n_seq = n_seq
    p.cu_seqlens = None if cu_seqlens is None else cu_seqlens.data_ptr()
    p._keepalive = cu_seqlens            # the struct only holds the address: keep the tensor alive with it
    p.n_in = n_in
    p.total_tokens = total_tokens
    p.n_layers, p.n_q_heads, p.n_kv_heads, p.head_dim = n_layers, n_q_heads, n_kv_heads, head_dim
    p.n_lookahead, p.n_window = n_lookahead, n_window
    p.softmax_scale = softmax_scale
    dflt = (n_kv_heads * total_tokens * head_dim, total_tokens * head_dim, head_dim)
    for name, t in (("k", k), ("v", v)):
        st = dflt
        if t is not None:
            assert t.dim() == 4 and t.stride(3) == 1
            st = (t.stride(0), t.stride(1), t.stride(2))
        setattr(p, name + "_stride_layer", st[0])
        setattr(p, name + "_stride_head", st[1])
        setattr(p, name + "_stride_token", st[2])
    return p


def spec_workspace_bytes(problem: spec_problem) -> int:
    return int(lib().spec_workspace_bytes(ctypes.byref(problem)))


def spec_last_error() -> str:
    return lib().spec_last_error().decode()


def spec_score(problem, q, k, scores_out, workspace, row_weight=None, reduce=REDUCE_SUM, causal_window=0,
               status_word=None):
    _check(lib().spec_score(ctypes.byref(problem), _ptr(q), _ptr(k), _ptr(row_weight), reduce, causal_window,
                            _ptr(scores_out), _ptr(workspace), workspace.numel() * workspace.element_size(),
                            _ptr(status_word), _stream()))


def spec_pool_topk(problem, scores, pool, pool_k, c_max, n_forced_tail, idx_out, count_out=None,
                   workspace=None, status_word=None):
    wsb = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().spec_pool_topk(ctypes.byref(problem), _ptr(scores), pool, pool_k, c_max, n_forced_tail,
                                _ptr(idx_out), _ptr(count_out), _ptr(workspace), wsb, _ptr(status_word), _stream()))


def spec_pool_topk_vert(problem, scores, pool, pool_k, c_max, n_forced_tail, idx_out, count_out, n_vert,
                        vert_idx_out, vert_count_out=None, workspace=None, status_word=None):
    wsb = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().spec_pool_topk_vert(ctypes.byref(problem), _ptr(scores), pool, pool_k, c_max, n_forced_tail,
                                     _ptr(idx_out), _ptr(count_out), n_vert, _ptr(vert_idx_out), _ptr(vert_count_out),
                                     _ptr(workspace), wsb, _ptr(status_word), _stream()))


def spec_compact_kv(problem, k, v, idx, c_max, k_out, v_out, block_table=None, page_size=0, n_pages=0,
                    status_word=None):
    _check(lib().spec_compact_kv(ctypes.byref(problem), _ptr(k), _ptr(v), _ptr(idx), c_max, _ptr(k_out),
                                 _ptr(v_out), _ptr(block_table), page_size, n_pages, _ptr(status_word), _stream()))


def specpc_token_select(problem, scores, layer_head_reduce, pool, pool_k, c_max, n_neighbor, n_forced_tail,
                        keep_out, keep_capacity, n_keep_out, workspace, status_word=None):
    _check(lib().specpc_token_select(ctypes.byref(problem), _ptr(scores), layer_head_reduce, pool, pool_k, c_max,
                                     n_neighbor, n_forced_tail, _ptr(keep_out), keep_capacity, _ptr(n_keep_out),
                                     _ptr(workspace), workspace.numel() * workspace.element_size(),
                                     _ptr(status_word), _stream()))


def spec_gather_tokens(problem, k, v, keep, keep_capacity, n_keep, k_out, v_out, out_tokens, cu_seqlens_out,
                       status_word=None):
    _check(lib().spec_gather_tokens(ctypes.byref(problem), _ptr(k), _ptr(v), _ptr(keep), keep_capacity, _ptr(n_keep),
                                    _ptr(k_out), _ptr(v_out), out_tokens, _ptr(cu_seqlens_out), _ptr(status_word),
                                    _stream()))


def specpc_token_select_static(problem, scores, layer_head_reduce, pool, pool_k, c_max, n_neighbor, n_forced_tail,
                               keep_out, keep_capacity, n_keep_out, status_word=None):
    """specpc_token_select without a workspace argument, for callers that cannot allocate device
    memory: the token-score scratch is an array inside the library (at most STATIC_MAX_TOKENS
    packed tokens).  Calls that overlap on the GPU race on that array."""
    _check(lib().specpc_token_select_static(ctypes.byref(problem), _ptr(scores), layer_head_reduce, pool, pool_k,
                                            c_max, n_neighbor, n_forced_tail, _ptr(keep_out), keep_capacity,
                                            _ptr(n_keep_out), _ptr(status_word), _stream()))
