"""ctypes front-end of the CPU oracle (``spec_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this package, and this package imports nothing from them.

All arrays are numpy; bf16 tensors are passed as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "spec_oracle.c")
_LIB = os.path.join(_DIR, "liboracle.so")
_lib = None

SUM, MAX = 0, 1          # reduction over query rows / over layers and heads
POOL_MAX, POOL_AVG, POOL_AVG_THEN_MAX = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP over independent (sequence, layer, head) units)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i32, i64, dbl, vp = ctypes.c_int, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.oracle_threads.restype = i32
        lib.oracle_spec_score.restype = i32
        lib.oracle_spec_score.argtypes = [vp, vp, i64, i64, i64, i32, vp, i32, i32, i32, i32, i32, i32,
                                          dbl, vp, i32, i32, i64, vp]
        lib.oracle_pool.restype = i32
        lib.oracle_pool.argtypes = [vp, i32, i32, i32, vp]
        lib.oracle_pool_topk.restype = i32
        lib.oracle_pool_topk.argtypes = [vp, i32, vp, i32, i32, i64, i32, i32, i32, i32, vp, vp, vp, vp]
        lib.oracle_compact.restype = i32
        lib.oracle_compact.argtypes = [vp, i64, i64, i64, i32, vp, i32, i32, i32, vp, i32, vp, vp, i32, i32]
        lib.oracle_specpc_select.restype = i32
        lib.oracle_specpc_select.argtypes = [vp, i32, vp, i32, i32, i64, i32, i32, i32, i32, i32, i32,
                                             vp, i32, vp, vp, vp]
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().oracle_threads())


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _cu(cu: Sequence[int]) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(cu, dtype=np.int32))


def spec_score(q: np.ndarray, k: np.ndarray, cu: Sequence[int], n_lookahead: int, n_window: int,
               scale: float, row_weight: Optional[np.ndarray] = None, mode: int = SUM,
               causal_window: bool = False) -> np.ndarray:
    """q uint16 [n_seq, L, Hq, R, d]; k uint16 [L, Hkv, T, d] -> float64 scores [L, Hkv, T]."""
    assert q.dtype == np.uint16 and k.dtype == np.uint16
    q = np.ascontiguousarray(q)
    k = np.ascontiguousarray(k)
    n_seq, L, Hq, R, d = q.shape
    L2, Hkv, T, d2 = k.shape
    assert L2 == L and d2 == d and R == n_lookahead + n_window
    cu = _cu(cu)
    assert len(cu) == n_seq + 1 and cu[-1] <= T
    rw = None if row_weight is None else np.ascontiguousarray(row_weight, dtype=np.float64)
    out = np.zeros((L, Hkv, T), dtype=np.float64)
    rc = _load().oracle_spec_score(_p(q), _p(k), Hkv * T * d, T * d, d, n_seq, _p(cu), L, Hq, Hkv, d,
                                   n_lookahead, n_window, float(scale), _p(rw), int(mode),
                                   int(bool(causal_window)), T, _p(out))
    if rc != 0:
        raise RuntimeError("oracle_spec_score failed: %d" % rc)
    return out


def pool(s: np.ndarray, k: int, kind: int = POOL_MAX) -> np.ndarray:
    s = np.ascontiguousarray(s, dtype=np.float64)
    out = np.empty_like(s)
    rc = _load().oracle_pool(_p(s), s.shape[0], int(kind), int(k), _p(out))
    if rc != 0:
        raise RuntimeError("oracle_pool failed: %d" % rc)
    return out


def pool_topk(scores: np.ndarray, cu: Sequence[int], pool_kind: int, k: int, c_max: int,
              n_forced_tail: int = 0):
    """scores float64 [L, Hkv, T] -> (idx int32 [n_seq, L, Hkv, c_max], count [n_seq, L, Hkv],
    pooled float64 [L, Hkv, T], thresh float64 [n_seq, L, Hkv])."""
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    L, Hkv, T = scores.shape
    cu = _cu(cu)
    n_seq = len(cu) - 1
    idx = np.empty((n_seq, L, Hkv, c_max), dtype=np.int32)
    cnt = np.empty((n_seq, L, Hkv), dtype=np.int32)
    pooled = np.zeros((L, Hkv, T), dtype=np.float64)
    th = np.empty((n_seq, L, Hkv), dtype=np.float64)
    rc = _load().oracle_pool_topk(_p(scores), n_seq, _p(cu), L, Hkv, T, int(pool_kind), int(k), int(c_max),
                                  int(n_forced_tail), _p(idx), _p(cnt), _p(pooled), _p(th))
    if rc != 0:
        raise RuntimeError("oracle_pool_topk failed: %d" % rc)
    return idx, cnt, pooled, th


def compact(src: np.ndarray, cu: Sequence[int], idx: np.ndarray, block_table: Optional[np.ndarray] = None,
            page_size: int = 0, n_pages: int = 0) -> np.ndarray:
    """src uint16 [L, Hkv, T, d]; idx int32 [n_seq, L, Hkv, c_max] -> compacted uint16 cache."""
    assert src.dtype == np.uint16
    src = np.ascontiguousarray(src)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    L, Hkv, T, d = src.shape
    n_seq, _, _, c_max = idx.shape
    cu = _cu(cu)
    if block_table is None:
        dst = np.full((n_seq, L, Hkv, c_max, d), 0xFFFF, dtype=np.uint16)
        bt = None
    else:
        bt = np.ascontiguousarray(block_table, dtype=np.int32)
        dst = np.full((L, n_pages, Hkv, page_size, d), 0xFFFF, dtype=np.uint16)
    rc = _load().oracle_compact(_p(src), Hkv * T * d, T * d, d, n_seq, _p(cu), L, Hkv, d, _p(idx), c_max,
                                _p(dst), _p(bt), int(page_size), int(n_pages))
    if rc != 0:
        raise RuntimeError("oracle_compact failed: %d" % rc)
    return dst


def gather_tokens(src: np.ndarray, cu: Sequence[int], keep: np.ndarray, n_keep: np.ndarray, out_tokens: int):
    """Prompt compression of the SpecKV-PC cascade (Section 4.3): the rows of the kept tokens of every
    sequence, packed back to back.  src uint16 [L, Hkv, T, d]; keep int32 [n_seq, cap] sequence-local;
    -> (dst uint16 [L, Hkv, out_tokens, d] with untouched rows 0xFFFF, cu_out int32 [n_seq + 1])."""
    assert src.dtype == np.uint16
    L, Hkv, T, d = src.shape
    cu = _cu(cu)
    n_seq = len(cu) - 1
    dst = np.full((L, Hkv, out_tokens, d), 0xFFFF, dtype=np.uint16)
    cu_out = np.zeros(n_seq + 1, dtype=np.int32)
    for s in range(n_seq):
        cu_out[s + 1] = cu_out[s] + int(n_keep[s])
        for c in range(int(n_keep[s])):
            dst[:, :, cu_out[s] + c, :] = src[:, :, cu[s] + int(keep[s, c]), :]
    return dst, cu_out


def specpc_select(scores: np.ndarray, cu: Sequence[int], reduce: int, pool_kind: int, k: int, c_max: int,
                  n_neighbor: int, n_forced_tail: int = 0, keep_capacity: Optional[int] = None):
    """scores float64 [L, Hkv, T] -> (keep int32 [n_seq, cap] (-1 padded), n_keep [n_seq],
    pooled token scores float64 [T], thresh float64 [n_seq])."""
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    L, Hkv, T = scores.shape
    cu = _cu(cu)
    n_seq = len(cu) - 1
    if keep_capacity is None:
        keep_capacity = int(max(1, max(cu[1:] - cu[:-1])))
    keep = np.empty((n_seq, keep_capacity), dtype=np.int32)
    n_keep = np.zeros((n_seq,), dtype=np.int32)
    tok = np.zeros((T,), dtype=np.float64)
    th = np.empty((n_seq,), dtype=np.float64)
    rc = _load().oracle_specpc_select(_p(scores), n_seq, _p(cu), L, Hkv, T, int(reduce), int(pool_kind),
                                      int(k), int(c_max), int(n_neighbor), int(n_forced_tail), _p(keep),
                                      int(keep_capacity), _p(n_keep), _p(tok), _p(th))
    if rc != 0:
        raise RuntimeError("oracle_specpc_select failed: %d" % rc)
    return keep, n_keep, tok, th
