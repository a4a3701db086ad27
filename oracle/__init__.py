"""ctypes wrapper around the fp64 CPU oracle (``fedattn_oracle.c``).

TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT PATH.  Only the tests, the smoke
check and the benchmark's cpu_baseline / reference legs import this package; the
CUDA package never does, and this package never imports the CUDA package.

The wrapper only marshals numpy arrays (converted exactly to float64) into the C
functions; the arithmetic lives in the C file, where each function cites the
passage of the paper it follows.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fedattn_oracle.c")
_LIB = os.path.join(_HERE, "libfedattn_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-ffp-contract=off", "-fPIC",
                               "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB)
        _lib.fedattn_oracle_threads.restype = C.c_int
    return _lib


def threads() -> int:
    return int(_load().fedattn_oracle_threads())


def _f64(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x), dtype=np.float64)


def _i32(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x), dtype=np.int32)


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _scale(scale, d) -> float:
    return float(scale) if scale else 1.0 / float(np.sqrt(np.float64(d)))


def offsets(seqlens) -> np.ndarray:
    s = _i32(seqlens)
    off = np.zeros(len(s) + 1, dtype=np.int32)
    _load().fedattn_oracle_offsets(_p(s), C.c_int32(len(s)), _p(off))
    return off


def local(q, k, v, seqlens, scale: float = 0.0, causal: bool = True,
          rows: Optional[Sequence[int]] = None):
    """Per-participant attention over packed Q [L,Hq,d], K/V [L,Hkv,d].
    Returns (o [R,Hq,d], lse [R,Hq]) for the listed rows (all rows when ``rows`` is None)."""
    q, k, v = _f64(q), _f64(k), _f64(v)
    L, hq, d = q.shape
    hkv = k.shape[1]
    off = offsets(seqlens)
    assert off[-1] == L and k.shape == (L, hkv, d) and v.shape == k.shape and hq % hkv == 0
    r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n_rows = L if r is None else len(r)
    o = np.zeros((n_rows, hq, d), dtype=np.float64)
    lse = np.zeros((n_rows, hq), dtype=np.float64)
    _load().fedattn_oracle_local(_p(q), _p(k), _p(v), _p(off), C.c_int32(len(off) - 1),
                                 C.c_int32(hq), C.c_int32(hkv), C.c_int32(d),
                                 C.c_double(_scale(scale, d)), C.c_int32(int(causal)),
                                 _p(r), C.c_int64(n_rows), _p(o), _p(lse))
    return o, lse


def _ptr_array(parts):
    arr = (C.c_void_p * len(parts))()
    for i, p in enumerate(parts):
        arr[i] = p.ctypes.data
    return arr


def aggregate_concat(k_parts, v_parts):
    """Dense aggregation: returns (k_agg [L,Hkv,d], v_agg, kv_pos [L], cu_kv [N+1])."""
    k_parts = [_f64(x) for x in k_parts]
    v_parts = [_f64(x) for x in v_parts]
    seqlens = _i32([x.shape[0] for x in k_parts])
    hkv, d = k_parts[0].shape[1:]
    L = int(seqlens.sum())
    k_agg = np.zeros((L, hkv, d)); v_agg = np.zeros((L, hkv, d))
    kv_pos = np.zeros(L, dtype=np.int32); cu_kv = np.zeros(len(seqlens) + 1, dtype=np.int32)
    _load().fedattn_oracle_aggregate_concat(_ptr_array(k_parts), _ptr_array(v_parts), _p(seqlens),
                                            C.c_int32(len(seqlens)), C.c_int32(hkv), C.c_int32(d),
                                            _p(k_agg), _p(v_agg), _p(kv_pos), _p(cu_kv))
    return k_agg, v_agg, kv_pos, cu_kv


def topk_knorm(k_part, k_sel: int, return_scores: bool = False):
    """Per-KV-head top ``k_sel`` token indices of one participant by squared key norm,
    ascending.  Returns sel_idx [Hkv, k_sel] (and scores [Hkv, L_n])."""
    k_part = _f64(k_part)
    ln, hkv, d = k_part.shape
    assert 0 <= k_sel <= ln
    sel = np.zeros((hkv, k_sel), dtype=np.int32)
    scores = np.zeros((hkv, ln), dtype=np.float64)
    _load().fedattn_oracle_topk_knorm(_p(k_part), C.c_int32(ln), C.c_int32(hkv), C.c_int32(d),
                                      C.c_int32(k_sel), _p(sel), _p(scores))
    return (sel, scores) if return_scores else sel


def aggregate_indexed(k_parts, v_parts, k_sel, sel_idx):
    """Sparse aggregation with given per-head local indices sel_idx [Hkv, sum k_sel].
    Returns (k_agg [Hkv,T,d], v_agg, kv_pos [Hkv,T], cu_kv [N+1])."""
    k_parts = [_f64(x) for x in k_parts]
    v_parts = [_f64(x) for x in v_parts]
    seqlens = _i32([x.shape[0] for x in k_parts])
    k_sel = _i32(k_sel)
    sel_idx = _i32(sel_idx)
    hkv, d = k_parts[0].shape[1:]
    T = int(k_sel.sum())
    assert sel_idx.shape == (hkv, T)
    k_agg = np.zeros((hkv, T, d)); v_agg = np.zeros((hkv, T, d))
    kv_pos = np.zeros((hkv, T), dtype=np.int32); cu_kv = np.zeros(len(seqlens) + 1, dtype=np.int32)
    _load().fedattn_oracle_aggregate_indexed(_ptr_array(k_parts), _ptr_array(v_parts), _p(seqlens),
                                             _p(k_sel), C.c_int32(len(seqlens)), C.c_int32(hkv),
                                             C.c_int32(d), _p(sel_idx), _p(k_agg), _p(v_agg),
                                             _p(kv_pos), _p(cu_kv))
    return k_agg, v_agg, kv_pos, cu_kv


def aggregate_topk(k_parts, v_parts, k_sel):
    """Sparse aggregation with the key-norm top-k selector.
    Returns (k_agg, v_agg, kv_pos, cu_kv, sel_idx [Hkv, sum k_sel])."""
    k_sel = _i32(k_sel)
    sels = [topk_knorm(kp, int(ks)) for kp, ks in zip(k_parts, k_sel)]
    hkv = np.asarray(k_parts[0]).shape[1]
    sel_idx = np.concatenate(sels, axis=1) if sels else np.zeros((hkv, 0), np.int32)
    return aggregate_indexed(k_parts, v_parts, k_sel, sel_idx) + (sel_idx,)


def aggregate_topk_token(k_parts, v_parts, k_sel):
    """Sparse aggregation with token-level selection (the selection matrix of the paper's adaptive
    aggregation picks whole tokens): one score per token, the squared norm of its whole key row
    [Hkv * d] accumulated in fp64 in memory order, same order and tie rule as the per-head selector;
    every KV head keeps the same tokens.  The definition is the per-head one applied to the row
    viewed as a single head.  Returns (k_agg [T,Hkv,d], v_agg, kv_pos [T], cu_kv [N+1], sel_idx [T])."""
    k_parts = [_f64(x) for x in k_parts]
    v_parts = [_f64(x) for x in v_parts]
    hkv, d = k_parts[0].shape[1:]
    flat_k = [x.reshape(x.shape[0], 1, hkv * d) for x in k_parts]
    flat_v = [x.reshape(x.shape[0], 1, hkv * d) for x in v_parts]
    k_agg, v_agg, kv_pos, cu_kv, sel = aggregate_topk(flat_k, flat_v, k_sel)
    T = k_agg.shape[1]
    return k_agg.reshape(T, hkv, d), v_agg.reshape(T, hkv, d), kv_pos[0], cu_kv, sel[0]


def sync(q, k_agg, v_agg, kv_pos=None, q_pos=None, kv_head_major: bool = False,
         scale: float = 0.0, causal: bool = True, rows: Optional[Sequence[int]] = None):
    """Global attention of packed queries Q [L,Hq,d] over the aggregated KV
    ([T,Hkv,d] token-major with kv_pos [T], or [Hkv,T,d] head-major with kv_pos [Hkv,T])."""
    q, k_agg, v_agg = _f64(q), _f64(k_agg), _f64(v_agg)
    L, hq, d = q.shape
    if kv_head_major:
        hkv, T, _ = k_agg.shape
        tok_stride, head_stride, pos_stride = d, T * d, T
    else:
        T, hkv, _ = k_agg.shape
        tok_stride, head_stride, pos_stride = hkv * d, d, 0
    kvp = None if kv_pos is None else _i32(kv_pos)
    if kvp is not None:
        assert kvp.shape == ((hkv, T) if kv_head_major else (T,))
    qp = None if q_pos is None else _i32(q_pos)
    r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n_rows = L if r is None else len(r)
    o = np.zeros((n_rows, hq, d)); lse = np.zeros((n_rows, hq))
    _load().fedattn_oracle_sync(_p(q), C.c_int64(L), _p(qp), _p(k_agg), _p(v_agg), C.c_int64(T),
                                C.c_int64(tok_stride), C.c_int64(head_stride), _p(kvp),
                                C.c_int64(pos_stride), C.c_int32(hq), C.c_int32(hkv), C.c_int32(d),
                                C.c_double(_scale(scale, d)), C.c_int32(int(causal)),
                                _p(r), C.c_int64(n_rows), _p(o), _p(lse))
    return o, lse


def sync_exchange(q, k, v, seqlens, k_agg, v_agg, kv_pos, cu_kv, scale: float = 0.0,
                  rows: Optional[Sequence[int]] = None, causal: bool = True):
    """Sync block with sparse KV exchange: every participant attends its own complete segment
    (causally, or all of it when ``causal`` is False) plus the exchanged, sparsified keys of the
    other participants (those not later than the query, or all of them when ``causal`` is False).
    q [L,Hq,d]; k, v [L,Hkv,d] local; k_agg, v_agg [Hkv,T,d] head-major aggregate with
    kv_pos [Hkv,T] and participant ranges cu_kv [N+1]."""
    q, k, v, k_agg, v_agg = _f64(q), _f64(k), _f64(v), _f64(k_agg), _f64(v_agg)
    L, hq, d = q.shape
    hkv, T, _ = k_agg.shape
    off = offsets(seqlens)
    kvp, cu = _i32(kv_pos), _i32(cu_kv)
    assert kvp.shape == (hkv, T) and len(cu) == len(off)
    r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    n_rows = L if r is None else len(r)
    o = np.zeros((n_rows, hq, d)); lse = np.zeros((n_rows, hq))
    _load().fedattn_oracle_sync_exchange(_p(q), _p(k), _p(v), _p(off), C.c_int32(len(off) - 1),
                                         _p(k_agg), _p(v_agg), _p(kvp), _p(cu), C.c_int64(T),
                                         C.c_int32(hq), C.c_int32(hkv), C.c_int32(d),
                                         C.c_double(_scale(scale, d)), C.c_int32(int(causal)), _p(r),
                                         C.c_int64(n_rows), _p(o), _p(lse))
    return o, lse


def decode(q, k_cache, v_cache, kv_len, sync_mode: bool, scale: float = 0.0):
    """Decode step.  LOCAL: caches [N,cap,Hkv,d], kv_len [N].  SYNC: cache [T,Hkv,d], kv_len [1].
    q [N,Hq,d].  Returns (o [N,Hq,d], lse [N,Hq])."""
    q, k_cache, v_cache = _f64(q), _f64(k_cache), _f64(v_cache)
    n, hq, d = q.shape
    kv_len = _i32(kv_len)
    if sync_mode:
        hkv = k_cache.shape[1]
        stride = 0
        assert len(kv_len) == 1
    else:
        hkv = k_cache.shape[2]
        stride = k_cache.shape[1] * hkv * d
        assert len(kv_len) == n
    o = np.zeros((n, hq, d)); lse = np.zeros((n, hq))
    _load().fedattn_oracle_decode(_p(q), _p(k_cache), _p(v_cache), C.c_int64(stride), _p(kv_len),
                                  C.c_int32(int(sync_mode)), C.c_int32(n), C.c_int32(hq),
                                  C.c_int32(hkv), C.c_int32(d), C.c_double(_scale(scale, d)),
                                  _p(o), _p(lse))
    return o, lse
