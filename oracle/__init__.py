"""fp64 CPU oracle for the Finch score / select / compact path -- TEST INFRASTRUCTURE.

Thin ctypes loader around ``finch_oracle.c`` (plain C, built with gcc on first
use).  Nothing in the product imports this package: only the tests, the smoke
check and the benchmark's CPU-baseline leg do.  It imports nothing from the
CUDA package and shares no code with it.

All arrays are dense numpy arrays in the packed layouts the C file documents.
Floating inputs are passed as their storage bit patterns: ``np.float32`` for
dtype "f32", ``np.uint16`` (bfloat16 bits) for dtype "bf16".
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "finch_oracle.c"
_LIB = _HERE / "libfinch_oracle.so"
_lib = None

DTYPES = {"f32": 0, "bf16": 1}


def build(force: bool = False) -> Path:
    """Compile finch_oracle.c into a shared library beside it (gcc, -O2, OpenMP)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-fno-fast-math",
             "-o", str(tmp), str(_SRC), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(str(build()))
        _lib.finch_oracle_max_threads.restype = ctypes.c_int
        for name in ("finch_oracle_score", "finch_oracle_select_unit", "finch_oracle_select",
                     "finch_oracle_compact", "finch_oracle_step"):
            getattr(_lib, name).restype = ctypes.c_int
    return _lib


def max_threads() -> int:
    return int(lib().finch_oracle_max_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a


def _check_storage(a, dtype):
    want = np.float32 if dtype == "f32" else np.uint16
    if a.dtype != want or not a.flags["C_CONTIGUOUS"]:
        raise TypeError(f"expected contiguous {want} storage for dtype {dtype}, got {a.dtype}")


def score(dtype, q, cache_k, chunk_k, *, n_q_heads, n_kv_heads, head_dim, group_mode=0, scale=None,
          q_off, chunk_off, cache_off, cache_len, apply_norm=False, want_lse=False, threads=1,
          prompt_self_lse=None, row_limit=None, row_norm=False):
    """A^agg for every (layer, group, request): returns scores [L][G][total_cand] fp64
    (and row_lse [L][Hq][total_q] fp64 when want_lse).  prompt_self_lse [L][Hq][total_q] (natural log, -inf = no
    term) adds the prompt's own keys to every row's softmax denominator.  row_limit [total_q] int32: row i attends to
    its request's first row_limit[i] candidates only (causal rows); row_norm scales a row's weights by the fraction of
    the candidates it sees."""
    for a in (q, cache_k, chunk_k):
        _check_storage(a, dtype)
    q_off, chunk_off, cache_off, cache_len = map(_i32, (q_off, chunk_off, cache_off, cache_len))
    batch = len(cache_len)
    L = q.shape[0]
    G = n_kv_heads if group_mode == 0 else 1
    total_cand = int(cache_off[batch]) + int(chunk_off[batch])
    scores = np.zeros((L, G, total_cand), dtype=np.float64)
    lse = np.full((L, n_q_heads, int(q_off[batch])), np.nan, dtype=np.float64) if want_lse else None
    if scale is None:
        scale = 1.0 / np.sqrt(float(head_dim))
    if prompt_self_lse is not None:
        prompt_self_lse = np.ascontiguousarray(prompt_self_lse, dtype=np.float64)
        assert prompt_self_lse.shape == (L, n_q_heads, int(q_off[batch]))
    rc = lib().finch_oracle_score(
        ctypes.c_int(DTYPES[dtype]), _p(q), _p(cache_k), _p(chunk_k),
        ctypes.c_int(L), ctypes.c_int(n_q_heads), ctypes.c_int(n_kv_heads), ctypes.c_int(head_dim),
        ctypes.c_int(group_mode), ctypes.c_double(scale), ctypes.c_int(batch),
        _p(q_off), _p(chunk_off), _p(cache_off), _p(cache_len), ctypes.c_int(int(apply_norm)),
        _p(prompt_self_lse), _p(None if row_limit is None else _i32(row_limit)), ctypes.c_int(int(row_norm)),
        _p(scores), _p(lse), ctypes.c_int(threads))
    if rc:
        raise ValueError(f"finch_oracle_score rc={rc}")
    return (scores, lse) if want_lse else scores


def select_unit(scores, r, rank_order=False):
    """top-r of one score vector (fp64): candidate indices, ascending unless rank_order."""
    s = np.ascontiguousarray(scores, dtype=np.float64)
    kept = np.zeros(max(min(int(r), len(s)), 0), dtype=np.int32)
    n = lib().finch_oracle_select_unit(_p(s), ctypes.c_int(len(s)), ctypes.c_int(int(r)),
                                       ctypes.c_int(int(rank_order)), _p(kept) if len(kept) else None)
    assert n == len(kept)
    return kept


def select(scores, *, chunk_off, cache_off, cache_len, budget, rank_order=False):
    """Batched top-r: scores [L][G][total_cand] fp64 -> (kept_idx [L][G][total_cache] int32, out_len [batch])."""
    scores = np.ascontiguousarray(scores, dtype=np.float64)
    chunk_off, cache_off, cache_len, budget = map(_i32, (chunk_off, cache_off, cache_len, budget))
    batch = len(cache_len)
    L, G = scores.shape[:2]
    kept = np.full((L, G, int(cache_off[batch])), -1, dtype=np.int32)
    out_len = np.zeros(batch, dtype=np.int32)
    rc = lib().finch_oracle_select(_p(scores), ctypes.c_int(L), ctypes.c_int(G), ctypes.c_int(batch),
                                   _p(chunk_off), _p(cache_off), _p(cache_len), _p(budget),
                                   ctypes.c_int(int(rank_order)), _p(kept), _p(out_len))
    if rc:
        raise ValueError(f"finch_oracle_select rc={rc}")
    return kept, out_len


def compact(dtype, kept_idx, out_len, cache_k, cache_v, cache_pos, chunk_k, chunk_v, chunk_pos, *,
            n_kv_heads, head_dim, group_mode=0, chunk_off, cache_off, cache_len, rope_theta=0.0, rope_pairing=0):
    """Gather kept rows: returns (out_k, out_v, out_pos) in the cache's packed layout.  rope_theta > 0 re-rotates the
    K rows from their candidate index to their output slot (pairing 0: coordinates (t, t + d/2); 1: (2t, 2t + 1))."""
    for a in (cache_k, cache_v, chunk_k, chunk_v):
        _check_storage(a, dtype)
    chunk_off, cache_off, cache_len = map(_i32, (chunk_off, cache_off, cache_len))
    kept_idx, out_len, cache_pos, chunk_pos = map(_i32, (kept_idx, out_len, cache_pos, chunk_pos))
    batch = len(cache_len)
    L = cache_k.shape[0]
    out_k = np.zeros_like(cache_k)
    out_v = np.zeros_like(cache_v)
    out_pos = np.full(kept_idx.shape, -1, dtype=np.int32)
    rc = lib().finch_oracle_compact(
        ctypes.c_int(DTYPES[dtype]), _p(kept_idx), _p(out_len), _p(cache_k), _p(cache_v), _p(cache_pos),
        _p(chunk_k), _p(chunk_v), _p(chunk_pos), ctypes.c_int(L), ctypes.c_int(n_kv_heads),
        ctypes.c_int(head_dim), ctypes.c_int(group_mode), ctypes.c_int(batch),
        _p(chunk_off), _p(cache_off), _p(cache_len), ctypes.c_double(rope_theta), ctypes.c_int(rope_pairing),
        _p(out_k), _p(out_v), _p(out_pos))
    if rc:
        raise ValueError(f"finch_oracle_compact rc={rc}")
    return out_k, out_v, out_pos


def step(dtype, q, cache_k, cache_v, cache_pos, chunk_k, chunk_v, chunk_pos, *, n_q_heads, n_kv_heads, head_dim,
         group_mode=0, scale=None, q_off, chunk_off, cache_off, cache_len, budget, threads=1):
    """score -> select -> compact in one C call.  Returns a dict with out_k, out_v, out_pos,
    kept_idx, out_len and the fp64 scores."""
    for a in (q, cache_k, cache_v, chunk_k, chunk_v):
        _check_storage(a, dtype)
    q_off, chunk_off, cache_off, cache_len, budget = map(_i32, (q_off, chunk_off, cache_off, cache_len, budget))
    cache_pos, chunk_pos = _i32(cache_pos), _i32(chunk_pos)
    batch = len(cache_len)
    L = q.shape[0]
    G = n_kv_heads if group_mode == 0 else 1
    total_cache = int(cache_off[batch])
    total_cand = total_cache + int(chunk_off[batch])
    scores = np.zeros((L, G, total_cand), dtype=np.float64)
    out_k = np.zeros_like(cache_k)
    out_v = np.zeros_like(cache_v)
    out_pos = np.full((L, G, total_cache), -1, dtype=np.int32)
    kept = np.full((L, G, total_cache), -1, dtype=np.int32)
    out_len = np.zeros(batch, dtype=np.int32)
    if scale is None:
        scale = 1.0 / np.sqrt(float(head_dim))
    rc = lib().finch_oracle_step(
        ctypes.c_int(DTYPES[dtype]), _p(q), _p(cache_k), _p(cache_v), _p(cache_pos), _p(chunk_k), _p(chunk_v),
        _p(chunk_pos), ctypes.c_int(L), ctypes.c_int(n_q_heads), ctypes.c_int(n_kv_heads), ctypes.c_int(head_dim),
        ctypes.c_int(group_mode), ctypes.c_double(scale), ctypes.c_int(batch), _p(q_off), _p(chunk_off),
        _p(cache_off), _p(cache_len), _p(budget), _p(out_k), _p(out_v), _p(out_pos), _p(kept), _p(out_len),
        _p(scores), ctypes.c_int(threads))
    if rc:
        raise ValueError(f"finch_oracle_step rc={rc}")
    return dict(out_k=out_k, out_v=out_v, out_pos=out_pos, kept_idx=kept, out_len=out_len, scores=scores)
