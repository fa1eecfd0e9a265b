"""ctypes binding of libfinch.so: the same entry points as include/finch.h, taking torch tensors.

Argument marshalling only -- every step of the path runs in the library's CUDA kernels.  torch is used for
device memory and stream handles.  Importing this module never builds anything; loading the library fails
loudly when libfinch.so is missing (build it with ``python -m paper_2408_00167_b200.build``).
"""
from __future__ import annotations

import ctypes as C
from dataclasses import dataclass
from pathlib import Path
from typing import Optional, Sequence

import numpy as np

import os

# FINCH_LIB lets a developer load an alternative build of the library (same ABI) for experiments
_LIB_PATH = Path(os.environ.get("FINCH_LIB") or Path(__file__).resolve().parent / "libfinch.so")
_lib = None

FINCH_OK = 0
FINCH_ERR_INVALID_ARG = 1
FINCH_ERR_UNSUPPORTED = 2
FINCH_ERR_BAD_LAYOUT = 3
FINCH_ERR_WORKSPACE_TOO_SMALL = 4
FINCH_ERR_OOM = 5
FINCH_ERR_CUDA = 6
FINCH_ERR_DEVICE_STATUS = 7
FINCH_F32, FINCH_BF16 = 0, 1
FINCH_GROUP_PER_KV_HEAD, FINCH_GROUP_PER_LAYER = 0, 1
FINCH_DEV_BAD_BATCH, FINCH_DEV_TIMEOUT, FINCH_DEV_BAD_INDEX = 1, 2, 4

EXPORTS = ("finch_ctx_create", "finch_ctx_destroy", "finch_workspace_bytes", "finch_score", "finch_select",
           "finch_compact", "finch_step", "finch_device_status", "finch_launch_count", "finch_status_string", "finch_score_static", "finch_score_static_max_rows", "finch_score_static_path",
           "finch_step_host", "finch_score_plan")


class finch_config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("dtype", C.c_int32), ("group_mode", C.c_int32), ("scale", C.c_float),
                ("max_batch", C.c_int32), ("max_prompt", C.c_int32), ("max_candidates", C.c_int32),
                ("device", C.c_int32), ("rope_theta", C.c_float), ("rope_pairing", C.c_int32)]


class finch_tensor(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("stride_layer", C.c_int64), ("stride_head", C.c_int64),
                ("stride_tok", C.c_int64)]


class finch_batch(C.Structure):
    _fields_ = [("batch", C.c_int32), ("q_off", C.c_void_p), ("chunk_off", C.c_void_p), ("cache_off", C.c_void_p),
                ("cache_len", C.c_void_p), ("budget", C.c_void_p), ("total_q", C.c_int32),
                ("total_chunk", C.c_int32), ("total_cache", C.c_int32), ("max_q", C.c_int32),
                ("max_cache", C.c_int32), ("max_chunk", C.c_int32), ("max_budget", C.c_int32),
                ("prompt_self_lse", C.c_void_p), ("row_limit", C.c_void_p),
                ("row_norm", C.c_int32)]


class FinchError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {finch_status_string(status)} (status {status})")


def load() -> C.CDLL:
    """Load libfinch.so; raises if it has not been built (there is no fallback path)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2408_00167_b200.build`")
        lib = C.CDLL(str(_LIB_PATH))
        for name in EXPORTS:
            getattr(lib, name).restype = C.c_int
        lib.finch_ctx_destroy.restype = None
        lib.finch_status_string.restype = C.c_char_p
        lib.finch_score_static_max_rows.restype = C.c_size_t
        _lib = lib
    return _lib


def finch_status_string(status: int) -> str:
    return load().finch_status_string(C.c_int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != FINCH_OK:
        raise FinchError(status, where)


# ------------------------------------------------------------------ marshalling helpers

def _tensor(t) -> finch_tensor:
    """[L][heads][tokens][d] torch tensor (head_dim contiguous) -> finch_tensor; None -> null view."""
    if t is None:
        return finch_tensor(None, 0, 0, 0)
    if t.dim() != 4 or (t.shape[3] > 1 and t.stride(3) != 1):
        raise ValueError("expected a [layers][heads][tokens][head_dim] tensor with head_dim contiguous")
    ptr = t.data_ptr() if t.numel() else None
    return finch_tensor(ptr, t.stride(0), t.stride(1), t.stride(2))


def _ptr(t) -> Optional[int]:
    return None if t is None or t.numel() == 0 else t.data_ptr()


def _nbytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return stream.cuda_stream or None


@dataclass
class Batch:
    """Device-side batch metadata plus the host bounds finch_batch carries."""
    q_off: object
    chunk_off: object
    cache_off: object
    cache_len: object
    budget: object
    c: finch_batch
    prompt_self_lse: object = None   # keeps the optional device tensors alive
    row_limit: object = None

    @property
    def batch(self) -> int:
        return self.c.batch


def make_batch(q_off: Sequence[int], chunk_off: Sequence[int], cache_off: Sequence[int], cache_len: Sequence[int],
               budget: Sequence[int], device="cuda", prompt_self_lse=None, row_limit=None, row_norm=False) -> Batch:
    """Copy the offset arrays to the device and fill in the host bounds.  prompt_self_lse: optional device tensor
    [n_layers][n_q_heads][total_q] fp32; row_limit: optional device tensor [total_q] int32 (see finch_batch in the
    header)."""
    import torch
    h = [np.ascontiguousarray(a, dtype=np.int32) for a in (q_off, chunk_off, cache_off, cache_len, budget)]
    B = len(h[3])
    assert len(h[0]) == len(h[1]) == len(h[2]) == B + 1 and len(h[4]) == B
    d = [torch.from_numpy(a).to(device) for a in h]

    def diff(a):
        return (a[1:] - a[:-1]) if B else np.zeros(0, np.int32)

    def mx(a):
        return int(a.max()) if len(a) else 0
    n_cand = h[3] + diff(h[1])
    cb = finch_batch(B, *[x.data_ptr() for x in d], int(h[0][B]), int(h[1][B]), int(h[2][B]),
                     mx(diff(h[0])), mx(h[3]), mx(diff(h[1])), mx(np.minimum(h[4], n_cand)) if B else 0,
                     prompt_self_lse.data_ptr() if prompt_self_lse is not None else None,
                     row_limit.data_ptr() if row_limit is not None else None, int(bool(row_norm)))
    return Batch(*d, cb, prompt_self_lse, row_limit)


# ------------------------------------------------------------------ the entry points

def finch_ctx_create(n_layers, n_q_heads, n_kv_heads, head_dim, dtype, group_mode=FINCH_GROUP_PER_KV_HEAD, scale=0.0,
                     max_batch=1, max_prompt=256, max_candidates=8192, device=0, rope_theta=0.0,
                     rope_pairing=0) -> C.c_void_p:
    cfg = finch_config(n_layers, n_q_heads, n_kv_heads, head_dim, dtype, group_mode, scale, max_batch, max_prompt,
                       max_candidates, device, rope_theta, rope_pairing)
    ctx = C.c_void_p()
    _check(load().finch_ctx_create(C.byref(cfg), C.byref(ctx)), "finch_ctx_create")
    return ctx


def finch_ctx_destroy(ctx) -> None:
    if ctx:
        load().finch_ctx_destroy(ctx)


def finch_workspace_bytes(ctx, batch: Batch) -> int:
    out = C.c_size_t()
    _check(load().finch_workspace_bytes(ctx, C.byref(batch.c), C.byref(out)), "finch_workspace_bytes")
    return int(out.value)


def finch_score(ctx, prompt_q, cache_k, chunk_k, batch: Batch, scores, row_lse=None, ws=None, stream=None) -> None:
    q, ck, hk = _tensor(prompt_q), _tensor(cache_k), _tensor(chunk_k)
    _check(load().finch_score(ctx, C.byref(q), C.byref(ck), C.byref(hk), C.byref(batch.c), C.c_void_p(_ptr(scores)),
                              C.c_void_p(_ptr(row_lse)), C.c_void_p(_ptr(ws)), C.c_size_t(_nbytes(ws)),
                              C.c_void_p(_stream(stream))), "finch_score")


def finch_select(ctx, scores, batch: Batch, kept_idx, out_len, ws=None, stream=None) -> None:
    _check(load().finch_select(ctx, C.c_void_p(_ptr(scores)), C.byref(batch.c), C.c_void_p(_ptr(kept_idx)),
                               C.c_void_p(_ptr(out_len)), C.c_void_p(_ptr(ws)), C.c_size_t(_nbytes(ws)),
                               C.c_void_p(_stream(stream))), "finch_select")


def finch_compact(ctx, kept_idx, out_len, cache_k, cache_v, cache_pos, chunk_k, chunk_v, chunk_pos, batch: Batch,
                  out_k, out_v, out_pos, stream=None) -> None:
    ts = [_tensor(t) for t in (cache_k, cache_v, chunk_k, chunk_v, out_k, out_v)]
    _check(load().finch_compact(ctx, C.c_void_p(_ptr(kept_idx)), C.c_void_p(_ptr(out_len)), C.byref(ts[0]),
                                C.byref(ts[1]), C.c_void_p(_ptr(cache_pos)), C.byref(ts[2]), C.byref(ts[3]),
                                C.c_void_p(_ptr(chunk_pos)), C.byref(batch.c), C.byref(ts[4]), C.byref(ts[5]),
                                C.c_void_p(_ptr(out_pos)), C.c_void_p(_stream(stream))), "finch_compact")


def finch_step(ctx, prompt_q, cache_k, cache_v, cache_pos, chunk_k, chunk_v, chunk_pos, batch: Batch, out_k, out_v,
               out_pos, kept_idx, out_len, scores=None, ws=None, stream=None) -> None:
    ts = [_tensor(t) for t in (prompt_q, cache_k, cache_v, chunk_k, chunk_v, out_k, out_v)]
    _check(load().finch_step(ctx, C.byref(ts[0]), C.byref(ts[1]), C.byref(ts[2]), C.c_void_p(_ptr(cache_pos)),
                             C.byref(ts[3]), C.byref(ts[4]), C.c_void_p(_ptr(chunk_pos)), C.byref(batch.c),
                             C.byref(ts[5]), C.byref(ts[6]), C.c_void_p(_ptr(out_pos)), C.c_void_p(_ptr(kept_idx)),
                             C.c_void_p(_ptr(out_len)), C.c_void_p(_ptr(scores)), C.c_void_p(_ptr(ws)),
                             C.c_size_t(_nbytes(ws)), C.c_void_p(_stream(stream))), "finch_step")


def finch_device_status(ctx, stream=None) -> int:
    """Synchronises the stream and returns the status word (0 = clean); the word is cleared."""
    out = C.c_int32()
    st = load().finch_device_status(ctx, C.c_void_p(_stream(stream)), C.byref(out))
    if st not in (FINCH_OK, FINCH_ERR_DEVICE_STATUS):
        raise FinchError(st, "finch_device_status")
    return int(out.value)


def finch_launch_count(ctx) -> int:
    """Kernels enqueued through this context since it was created."""
    out = C.c_uint64()
    _check(load().finch_launch_count(ctx, C.byref(out)), "finch_launch_count")
    return int(out.value)


def finch_score_static(ctx, prompt_q, cache_k, chunk_k, batch: Batch, scores, row_lse=None, stream=None) -> None:
    """finch_score without a workspace: the scratch is a fixed array inside the library (see finch.h for the
    row limit and the sharing rules).  For callers that may not allocate device memory."""
    q, ck, hk = _tensor(prompt_q), _tensor(cache_k), _tensor(chunk_k)
    _check(load().finch_score_static(ctx, C.byref(q), C.byref(ck), C.byref(hk), C.byref(batch.c),
                                     C.c_void_p(_ptr(scores)), C.c_void_p(_ptr(row_lse)),
                                     C.c_void_p(_stream(stream))), "finch_score_static")


def finch_score_static_max_rows() -> int:
    return int(load().finch_score_static_max_rows())


FINCH_SCORE_WARP_LEVEL, FINCH_SCORE_TWO_LAUNCH, FINCH_SCORE_ONE_KERNEL = 0, 1, 2


def finch_score_plan(ctx, batch: Batch):
    """(path, window): which kernels finch_score / finch_step run for this batch and, on the one-kernel path, the
    window length in key tiles."""
    path, window = C.c_int32(), C.c_int32()
    _check(load().finch_score_plan(ctx, C.byref(batch.c), C.byref(path), C.byref(window)), "finch_score_plan")
    return path.value, window.value


def finch_score_static_path(ctx, batch: Batch) -> bool:
    """True when finch_score_static would run this batch on the tensor-core kernels, False: warp-level kernels."""
    out = C.c_int32()
    _check(load().finch_score_static_path(ctx, C.byref(batch.c), C.byref(out)), "finch_score_static_path")
    return bool(out.value)


def finch_step_host(ctx, host_prompt_q, host_chunk_k, host_chunk_v, host_chunk_pos, stage_q, stage_chunk_k,
                    stage_chunk_v, stage_chunk_pos, cache_k, cache_v, cache_pos, batch: Batch, out_k, out_v, out_pos,
                    kept_idx, out_len, host_kept_idx, host_out_len, ws, stream=None) -> None:
    """finch_step with this step's inputs in host memory (torch CPU tensors, ideally pinned) and the kept indices
    and lengths returned to host tensors; the call returns after the stream has finished."""
    ts = [_tensor(t) for t in (stage_q, stage_chunk_k, stage_chunk_v, cache_k, cache_v, out_k, out_v)]
    _check(load().finch_step_host(
        ctx, C.c_void_p(_ptr(host_prompt_q)), C.c_void_p(_ptr(host_chunk_k)), C.c_void_p(_ptr(host_chunk_v)),
        C.c_void_p(_ptr(host_chunk_pos)), C.byref(ts[0]), C.byref(ts[1]), C.byref(ts[2]),
        C.c_void_p(_ptr(stage_chunk_pos)), C.byref(ts[3]), C.byref(ts[4]), C.c_void_p(_ptr(cache_pos)),
        C.byref(batch.c), C.byref(ts[5]), C.byref(ts[6]), C.c_void_p(_ptr(out_pos)), C.c_void_p(_ptr(kept_idx)),
        C.c_void_p(_ptr(out_len)), C.c_void_p(_ptr(host_kept_idx)), C.c_void_p(_ptr(host_out_len)),
        C.c_void_p(_ptr(ws)), C.c_size_t(_nbytes(ws)), C.c_void_p(_stream(stream))), "finch_step_host")
