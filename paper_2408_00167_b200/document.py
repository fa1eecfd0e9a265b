"""Whole-document compression: the chunk loop around the step (Finch, Section "Method").

"Document Segmentation" feeds the document chunk by chunk; every step scores the compressed cache plus the new chunk
against the prompt, keeps `budget` candidates and carries them to the next step ("Selection of top r position",
"Managing the Cache").  This module only orchestrates: two caches on the device that swap roles each step, the batch
metadata, and the budget schedule.  Every step is one finch_step call; nothing is computed here, and the loop never
waits for the device: the lengths a step will produce are known on the host (out_len = min(budget, cache + chunk))
and kept in a host mirror.  The mirror is only a prediction -- a step the device refused (status word set) writes
length 0 -- so `verify` compares it with the device at the end of a document, and `reset` / `close` call it.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np

from . import binding as fb


def fixed_budgets(n_steps: int, k: int) -> List[int]:
    """The same target size at every step (the cache fills up to k and stays there)."""
    return [int(k)] * int(n_steps)


def paper_budgets(chunk_lens: Sequence[int], sigma: float, k: int) -> List[int]:
    """The paper's growing schedule, r_{it+1} = m_{it+1} / sigma + c_it, with the final step's r equal to the target
    size k ("Selection of top r position").  c_it is the cache length after step it (c_0 = 0); the division is
    rounded down (the paper does not say)."""
    budgets, c = [], 0
    for it, m in enumerate(chunk_lens):
        r = int(m // sigma) + c if it + 1 < len(chunk_lens) else int(k)
        budgets.append(r)
        c = min(r, c + int(m))
    return budgets


class DocumentCompressor:
    """Device-resident state of one batch of documents being compressed.

    capacity[b] rows of cache per request (at least the largest budget that request will see).  `step` takes the
    chunk's K, V, positions (device tensors in the library's packed layout) and this step's budgets; afterwards
    `cache_k / cache_v / cache_pos / cache_len` describe the compressed cache.
    """

    def __init__(self, n_layers: int, n_q_heads: int, n_kv_heads: int, head_dim: int, dtype: int,
                 capacity: Sequence[int], max_prompt: int, max_chunk: int, group_mode: int = fb.FINCH_GROUP_PER_KV_HEAD,
                 scale: float = 0.0, rope_theta: float = 0.0, rope_pairing: int = 0, device="cuda"):
        import torch
        self.torch = torch
        self.device = device
        self.L, self.Hq, self.Hkv, self.d = n_layers, n_q_heads, n_kv_heads, head_dim
        self.G = n_kv_heads if group_mode == fb.FINCH_GROUP_PER_KV_HEAD else 1
        self.capacity = np.asarray(capacity, dtype=np.int32)
        self.B = len(self.capacity)
        self.cache_off = np.concatenate([[0], np.cumsum(self.capacity)]).astype(np.int32)
        total_cap = int(self.cache_off[-1])
        tdtype = torch.float32 if dtype == fb.FINCH_F32 else torch.bfloat16
        self.ctx = fb.finch_ctx_create(n_layers, n_q_heads, n_kv_heads, head_dim, dtype, group_mode, scale,
                                       max_batch=max(self.B, 1), max_prompt=max(max_prompt, 1),
                                       max_candidates=max(int(self.capacity.max(initial=0)) + max_chunk, 1),
                                       device=torch.device(device).index or 0, rope_theta=rope_theta,
                                       rope_pairing=rope_pairing)
        mk = lambda: dict(k=torch.zeros((n_layers, n_kv_heads, total_cap, head_dim), dtype=tdtype, device=device),
                          v=torch.zeros((n_layers, n_kv_heads, total_cap, head_dim), dtype=tdtype, device=device),
                          pos=torch.full((n_layers, self.G, total_cap), -1, dtype=torch.int32, device=device),
                          len=torch.zeros(max(self.B, 1), dtype=torch.int32, device=device))
        self._bufs = [mk(), mk()]
        self._cur = 0
        self.kept_idx = torch.full((n_layers, self.G, total_cap), -1, dtype=torch.int32, device=device)
        self.cache_len = np.zeros(self.B, dtype=np.int32)       # host mirror of the device lengths
        self._ws = None
        self._meta = {}
        self.steps = 0
        self._unverified = 0    # steps enqueued since the device was last compared with the host mirror

    # the cache the next step will read
    @property
    def cache_k(self):
        return self._bufs[self._cur]["k"]

    @property
    def cache_v(self):
        return self._bufs[self._cur]["v"]

    @property
    def cache_pos(self):
        return self._bufs[self._cur]["pos"]

    def verify(self) -> None:
        """Wait for the steps enqueued so far and check them: raises RuntimeError when the device status word is set
        or when the lengths on the device differ from the host mirror the later steps were sized with."""
        if self._unverified == 0:
            return
        self._unverified = 0
        word = fb.finch_device_status(self.ctx)            # synchronises the stream
        dev_len = self._bufs[self._cur]["len"][:self.B].cpu().numpy()
        if word != 0:
            raise RuntimeError(f"document loop: device status word {word:#x} after {self.steps} steps "
                               f"(lengths on the device {dev_len.tolist()}, expected {self.cache_len.tolist()})")
        if not np.array_equal(dev_len, self.cache_len):
            raise RuntimeError(f"document loop: cache lengths on the device {dev_len.tolist()} differ from the "
                               f"host mirror {self.cache_len.tolist()} after {self.steps} steps")

    def reset(self) -> None:
        """Start a new batch of documents in the same buffers (empty caches).  Checks the finished one first."""
        self.verify()
        self.cache_len = np.zeros(self.B, dtype=np.int32)
        self._bufs[0]["len"].zero_()
        self._cur = 0
        self.steps = 0

    def close(self) -> None:
        """Check the steps still unverified, then free the context (the check's error, if any, is raised after)."""
        if self.ctx:
            try:
                self.verify()
            finally:
                fb.finch_ctx_destroy(self.ctx)
                self.ctx = None

    def _device_i32(self, a: np.ndarray):
        """Device copy of a small int32 array, cached by content (offsets and budgets repeat from step to step)."""
        key = a.tobytes()
        t = self._meta.get(key)
        if t is None:
            if len(self._meta) > 256:
                self._meta.clear()
            t = self.torch.from_numpy(a.copy()).to(self.device)
            self._meta[key] = t
        return t

    def step(self, q, q_off: Sequence[int], chunk_k, chunk_v, chunk_pos, chunk_off: Sequence[int],
             budget: Sequence[int], scores=None, prompt_self_lse=None, row_limit=None, row_norm=False) -> None:
        """One finch_step: [cache ; chunk] -> the other cache.  Enqueues and returns.

        The lengths the previous step wrote on the device are this step's cache lengths as they are: nothing comes
        back to the host between steps, and the only host-to-device traffic is metadata that has not been seen yet."""
        torch = self.torch
        src, dst = self._bufs[self._cur], self._bufs[self._cur ^ 1]
        B = self.B
        q_off = np.ascontiguousarray(q_off, dtype=np.int32)
        chunk_off = np.ascontiguousarray(chunk_off, dtype=np.int32)
        budget = np.minimum(np.asarray(budget, dtype=np.int32), self.capacity).astype(np.int32)
        assert len(q_off) == len(chunk_off) == B + 1 and len(budget) == B
        n_q, chunk_len = np.diff(q_off), np.diff(chunk_off)
        n_cand = self.cache_len + chunk_len
        mx = lambda a: int(a.max()) if len(a) else 0
        c = fb.finch_batch(B, self._device_i32(q_off).data_ptr(), self._device_i32(chunk_off).data_ptr(),
                           self._device_i32(self.cache_off).data_ptr(), src["len"].data_ptr(),
                           self._device_i32(budget).data_ptr(), int(q_off[B]), int(chunk_off[B]), int(self.cache_off[B]),
                           mx(n_q), mx(self.cache_len), mx(chunk_len), mx(np.minimum(budget, n_cand)),
                           prompt_self_lse.data_ptr() if prompt_self_lse is not None else None,
                           row_limit.data_ptr() if row_limit is not None else None, int(bool(row_norm)))
        batch = fb.Batch(None, None, None, None, None, c, prompt_self_lse, row_limit)
        need = fb.finch_workspace_bytes(self.ctx, batch)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        fb.finch_step(self.ctx, q, src["k"], src["v"], src["pos"], chunk_k, chunk_v, chunk_pos, batch, dst["k"], dst["v"],
                      dst["pos"], self.kept_idx, dst["len"], scores, self._ws)
        self.cache_len = np.minimum(budget, n_cand).astype(np.int32)   # what the step writes to dst["len"]
        self._cur ^= 1
        self.steps += 1
        self._unverified += 1

    def status(self) -> int:
        """Wait for the stream and return (and clear) the device status word; 0 = clean."""
        return fb.finch_device_status(self.ctx)
