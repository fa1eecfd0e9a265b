"""Shared test harness: run one step through the C ABI on the GPU and compare it with the fp64 oracle.

Used by the gpu-marked tests and by the smoke check.  The oracle is called here (test infrastructure); the
library side goes through ``paper_2408_00167_b200.binding`` only.
"""
from __future__ import annotations

import numpy as np

import oracle
from paper_2408_00167_b200 import binding as fb
from paper_2408_00167_b200 import workloads as wl

REL_TOL, ABS_TOL = 1e-3, 1e-5   # per-key score tolerance for bf16/fp32 inputs with fp32 accumulation

# Every output buffer starts out filled with a value the kernels never produce, and sits between two guard zones
# of GUARD elements holding the same value: whatever is still there afterwards was not written.
GUARD = 4096
SENTINEL_I32 = -1          # kept_idx, out_pos
SENTINEL_LEN = -7          # out_len
SENTINEL_BF16 = 0x7FC5     # a NaN bit pattern no rounding produces (out_k / out_v rows, bf16 storage)
SENTINEL_F32 = 0x7FC00005  # the same for fp32 storage (scores and row_lse use it as well)


def to_device(a: np.ndarray, dtype: str, device="cuda"):
    """Storage bit patterns (float32 or uint16-as-bf16) -> torch tensor of the matching dtype on the device."""
    import torch
    if dtype == "f32":
        return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device).view(torch.bfloat16)


def to_host(t, dtype: str) -> np.ndarray:
    import torch
    if dtype == "f32":
        return t.detach().cpu().numpy()
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)


class GpuStep:
    """Device buffers of one step plus the context; `run` calls finch_step, `run_parts` the three calls."""

    def __init__(self, cfg: wl.Config, st: dict, n_layers: int, device="cuda", group_mode=None, scale=0.0,
                 prompt_self_lse=None, row_limit=None, row_norm=False):
        import torch
        self.cfg, self.st, self.dtype, self.device = cfg, st, cfg.dtype, device
        gm = cfg.group_mode if group_mode is None else group_mode
        self.G = cfg.n_kv_heads if gm == 0 else 1
        self.L = n_layers
        B = len(st["cache_len"])
        self_lse = None
        if prompt_self_lse is not None:
            self_lse = torch.from_numpy(np.ascontiguousarray(prompt_self_lse, dtype=np.float32)).to(device)
        limit = None
        if row_limit is not None:
            limit = torch.from_numpy(np.ascontiguousarray(row_limit, dtype=np.int32)).to(device)
        self.batch = fb.make_batch(st["q_off"], st["chunk_off"], st["cache_off"], st["cache_len"], st["budget"],
                                   device, prompt_self_lse=self_lse, row_limit=limit, row_norm=row_norm)
        c = self.batch.c
        self.ctx = fb.finch_ctx_create(n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim,
                                       fb.FINCH_F32 if cfg.dtype == "f32" else fb.FINCH_BF16, gm, scale,
                                       max_batch=max(B, 1), max_prompt=max(c.max_q, 1),
                                       max_candidates=max(c.max_cache + c.max_chunk, 1), device=0)
        td = lambda k: to_device(st[k], cfg.dtype, device)
        self.q, self.cache_k, self.cache_v = td("q"), td("cache_k"), td("cache_v")
        self.chunk_k, self.chunk_v = td("chunk_k"), td("chunk_v")
        self.cache_pos = torch.from_numpy(np.ascontiguousarray(st["cache_pos"], dtype=np.int32)).to(device)
        self.chunk_pos = torch.from_numpy(np.ascontiguousarray(st["chunk_pos"], dtype=np.int32)).to(device)
        total_cache, total_cand = c.total_cache, c.total_cache + c.total_chunk
        self._guarded = []      # (flat integer tensor with the guard zones, sentinel) of every output buffer
        store = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
        store_bits = SENTINEL_F32 if cfg.dtype == "f32" else SENTINEL_BF16
        self.out_k = self._output(self.cache_k.shape, store, store_bits)
        self.out_v = self._output(self.cache_v.shape, store, store_bits)
        self.out_pos = self._output((n_layers, self.G, total_cache), torch.int32, SENTINEL_I32)
        self.kept_idx = self._output((n_layers, self.G, total_cache), torch.int32, SENTINEL_I32)
        self.out_len = self._output((max(B, 1),), torch.int32, SENTINEL_LEN)
        self.scores = self._output((n_layers, self.G, total_cand), torch.float32, SENTINEL_F32)
        self.row_lse = self._output((n_layers, cfg.n_q_heads, c.total_q), torch.float32, SENTINEL_F32)
        self.ws = torch.empty(fb.finch_workspace_bytes(self.ctx, self.batch), dtype=torch.uint8, device=device)

    def _output(self, shape, dtype, sentinel: int):
        """A contiguous output tensor of `shape`, sentinel-filled, with a guard zone of GUARD elements on each side."""
        import torch
        bits = {torch.float32: torch.int32, torch.bfloat16: torch.int16, torch.int32: torch.int32}[dtype]
        n = int(np.prod(shape))
        signed = sentinel - (1 << 16) if bits == torch.int16 and sentinel >= (1 << 15) else sentinel
        flat = torch.full((n + 2 * GUARD,), signed, dtype=bits, device=self.device)
        self._guarded.append((flat, n, signed))
        return flat[GUARD:GUARD + n].view(dtype).view(*shape)

    def guards_intact(self) -> bool:
        """True when no kernel wrote before the start or past the end of any output buffer."""
        return all(bool((flat[:GUARD] == s).all()) and bool((flat[GUARD + n:] == s).all())
                   for flat, n, s in self._guarded)

    def close(self):
        fb.finch_ctx_destroy(self.ctx)
        self.ctx = None

    def run(self, scores=True):
        fb.finch_step(self.ctx, self.q, self.cache_k, self.cache_v, self.cache_pos, self.chunk_k, self.chunk_v,
                      self.chunk_pos, self.batch, self.out_k, self.out_v, self.out_pos, self.kept_idx, self.out_len,
                      self.scores if scores else None, self.ws)
        return self

    def run_parts(self):
        fb.finch_score(self.ctx, self.q, self.cache_k, self.chunk_k, self.batch, self.scores, self.row_lse, self.ws)
        fb.finch_select(self.ctx, self.scores, self.batch, self.kept_idx, self.out_len)
        fb.finch_compact(self.ctx, self.kept_idx, self.out_len, self.cache_k, self.cache_v, self.cache_pos,
                         self.chunk_k, self.chunk_v, self.chunk_pos, self.batch, self.out_k, self.out_v, self.out_pos)
        return self

    def status(self) -> int:
        return fb.finch_device_status(self.ctx)

    def results(self) -> dict:
        """Host copies of the outputs.  `sentinels` tells check_parity that everything outside the valid regions
        must still hold the initial fill; the guard zones around the buffers are checked right here."""
        assert self.guards_intact(), "a kernel wrote outside an output buffer"
        return dict(scores=self.scores.cpu().numpy(), kept_idx=self.kept_idx.cpu().numpy(),
                    out_len=self.out_len.cpu().numpy(), out_pos=self.out_pos.cpu().numpy(),
                    out_k=to_host(self.out_k, self.dtype), out_v=to_host(self.out_v, self.dtype),
                    row_lse=self.row_lse.cpu().numpy(), sentinels=True)


def oracle_scores(cfg: wl.Config, st: dict, group_mode=None, scale=None, threads=8, want_lse=False,
                  prompt_self_lse=None, row_limit=None, row_norm=False):
    gm = cfg.group_mode if group_mode is None else group_mode
    return oracle.score(cfg.dtype, st["q"], st["cache_k"], st["chunk_k"], n_q_heads=cfg.n_q_heads,
                        n_kv_heads=cfg.n_kv_heads, head_dim=cfg.head_dim, group_mode=gm, scale=scale,
                        q_off=st["q_off"], chunk_off=st["chunk_off"], cache_off=st["cache_off"],
                        cache_len=st["cache_len"], threads=threads, want_lse=want_lse,
                        prompt_self_lse=prompt_self_lse, row_limit=row_limit, row_norm=row_norm)


def check_parity(cfg: wl.Config, st: dict, res: dict, ref_scores: np.ndarray, group_mode=None, check_scores=True):
    """The parity procedure.  Returns a summary dict (band occupancy etc.); raises AssertionError on a mismatch.

    (i)   per-key scores within max(1e-3 relative, 1e-5 absolute) of the oracle
    (ii)  kept set: everything the oracle scores above tau + delta is kept, nothing below tau - delta is, the count
          is exactly r' and the indices strictly increase (tau = the oracle's r'-th largest score)
    (iii) the oracle's selection applied to the GPU's own fp32 scores reproduces kept_idx bit for bit (tie rule)
    (iv)  gathered K / V / position rows equal the source rows at the GPU's kept_idx, bit for bit
    (v)   with res["sentinels"] (buffers of a GpuStep): nothing was written outside the valid regions -- rows at or
          beyond r' of kept_idx / out_pos / out_k / out_v up to the request's capacity and score entries at or beyond
          N_b still hold the initial fill
    """
    gm = cfg.group_mode if group_mode is None else group_mode
    G = cfg.n_kv_heads if gm == 0 else 1
    kvpg = cfg.n_kv_heads // G
    L = ref_scores.shape[0]
    B = len(st["cache_len"])
    q_off, chunk_off, cache_off = st["q_off"], st["chunk_off"], st["cache_off"]
    summary = dict(units=0, band_keys=0, max_rel_err=0.0, swapped_units=0)
    sentinels = bool(res.get("sentinels"))
    if sentinels:
        store_fill = np.uint32(SENTINEL_F32) if cfg.dtype == "f32" else np.uint16(SENTINEL_BF16)
        store_bits = (lambda a: a.view(np.uint32)) if cfg.dtype == "f32" else (lambda a: a)
        f32_bits = lambda a: np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    for b in range(B):
        c = int(st["cache_len"][b])
        m = int(chunk_off[b + 1] - chunk_off[b])
        N = c + m
        r = max(0, min(int(st["budget"][b]), N))
        assert int(res["out_len"][b]) == r, (b, res["out_len"][b], r)
        so, co, ho = int(cache_off[b] + chunk_off[b]), int(cache_off[b]), int(chunk_off[b])
        cap = int(cache_off[b + 1] - cache_off[b])
        for l in range(L):
            for g in range(G):
                summary["units"] += 1
                if sentinels:
                    assert np.all(f32_bits(res["scores"][l, g, so + N:so + cap + m]) == SENTINEL_F32), \
                        f"scores written beyond the candidates b={b} l={l} g={g}"
                    assert np.all(res["kept_idx"][l, g, co + r:co + cap] == SENTINEL_I32), "kept_idx beyond r'"
                    assert np.all(res["out_pos"][l, g, co + r:co + cap] == SENTINEL_I32), "out_pos beyond r'"
                    for kk in range(kvpg):
                        for name_out in ("out_k", "out_v"):
                            tail = store_bits(np.ascontiguousarray(res[name_out][l, g * kvpg + kk, co + r:co + cap]))
                            assert np.all(tail == store_fill), f"{name_out} rows written beyond r' b={b} l={l}"

                ref = ref_scores[l, g, so:so + N]
                got = res["scores"][l, g, so:so + N].astype(np.float64)
                if check_scores and N:
                    err = np.abs(got - ref)
                    tol = np.maximum(REL_TOL * np.abs(ref), ABS_TOL)
                    bad = np.nonzero(err > tol)[0]
                    assert bad.size == 0, f"score mismatch b={b} l={l} g={g} j={bad[:5]} got={got[bad[:5]]} " \
                                          f"ref={ref[bad[:5]]}"
                    summary["max_rel_err"] = max(summary["max_rel_err"],
                                                 float((err / np.maximum(np.abs(ref), ABS_TOL / REL_TOL)).max()))
                kept = res["kept_idx"][l, g, co:co + r]
                if r:
                    assert kept.min() >= 0 and kept.max() < N
                    assert np.all(np.diff(kept) > 0), "kept indices must strictly increase"
                    tau = np.sort(ref)[N - r]
                    delta = max(REL_TOL * abs(tau), ABS_TOL)
                    mask = np.zeros(N, bool)
                    mask[kept] = True
                    assert mask[ref > tau + delta].all(), "a clear top-r key was dropped"
                    assert not mask[ref < tau - delta].any(), "a clearly low key was kept"
                    summary["band_keys"] += int(((ref >= tau - delta) & (ref <= tau + delta)).sum())
                    ref_kept = oracle.select_unit(ref, r)
                    summary["swapped_units"] += int(not np.array_equal(ref_kept, kept))
                    self_kept = oracle.select_unit(res["scores"][l, g, so:so + N].astype(np.float64), r)
                    np.testing.assert_array_equal(kept, self_kept, err_msg="tie-break / selection on own scores")
                # gathered rows
                cpos = st["cache_pos"][l, g, co:co + c]
                cand_pos = np.concatenate([cpos, st["chunk_pos"][ho:ho + m]])
                np.testing.assert_array_equal(res["out_pos"][l, g, co:co + r], cand_pos[kept])
                for kk in range(kvpg):
                    h = g * kvpg + kk
                    for name_in, name_chunk, name_out in (("cache_k", "chunk_k", "out_k"),
                                                          ("cache_v", "chunk_v", "out_v")):
                        cand = np.concatenate([st[name_in][l, h, co:co + c], st[name_chunk][l, h, ho:ho + m]])
                        np.testing.assert_array_equal(res[name_out][l, h, co:co + r], cand[kept],
                                                      err_msg=f"{name_out} rows b={b} l={l} h={h}")
    return summary
