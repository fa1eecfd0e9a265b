"""Seeded synthetic inputs shaped like the paper's workloads.

This module only *draws inputs*: random Q/K/V tensors, request length mixes,
chunk schedules and planted high-relevance keys.  It holds none of the method's
arithmetic (no logits, softmax, ranking or gathering) and imports neither the
CUDA binding nor the CPU oracle, so both sides can be fed the same bits.

Shapes follow the paper's experimental setup: chunk sizes of 64..2048 tokens
(Appendix, chunk-size table), prompts of at most 128/256 tokens (Appendix,
prompt-length table), target cache sizes of 512..2000 tokens (LongBench tables)
and compression ratios from 2x to 93x (Results).  The data themselves are
Gaussian or Student-t draws that stand in for the benchmark documents.

Floating tensors are produced as float32 arrays whose values are exactly
representable in the configuration's storage type; ``to_storage`` turns them
into the bit patterns the library and the oracle consume (float32, or uint16
holding bfloat16).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence

import numpy as np

# tensor ids for seeding
_T_Q, _T_K, _T_V, _T_PLANT, _T_REQ, _T_CACHE_K, _T_CACHE_V, _T_CACHE_POS, _T_BETA = range(9)


@dataclass(frozen=True)
class Request:
    n_q: int        # prompt length n^que (query rows used for scoring)
    text_len: int   # n^cont, tokens of the long text
    chunk: int      # m, chunk length
    budget: int     # k, target tokens of the compressed cache (also the per-step r)

    @property
    def n_steps(self) -> int:
        return -(-self.text_len // self.chunk)

    def chunk_len(self, step: int) -> int:
        return max(0, min(self.chunk, self.text_len - step * self.chunk))


@dataclass(frozen=True)
class Config:
    name: str
    cfg_id: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str                 # "f32" | "bf16"
    dist: str                  # "normal" | "student_t3"
    planted_frac: float        # fraction of candidate positions carrying a planted key
    planted_mode: str          # "replace" (k = 3 sqrt(d) u) | "bias" (k += beta sqrt(d) u, beta ~ U(2,4) per head)
    requests: Sequence[Request] = field(default_factory=tuple)
    planted_count: Optional[int] = None   # fixed count per head instead of a fraction
    group_mode: int = 0        # 0: one selection group per KV head; 1: one per layer (sum over all heads)

    @property
    def batch(self) -> int:
        return len(self.requests)

    @property
    def n_groups(self) -> int:
        return self.n_kv_heads if self.group_mode == 0 else 1

    @property
    def n_steps(self) -> int:
        return max(r.n_steps for r in self.requests)


def _rng(*key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([0xF17C, *key])))


def _ragged_requests(cfg_id: int, batch: int) -> List[Request]:
    g = _rng(cfg_id, _T_REQ)
    lens = g.integers(4096, 32768, size=batch, endpoint=True)
    nqs = g.integers(16, 256, size=batch, endpoint=True)
    return [Request(int(nq), int(n), 1024, int(-(-int(n) // 8))) for n, nq in zip(lens, nqs)]


def _make_configs() -> Dict[str, Config]:
    c = {}
    c["c1"] = Config("c1", 1, 1, 8, 8, 64, "f32", "normal", 0.0, "replace",
                     (Request(16, 512, 256, 256),), planted_count=8)
    c["c2"] = Config("c2", 2, 32, 32, 32, 128, "bf16", "normal", 0.02, "bias",
                     (Request(64, 4096, 512, 512),))
    c["c3"] = Config("c3", 3, 32, 32, 8, 128, "bf16", "normal", 0.01, "bias",
                     (Request(128, 32768, 2048, 2048),))
    c["c4"] = Config("c4", 4, 32, 32, 8, 128, "bf16", "normal", 0.01, "bias",
                     tuple(_ragged_requests(4, 16)))
    c["c5"] = Config("c5", 5, 32, 32, 8, 128, "bf16", "student_t3", 0.005, "bias",
                     (Request(64, 131072, 2048, 1408),))
    return c


CONFIGS: Dict[str, Config] = _make_configs()


def scaled(cfg: Config, **changes) -> Config:
    """A copy of a configuration with some fields replaced (fewer layers, other requests...)."""
    d = {f: getattr(cfg, f) for f in cfg.__dataclass_fields__}
    d.update(changes)
    return Config(**d)


# ------------------------------------------------------------------ storage types

def round_to_dtype(a: np.ndarray, dtype: str) -> np.ndarray:
    """float32 array whose values are exactly representable in `dtype` (round to nearest even)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "f32":
        return a
    u = a.view(np.uint32)
    r = ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000))
    return r.view(np.float32)


def to_storage(a: np.ndarray, dtype: str) -> np.ndarray:
    """Bit patterns of `a` in the storage type: float32, or uint16 holding bfloat16."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "f32":
        return a
    return (round_to_dtype(a, dtype).view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def from_storage(s: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "f32":
        return np.ascontiguousarray(s, dtype=np.float32)
    return (s.astype(np.uint32) << np.uint32(16)).view(np.float32)


# ------------------------------------------------------------------ draws

def _draw(g: np.random.Generator, shape, dist: str) -> np.ndarray:
    if dist == "normal":
        return g.standard_normal(shape, dtype=np.float32)
    if dist == "student_t3":
        return g.standard_t(3.0, shape).astype(np.float32)
    raise ValueError(dist)


def offsets(lengths: Sequence[int]) -> np.ndarray:
    off = np.zeros(len(lengths) + 1, dtype=np.int32)
    off[1:] = np.cumsum(np.asarray(lengths, dtype=np.int64))
    return off


def prompt_q(cfg: Config, layer: int) -> np.ndarray:
    """Prompt queries of one layer, [Hq][total_q][d]; fixed for all steps of a request."""
    parts = []
    for b, r in enumerate(cfg.requests):
        parts.append(_draw(_rng(cfg.cfg_id, layer, b, 0, _T_Q), (cfg.n_q_heads, r.n_q, cfg.head_dim), "normal"))
    return round_to_dtype(np.concatenate(parts, axis=1), cfg.dtype)


def q_offsets(cfg: Config) -> np.ndarray:
    return offsets([r.n_q for r in cfg.requests])


def _plant_directions(cfg: Config, q_layer: np.ndarray, b: int) -> np.ndarray:
    """Unit vector along the mean prompt query of each KV head's query group, [Hkv][d]."""
    qo = q_offsets(cfg)
    g = cfg.n_q_heads // cfg.n_kv_heads
    qb = q_layer[:, qo[b]:qo[b + 1], :].reshape(cfg.n_kv_heads, g * (qo[b + 1] - qo[b]), cfg.head_dim)
    mean = qb.astype(np.float64).mean(axis=1)
    return (mean / np.linalg.norm(mean, axis=1, keepdims=True)).astype(np.float32)


def _plant(cfg: Config, k: np.ndarray, u: np.ndarray, positions: np.ndarray, beta: np.ndarray) -> None:
    """Write planted keys into k [Hkv][n][d] at `positions` (same positions for every head)."""
    root_d = np.float32(np.sqrt(cfg.head_dim))
    if len(positions) == 0:
        return
    if cfg.planted_mode == "replace":
        k[:, positions, :] = (np.float32(3.0) * root_d * u)[:, None, :]
    else:
        k[:, positions, :] += (beta[:, None] * root_d * u)[:, None, :]


def _n_planted(cfg: Config, n: int) -> int:
    if cfg.planted_count is not None:
        return min(cfg.planted_count, n)
    return int(round(cfg.planted_frac * n))


def chunk_kv(cfg: Config, layer: int, step: int, q_layer: Optional[np.ndarray] = None):
    """Keys/values of the `step`-th chunk of every request for one layer.

    Returns dict(k, v [Hkv][total_chunk][d] float32, chunk_off int32[B+1], chunk_pos int32[total_chunk],
    planted int32 chunk-local row numbers per request).  Requests whose text is exhausted contribute 0 rows."""
    if q_layer is None:
        q_layer = prompt_q(cfg, layer)
    ks, vs, pos, planted = [], [], [], []
    lens = [r.chunk_len(step) for r in cfg.requests]
    for b, r in enumerate(cfg.requests):
        m = lens[b]
        k = _draw(_rng(cfg.cfg_id, layer, b, step, _T_K), (cfg.n_kv_heads, m, cfg.head_dim), cfg.dist)
        v = _draw(_rng(cfg.cfg_id, layer, b, step, _T_V), (cfg.n_kv_heads, m, cfg.head_dim), cfg.dist)
        gp = _rng(cfg.cfg_id, 0, b, step, _T_PLANT)          # same planted positions in every layer
        pl = np.sort(gp.choice(m, size=_n_planted(cfg, m), replace=False)).astype(np.int32) if m else \
            np.zeros(0, np.int32)
        beta = _rng(cfg.cfg_id, layer, b, 0, _T_BETA).uniform(2.0, 4.0, cfg.n_kv_heads).astype(np.float32)
        _plant(cfg, k, _plant_directions(cfg, q_layer, b), pl, beta)
        ks.append(k)
        vs.append(v)
        pos.append(np.arange(step * r.chunk, step * r.chunk + m, dtype=np.int32))
        planted.append(pl)
    return dict(k=round_to_dtype(np.concatenate(ks, axis=1), cfg.dtype),
                v=round_to_dtype(np.concatenate(vs, axis=1), cfg.dtype),
                chunk_off=offsets(lens), chunk_pos=np.concatenate(pos), planted=planted)


def steady_state(cfg: Config, layers: Sequence[int], step: int = 1):
    """One full-cache step for the given layers, in storage bit patterns.

    The cache holds `budget` synthetic rows per request (same distribution as the chunk, with planted keys,
    increasing positions below the chunk's); the chunk is the `step`-th chunk.  Returns a dict with
    q, cache_k, cache_v, chunk_k, chunk_v (storage arrays, leading axis = len(layers)), cache_pos [L][G][total_cache],
    chunk_pos, q_off, chunk_off, cache_off, cache_len, budget, planted (per request: candidate indices)."""
    B = cfg.batch
    caps = [r.budget for r in cfg.requests]
    cache_off = offsets(caps)
    cache_len = np.asarray(caps, dtype=np.int32)
    budget = np.asarray(caps, dtype=np.int32)
    q_all, ck_all, cv_all, hk_all, hv_all, cpos_all = [], [], [], [], [], []
    chunk_off = chunk_pos = None
    planted = None
    for layer in layers:
        q_layer = prompt_q(cfg, layer)
        ch = chunk_kv(cfg, layer, step, q_layer)
        chunk_off, chunk_pos = ch["chunk_off"], ch["chunk_pos"]
        cks, cvs, cps, pl_all = [], [], [], []
        for b, r in enumerate(cfg.requests):
            c = caps[b]
            k = _draw(_rng(cfg.cfg_id, layer, b, step, _T_CACHE_K), (cfg.n_kv_heads, c, cfg.head_dim), cfg.dist)
            v = _draw(_rng(cfg.cfg_id, layer, b, step, _T_CACHE_V), (cfg.n_kv_heads, c, cfg.head_dim), cfg.dist)
            gp = _rng(cfg.cfg_id, 0, b, step, _T_CACHE_POS)
            m = r.chunk_len(step)
            n_pl_total = _n_planted(cfg, c + m)
            n_pl_cache = max(0, n_pl_total - len(ch["planted"][b]))
            pl = np.sort(gp.choice(c, size=min(n_pl_cache, c), replace=False)).astype(np.int32) if c else \
                np.zeros(0, np.int32)
            beta = _rng(cfg.cfg_id, layer, b, 0, _T_BETA).uniform(2.0, 4.0, cfg.n_kv_heads).astype(np.float32)
            _plant(cfg, k, _plant_directions(cfg, q_layer, b), pl, beta)
            cks.append(k)
            cvs.append(v)
            # kept positions of earlier chunks: an increasing sample of [0, step*chunk), identical per group here
            hi = max(step * r.chunk, c)
            cps.append(np.sort(gp.choice(hi, size=c, replace=False)).astype(np.int32))
            pl_all.append(np.concatenate([pl, c + ch["planted"][b]]).astype(np.int32))
        planted = pl_all
        q_all.append(to_storage(q_layer, cfg.dtype))
        ck_all.append(to_storage(np.concatenate(cks, axis=1), cfg.dtype))
        cv_all.append(to_storage(np.concatenate(cvs, axis=1), cfg.dtype))
        hk_all.append(to_storage(ch["k"], cfg.dtype))
        hv_all.append(to_storage(ch["v"], cfg.dtype))
        cpos_all.append(np.broadcast_to(np.concatenate(cps)[None, :], (cfg.n_groups, int(cache_off[B]))).copy())
    return dict(q=np.stack(q_all), cache_k=np.stack(ck_all), cache_v=np.stack(cv_all),
                chunk_k=np.stack(hk_all), chunk_v=np.stack(hv_all), cache_pos=np.stack(cpos_all),
                chunk_pos=chunk_pos, q_off=q_offsets(cfg), chunk_off=chunk_off, cache_off=cache_off,
                cache_len=cache_len, budget=budget, planted=planted)
