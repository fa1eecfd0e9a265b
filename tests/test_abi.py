"""Host-side checks of the C ABI that need no GPU: exported symbols, argument validation, workspace sizing.

A context created with device = -1 validates arguments exactly like a real one and then refuses to enqueue
(FINCH_ERR_UNSUPPORTED), so every error path below runs without touching a device.
"""
import ctypes as C
import re
from pathlib import Path

import pytest

from paper_2408_00167_b200 import binding as fb
from paper_2408_00167_b200 import build as fbuild

ROOT = Path(__file__).resolve().parents[1]


@pytest.fixture(scope="module")
def lib():
    fbuild.build()
    return fb.load()


def test_library_exports_every_declared_symbol(lib):
    header = (ROOT / "include" / "finch.h").read_text()
    declared = set(re.findall(r"\b(finch_[a-z_]+)\s*\(", header))
    assert declared == set(fb.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings(lib):
    seen = {fb.finch_status_string(s) for s in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert fb.finch_status_string(99) == "unknown status"


def _cfg(**kw):
    base = dict(n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64, dtype=fb.FINCH_BF16,
                group_mode=fb.FINCH_GROUP_PER_KV_HEAD, scale=0.0, max_batch=4, max_prompt=64, max_candidates=1024,
                device=-1)
    base.update(kw)
    return base


@pytest.mark.parametrize("bad,status", [
    (dict(n_layers=0), fb.FINCH_ERR_INVALID_ARG),
    (dict(n_q_heads=6, n_kv_heads=4), fb.FINCH_ERR_INVALID_ARG),
    (dict(dtype=7), fb.FINCH_ERR_INVALID_ARG),
    (dict(group_mode=3), fb.FINCH_ERR_INVALID_ARG),
    (dict(scale=-1.0), fb.FINCH_ERR_INVALID_ARG),
    (dict(scale=float("nan")), fb.FINCH_ERR_INVALID_ARG),
    (dict(max_batch=0), fb.FINCH_ERR_INVALID_ARG),
    (dict(rope_theta=-1.0), fb.FINCH_ERR_INVALID_ARG),
    (dict(rope_theta=0.5), fb.FINCH_ERR_INVALID_ARG),
    (dict(rope_theta=float("inf")), fb.FINCH_ERR_INVALID_ARG),
    (dict(rope_theta=10000.0, rope_pairing=2), fb.FINCH_ERR_INVALID_ARG),
    (dict(head_dim=48), fb.FINCH_ERR_UNSUPPORTED),
    (dict(head_dim=512), fb.FINCH_ERR_UNSUPPORTED),
])
def test_ctx_create_rejects_bad_configs(lib, bad, status):
    with pytest.raises(fb.FinchError) as e:
        fb.finch_ctx_create(**_cfg(**bad))
    assert e.value.status == status


def test_ctx_create_accepts_the_rotary_options_without_a_device(lib):
    ctx = fb.finch_ctx_create(**_cfg(rope_theta=10000.0, rope_pairing=1))     # validation-only: no table is built
    fb.finch_ctx_destroy(ctx)


def test_ctx_create_null_arguments(lib):
    assert lib.finch_ctx_create(None, None) == fb.FINCH_ERR_INVALID_ARG
    lib.finch_ctx_destroy(None)   # ignored


def test_real_device_is_refused_without_a_b200(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(fb.FinchError) as e:
        fb.finch_ctx_create(**_cfg(device=0))
    assert e.value.status == fb.FINCH_ERR_UNSUPPORTED


class _Fake:
    """Stand-ins for device buffers: validation only looks at addresses, never dereferences them."""
    base = 0x7000_0000_0000

    @classmethod
    def batch(cls, B=2, total_q=96, total_chunk=512, total_cache=256, max_q=64, max_cache=128, max_chunk=256,
              max_budget=128):
        p = cls.base
        return fb.Batch(None, None, None, None, None,
                        fb.finch_batch(B, p, p + 256, p + 512, p + 768, p + 1024, total_q, total_chunk, total_cache,
                                       max_q, max_cache, max_chunk, max_budget))

    @classmethod
    def tensor(cls, slot, tokens, d=64, heads=2, misalign=0, stride_tok=None):
        st = d if stride_tok is None else stride_tok
        return fb.finch_tensor(cls.base + 0x1000_0000 * (slot + 1) + misalign, heads * tokens * st, tokens * st, st)


def _step(lib, ctx, batch, q=None, ck=None, cv=None, hk=None, hv=None, ok=None, ov=None, ws=_Fake.base + 0x9000_0000,
          ws_bytes=1 << 30, scores=None, kept=_Fake.base + 0xA000_0000, out_len=_Fake.base + 0xA100_0000,
          cache_pos=_Fake.base + 0xA200_0000, chunk_pos=_Fake.base + 0xA300_0000, out_pos=_Fake.base + 0xA400_0000):
    c = batch.c
    q = q or _Fake.tensor(0, c.total_q, heads=8)
    ck, cv = ck or _Fake.tensor(1, c.total_cache), cv or _Fake.tensor(2, c.total_cache)
    hk, hv = hk or _Fake.tensor(3, c.total_chunk), hv or _Fake.tensor(4, c.total_chunk)
    ok, ov = ok or _Fake.tensor(5, c.total_cache), ov or _Fake.tensor(6, c.total_cache)
    return lib.finch_step(ctx, C.byref(q), C.byref(ck), C.byref(cv), C.c_void_p(cache_pos), C.byref(hk), C.byref(hv),
                          C.c_void_p(chunk_pos), C.byref(c), C.byref(ok), C.byref(ov), C.c_void_p(out_pos),
                          C.c_void_p(kept), C.c_void_p(out_len), C.c_void_p(scores), C.c_void_p(ws),
                          C.c_size_t(ws_bytes), None)


def test_step_validation_paths(lib):
    ctx = fb.finch_ctx_create(**_cfg())
    try:
        good = _Fake.batch()
        # a fully valid call reaches the launch stage, where a validation-only context stops
        assert _step(lib, ctx, good) == fb.FINCH_ERR_UNSUPPORTED
        assert _step(lib, ctx, good, ws=None) == fb.FINCH_ERR_INVALID_ARG
        assert _step(lib, ctx, good, ws=_Fake.base + 8) == fb.FINCH_ERR_BAD_LAYOUT
        assert _step(lib, ctx, good, ws_bytes=16) == fb.FINCH_ERR_WORKSPACE_TOO_SMALL
        assert _step(lib, ctx, good, kept=None) == fb.FINCH_ERR_INVALID_ARG
        assert _step(lib, ctx, good, out_len=None) == fb.FINCH_ERR_INVALID_ARG
        assert _step(lib, ctx, good, cache_pos=None) == fb.FINCH_ERR_INVALID_ARG
        assert _step(lib, ctx, good, chunk_pos=None) == fb.FINCH_ERR_INVALID_ARG
        assert _step(lib, ctx, good, q=_Fake.tensor(0, 96, heads=8, misalign=4)) == fb.FINCH_ERR_BAD_LAYOUT
        assert _step(lib, ctx, good, hk=_Fake.tensor(3, 512, stride_tok=68)) == fb.FINCH_ERR_BAD_LAYOUT
        assert _step(lib, ctx, good, hk=_Fake.tensor(3, 512, stride_tok=32)) == fb.FINCH_ERR_INVALID_ARG
        # outputs may not alias inputs (parallel gather)
        assert _step(lib, ctx, good, ok=_Fake.tensor(1, 256)) == fb.FINCH_ERR_INVALID_ARG
        assert _step(lib, ctx, good, ov=_Fake.tensor(5, 256)) == fb.FINCH_ERR_INVALID_ARG
        # ... nor overlap them partially: an output that starts inside cache_k's extent, or ends inside chunk_v's
        assert _step(lib, ctx, good, ok=_Fake.tensor(1, 256, misalign=64 * 2 * 100)) == fb.FINCH_ERR_INVALID_ARG
        assert _step(lib, ctx, good, ov=_Fake.tensor(4, 256, misalign=-64 * 2 * 200)) == fb.FINCH_ERR_INVALID_ARG
        assert _step(lib, ctx, good, ov=_Fake.tensor(5, 256, misalign=16)) == fb.FINCH_ERR_INVALID_ARG
        # K and V rows interleaved in one buffer (token stride 2 * head_dim, V shifted by one row) share no byte
        inter = lambda slot, shift: _Fake.tensor(slot, 256, stride_tok=128, misalign=shift)
        assert _step(lib, ctx, good, ok=inter(5, 0), ov=inter(5, 128)) == fb.FINCH_ERR_UNSUPPORTED
        assert _step(lib, ctx, good, ok=inter(5, 0), ov=inter(5, 64)) == fb.FINCH_ERR_INVALID_ARG   # half a row
        assert _step(lib, ctx, good, ck=inter(1, 0), ok=inter(1, 128)) == fb.FINCH_ERR_UNSUPPORTED
        # batch bounds against the context and against themselves
        assert _step(lib, ctx, _Fake.batch(B=5)) == fb.FINCH_ERR_INVALID_ARG
        assert _step(lib, ctx, _Fake.batch(max_q=65, total_q=128)) == fb.FINCH_ERR_INVALID_ARG
        assert _step(lib, ctx, _Fake.batch(max_cache=900, total_cache=900, max_chunk=256)) == fb.FINCH_ERR_INVALID_ARG
        assert _step(lib, ctx, _Fake.batch(max_q=0)) == fb.FINCH_ERR_INVALID_ARG
        assert _step(lib, ctx, _Fake.batch(max_budget=300)) == fb.FINCH_ERR_INVALID_ARG
        nullb = _Fake.batch()
        nullb.c.q_off = None
        assert _step(lib, ctx, nullb) == fb.FINCH_ERR_INVALID_ARG
    finally:
        fb.finch_ctx_destroy(ctx)


def test_workspace_bytes_is_host_arithmetic(lib):
    ctx = fb.finch_ctx_create(**_cfg())
    try:
        b = _Fake.batch()
        n = fb.finch_workspace_bytes(ctx, b)
        lse = 2 * 8 * 96 * 8 * 33 + 4 * 2 * 2 * (256 + 512) * 4
        scores = 2 * 2 * (256 + 512) * 4
        assert n >= lse + scores and n % 256 == 0
        bigger = _Fake.batch(total_q=192)
        assert fb.finch_workspace_bytes(ctx, bigger) > n
        out = C.c_size_t()
        assert lib.finch_workspace_bytes(ctx, C.byref(b.c), None) == fb.FINCH_ERR_INVALID_ARG
        assert lib.finch_workspace_bytes(None, C.byref(b.c), C.byref(out)) == fb.FINCH_ERR_INVALID_ARG
        status = C.c_int32()
        assert lib.finch_device_status(ctx, None, C.byref(status)) == fb.FINCH_ERR_UNSUPPORTED
    finally:
        fb.finch_ctx_destroy(ctx)


def test_step_host_validation(lib):
    """finch_step_host checks its staging tensors and host pointers before anything is copied."""
    ctx = fb.finch_ctx_create(**_cfg())
    try:
        b = _Fake.batch()
        c = b.c
        host = _Fake.base + 0xB000_0000

        def call(stage_q=None, host_q=host, host_len=host + 0x100_0000, ws_bytes=1 << 30):
            sq = stage_q or _Fake.tensor(0, c.total_q, heads=8)
            sk, sv = _Fake.tensor(3, c.total_chunk), _Fake.tensor(4, c.total_chunk)
            ck, cv = _Fake.tensor(1, c.total_cache), _Fake.tensor(2, c.total_cache)
            ok, ov = _Fake.tensor(5, c.total_cache), _Fake.tensor(6, c.total_cache)
            p = lambda x: C.c_void_p(x)
            return lib.finch_step_host(ctx, p(host_q), p(host + 0x10_0000), p(host + 0x20_0000), p(host + 0x30_0000),
                                       C.byref(sq), C.byref(sk), C.byref(sv), p(_Fake.base + 0xA300_0000), C.byref(ck),
                                       C.byref(cv), p(_Fake.base + 0xA200_0000), C.byref(c), C.byref(ok), C.byref(ov),
                                       p(_Fake.base + 0xA400_0000), p(_Fake.base + 0xA000_0000),
                                       p(_Fake.base + 0xA100_0000), p(host + 0x40_0000), p(host_len),
                                       p(_Fake.base + 0x9000_0000), C.c_size_t(ws_bytes), None)
        assert call() == fb.FINCH_ERR_UNSUPPORTED                      # valid: stops at the launch stage
        assert call(stage_q=_Fake.tensor(0, c.total_q, heads=8, stride_tok=128)) == fb.FINCH_ERR_BAD_LAYOUT
        assert call(host_q=None) == fb.FINCH_ERR_INVALID_ARG
        assert call(host_len=None) == fb.FINCH_ERR_INVALID_ARG
        assert call(ws_bytes=1024) == fb.FINCH_ERR_WORKSPACE_TOO_SMALL
    finally:
        fb.finch_ctx_destroy(ctx)


# ---------------------------------------------------------------------------------------------- the score plan

def _plan(n_layers, n_q_heads, n_kv_heads, head_dim, n_q, cache, chunk, dtype=None, requests=1, row_limit=None):
    dtype = fb.FINCH_BF16 if dtype is None else dtype
    ctx = fb.finch_ctx_create(n_layers=n_layers, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, head_dim=head_dim,
                              dtype=dtype, group_mode=fb.FINCH_GROUP_PER_KV_HEAD, scale=0.0, max_batch=requests,
                              max_prompt=n_q, max_candidates=cache + chunk, device=-1)
    try:
        off = lambda n: [n * i for i in range(requests + 1)]
        batch = fb.make_batch(off(n_q), off(chunk), off(cache), [cache] * requests, [cache] * requests, device="cpu",
                              row_limit=row_limit)
        return fb.finch_score_plan(ctx, batch)
    finally:
        fb.finch_ctx_destroy(ctx)


def test_score_plan_of_the_benchmark_configurations(lib):
    """Host arithmetic only: which kernels a batch takes and the window length of the one-kernel path."""
    one, two, warp = fb.FINCH_SCORE_ONE_KERNEL, fb.FINCH_SCORE_TWO_LAUNCH, fb.FINCH_SCORE_WARP_LEVEL
    # 32 layers x 32q/8kv, 128 prompt rows, 2048 + 2048 candidates: 32 key tiles per unit, windows of 8 (98.8 % full)
    assert _plan(32, 32, 8, 128, 128, 2048, 2048) == (one, 8)
    # 32 x 32 MHA, 64 prompt rows, 512 + 512 candidates: 8 key tiles per unit, one window per unit
    assert _plan(32, 32, 32, 128, 64, 512, 512) == (one, 8)
    # 27 key tiles per unit (1408 cache rows = 11 tiles, 2048 chunk rows = 16): windows of 9, 86 % full
    assert _plan(32, 32, 8, 128, 64, 1408, 2048) == (one, 9)
    # 29 key tiles per unit on 256 units: 29 is prime and a whole unit per window fills 148 CTAs to 86.5 % ...
    assert _plan(32, 32, 8, 128, 64, 1664, 2048)[0] in (one, two)
    # ... but 31 tiles per unit, 24 layers: 192 units on 148 CTAs, two windows, 65 % full: no window
    assert _plan(24, 32, 8, 128, 64, 1920, 2048) == (two, 0)
    # several requests, fp32 inputs, other head dimensions, more than four query tiles per KV head
    assert _plan(32, 32, 8, 128, 128, 2048, 2048, requests=2) == (two, 0)
    assert _plan(32, 32, 8, 128, 128, 2048, 2048, dtype=fb.FINCH_F32) == (warp, 0)
    assert _plan(2, 8, 8, 96, 64, 512, 512) == (warp, 0)
    assert _plan(32, 32, 8, 128, 192, 2048, 2048) == (two, 0)     # 4 heads x 3 sub-blocks = 12 > 8
    assert _plan(32, 32, 8, 128, 128, 2048, 2048)[1] * 128 * 4 == 4096  # four windows per unit


def test_score_plan_null_arguments(lib):
    ctx = fb.finch_ctx_create(**_cfg())
    batch = fb.make_batch([0, 8], [0, 64], [0, 64], [64], [64], device="cpu")
    assert lib.finch_score_plan(ctx, C.byref(batch.c), None, None) == fb.FINCH_ERR_INVALID_ARG
    path = C.c_int32(-1)
    assert lib.finch_score_plan(ctx, C.byref(batch.c), C.byref(path), None) == fb.FINCH_OK and path.value >= 0
    fb.finch_ctx_destroy(ctx)
