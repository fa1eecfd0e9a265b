"""GPU parity on the five workload configurations, the standalone select / compact calls and the chunk loop."""
import numpy as np
import pytest

import oracle
from paper_2408_00167_b200 import binding as fb
from paper_2408_00167_b200 import build as fbuild
from paper_2408_00167_b200 import workloads as wl
from parity_harness import GpuStep, check_parity, oracle_scores, to_device, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    fbuild.build()
    fb.load()


def _slice_layers(st, layers):
    out = dict(st)
    for k in ("q", "cache_k", "cache_v", "chunk_k", "chunk_v", "cache_pos"):
        out[k] = np.ascontiguousarray(st[k][layers])
    return out


def _slice_results(res, layers):
    out = dict(res)
    for k in ("scores", "kept_idx", "out_pos", "out_k", "out_v", "row_lse"):
        out[k] = res[k][layers]
    return out


@pytest.mark.parametrize("name,layers_gpu,layers_checked", [
    ("c2", [0, 1, 31], [0, 2]),
    ("c3", [0, 17], [1]),
    ("c5", [0, 5], [0]),
])
def test_config_layers_full_width(name, layers_gpu, layers_checked):
    """Every unit of some layers at the configuration's full per-layer size (all heads, full N, full budget)."""
    cfg = wl.CONFIGS[name]
    st = wl.steady_state(cfg, layers_gpu)
    g = GpuStep(cfg, st, len(layers_gpu))
    try:
        g.run()
        assert g.status() == 0
        res = g.results()
    finally:
        g.close()
    sub = _slice_layers(st, layers_checked)
    ref = oracle_scores(cfg, sub, threads=oracle.max_threads())
    summary = check_parity(cfg, sub, _slice_results(res, layers_checked), ref)
    planted = set(st["planted"][0].tolist())
    r = int(st["budget"][0])
    for l in layers_checked:
        for grp in range(cfg.n_groups):
            assert planted <= set(res["kept_idx"][l, grp, :r].tolist()), "a planted key was dropped"
    print(name, summary)


@pytest.mark.parametrize("name,layers_checked", [
    ("c2", [0, 7, 15, 31]),
    ("c3", [0, 7, 15, 31]),
    ("c5", [0, 7, 15, 31]),
])
def test_config_all_layers_in_the_benchmarked_geometry(name, layers_checked):
    """The whole configuration -- all 32 layers in one step, i.e. the launch geometry bench.py times -- with the
    oracle checking the first, the last and two inner layers.  Work is dealt to the persistent CTAs in contiguous
    ranges of key tiles that do not line up with layers, so every checked layer holds units that straddle a range
    boundary.  All layers are checked for what needs no oracle: the exact selection on the GPU's own scores, the
    gathered rows, the planted keys and the untouched sentinels."""
    cfg = wl.CONFIGS[name]
    layers = list(range(cfg.n_layers))
    st = wl.steady_state(cfg, layers)
    g = GpuStep(cfg, st, len(layers))
    try:
        # the geometry that is benchmarked runs both sweeps in one kernel: a silent detour would show here
        path, window = fb.finch_score_plan(g.ctx, g.batch)
        assert path == fb.FINCH_SCORE_ONE_KERNEL and window == {"c2": 8, "c3": 8, "c5": 9}[name]
        g.run()
        assert g.status() == 0
        res = g.results()
    finally:
        g.close()
    sub = _slice_layers(st, layers_checked)
    ref = oracle_scores(cfg, sub, threads=oracle.max_threads())
    summary = check_parity(cfg, sub, _slice_results(res, layers_checked), ref)
    # every layer: selection, gather and sentinels against the GPU's own scores (no oracle scores needed)
    check_parity(cfg, st, res, res["scores"].astype(np.float64), check_scores=False)
    planted = set(st["planted"][0].tolist())
    r = int(st["budget"][0])
    for l in layers:
        for grp in range(cfg.n_groups):
            assert planted <= set(res["kept_idx"][l, grp, :r].tolist()), "a planted key was dropped"
    print(name, summary)


def test_config4_ragged_batch_layer():
    """The ragged batch at full shape for one layer; the oracle checks every request."""
    cfg = wl.CONFIGS["c4"]
    st = wl.steady_state(cfg, [3])
    g = GpuStep(cfg, st, 1)
    try:
        g.run()
        assert g.status() == 0
        res = g.results()
    finally:
        g.close()
    nqs = [r.n_q for r in cfg.requests]
    for b in range(cfg.batch):
        one = wl.scaled(cfg, requests=(cfg.requests[b],))
        sl = lambda off, a, ax: np.ascontiguousarray(np.take(a, np.arange(off[b], off[b + 1]), axis=ax))
        sub = dict(q=sl(st["q_off"], st["q"], 2), cache_k=sl(st["cache_off"], st["cache_k"], 2),
                   cache_v=sl(st["cache_off"], st["cache_v"], 2), chunk_k=sl(st["chunk_off"], st["chunk_k"], 2),
                   chunk_v=sl(st["chunk_off"], st["chunk_v"], 2), cache_pos=sl(st["cache_off"], st["cache_pos"], 2),
                   chunk_pos=st["chunk_pos"][st["chunk_off"][b]:st["chunk_off"][b + 1]],
                   q_off=wl.offsets([nqs[b]]), chunk_off=wl.offsets([st["chunk_off"][b + 1] - st["chunk_off"][b]]),
                   cache_off=wl.offsets([st["cache_off"][b + 1] - st["cache_off"][b]]),
                   cache_len=st["cache_len"][b:b + 1], budget=st["budget"][b:b + 1])
        so = int(st["cache_off"][b] + st["chunk_off"][b])
        n_cand = int(sub["cache_off"][1] + sub["chunk_off"][1])
        co, cap = int(st["cache_off"][b]), int(sub["cache_off"][1])
        rsub = dict(scores=res["scores"][:, :, so:so + n_cand], kept_idx=res["kept_idx"][:, :, co:co + cap],
                    out_len=res["out_len"][b:b + 1], out_pos=res["out_pos"][:, :, co:co + cap],
                    out_k=res["out_k"][:, :, co:co + cap], out_v=res["out_v"][:, :, co:co + cap], sentinels=True)
        ref = oracle_scores(one, sub, threads=oracle.max_threads())
        check_parity(one, sub, rsub, ref)


def _select_only(scores_np, chunk_lens, cache_caps, cache_lens, budgets, L, G):
    import torch
    B = len(budgets)
    batch = fb.make_batch(wl.offsets([1] * B), wl.offsets(chunk_lens), wl.offsets(cache_caps), cache_lens, budgets)
    c = batch.c
    ctx = fb.finch_ctx_create(L, G, G, 64, fb.FINCH_F32, max_batch=B, max_prompt=1,
                              max_candidates=max(c.max_cache + c.max_chunk, 1))
    try:
        # the score rows are laid out with the full candidate stride (cache capacity + chunk rows)
        padded = np.full((L, G, c.total_cache + c.total_chunk), np.nan, np.float32)
        padded[:, :, :scores_np.shape[2]] = scores_np
        scores = torch.from_numpy(padded).cuda()
        kept = torch.full((L, G, c.total_cache), -1, dtype=torch.int32, device="cuda")
        out_len = torch.zeros(B, dtype=torch.int32, device="cuda")
        fb.finch_select(ctx, scores, batch, kept, out_len)
        assert fb.finch_device_status(ctx) == 0
        return kept.cpu().numpy(), out_len.cpu().numpy()
    finally:
        fb.finch_ctx_destroy(ctx)


@pytest.mark.parametrize("n,r,kind", [(1, 1, "rand"), (33, 7, "ties"), (1000, 999, "rand"), (4096, 2048, "ties"),
                                      (1024, 512, "ties"), (1025, 500, "ties"), (4097, 4000, "special"),
                                      (5000, 1234, "special"), (50000, 30000, "rand"), (50000, 777, "ties")])
def test_select_matches_oracle_exactly(n, r, kind):
    rng = np.random.default_rng(n * 7 + r)
    L, G = 2, 3
    if kind == "rand":
        s = rng.random((L, G, n), dtype=np.float32)
    elif kind == "ties":
        s = rng.integers(0, 5, size=(L, G, n)).astype(np.float32) / 4
    else:
        s = rng.standard_normal((L, G, n)).astype(np.float32)
        s[:, :, ::7] = 0.0
        s[:, :, 3::11] = -0.0
        s[:, :, 5::13] = np.nan
        s[:, :, 1::17] = np.inf
        s[:, :, 2::19] = -np.inf
        s[:, :, 4::23] = 1e-42      # subnormal
    kept, out_len = _select_only(s, [n], [n], [0], [r], L, G)
    assert out_len.tolist() == [min(r, n)]
    for l in range(L):
        for g in range(G):
            np.testing.assert_array_equal(kept[l, g, :r], oracle.select_unit(s[l, g].astype(np.float64), r))


def test_compact_with_strided_tensors_and_per_layer_groups():
    import torch
    rng = np.random.default_rng(5)
    L, Hkv, d = 2, 4, 64
    caps, lens, ms, budgets = [40, 24], [33, 24], [17, 30], [35, 20]
    cache_off, chunk_off = wl.offsets(caps), wl.offsets(ms)
    mk = lambda n: wl.to_storage(rng.standard_normal((L, Hkv, n, d)).astype(np.float32), "bf16")
    ck, cv, hk, hv = mk(cache_off[-1]), mk(cache_off[-1]), mk(chunk_off[-1]), mk(chunk_off[-1])
    cpos = rng.integers(0, 1000, size=(L, 1, cache_off[-1])).astype(np.int32)
    hpos = rng.integers(1000, 2000, size=chunk_off[-1]).astype(np.int32)
    scores = rng.random((L, 1, cache_off[-1] + chunk_off[-1]))
    kept, out_len = oracle.select(scores, chunk_off=chunk_off, cache_off=cache_off, cache_len=lens, budget=budgets)
    want_k, want_v, want_p = oracle.compact("bf16", kept, out_len, ck, cv, cpos, hk, hv, hpos, n_kv_heads=Hkv,
                                            head_dim=d, group_mode=1, chunk_off=chunk_off, cache_off=cache_off,
                                            cache_len=lens)

    def strided(a):     # token stride 2*d, extra head padding: exercises the element strides
        t = to_device(a, "bf16")
        big = torch.zeros((L, Hkv + 1, a.shape[2], 2 * d), dtype=torch.bfloat16, device="cuda")
        view = big[:, :Hkv, :, :d]
        view.copy_(t)
        return view
    batch = fb.make_batch(wl.offsets([1, 1]), chunk_off, cache_off, lens, budgets)
    ctx = fb.finch_ctx_create(L, Hkv, Hkv, d, fb.FINCH_BF16, fb.FINCH_GROUP_PER_LAYER, max_batch=2, max_prompt=1,
                              max_candidates=128)
    try:
        out_k, out_v = strided(np.zeros_like(ck)), strided(np.zeros_like(cv))
        out_pos = torch.full((L, 1, int(cache_off[-1])), -1, dtype=torch.int32, device="cuda")
        fb.finch_compact(ctx, torch.from_numpy(kept).cuda(), torch.from_numpy(out_len).cuda(), strided(ck), strided(cv),
                         torch.from_numpy(cpos).cuda(), strided(hk), strided(hv), torch.from_numpy(hpos).cuda(), batch,
                         out_k, out_v, out_pos)
        assert fb.finch_device_status(ctx) == 0
        np.testing.assert_array_equal(to_host(out_k.contiguous(), "bf16"), want_k)
        np.testing.assert_array_equal(to_host(out_v.contiguous(), "bf16"), want_v)
        np.testing.assert_array_equal(out_pos.cpu().numpy(), want_p)
        # a kept index outside [0, N) is reported, not dereferenced
        bad = kept.copy()
        bad[0, 0, 1] = 10_000
        fb.finch_compact(ctx, torch.from_numpy(bad).cuda(), torch.from_numpy(out_len).cuda(), strided(ck), strided(cv),
                         torch.from_numpy(cpos).cuda(), strided(hk), strided(hv), torch.from_numpy(hpos).cuda(), batch,
                         out_k, out_v, out_pos)
        assert fb.finch_device_status(ctx) == fb.FINCH_DEV_BAD_INDEX
        assert fb.finch_device_status(ctx) == 0      # reading clears the word
    finally:
        fb.finch_ctx_destroy(ctx)


def test_inconsistent_device_metadata_sets_the_status_word():
    cfg = wl.scaled(wl.CONFIGS["c3"], n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=64,
                    requests=(wl.Request(8, 9999, 40, 16),))
    st = wl.steady_state(cfg, [0])
    g = GpuStep(cfg, st, 1)
    try:
        g.batch.cache_len.fill_(17)      # exceeds both the declared max_cache (16) and the capacity
        g.run()
        assert g.status() & fb.FINCH_DEV_BAD_BATCH
        assert int(g.out_len.cpu()[0]) == 0
        assert g.guards_intact()
    finally:
        g.close()


@pytest.mark.parametrize("which", ["q_off", "chunk_off", "cache_off"])
def test_device_offsets_outside_the_packed_tensors_set_the_status_word(which):
    """Offsets live in device memory and are only bounded by the host totals: a region that would start or end
    outside its packed tensor is refused by every kernel (status word, unit skipped), never dereferenced."""
    cfg = wl.scaled(wl.CONFIGS["c3"], n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=64,
                    requests=(wl.Request(8, 9999, 40, 16),))
    st = wl.steady_state(cfg, [0])
    g = GpuStep(cfg, st, 1)
    try:
        getattr(g.batch, which).add_(5)      # same lengths, shifted past the end of the packed tensor
        g.run()
        assert g.status() & fb.FINCH_DEV_BAD_BATCH
        assert int(g.out_len.cpu()[0]) == 0
        assert g.guards_intact()
        kept = g.kept_idx.cpu().numpy()
        assert (kept == -1).all(), "a refused unit must leave its outputs alone"
    finally:
        g.close()


def test_chunk_loop_on_gpu_matches_oracle_and_keeps_planted_keys():
    """Drive the whole document (Method, "Document Segmentation") with ping-pong caches that never leave the GPU.
    After every step the oracle re-scores the cache the GPU actually held, so the comparison stays within the
    stated tolerances even if a near-threshold key is swapped along the way."""
    import torch
    cfg = wl.scaled(wl.CONFIGS["c2"], n_layers=2, n_q_heads=8, n_kv_heads=4, head_dim=64,
                    requests=(wl.Request(64, 1024, 128, 96), wl.Request(20, 700, 128, 64)), planted_frac=0.03)
    L, B, Hkv, d = 2, cfg.batch, cfg.n_kv_heads, cfg.head_dim
    caps = [r.budget for r in cfg.requests]
    cache_off = wl.offsets(caps)
    q_np = np.stack([wl.to_storage(wl.prompt_q(cfg, l), cfg.dtype) for l in range(L)])
    q = to_device(q_np, cfg.dtype)
    zeros = np.zeros((L, Hkv, cache_off[-1], d), np.uint16)
    dev = [dict(k=to_device(zeros, "bf16"), v=to_device(zeros, "bf16"),
                pos=torch.full((L, cfg.n_groups, int(cache_off[-1])), -1, dtype=torch.int32, device="cuda"))
           for _ in range(2)]
    cache_len = np.zeros(B, np.int32)
    planted = [set() for _ in range(B)]
    budget = np.asarray(caps, np.int32)
    ctx = fb.finch_ctx_create(L, cfg.n_q_heads, Hkv, d, fb.FINCH_BF16, max_batch=B, max_prompt=64, max_candidates=256)
    try:
        for step in range(cfg.n_steps):
            chunks = [wl.chunk_kv(cfg, l, step) for l in range(L)]
            hk_np = np.stack([wl.to_storage(c["k"], cfg.dtype) for c in chunks])
            hv_np = np.stack([wl.to_storage(c["v"], cfg.dtype) for c in chunks])
            chunk_off, chunk_pos = chunks[0]["chunk_off"], chunks[0]["chunk_pos"]
            for b, r in enumerate(cfg.requests):
                planted[b] |= set((step * r.chunk + chunks[0]["planted"][b]).tolist())
            src, dst = dev[step % 2], dev[(step + 1) % 2]
            batch = fb.make_batch(wl.q_offsets(cfg), chunk_off, cache_off, cache_len, budget)
            ws = torch.empty(fb.finch_workspace_bytes(ctx, batch), dtype=torch.uint8, device="cuda")
            kept = torch.full((L, cfg.n_groups, int(cache_off[-1])), -1, dtype=torch.int32, device="cuda")
            out_len = torch.zeros(B, dtype=torch.int32, device="cuda")
            scores = torch.zeros((L, cfg.n_groups, int(cache_off[-1] + chunk_off[-1])), dtype=torch.float32,
                                 device="cuda")
            fb.finch_step(ctx, q, src["k"], src["v"], src["pos"], to_device(hk_np, "bf16"), to_device(hv_np, "bf16"),
                          torch.from_numpy(chunk_pos).cuda(), batch, dst["k"], dst["v"], dst["pos"], kept, out_len,
                          scores, ws)
            assert fb.finch_device_status(ctx) == 0
            st = dict(q=q_np, cache_k=to_host(src["k"], "bf16"), cache_v=to_host(src["v"], "bf16"),
                      cache_pos=src["pos"].cpu().numpy(), chunk_k=hk_np, chunk_v=hv_np, chunk_pos=chunk_pos,
                      q_off=wl.q_offsets(cfg), chunk_off=chunk_off, cache_off=cache_off, cache_len=cache_len,
                      budget=budget)
            res = dict(scores=scores.cpu().numpy(), kept_idx=kept.cpu().numpy(), out_len=out_len.cpu().numpy(),
                       out_pos=dst["pos"].cpu().numpy(), out_k=to_host(dst["k"], "bf16"),
                       out_v=to_host(dst["v"], "bf16"))
            check_parity(cfg, st, res, oracle_scores(cfg, st))
            cache_len = res["out_len"].copy()
    finally:
        fb.finch_ctx_destroy(ctx)
    assert cache_len.tolist() == caps
    final = dev[cfg.n_steps % 2]["pos"].cpu().numpy()
    for b in range(B):
        for l in range(L):
            for g in range(cfg.n_groups):
                assert planted[b] <= set(final[l, g, cache_off[b]:cache_off[b] + cache_len[b]].tolist())


def test_step_host_matches_step():
    """finch_step_host (inputs in pinned host memory, results read back) against finch_step on resident inputs."""
    import torch
    cfg = wl.scaled(wl.CONFIGS["c3"], n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=128,
                    requests=(wl.Request(128, 9999, 300, 200), wl.Request(40, 9999, 70, 90)))
    st = wl.steady_state(cfg, [0, 1], step=2)
    g = GpuStep(cfg, st, 2)
    try:
        g.run(scores=False)
        assert g.status() == 0
        want = g.results()
        host = {k: to_device(st[k], "bf16", "cpu").pin_memory() for k in ("q", "chunk_k", "chunk_v")}
        host_pos = torch.from_numpy(st["chunk_pos"]).pin_memory()
        stage = {k: torch.zeros_like(getattr(g, k)) for k in ("q", "chunk_k", "chunk_v")}
        stage_pos = torch.zeros_like(g.chunk_pos)
        out_k, out_v = torch.zeros_like(g.out_k), torch.zeros_like(g.out_v)
        out_pos, kept, out_len = torch.full_like(g.out_pos, -1), torch.full_like(g.kept_idx, -1), torch.zeros_like(g.out_len)
        host_kept = torch.full(kept.shape, -5, dtype=torch.int32).pin_memory()
        host_len = torch.full(out_len.shape, -5, dtype=torch.int32).pin_memory()
        for _ in range(2):
            fb.finch_step_host(g.ctx, host["q"], host["chunk_k"], host["chunk_v"], host_pos, stage["q"],
                               stage["chunk_k"], stage["chunk_v"], stage_pos, g.cache_k, g.cache_v, g.cache_pos,
                               g.batch, out_k, out_v, out_pos, kept, out_len, host_kept, host_len, g.ws)
            assert g.status() == 0
            np.testing.assert_array_equal(host_len.numpy(), want["out_len"])
            np.testing.assert_array_equal(host_kept.numpy(), want["kept_idx"])
            np.testing.assert_array_equal(to_host(out_k, "bf16"), want["out_k"])
            np.testing.assert_array_equal(to_host(out_v, "bf16"), want["out_v"])
            np.testing.assert_array_equal(out_pos.cpu().numpy(), want["out_pos"])
        # a staging tensor that is not dense is refused before anything is copied
        padded = torch.zeros((2, 8, g.q.shape[2], 256), dtype=torch.bfloat16, device="cuda")[:, :, :, :128]
        with pytest.raises(fb.FinchError) as e:
            fb.finch_step_host(g.ctx, host["q"], host["chunk_k"], host["chunk_v"], host_pos, padded,
                               stage["chunk_k"], stage["chunk_v"], stage_pos, g.cache_k, g.cache_v, g.cache_pos,
                               g.batch, out_k, out_v, out_pos, kept, out_len, host_kept, host_len, g.ws)
        assert e.value.status == fb.FINCH_ERR_BAD_LAYOUT
    finally:
        g.close()


@pytest.mark.parametrize("dtype,d,pairing,group_mode", [("bf16", 128, 0, 0), ("bf16", 64, 1, 1), ("f32", 64, 0, 0),
                                                        ("f32", 32, 1, 0)])
def test_compact_repositions_rotary_keys(dtype, d, pairing, group_mode):
    """Managing the Cache: with a rotary base configured, kept K rows are rotated by (output slot - candidate index)
    positions; V rows, positions and the plain-copy configuration are untouched.  Compared with the fp64 oracle: the
    GPU rotates in fp32 (angle reduced in double), so a stored value may differ from the oracle's rounding by one unit
    in the last place of the storage type on rare near-ties, never by more."""
    import torch
    rng = np.random.default_rng(7)
    L, Hkv, theta = 2, 4, 10000.0
    G = Hkv if group_mode == 0 else 1
    caps, lens, ms, budgets = [300, 64], [290, 50], [260, 70], [300, 40]
    cache_off, chunk_off = wl.offsets(caps), wl.offsets(ms)
    mk = lambda n: wl.to_storage(rng.standard_normal((L, Hkv, n, d)).astype(np.float32), dtype)
    ck, cv, hk, hv = mk(cache_off[-1]), mk(cache_off[-1]), mk(chunk_off[-1]), mk(chunk_off[-1])
    cpos = rng.integers(0, 1000, size=(L, G, cache_off[-1])).astype(np.int32)
    hpos = rng.integers(1000, 2000, size=chunk_off[-1]).astype(np.int32)
    scores = rng.random((L, G, cache_off[-1] + chunk_off[-1]))
    kept, out_len = oracle.select(scores, chunk_off=chunk_off, cache_off=cache_off, cache_len=lens, budget=budgets)
    kw = dict(n_kv_heads=Hkv, head_dim=d, group_mode=group_mode, chunk_off=chunk_off, cache_off=cache_off, cache_len=lens)
    want_k, want_v, want_p = oracle.compact(dtype, kept, out_len, ck, cv, cpos, hk, hv, hpos, rope_theta=theta,
                                            rope_pairing=pairing, **kw)
    plain_k, _, _ = oracle.compact(dtype, kept, out_len, ck, cv, cpos, hk, hv, hpos, **kw)
    assert not np.array_equal(want_k, plain_k)
    batch = fb.make_batch(wl.offsets([1, 1]), chunk_off, cache_off, lens, budgets)
    ctx = fb.finch_ctx_create(L, Hkv, Hkv, d, fb.FINCH_F32 if dtype == "f32" else fb.FINCH_BF16, group_mode,
                              max_batch=2, max_prompt=1, max_candidates=1024, rope_theta=theta, rope_pairing=pairing)
    try:
        dev = lambda a: to_device(a, dtype)
        out_k, out_v = dev(np.zeros_like(ck)), dev(np.zeros_like(cv))
        out_pos = torch.full((L, G, int(cache_off[-1])), -1, dtype=torch.int32, device="cuda")
        fb.finch_compact(ctx, torch.from_numpy(kept).cuda(), torch.from_numpy(out_len).cuda(), dev(ck), dev(cv),
                         torch.from_numpy(cpos).cuda(), dev(hk), dev(hv), torch.from_numpy(hpos).cuda(), batch,
                         out_k, out_v, out_pos)
        assert fb.finch_device_status(ctx) == 0
        np.testing.assert_array_equal(to_host(out_v, dtype), want_v)
        np.testing.assert_array_equal(out_pos.cpu().numpy(), want_p)
        got_bits, want_bits = to_host(out_k, dtype), want_k
        got = wl.from_storage(got_bits, dtype).astype(np.float64)
        want = wl.from_storage(want_bits, dtype).astype(np.float64)
        # fp32 sine, cosine and rotation: an absolute error of a few 1e-7 of the pair's length (bounded here by the
        # row's), which moves a stored bfloat16 by at most one unit in the last place, and only on near-ties
        row_scale = np.sqrt((want ** 2).sum(axis=-1, keepdims=True)) + 1e-30
        if dtype == "bf16":
            assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -7 + 2e-6 * row_scale)
            assert np.mean(got_bits != want_bits) < 2e-3                  # nearly all values identical
        else:
            assert np.all(np.abs(got - want) <= 2e-6 * row_scale)
    finally:
        fb.finch_ctx_destroy(ctx)
