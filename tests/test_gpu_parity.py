"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded inputs."""
import numpy as np
import pytest

import oracle
from paper_2408_00167_b200 import binding as fb
from paper_2408_00167_b200 import build as fbuild
from paper_2408_00167_b200 import workloads as wl
from parity_harness import GpuStep, check_parity, oracle_scores

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    fbuild.build()
    fb.load()


def _small(name, dtype, Hq, Hkv, d, reqs, L=2, group_mode=0, **kw):
    return wl.scaled(wl.CONFIGS[name], n_layers=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, dtype=dtype,
                     requests=tuple(wl.Request(*r) for r in reqs), group_mode=group_mode, **kw)


def _run_and_check(cfg, st, L, parts=False, group_mode=None, check_scores=True):
    g = GpuStep(cfg, st, L, group_mode=group_mode)
    try:
        (g.run_parts() if parts else g.run())
        assert g.status() == 0
        res = g.results()
        ref = oracle_scores(cfg, st, group_mode=group_mode)
        summary = check_parity(cfg, st, res, ref, group_mode=group_mode, check_scores=check_scores)
        # determinism: a second run gives identical bytes
        (g.run_parts() if parts else g.run())
        res2 = g.results()
        for k in ("scores", "kept_idx", "out_k", "out_v", "out_pos"):
            np.testing.assert_array_equal(res[k], res2[k], err_msg=f"{k} differs between two runs")
        return summary, res, g
    finally:
        g.close()


def test_config1_tiny_fp32_step():
    cfg = wl.CONFIGS["c1"]
    st = wl.steady_state(cfg, [0])
    summary, res, _ = _run_and_check(cfg, st, 1)
    assert summary["units"] == 8
    for g in range(8):     # planted keys are always retained
        assert set(st["planted"][0].tolist()) <= set(res["kept_idx"][0, g, :256].tolist())


# (n_q, text_len, chunk, budget): candidates = budget + chunk, chosen to leave ragged tails in every tile size
SHAPES = [
    ("f32", 4, 2, 64, [(1, 999, 37, 50)]),
    ("f32", 2, 2, 32, [(70, 999, 130, 65)]),
    ("bf16", 8, 2, 128, [(16, 9999, 200, 100)]),
    ("bf16", 4, 4, 64, [(63, 9999, 129, 64)]),
    ("bf16", 8, 2, 128, [(5, 9999, 64, 17), (33, 9999, 100, 300), (20, 9999, 1, 1)]),
    # partial row blocks, partial key tiles on both sides of the cache/chunk seam
    ("bf16", 8, 2, 128, [(130, 9999, 300, 333)]),
    ("bf16", 4, 2, 64, [(64, 9999, 1, 129), (257, 9999, 257, 255), (40, 9999, 90, 70)]),
    # single requests whose query rows fill three and two 128-row tiles per KV head (three heads x 100 rows: the
    # tiles do not divide the four softmax groups; two heads x 100 rows: two groups per tile)
    ("bf16", 6, 2, 64, [(100, 9999, 290, 260)]),
    ("bf16", 4, 2, 128, [(100, 9999, 390, 270)]),
]


@pytest.mark.parametrize("dtype,Hq,Hkv,d,reqs", SHAPES)
@pytest.mark.parametrize("group_mode", [0, 1])
def test_small_shapes_with_ragged_tails(dtype, Hq, Hkv, d, reqs, group_mode):
    cfg = _small("c3", dtype, Hq, Hkv, d, reqs, group_mode=group_mode, planted_frac=0.03)
    st = wl.steady_state(cfg, [0, 1], step=3)
    _run_and_check(cfg, st, 2, parts=(group_mode == 1))


@pytest.mark.parametrize("scale", [6.0, 40.0])
def test_wide_logit_range_on_the_tensor_core_path(scale):
    # logits spread over hundreds (scale 6) or thousands (scale 40) of binary orders: the row sums, taken against the
    # maximum of the first 32 keys only, overflow in later chunks and have to move their reference
    cfg = _small("c3", "bf16", 8, 2, 128, [(130, 9999, 300, 333), (20, 9999, 40, 250)], planted_frac=0.03)
    st = wl.steady_state(cfg, [0, 1], step=2)
    g = GpuStep(cfg, st, 2, scale=scale)
    try:
        g.run_parts()
        assert g.status() == 0
        res = g.results()
        ref, ref_lse = oracle_scores(cfg, st, scale=scale, want_lse=True)
        summary = check_parity(cfg, st, res, ref)
        assert summary["max_rel_err"] < 1e-3
        valid = ~np.isnan(res["row_lse"])
        np.testing.assert_allclose(res["row_lse"][valid], ref_lse[valid], rtol=2e-6, atol=2e-4)
    finally:
        g.close()


@pytest.mark.parametrize("dtype,Hq,Hkv,d,reqs,group_mode", [
    ("bf16", 8, 2, 128, [(130, 9999, 300, 333), (20, 9999, 40, 250)], 0),   # tensor-core path
    ("f32", 4, 2, 64, [(70, 999, 130, 65), (3, 999, 20, 10)], 0),            # warp-level path
    ("f32", 4, 2, 32, [(33, 999, 50, 40)], 1),                               # warp-level path, per-layer groups
    ("bf16", 4, 2, 64, [(40, 9999, 90, 70)], 1),                             # per-layer groups (tensor-core path, heads summed)
])
def test_prompt_self_term_in_the_softmax_denominator(dtype, Hq, Hkv, d, reqs, group_mode):
    # the full attention row of a prompt token also covers the prompt's own keys (Method, "N = m + n^que + c"):
    # their log-sum-exp per row enters the denominator; rows with -inf behave as without the term
    cfg = _small("c3", dtype, Hq, Hkv, d, reqs, group_mode=group_mode, planted_frac=0.03)
    st = wl.steady_state(cfg, [0, 1], step=2)
    rng = np.random.default_rng(5)
    total_q = int(st["q_off"][-1])
    _, base_lse = oracle_scores(cfg, st, group_mode=group_mode, want_lse=True)
    self_lse = base_lse + rng.normal(0.0, 2.0, size=base_lse.shape)      # comparable to the candidates' own mass
    self_lse[rng.random(self_lse.shape) < 0.2] = -np.inf
    self_lse = self_lse.astype(np.float32).astype(np.float64)
    assert self_lse.shape == (2, Hq, total_q)
    g = GpuStep(cfg, st, 2, group_mode=group_mode, prompt_self_lse=self_lse)
    try:
        g.run_parts()
        assert g.status() == 0
        res = g.results()
        ref, ref_lse = oracle_scores(cfg, st, group_mode=group_mode, want_lse=True, prompt_self_lse=self_lse)
        plain = oracle_scores(cfg, st, group_mode=group_mode)
        assert np.abs(ref - plain).max() > 0.05                           # the term matters in this test
        summary = check_parity(cfg, st, res, ref, group_mode=group_mode)
        assert summary["max_rel_err"] < 1e-4
        np.testing.assert_allclose(res["row_lse"], ref_lse, rtol=2e-5, atol=2e-5)
    finally:
        g.close()


@pytest.mark.parametrize("dtype,Hq,Hkv,d,reqs,group_mode,row_norm", [
    ("bf16", 8, 2, 128, [(150, 9999, 120, 60), (20, 9999, 15, 30)], 0, False),
    ("bf16", 4, 2, 64, [(90, 9999, 70, 40)], 1, True),
    ("f32", 4, 4, 32, [(70, 999, 64, 10), (5, 999, 3, 8)], 0, True),
])
def test_causal_query_rows_and_per_row_normalisation(dtype, Hq, Hkv, d, reqs, group_mode, row_norm):
    # the conditioning ablation: the chunk's own tokens are query rows, each seeing the cache and the chunk up to
    # itself; the last rows of every request stand for prompt rows and see everything; one row sees nothing at all
    cfg = _small("c3", dtype, Hq, Hkv, d, reqs, group_mode=group_mode, planted_frac=0.03)
    st = wl.steady_state(cfg, [0, 1], step=2)
    limit = np.zeros(int(st["q_off"][-1]), np.int32)
    for b in range(cfg.batch):
        n_q = int(st["q_off"][b + 1] - st["q_off"][b])
        c = int(st["cache_len"][b])
        N = c + int(st["chunk_off"][b + 1] - st["chunk_off"][b])
        rows = np.minimum(c + np.arange(n_q) + 1, N)
        rows[-3:] = N + 7                                   # "prompt" rows; a limit beyond N is no limit
        limit[st["q_off"][b]:st["q_off"][b + 1]] = rows
    limit[1] = 0                                            # sees nothing: contributes nothing
    g = GpuStep(cfg, st, 2, group_mode=group_mode, row_limit=limit, row_norm=row_norm)
    try:
        g.run_parts()
        assert g.status() == 0
        res = g.results()
        ref, ref_lse = oracle_scores(cfg, st, group_mode=group_mode, want_lse=True, row_limit=limit, row_norm=row_norm)
        assert np.abs(ref - oracle_scores(cfg, st, group_mode=group_mode)).max() > 0.05
        summary = check_parity(cfg, st, res, ref, group_mode=group_mode)
        assert summary["max_rel_err"] < 1e-4
        finite = np.isfinite(ref_lse)
        np.testing.assert_allclose(res["row_lse"][finite], ref_lse[finite], rtol=2e-5, atol=2e-5)
        assert np.all(np.isneginf(res["row_lse"][np.isneginf(ref_lse)]))
    finally:
        g.close()


def test_row_lse_output_matches_oracle():
    cfg = _small("c3", "bf16", 4, 2, 64, [(9, 9999, 70, 40), (64, 9999, 30, 90)])
    st = wl.steady_state(cfg, [0, 1], step=2)
    g = GpuStep(cfg, st, 2)
    try:
        g.run_parts()
        assert g.status() == 0
        _, lse = oracle_scores(cfg, st, want_lse=True)
        np.testing.assert_allclose(g.results()["row_lse"], lse, rtol=2e-5, atol=2e-5)
    finally:
        g.close()


def test_empty_and_degenerate_requests():
    # request 0: empty cache; request 1: empty chunk; request 2: nothing at all; request 3: budget 0
    cfg = _small("c3", "bf16", 4, 2, 64, [(8, 9999, 40, 16), (8, 9999, 40, 16), (8, 9999, 40, 16), (8, 9999, 40, 16)])
    st = wl.steady_state(cfg, [0], step=2)
    st["cache_len"] = np.array([0, 16, 0, 16], np.int32)
    chunk_lens = [40, 0, 0, 40]
    new_off = wl.offsets(chunk_lens)
    keep = np.concatenate([np.arange(st["chunk_off"][b], st["chunk_off"][b] + chunk_lens[b]) for b in range(4)])
    for k in ("chunk_k", "chunk_v"):
        st[k] = np.ascontiguousarray(st[k][:, :, keep])
    st["chunk_pos"] = st["chunk_pos"][keep]
    st["chunk_off"] = new_off
    st["budget"] = np.array([16, 10, 5, 0], np.int32)
    summary, res, _ = _run_and_check(cfg, st, 1)
    assert res["out_len"].tolist() == [16, 10, 0, 0]


def test_request_without_prompt_rows_scores_zero_and_keeps_the_first_rows():
    # the sum over no prompt rows is zero for every key: all candidates tie and the lowest indices are kept
    cfg = _small("c3", "bf16", 4, 2, 64, [(70, 9999, 40, 16), (0, 9999, 30, 16), (8, 9999, 20, 16)], planted_frac=0.0)
    st = wl.steady_state(cfg, [0, 1], step=2)
    summary, res, _ = _run_and_check(cfg, st, 2)
    lo = int(st["cache_off"][1] + st["chunk_off"][1])
    assert np.all(res["scores"][:, :, lo:lo + 46] == 0.0)
    np.testing.assert_array_equal(res["kept_idx"][:, :, 16:32], np.broadcast_to(np.arange(16), (2, 2, 16)))


@pytest.mark.parametrize("budget", [0, 1, 63, 104, 105, 500])
def test_budget_edges(budget):
    cfg = _small("c3", "bf16", 4, 2, 64, [(12, 9999, 65, 40)])
    st = wl.steady_state(cfg, [0], step=2)
    st["budget"] = np.array([min(budget, 40)], np.int32)   # capacity is 40 rows
    _run_and_check(cfg, st, 1)
    # a budget at or above the candidate count is the identity: needs capacity >= N
    cfg2 = _small("c3", "bf16", 4, 2, 64, [(12, 9999, 25, 120)])
    st2 = wl.steady_state(cfg2, [0], step=2)
    st2["cache_len"] = np.array([80], np.int32)            # N = 105 <= capacity 120
    st2["budget"] = np.array([min(budget, 120)], np.int32)
    _, res, _ = _run_and_check(cfg2, st2, 1)
    if budget >= 105:
        np.testing.assert_array_equal(res["kept_idx"][0, :, :105], np.broadcast_to(np.arange(105), (2, 105)))


def test_large_scale_gives_massive_exact_ties():
    # a huge logit scale makes every softmax row an indicator: scores are small integers with many ties
    cfg = _small("c3", "bf16", 4, 2, 64, [(24, 9999, 300, 200)], planted_frac=0.0)
    st = wl.steady_state(cfg, [0], step=2)
    g = GpuStep(cfg, st, 1, scale=4096.0)
    try:
        g.run()
        assert g.status() == 0
        res = g.results()
        ref = oracle_scores(cfg, st, scale=4096.0)
        assert np.abs(np.round(ref[0, :, :500]) - ref[0, :, :500]).max() < 1e-30        # integers
        assert len(np.unique(ref[0, 0, :500])) < 12
        np.testing.assert_allclose(res["scores"][0, :, :500], ref[0, :, :500], rtol=2e-6, atol=1e-6)
        check_parity(cfg, st, res, ref)
    finally:
        g.close()
