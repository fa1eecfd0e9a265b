"""finch_score_static: the scoring call for hosts that may not allocate device memory.

Some users of the library run where cudaMalloc is not an option (a plugin inside a server whose memory pool owns
the device, a step that must not touch the driver's allocator).  They call finch_score_static, whose scratch is a
fixed array inside the library instead of a caller-supplied workspace.  These tests check that it returns what
finch_score returns, call after call, although every call reuses the same array, and that it refuses batches that
do not fit the array.  The array is 8 MiB; the tensor-core kernels need more of it than one entry per prompt row, so a
batch with few prompt rows but very many candidates stays within the row limit and still has to run on the warp-level
kernels: that case is driven on purpose, and both kinds of batch are compared with the fp64 oracle, not only with
finch_score.  The file is named to be collected last.
"""
import ctypes as C

import numpy as np
import pytest

from paper_2408_00167_b200 import binding as fb
from paper_2408_00167_b200 import build as fbuild
from paper_2408_00167_b200 import workloads as wl
from parity_harness import ABS_TOL, REL_TOL, GpuStep, oracle_scores


@pytest.fixture(scope="module", autouse=True)
def _built():
    fbuild.build()
    fb.load()


def _case(reqs, step):
    cfg = wl.scaled(wl.CONFIGS["c3"], n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64,
                    requests=tuple(wl.Request(*r) for r in reqs), planted_frac=0.02)
    return cfg, wl.steady_state(cfg, [0, 1], step=step)


@pytest.mark.gpu
def test_static_scratch_matches_workspace_version_on_consecutive_calls():
    import torch
    # two different batches back to back: the second call finds the first call's leftovers in the shared array
    cases = [_case([(70, 9999, 150, 90), (9, 9999, 40, 33)], 2), _case([(33, 9999, 100, 260)], 3)]
    for cfg, st in cases:
        g = GpuStep(cfg, st, 2)
        try:
            fb.finch_score(g.ctx, g.q, g.cache_k, g.chunk_k, g.batch, g.scores, g.row_lse, g.ws)
            want, want_lse = g.scores.clone(), g.row_lse.clone()
            for _ in range(2):                                   # and the same batch twice in a row
                got = torch.full_like(g.scores, float("nan"))
                got_lse = torch.full_like(g.row_lse, float("nan"))
                fb.finch_score_static(g.ctx, g.q, g.cache_k, g.chunk_k, g.batch, got, got_lse)
                assert g.status() == 0
                w, x = want.cpu().numpy(), got.cpu().numpy()
                valid = ~np.isnan(w)
                assert valid.any() and np.array_equal(valid, ~np.isnan(x))
                err = np.abs(x[valid] - w[valid])
                assert np.all(err <= np.maximum(REL_TOL * np.abs(w[valid]), ABS_TOL))
                np.testing.assert_allclose(got_lse.cpu().numpy(), want_lse.cpu().numpy(), rtol=1e-5, atol=1e-5)
        finally:
            g.close()


@pytest.mark.gpu
@pytest.mark.parametrize("reqs,tensor_cores", [
    ([(40, 10 ** 7, 700, 300)], True),          # a small batch: the tensor-core kernels fit the array
    ([(33, 10 ** 7, 140_000, 200)], False),     # 4 units x 140 200 candidates of partial sums do not: warp-level kernels
])
def test_static_scratch_on_both_kernel_paths_against_the_oracle(reqs, tensor_cores):
    import torch
    cfg, st = _case(reqs, 1)
    g = GpuStep(cfg, st, 2)
    try:
        assert fb.finch_score_static_path(g.ctx, g.batch) is tensor_cores
        ref = oracle_scores(cfg, st, threads=8)
        fb.finch_score(g.ctx, g.q, g.cache_k, g.chunk_k, g.batch, g.scores, g.row_lse, g.ws)   # always tensor cores
        want = g.scores.clone()
        for _ in range(2):
            got = torch.full_like(g.scores, float("nan"))
            fb.finch_score_static(g.ctx, g.q, g.cache_k, g.chunk_k, g.batch, got, None)
            assert g.status() == 0
            for name, x in (("static", got), ("workspace", want)):
                x = x.cpu().numpy().astype(np.float64)
                assert not np.isnan(x).any()
                bad = np.abs(x - ref) > np.maximum(REL_TOL * np.abs(ref), ABS_TOL)
                assert not bad.any(), f"{name}: {int(bad.sum())} scores outside the tolerance"
    finally:
        g.close()


def test_static_scratch_rejects_batches_beyond_its_size():
    """Host-side check, no GPU needed: a validation-only context still applies the size limit first."""
    limit = fb.finch_score_static_max_rows()
    assert limit == 1 << 20
    ctx = fb.finch_ctx_create(32, 32, 8, 64, fb.FINCH_BF16, max_batch=1, max_prompt=4096, max_candidates=8192,
                              device=-1)
    try:
        base = 0x7000_0000_0000

        def call(total_q):
            b = fb.finch_batch(1, base, base + 256, base + 512, base + 768, base + 1024, total_q, 512, 256,
                               min(total_q, 4096), 256, 512, 256)
            t = lambda slot, tok, heads: fb.finch_tensor(base + 0x1000_0000 * slot, heads * tok * 64, tok * 64, 64)
            q, ck, hk = t(1, total_q, 32), t(2, 256, 8), t(3, 512, 8)
            return fb.load().finch_score_static(ctx, C.byref(q), C.byref(ck), C.byref(hk), C.byref(b),
                                                C.c_void_p(base + 0x9000_0000), None, None)
        assert call(limit // (32 * 32)) == fb.FINCH_ERR_UNSUPPORTED            # fits: stops only at the launch
        assert call(limit // (32 * 32) + 1) == fb.FINCH_ERR_WORKSPACE_TOO_SMALL
    finally:
        fb.finch_ctx_destroy(ctx)
