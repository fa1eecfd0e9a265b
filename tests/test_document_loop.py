"""The chunk loop around the step: budget schedules (host logic) and the device-resident driver."""
import numpy as np
import pytest

from paper_2408_00167_b200 import document as doc


def test_paper_schedule_grows_linearly_and_ends_at_the_target():
    # r_{it+1} = m/sigma + c_it with equal chunks: the cache grows by m/sigma per step ("Selection of top r
    # position"); the last step's r is the target size k
    budgets = doc.paper_budgets([2048] * 16, sigma=16, k=2048)
    assert budgets[:15] == [128 * (it + 1) for it in range(15)]
    assert budgets[-1] == 2048
    # a ragged last chunk and a non-integer ratio: rounded down, never above what is available
    budgets = doc.paper_budgets([100, 100, 37], sigma=3, k=50)
    assert budgets == [33, 66, 50]
    assert doc.fixed_budgets(3, 7) == [7, 7, 7]


def test_paper_schedule_first_step_keeps_a_sigma_th_of_the_chunk():
    assert doc.paper_budgets([512, 512], sigma=4, k=200)[0] == 128


@pytest.mark.gpu
@pytest.mark.parametrize("group_mode,schedule", [(0, "fixed"), (1, "paper")])
def test_document_driver_matches_the_oracle_step_by_step(group_mode, schedule):
    """The driver's caches never leave the GPU between steps; after every step the oracle re-scores the cache the GPU
    actually held, so the comparison stays within tolerance even if a near-threshold key was swapped earlier."""
    import torch
    from paper_2408_00167_b200 import binding as fb, workloads as wl
    from parity_harness import check_parity, oracle_scores, to_device, to_host
    cfg = wl.scaled(wl.CONFIGS["c2"], n_layers=2, n_q_heads=8, n_kv_heads=4, head_dim=64, group_mode=group_mode,
                    requests=(wl.Request(64, 1024, 128, 96), wl.Request(20, 700, 128, 64)), planted_frac=0.03)
    L, B = 2, cfg.batch
    caps = [r.budget for r in cfg.requests]
    if schedule == "paper":
        per_req = [doc.paper_budgets([r.chunk_len(s) for s in range(r.n_steps)], sigma=r.text_len / r.budget, k=r.budget)
                   for r in cfg.requests]
    else:
        per_req = [doc.fixed_budgets(r.n_steps, r.budget) for r in cfg.requests]
    q_np = np.stack([wl.to_storage(wl.prompt_q(cfg, l), cfg.dtype) for l in range(L)])
    q = to_device(q_np, cfg.dtype)
    drv = doc.DocumentCompressor(L, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, fb.FINCH_BF16, caps, max_prompt=64,
                                 max_chunk=128, group_mode=group_mode)
    planted = [set() for _ in range(B)]
    try:
        for step in range(cfg.n_steps):
            chunks = [wl.chunk_kv(cfg, l, step) for l in range(L)]
            hk_np = np.stack([wl.to_storage(c["k"], cfg.dtype) for c in chunks])
            hv_np = np.stack([wl.to_storage(c["v"], cfg.dtype) for c in chunks])
            chunk_off, chunk_pos = chunks[0]["chunk_off"], chunks[0]["chunk_pos"]
            budget = np.array([per_req[b][min(step, len(per_req[b]) - 1)] for b in range(B)], np.int32)
            for b, r in enumerate(cfg.requests):
                planted[b] |= set((step * r.chunk + chunks[0]["planted"][b]).tolist())
            before = dict(cache_k=to_host(drv.cache_k, "bf16"), cache_v=to_host(drv.cache_v, "bf16"),
                          cache_pos=drv.cache_pos.cpu().numpy(), cache_len=drv.cache_len.copy())
            scores = torch.zeros((L, cfg.n_groups, int(drv.cache_off[-1] + chunk_off[-1])), dtype=torch.float32,
                                 device="cuda")
            drv.step(q, wl.q_offsets(cfg), to_device(hk_np, "bf16"), to_device(hv_np, "bf16"),
                     torch.from_numpy(chunk_pos).cuda(), chunk_off, budget, scores=scores)
            assert drv.status() == 0
            st = dict(q=q_np, chunk_k=hk_np, chunk_v=hv_np, chunk_pos=chunk_pos, q_off=wl.q_offsets(cfg),
                      chunk_off=chunk_off, cache_off=drv.cache_off, budget=budget, **before)
            out_len = drv._bufs[drv._cur]["len"].cpu().numpy()
            np.testing.assert_array_equal(out_len[:B], drv.cache_len)      # the host mirror is exact
            res = dict(scores=scores.cpu().numpy(), kept_idx=drv.kept_idx.cpu().numpy(), out_len=out_len,
                       out_pos=drv.cache_pos.cpu().numpy(), out_k=to_host(drv.cache_k, "bf16"),
                       out_v=to_host(drv.cache_v, "bf16"))
            check_parity(cfg, st, res, oracle_scores(cfg, st))
        assert drv.cache_len.tolist() == caps
        final = drv.cache_pos.cpu().numpy()
        if schedule == "fixed":      # with the full target at every step no planted key is ever at risk
            for b in range(B):
                for l in range(L):
                    for g in range(cfg.n_groups):
                        lo = int(drv.cache_off[b])
                        assert planted[b] <= set(final[l, g, lo:lo + caps[b]].tolist())
    finally:
        drv.close()
