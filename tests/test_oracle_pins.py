"""Pins for the fp64 CPU oracle: what the paper and the mathematics fix, independent of the oracle's own code.

Each test is chosen so that a plausible mistake in the oracle (dropped term, wrong sign or index, transposed
operand, wrong head-to-KV-head map, wrong tie rule) fails at least one of them.
"""
import itertools
import math
from fractions import Fraction
from pathlib import Path

import numpy as np
import pytest

import oracle
from paper_2408_00167_b200 import workloads as wl

GOLDEN = Path(__file__).resolve().parent / "golden"


def _dense(rng, L, Hq, Hkv, nq, c, m, d, dtype="f32", cap=None):
    """Single-request dense inputs in storage form."""
    cap = c if cap is None else cap
    q = wl.to_storage(rng.standard_normal((L, Hq, nq, d)), dtype)
    ck = wl.to_storage(rng.standard_normal((L, Hkv, cap, d)), dtype)
    hk = wl.to_storage(rng.standard_normal((L, Hkv, m, d)), dtype)
    meta = dict(q_off=[0, nq], chunk_off=[0, m], cache_off=[0, cap], cache_len=[c])
    return q, ck, hk, meta


def _score(dtype, q, ck, hk, meta, Hq, Hkv, d, **kw):
    return oracle.score(dtype, q, ck, hk, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, **meta, **kw)


def _numpy_scores(q, ck, hk, c, Hq, Hkv, scale, group_mode=0):
    """Textbook restatement with numpy: softmax(QK^T * scale) over keys, summed over prompt rows and group heads."""
    qf, kf = q.astype(np.float64), np.concatenate([ck[:, :, :c], hk], axis=2).astype(np.float64)
    g = Hq // Hkv
    k_per_qhead = np.repeat(kf, g, axis=1)                       # query head h reads KV head h // g
    s = np.einsum("lhpd,lhjd->lhpj", qf, k_per_qhead) * scale
    s = s - s.max(axis=-1, keepdims=True)
    w = np.exp(s)
    w /= w.sum(axis=-1, keepdims=True)
    per_head = w.sum(axis=2)                                     # [L][Hq][N]
    if group_mode == 0:
        return per_head.reshape(per_head.shape[0], Hkv, g, -1).sum(axis=2)
    return per_head.sum(axis=1, keepdims=True)


# ----------------------------------------------------------------------------- scoring

def test_single_candidate_scores_group_rows():
    # A key that is the only visible one gets softmax weight 1 from every row (Method, positional-bias paragraph).
    rng = np.random.default_rng(1)
    q, ck, hk, meta = _dense(rng, 2, 4, 2, 5, 0, 1, 8)
    s = _score("f32", q, ck, hk, meta, 4, 2, 8)
    assert s.shape == (2, 2, 1)
    np.testing.assert_array_equal(s, np.full((2, 2, 1), 2 * 5.0))


def test_two_candidates_logistic_closed_form():
    rng = np.random.default_rng(2)
    d, nq = 16, 3
    q, ck, hk, meta = _dense(rng, 1, 1, 1, nq, 1, 1, d)
    s = _score("f32", q, ck, hk, meta, 1, 1, d)[0, 0]
    k0, k1 = ck[0, 0, 0].astype(np.float64), hk[0, 0, 0].astype(np.float64)
    expect0 = sum(1.0 / (1.0 + math.exp(float(np.dot(q[0, 0, p].astype(np.float64), k1 - k0)) / math.sqrt(d)))
                  for p in range(nq))
    assert s[0] == pytest.approx(expect0, rel=1e-13)
    assert s[1] == pytest.approx(nq - expect0, rel=1e-13)


def test_uniform_when_keys_identical_or_queries_zero():
    rng = np.random.default_rng(3)
    L, Hq, Hkv, nq, c, m, d = 1, 4, 2, 3, 4, 5, 8
    q, ck, hk, meta = _dense(rng, L, Hq, Hkv, nq, c, m, d)
    ck[:] = ck[:, :, :1]
    hk[:] = ck[:, :, :1]
    s = _score("f32", q, ck, hk, meta, Hq, Hkv, d)
    np.testing.assert_allclose(s, (Hq // Hkv) * nq / (c + m), rtol=1e-14)
    q2, ck2, hk2, meta2 = _dense(rng, L, Hq, Hkv, nq, c, m, d)
    q2[:] = 0
    s2 = _score("f32", q2, ck2, hk2, meta2, Hq, Hkv, d)
    np.testing.assert_allclose(s2, (Hq // Hkv) * nq / (c + m), rtol=1e-14)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("group_mode", [0, 1])
def test_matches_numpy_restatement_and_rows_sum_to_one(dtype, group_mode):
    rng = np.random.default_rng(4)
    L, Hq, Hkv, nq, c, m, d, cap = 2, 6, 3, 7, 9, 6, 16, 12
    q, ck, hk, meta = _dense(rng, L, Hq, Hkv, nq, c, m, d, dtype, cap=cap)
    s = _score(dtype, q, ck, hk, meta, Hq, Hkv, d, group_mode=group_mode)
    G = Hkv if group_mode == 0 else 1
    assert s.shape == (L, G, cap + m)
    ref = _numpy_scores(wl.from_storage(q, dtype), wl.from_storage(ck, dtype), wl.from_storage(hk, dtype),
                        c, Hq, Hkv, 1 / math.sqrt(d), group_mode)
    np.testing.assert_allclose(s[:, :, :c + m], ref, rtol=1e-12, atol=1e-15)
    np.testing.assert_array_equal(s[:, :, c + m:], 0.0)            # capacity slack is left untouched
    np.testing.assert_allclose(s.sum(axis=-1), (Hq // G) * nq, rtol=1e-13)   # softmax rows sum to 1


def test_mpmath_second_opinion():
    mp = pytest.importorskip("mpmath")
    mp.mp.dps = 50
    rng = np.random.default_rng(5)
    Hq, Hkv, nq, c, m, d = 2, 1, 2, 2, 3, 4
    q, ck, hk, meta = _dense(rng, 1, Hq, Hkv, nq, c, m, d)
    q *= 6                                                       # peaked softmax: exercises the max-shift
    s = _score("f32", q, ck, hk, meta, Hq, Hkv, d, scale=0.5)[0, 0]
    keys = [ck[0, 0, j] for j in range(c)] + [hk[0, 0, j] for j in range(m)]
    acc = [mp.mpf(0)] * (c + m)
    for h in range(Hq):
        for p in range(nq):
            logits = [mp.mpf("0.5") * sum(mp.mpf(float(a)) * mp.mpf(float(b)) for a, b in zip(q[0, h, p], k))
                      for k in keys]
            Z = sum(mp.e ** x for x in logits)
            acc = [a + mp.e ** x / Z for a, x in zip(acc, logits)]
    for j in range(c + m):
        assert float(abs(mp.mpf(float(s[j])) - acc[j]) / acc[j]) < 1e-13


def test_shift_invariance_and_permutation_equivariance():
    rng = np.random.default_rng(6)
    L, Hq, Hkv, nq, c, m, d = 1, 4, 2, 5, 6, 7, 8
    q, ck, hk, meta = _dense(rng, L, Hq, Hkv, nq, c, m, d)
    base = _score("f32", q, ck, hk, meta, Hq, Hkv, d)
    u = rng.integers(-2, 3, size=d).astype(np.float32)           # exactly representable shift
    ck_i = np.round(ck * 4) / 4
    hk_i = np.round(hk * 4) / 4
    q_i = np.round(q * 4) / 4
    s0 = _score("f32", q_i, ck_i, hk_i, meta, Hq, Hkv, d)
    s1 = _score("f32", q_i, ck_i + u, hk_i + u, meta, Hq, Hkv, d)
    np.testing.assert_allclose(s1, s0, rtol=1e-12)               # a per-row constant cancels in the softmax
    perm = rng.permutation(c + m)
    allk = np.concatenate([ck, hk], axis=2)[:, :, perm]
    sp = _score("f32", q, np.ascontiguousarray(allk[:, :, :c]), np.ascontiguousarray(allk[:, :, c:]), meta,
                Hq, Hkv, d)
    np.testing.assert_allclose(sp, base[:, :, perm], rtol=1e-12)


def test_gqa_head_mapping_is_block_not_interleaved():
    # Only query heads 2,3 (KV head 1) see a distinguishing key; group 1 must react, group 0 must stay uniform.
    d, nq, N = 8, 2, 4
    q = np.zeros((1, 4, nq, d), np.float32)
    q[0, 2:, :, 0] = 5.0
    ck = np.zeros((1, 2, 0, d), np.float32)
    hk = np.zeros((1, 2, N, d), np.float32)
    hk[0, :, 1, 0] = 4.0
    meta = dict(q_off=[0, nq], chunk_off=[0, N], cache_off=[0, 0], cache_len=[0])
    s = _score("f32", q, ck, hk, meta, 4, 2, d)
    np.testing.assert_allclose(s[0, 0], 2 * nq / N, rtol=1e-14)
    assert s[0, 1, 1] > 0.99 * 2 * nq


def test_row_lse_matches_definition():
    rng = np.random.default_rng(7)
    L, Hq, Hkv, nq, c, m, d = 1, 4, 2, 3, 2, 4, 8
    q, ck, hk, meta = _dense(rng, L, Hq, Hkv, nq, c, m, d)
    _, lse = _score("f32", q, ck, hk, meta, Hq, Hkv, d, want_lse=True)
    kf = np.repeat(np.concatenate([ck, hk], axis=2).astype(np.float64), 2, axis=1)
    logits = np.einsum("lhpd,lhjd->lhpj", q.astype(np.float64), kf) / math.sqrt(d)
    np.testing.assert_allclose(lse, np.log(np.exp(logits).sum(-1)), rtol=1e-13)


def test_prompt_self_term_equals_full_row_softmax_over_candidates_and_prompt_keys():
    # In the full forward pass a prompt row attends to the candidates and, causally, to the prompt's own keys
    # ("N = m + n^que + c", Method).  Restated with numpy on the explicit concatenated key set: the candidate columns
    # of that softmax, summed over rows and heads, must equal the oracle fed with the prompt keys' log-sum-exp only.
    rng = np.random.default_rng(21)
    L, Hq, Hkv, nq, c, m, d = 2, 4, 2, 6, 7, 5, 8
    q, ck, hk, meta = _dense(rng, L, Hq, Hkv, nq, c, m, d)
    kp = rng.standard_normal((L, Hkv, nq, d)).astype(np.float32)          # the prompt's own keys
    scale, g = 1.0 / math.sqrt(d), Hq // Hkv
    cand = np.concatenate([ck[:, :, :c], hk], axis=2).astype(np.float64)
    keys = np.repeat(np.concatenate([cand, kp.astype(np.float64)], axis=2), g, axis=1)   # [L][Hq][N + nq][d]
    s = np.einsum("lhpd,lhjd->lhpj", q.astype(np.float64), keys) * scale
    causal = np.tril(np.ones((nq, nq), bool))                              # prompt row p sees prompt keys t <= p
    s[..., c + m:] = np.where(causal, s[..., c + m:], -np.inf)
    w = np.exp(s - s.max(axis=-1, keepdims=True))
    w /= w.sum(axis=-1, keepdims=True)
    want = w[..., :c + m].sum(axis=2).reshape(L, Hkv, g, c + m).sum(axis=2)
    sp = s[..., c + m:]
    self_lse = sp.max(axis=-1) + np.log(np.exp(sp - sp.max(axis=-1, keepdims=True)).sum(axis=-1))
    got, lse = _score("f32", q, ck, hk, meta, Hq, Hkv, d, prompt_self_lse=self_lse, want_lse=True)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)
    full_lse = s.max(axis=-1) + np.log(np.exp(s - s.max(axis=-1, keepdims=True)).sum(axis=-1))
    np.testing.assert_allclose(lse, full_lse, rtol=1e-12)
    # the prompt takes its share: the candidates' total is below the number of rows, by exactly the prompt's mass
    np.testing.assert_allclose(got.sum(axis=-1), (1.0 - w[..., c + m:].sum(axis=-1)).sum(axis=2).reshape(L, Hkv, g).sum(axis=2),
                               rtol=1e-12)
    assert np.all(got.sum(axis=-1) < g * nq)


def test_prompt_self_term_of_minus_infinity_changes_nothing_and_a_huge_one_takes_everything():
    rng = np.random.default_rng(22)
    q, ck, hk, meta = _dense(rng, 1, 2, 2, 3, 4, 4, 8)
    base, base_lse = _score("f32", q, ck, hk, meta, 2, 2, 8, want_lse=True)
    none = np.full((1, 2, 3), -np.inf)
    same, same_lse = _score("f32", q, ck, hk, meta, 2, 2, 8, prompt_self_lse=none, want_lse=True)
    np.testing.assert_array_equal(same, base)
    np.testing.assert_array_equal(same_lse, base_lse)
    # a term equal to the candidates' own log-sum-exp halves every weight
    half = _score("f32", q, ck, hk, meta, 2, 2, 8, prompt_self_lse=base_lse)
    np.testing.assert_allclose(half, base / 2, rtol=1e-13)
    # one row with an overwhelming term drops out of the sum; the other rows are untouched
    big = none.copy()
    big[0, 1, 2] = 1e4
    got = _score("f32", q, ck, hk, meta, 2, 2, 8, prompt_self_lse=big)
    np.testing.assert_array_equal(got[0, 0], base[0, 0])
    assert np.all(got[0, 1] < base[0, 1]) and np.all(got[0, 1] > 0)


def test_causal_rows_equal_a_masked_numpy_softmax_and_the_first_token_scores_one():
    # Whole-input conditioning (the paper's ablation): the chunk's own tokens are query rows too, each attending to
    # the cache and to the chunk up to itself; prompt rows see every candidate.  "For the first token, its attention
    # score is maximal since it only considers itself, leading to a score of 1" (Method, positional bias).
    rng = np.random.default_rng(41)
    L, Hq, Hkv, d, c, m, nq = 1, 4, 2, 8, 3, 5, 2
    rows = m + nq                                                    # chunk rows, then prompt rows
    q, ck, hk, meta = _dense(rng, L, Hq, Hkv, rows, c, m, d)
    limit = np.array([c + i + 1 for i in range(m)] + [c + m] * nq, np.int32)
    got, lse = _score("f32", q, ck, hk, meta, Hq, Hkv, d, row_limit=limit, want_lse=True)
    g, scale = Hq // Hkv, 1.0 / math.sqrt(d)
    keys = np.repeat(np.concatenate([ck[:, :, :c], hk], axis=2).astype(np.float64), g, axis=1)
    s = np.einsum("lhpd,lhjd->lhpj", q.astype(np.float64), keys) * scale
    visible = np.arange(c + m)[None, :] < limit[:, None]
    s = np.where(visible, s, -np.inf)
    w = np.exp(s - s.max(axis=-1, keepdims=True))
    w /= w.sum(axis=-1, keepdims=True)
    want = w.sum(axis=2).reshape(L, Hkv, g, c + m).sum(axis=2)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)
    # per-row normalisation: every row's weights times the fraction of the candidates it sees
    normed = _score("f32", q, ck, hk, meta, Hq, Hkv, d, row_limit=limit, row_norm=True)
    want_n = (w * (limit / (c + m))[None, None, :, None]).sum(axis=2).reshape(L, Hkv, g, c + m).sum(axis=2)
    np.testing.assert_allclose(normed, want_n, rtol=1e-12, atol=1e-15)
    # the paper's example: with an empty cache the first document token sees only itself and gives it a score of 1
    q1, ck1, hk1, meta1 = _dense(rng, 1, 1, 1, 4, 0, 4, d)
    lim1 = np.array([1, 2, 3, 4], np.int32)
    only_first_row = _score("f32", q1[:, :, :1], ck1, hk1, dict(meta1, q_off=[0, 1]), 1, 1, d, row_limit=lim1[:1])
    np.testing.assert_array_equal(only_first_row[0, 0], [1.0, 0.0, 0.0, 0.0])
    scaled = _score("f32", q1[:, :, :1], ck1, hk1, dict(meta1, q_off=[0, 1]), 1, 1, d, row_limit=lim1[:1], row_norm=True)
    np.testing.assert_array_equal(scaled[0, 0], [0.25, 0.0, 0.0, 0.0])          # count(row != 0) / (m + c) = 1/4
    # later tokens lose the head start: unnormalised column sums favour early columns, the normalised ones less so
    full = _score("f32", q1, ck1, hk1, meta1, 1, 1, d, row_limit=lim1)
    np.testing.assert_allclose(full.sum(), 4.0, rtol=1e-12)                     # four rows, each summing to 1
    # limits at or beyond N are no limits
    same = _score("f32", q, ck, hk, meta, Hq, Hkv, d, row_limit=np.full(rows, 99, np.int32))
    np.testing.assert_array_equal(same, _score("f32", q, ck, hk, meta, Hq, Hkv, d))


def test_bf16_widening_is_exact():
    # 1.0 + 2^-7 is representable in bfloat16; the dot product must see exactly that value.
    bits = np.array([[[[0x3F81]]]], dtype=np.uint16)              # q = 1.0078125
    one = np.array([[[[0x3F80]]]], dtype=np.uint16)               # k = 1
    two = np.array([[[[0x4000]]]], dtype=np.uint16)               # k = 2
    meta = dict(q_off=[0, 1], chunk_off=[0, 1], cache_off=[0, 1], cache_len=[1])
    s = oracle.score("bf16", bits, one, two, n_q_heads=1, n_kv_heads=1, head_dim=1, scale=1.0, **meta)[0, 0]
    assert s[1] == pytest.approx(1 / (1 + math.exp(-1.0078125)), rel=1e-15)


def test_normalisation_factor_is_rank_neutral():
    # Prompt rows see every candidate, so count(A != 0)/(m + c) is the constant n_q (Method, bullet "Normalization").
    rng = np.random.default_rng(8)
    L, Hq, Hkv, nq, c, m, d = 1, 2, 1, 5, 4, 6, 8
    q, ck, hk, meta = _dense(rng, L, Hq, Hkv, nq, c, m, d)
    plain = _score("f32", q, ck, hk, meta, Hq, Hkv, d)
    normed = _score("f32", q, ck, hk, meta, Hq, Hkv, d, apply_norm=True)
    np.testing.assert_allclose(normed, plain * nq, rtol=1e-13)
    for r in range(1, c + m):
        np.testing.assert_array_equal(oracle.select_unit(plain[0, 0], r), oracle.select_unit(normed[0, 0], r))


def test_ragged_batch_equals_separate_requests():
    rng = np.random.default_rng(9)
    L, Hq, Hkv, d = 2, 4, 2, 8
    nqs, caps, lens, ms = [3, 1, 4], [5, 2, 6], [4, 0, 6], [3, 5, 0]
    q_off, cache_off, chunk_off = wl.offsets(nqs), wl.offsets(caps), wl.offsets(ms)
    q = rng.standard_normal((L, Hq, q_off[-1], d)).astype(np.float32)
    ck = rng.standard_normal((L, Hkv, cache_off[-1], d)).astype(np.float32)
    hk = rng.standard_normal((L, Hkv, chunk_off[-1], d)).astype(np.float32)
    s = oracle.score("f32", q, ck, hk, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, q_off=q_off, chunk_off=chunk_off,
                     cache_off=cache_off, cache_len=lens)
    for b in range(3):
        qb = np.ascontiguousarray(q[:, :, q_off[b]:q_off[b + 1]])
        cb = np.ascontiguousarray(ck[:, :, cache_off[b]:cache_off[b] + lens[b]])
        hb = np.ascontiguousarray(hk[:, :, chunk_off[b]:chunk_off[b + 1]])
        sb = oracle.score("f32", qb, cb, hb, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, q_off=[0, nqs[b]],
                          chunk_off=[0, ms[b]], cache_off=[0, lens[b]], cache_len=[lens[b]])
        o = cache_off[b] + chunk_off[b]
        np.testing.assert_array_equal(s[:, :, o:o + lens[b] + ms[b]], sb)


# ----------------------------------------------------------------------------- selection

def _brute_force_best_subset(scores, r):
    """Exact arithmetic: among all r-subsets the maximum total score, ties -> lexicographically smallest indices."""
    fr = [Fraction(float(x)) for x in scores]
    best, best_sum = None, None
    for sub in itertools.combinations(range(len(fr)), r):        # generated in lexicographic order
        tot = sum(fr[i] for i in sub)
        if best is None or tot > best_sum:
            best, best_sum = sub, tot
    return list(best)


@pytest.mark.parametrize("seed", range(6))
def test_select_against_exhaustive_subsets(seed):
    rng = np.random.default_rng(100 + seed)
    N = int(rng.integers(1, 11))
    levels = int(rng.integers(1, 5))
    scores = rng.integers(0, levels, size=N).astype(np.float64) / 4 + (rng.random(N) if seed % 2 else 0.0)
    for r in range(0, N + 3):
        kept = oracle.select_unit(scores, r)
        rr = min(r, N)
        assert len(kept) == rr
        assert np.all(np.diff(kept) > 0)
        if 0 < rr:
            assert kept.tolist() == _brute_force_best_subset(scores, rr)


def test_select_budget_at_or_above_candidates_is_identity():
    s = np.array([0.3, 0.1, 0.2, 0.9])
    for r in (4, 5, 100):
        np.testing.assert_array_equal(oracle.select_unit(s, r), np.arange(4))
    assert len(oracle.select_unit(s, 0)) == 0
    assert len(oracle.select_unit(np.zeros(0), 3)) == 0


def test_select_ties_go_to_lower_position_and_nan_ranks_last():
    np.testing.assert_array_equal(oracle.select_unit(np.array([1.0, 2.0, 1.0, 2.0, 1.0]), 3), [0, 1, 3])
    np.testing.assert_array_equal(oracle.select_unit(np.array([np.nan, 0.0, np.nan, 0.0]), 2), [1, 3])
    np.testing.assert_array_equal(oracle.select_unit(np.array([np.nan, -1.0, np.nan]), 2), [0, 1])
    np.testing.assert_array_equal(oracle.select_unit(np.array([0.0, -0.0, 0.0]), 2), [0, 1])     # -0 == +0


def test_huge_scale_gives_integer_argmax_counts():
    # scale -> large turns each softmax row into an indicator of its arg-max key: scores are exact integers.
    rng = np.random.default_rng(11)
    Hq, Hkv, nq, c, m, d = 2, 1, 9, 3, 5, 4
    q, ck, hk, meta = _dense(rng, 1, Hq, Hkv, nq, c, m, d)
    s = _score("f32", q, ck, hk, meta, Hq, Hkv, d, scale=1e6)[0, 0]
    keys = np.concatenate([ck, hk], axis=2)[0, 0].astype(np.float64)
    counts = np.bincount(np.argmax(q[0].astype(np.float64).reshape(-1, d) @ keys.T, axis=1), minlength=c + m)
    np.testing.assert_array_equal(s, counts.astype(np.float64))
    kept = oracle.select_unit(s, 4)
    order = sorted(range(c + m), key=lambda j: (-counts[j], j))[:4]
    assert kept.tolist() == sorted(order)


def test_paper_worked_cache_example():
    txt = dict(line.split(":") for line in (GOLDEN / "cache_example.txt").read_text().splitlines()
               if line and not line.startswith("#"))
    positions = [int(x) for x in txt["cache_positions"].split()]
    ranking = [int(x) for x in txt["ranking"].split()]
    shifts = [int(x) for x in txt["shifts"].split()]
    discarded = [int(x) for x in txt["discarded"].split()]
    scores = np.zeros(len(positions))
    for rank, tok in enumerate(ranking):
        scores[positions.index(tok)] = 10.0 - rank               # any scores that realise the printed ranking
    in_rank_order = oracle.select_unit(scores, len(ranking), rank_order=True)
    assert in_rank_order.tolist() == ranking
    assert [slot - tok for slot, tok in enumerate(in_rank_order.tolist())] == shifts
    ascending = oracle.select_unit(scores, len(ranking))
    assert ascending.tolist() == sorted(ranking)                 # same kept set, original order
    assert sorted(set(positions) - set(ascending.tolist())) == discarded


def _rope_numpy(x, pos, theta, pairing):
    """RoFormer's rotation restated with complex numbers: pair t is the complex number x_t + i y_t, multiplied by
    exp(i * pos * theta^(-2t/d)).  x: [..., d] float64."""
    d = x.shape[-1]
    if pairing == 0:
        z = x[..., :d // 2] + 1j * x[..., d // 2:]
    else:
        z = x[..., 0::2] + 1j * x[..., 1::2]
    z = z * np.exp(1j * pos * theta ** (-2.0 * np.arange(d // 2) / d))
    out = np.empty_like(x)
    if pairing == 0:
        out[..., :d // 2], out[..., d // 2:] = z.real, z.imag
    else:
        out[..., 0::2], out[..., 1::2] = z.real, z.imag
    return out


@pytest.mark.parametrize("pairing", [0, 1])
def test_rerotation_moves_keys_to_their_new_slots_and_keeps_relative_logits(pairing):
    # keys carry rotary embeddings at their candidate index; after compaction a kept key must look exactly like the
    # same raw key embedded at its new slot, so that a query at any position sees the logit of the NEW distance
    rng = np.random.default_rng(31)
    L, Hkv, d, c, m, theta = 1, 2, 16, 6, 4, 10000.0
    raw = rng.standard_normal((L, Hkv, c + m, d))
    rotated = np.stack([_rope_numpy(raw[:, :, j], j, theta, pairing) for j in range(c + m)], axis=2).astype(np.float32)
    ck, hk = np.ascontiguousarray(rotated[:, :, :c]), np.ascontiguousarray(rotated[:, :, c:])
    cv, hv = rng.standard_normal((L, Hkv, c, d)).astype(np.float32), rng.standard_normal((L, Hkv, m, d)).astype(np.float32)
    kept = np.full((L, Hkv, c), -1, np.int32)
    kept[0, 0, :4] = [0, 3, 5, 8]
    kept[0, 1, :4] = [1, 2, 7, 9]
    meta = dict(chunk_off=[0, m], cache_off=[0, c], cache_len=[c])
    args = ("f32", kept, [4], ck, cv, np.zeros((L, Hkv, c), np.int32), hk, hv, np.zeros(m, np.int32))
    out_k, out_v, _ = oracle.compact(*args, n_kv_heads=Hkv, head_dim=d, rope_theta=theta, rope_pairing=pairing, **meta)
    plain_k, plain_v, _ = oracle.compact(*args, n_kv_heads=Hkv, head_dim=d, **meta)
    np.testing.assert_array_equal(out_v, plain_v)                          # values are never rotated
    q_raw = rng.standard_normal(d)
    for g in range(Hkv):
        for slot, j in enumerate(kept[0, g, :4]):
            want = _rope_numpy(raw[0, g, j], slot, theta, pairing)         # the raw key embedded at its new slot
            np.testing.assert_allclose(out_k[0, g, slot], want, rtol=0, atol=2e-6)
            np.testing.assert_allclose(np.linalg.norm(out_k[0, g, slot]), np.linalg.norm(raw[0, g, j]), rtol=1e-6)
            # rotary logits depend on the distance only: a query at position 20 against the moved key
            q_rot = _rope_numpy(q_raw, 20, theta, pairing)
            same_distance = _rope_numpy(q_raw, 0, theta, pairing) @ _rope_numpy(raw[0, g, j], slot - 20, theta, pairing)
            np.testing.assert_allclose(q_rot @ out_k[0, g, slot].astype(np.float64), same_distance, atol=1e-5)
    # a key that stays where it is (slot 0 <- candidate 0) is copied bit for bit
    np.testing.assert_array_equal(out_k[0, 0, 0], ck[0, 0, 0])
    assert not np.array_equal(out_k[0, 0, 1], plain_k[0, 0, 1])


def test_rerotation_shifts_of_the_paper_example_and_bf16_rounding():
    # Managing the Cache: ranking [3, 5, 0] of cache [0..5] moves 3 by -3, 5 by -4 and 0 by +2 when the kept keys are
    # placed in rank order; the oracle's rotation by exactly these shifts must undo/redo the embedding
    txt = dict(line.split(":") for line in (GOLDEN / "cache_example.txt").read_text().splitlines()
               if line and not line.startswith("#"))
    ranking = [int(x) for x in txt["ranking"].split()]
    shifts = [int(x) for x in txt["shifts"].split()]
    rng = np.random.default_rng(32)
    d, theta = 8, 100.0
    raw = rng.standard_normal((1, 1, 6, d))
    rotated = np.stack([_rope_numpy(raw[:, :, j], j, theta, 0) for j in range(6)], axis=2)
    ck = wl.to_storage(rotated, "bf16")
    kept = np.array(ranking, np.int32).reshape(1, 1, 3).copy()
    kept = np.concatenate([kept, np.full((1, 1, 3), -1, np.int32)], axis=2)
    empty = np.zeros((1, 1, 0, d), np.uint16)
    out_k, _, _ = oracle.compact("bf16", kept, [3], ck, ck, np.zeros((1, 1, 6), np.int32), empty, empty,
                                 np.zeros(0, np.int32), n_kv_heads=1, head_dim=d, chunk_off=[0, 0], cache_off=[0, 6],
                                 cache_len=[6], rope_theta=theta)
    stored = wl.from_storage(ck, "bf16").astype(np.float64)
    for slot, (tok, shift) in enumerate(zip(ranking, shifts)):
        assert slot - tok == shift
        exact = _rope_numpy(stored[0, 0, tok], shift, theta, 0)
        got = wl.from_storage(out_k[0, 0, slot], "bf16").astype(np.float64)
        # the stored value is the exact rotation rounded to bfloat16: within half a unit in the last place
        assert np.all(np.abs(got - exact) <= np.abs(exact) * 2.0 ** -8 + 1e-30)
        np.testing.assert_array_equal(out_k[0, 0, slot], wl.to_storage(exact, "bf16"))


def test_batched_select_layout_and_budget_clamp():
    rng = np.random.default_rng(12)
    L, G = 2, 3
    caps, lens, ms, budget = [4, 3], [2, 3], [3, 1], [4, 2]
    cache_off, chunk_off = wl.offsets(caps), wl.offsets(ms)
    scores = rng.random((L, G, cache_off[-1] + chunk_off[-1]))
    kept, out_len = oracle.select(scores, chunk_off=chunk_off, cache_off=cache_off, cache_len=lens, budget=budget)
    assert out_len.tolist() == [4, 2]
    for l in range(L):
        for g in range(G):
            for b in range(2):
                o = cache_off[b] + chunk_off[b]
                N = lens[b] + ms[b]
                want = oracle.select_unit(scores[l, g, o:o + N], budget[b])
                got = kept[l, g, cache_off[b]:cache_off[b] + out_len[b]]
                np.testing.assert_array_equal(got, want)
                np.testing.assert_array_equal(kept[l, g, cache_off[b] + out_len[b]:cache_off[b + 1]], -1)


# ----------------------------------------------------------------------------- compaction and the whole step

@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("group_mode", [0, 1])
def test_compact_is_a_bit_exact_gather(dtype, group_mode):
    rng = np.random.default_rng(13)
    L, Hkv, d = 2, 4, 8
    G = Hkv if group_mode == 0 else 1
    caps, lens, ms, budget = [6, 5], [4, 5], [3, 2], [5, 4]
    cache_off, chunk_off = wl.offsets(caps), wl.offsets(ms)

    def rnd(n):
        a = rng.standard_normal((L, Hkv, n, d)).astype(np.float32)
        return wl.to_storage(a, dtype)
    ck, cv, hk, hv = rnd(cache_off[-1]), rnd(cache_off[-1]), rnd(chunk_off[-1]), rnd(chunk_off[-1])
    cpos = rng.integers(0, 1000, size=(L, G, cache_off[-1])).astype(np.int32)
    hpos = rng.integers(1000, 2000, size=chunk_off[-1]).astype(np.int32)
    scores = rng.random((L, G, cache_off[-1] + chunk_off[-1]))
    kept, out_len = oracle.select(scores, chunk_off=chunk_off, cache_off=cache_off, cache_len=lens, budget=budget)
    ok, ov, op = oracle.compact(dtype, kept, out_len, ck, cv, cpos, hk, hv, hpos, n_kv_heads=Hkv, head_dim=d,
                                group_mode=group_mode, chunk_off=chunk_off, cache_off=cache_off, cache_len=lens)
    for l in range(L):
        for h in range(Hkv):
            g = h if group_mode == 0 else 0
            for b in range(2):
                cand_k = np.concatenate([ck[l, h, cache_off[b]:cache_off[b] + lens[b]],
                                         hk[l, h, chunk_off[b]:chunk_off[b + 1]]])
                cand_v = np.concatenate([cv[l, h, cache_off[b]:cache_off[b] + lens[b]],
                                         hv[l, h, chunk_off[b]:chunk_off[b + 1]]])
                cand_p = np.concatenate([cpos[l, g, cache_off[b]:cache_off[b] + lens[b]],
                                         hpos[chunk_off[b]:chunk_off[b + 1]]])
                idx = kept[l, g, cache_off[b]:cache_off[b] + out_len[b]]
                sl = slice(cache_off[b], cache_off[b] + out_len[b])
                np.testing.assert_array_equal(ok[l, h, sl], cand_k[idx])
                np.testing.assert_array_equal(ov[l, h, sl], cand_v[idx])
                np.testing.assert_array_equal(op[l, g, sl], cand_p[idx])


def test_rescoring_a_kept_subset_equals_scoring_the_subset():
    rng = np.random.default_rng(14)
    Hq, Hkv, nq, c, m, d = 2, 1, 3, 5, 6, 8
    q, ck, hk, meta = _dense(rng, 1, Hq, Hkv, nq, c, m, d)
    s = _score("f32", q, ck, hk, meta, Hq, Hkv, d)
    kept = oracle.select_unit(s[0, 0], 4)
    allk = np.concatenate([ck, hk], axis=2)
    sub = np.ascontiguousarray(allk[:, :, kept])
    empty = np.zeros((1, Hkv, 0, d), np.float32)
    s_sub = oracle.score("f32", q, sub, empty, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, q_off=[0, nq],
                         chunk_off=[0, 0], cache_off=[0, 4], cache_len=[4])
    ref = _numpy_scores(q, sub, empty, 4, Hq, Hkv, 1 / math.sqrt(d))
    np.testing.assert_allclose(s_sub, ref, rtol=1e-12)


def _run_document(cfg, layer, budgets_per_step=None):
    """Drive the chunk loop of the Method section with the oracle for one layer; returns final positions per group."""
    q = wl.prompt_q(cfg, layer)
    B, Hkv, d = cfg.batch, cfg.n_kv_heads, cfg.head_dim
    caps = [max(r.budget, 1) for r in cfg.requests] if budgets_per_step is None else \
        [max(max(bs), 1) for bs in budgets_per_step]
    cache_off = wl.offsets(caps)
    ck = wl.to_storage(np.zeros((1, Hkv, cache_off[-1], d), np.float32), cfg.dtype)
    cv = ck.copy()
    cpos = np.full((1, cfg.n_groups, cache_off[-1]), -1, np.int32)
    cache_len = np.zeros(B, np.int32)
    planted_pos = [set() for _ in range(B)]
    lens_seen = []
    for step in range(cfg.n_steps):
        ch = wl.chunk_kv(cfg, layer, step, q)
        for b, r in enumerate(cfg.requests):
            planted_pos[b] |= set((step * r.chunk + ch["planted"][b]).tolist())
        budget = [r.budget for r in cfg.requests] if budgets_per_step is None else \
            [bs[min(step, len(bs) - 1)] for bs in budgets_per_step]
        out = oracle.step(cfg.dtype, wl.to_storage(q, cfg.dtype)[None], ck, cv, cpos,
                          wl.to_storage(ch["k"], cfg.dtype)[None], wl.to_storage(ch["v"], cfg.dtype)[None],
                          ch["chunk_pos"], n_q_heads=cfg.n_q_heads, n_kv_heads=Hkv, head_dim=d,
                          group_mode=cfg.group_mode, q_off=wl.q_offsets(cfg), chunk_off=ch["chunk_off"],
                          cache_off=cache_off, cache_len=cache_len, budget=budget, threads=4)
        ck, cv, cpos, cache_len = out["out_k"], out["out_v"], out["out_pos"], out["out_len"]
        lens_seen.append(cache_len.copy())
    return cpos, cache_len, planted_pos, cache_off, lens_seen


def test_planted_keys_survive_the_whole_document():
    base = wl.CONFIGS["c2"]
    cfg = wl.scaled(base, n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=32,
                    requests=(wl.Request(8, 512, 64, 48), wl.Request(5, 200, 64, 32)), planted_frac=0.04)
    cpos, cache_len, planted, cache_off, _ = _run_document(cfg, 0)
    assert cache_len.tolist() == [48, 32]
    for b in range(cfg.batch):
        assert 0 < len(planted[b]) <= cfg.requests[b].budget // 2
        for g in range(cfg.n_groups):
            final = cpos[0, g, cache_off[b]:cache_off[b] + cache_len[b]]
            assert np.all(np.diff(final) > 0)
            assert planted[b] <= set(final.tolist())


def test_paper_schedule_gives_linear_cache_growth():
    # r_{it+1} = m/sigma + c_it with c_0 = 0 gives c_it = it*m/sigma and a final size k = n/sigma (Method; Table 1).
    sigma, m, n = 4, 64, 512
    k = n // sigma
    steps = n // m
    schedule = [min(k, (it + 1) * m // sigma) for it in range(steps)]
    schedule[-1] = k
    cfg = wl.scaled(wl.CONFIGS["c2"], n_layers=1, n_q_heads=2, n_kv_heads=1, head_dim=16,
                    requests=(wl.Request(4, n, m, k),))
    _, cache_len, _, _, lens_seen = _run_document(cfg, 0, budgets_per_step=[schedule])
    assert [int(x[0]) for x in lens_seen] == [(it + 1) * m // sigma for it in range(steps)]
    assert int(cache_len[0]) == k


def test_step_equals_its_three_parts():
    rng = np.random.default_rng(15)
    st = wl.steady_state(wl.scaled(wl.CONFIGS["c4"], n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=16,
                                   requests=(wl.Request(3, 64, 16, 8), wl.Request(6, 40, 16, 5))), [0])
    kw = dict(n_kv_heads=2, head_dim=16)
    meta = dict(chunk_off=st["chunk_off"], cache_off=st["cache_off"], cache_len=st["cache_len"])
    out = oracle.step("bf16", st["q"], st["cache_k"], st["cache_v"], st["cache_pos"], st["chunk_k"], st["chunk_v"],
                      st["chunk_pos"], n_q_heads=4, q_off=st["q_off"], budget=st["budget"], **kw, **meta)
    s = oracle.score("bf16", st["q"], st["cache_k"], st["chunk_k"], n_q_heads=4, q_off=st["q_off"], **kw, **meta)
    kept, out_len = oracle.select(s, budget=st["budget"], **meta)
    ok, ov, op = oracle.compact("bf16", kept, out_len, st["cache_k"], st["cache_v"], st["cache_pos"], st["chunk_k"],
                                st["chunk_v"], st["chunk_pos"], **kw, **meta)
    np.testing.assert_array_equal(out["scores"], s)
    np.testing.assert_array_equal(out["kept_idx"], kept)
    np.testing.assert_array_equal(out["out_k"], ok)
    np.testing.assert_array_equal(out["out_v"], ov)
    np.testing.assert_array_equal(out["out_pos"], op)
    del rng


# ----------------------------------------------------------------------------- the input recipe

@pytest.mark.parametrize("name,shrink", [("c1", {}),
                                         ("c2", dict(n_layers=1, n_q_heads=4, n_kv_heads=4)),
                                         ("c3", dict(n_layers=1, n_q_heads=8, n_kv_heads=2,
                                                     requests=(wl.Request(128, 4096, 512, 512),))),
                                         ("c5", dict(n_layers=1, n_q_heads=8, n_kv_heads=2,
                                                     requests=(wl.Request(64, 8192, 512, 352),)))])
def test_planted_keys_are_clear_top_scores(name, shrink):
    cfg = wl.scaled(wl.CONFIGS[name], **shrink)
    st = wl.steady_state(cfg, [0])
    s = oracle.score(cfg.dtype, st["q"], st["cache_k"], st["chunk_k"], n_q_heads=cfg.n_q_heads,
                     n_kv_heads=cfg.n_kv_heads, head_dim=cfg.head_dim, q_off=st["q_off"], chunk_off=st["chunk_off"],
                     cache_off=st["cache_off"], cache_len=st["cache_len"], threads=8)
    planted = st["planted"][0]
    assert len(planted) > 0
    mask = np.zeros(s.shape[-1], bool)
    mask[planted] = True
    for g in range(cfg.n_groups):
        if cfg.dist == "normal":
            assert s[0, g, mask].min() >= 2.0 * s[0, g, ~mask].max()
        else:
            # heavy-tailed keys: an outlier may outscore a planted key, but every planted key is retained
            kept = oracle.select_unit(s[0, g, :int(st["cache_len"][0] + st["chunk_off"][1])], int(st["budget"][0]))
            assert set(planted.tolist()) <= set(kept.tolist())
