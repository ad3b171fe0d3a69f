"""Pins for the CPU oracle: each test checks it against something other than itself
(a library routine, a closed form, brute force, an invariant), so that a dropped
term, a wrong sign or index, or a transposed operand fails at least one of them.
No GPU needed."""
import math
import os

import numpy as np
import pytest
import torch

from paper_2506_05096_b200 import synth


def _rand(rng, *shape):
    return rng.standard_normal(shape)


# ---------------------------------------------------------------- attention pins
def test_dense_special_case_matches_library_attention(oracle):
    """Keep-ratio 1 (all queries) is plain Softmax(QK^T/sqrt(d))V (Section 3.1 equations):
    compare with torch's fp64 scaled_dot_product_attention and a numpy einsum."""
    rng = np.random.default_rng(1)
    B, N, H, d = 2, 37, 3, 8
    q, k, v = (_rand(rng, B, N, H, d) for _ in range(3))
    o, lse, p = oracle.sparse_attn(q, k, v, want_probs=True)
    tq, tk, tv = (torch.from_numpy(a).permute(0, 2, 1, 3) for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(0, 2, 1, 3).numpy()
    assert np.abs(o - ref).max() < 1e-12
    s = np.einsum("bihc,bjhc->bhij", q, k) / math.sqrt(d)
    ref_lse = np.log(np.exp(s).sum(-1))
    assert np.abs(lse - ref_lse).max() < 1e-12
    ref_p = np.exp(s - ref_lse[..., None])
    assert np.abs(p - ref_p).max() < 1e-13
    assert np.abs(o - np.einsum("bhij,bjhc->bihc", ref_p, v)).max() < 1e-12


def test_selected_rows_equal_rows_of_dense(oracle):
    """Each selected output row depends only on its own query and all K/V."""
    rng = np.random.default_rng(2)
    B, N, H, d = 2, 50, 2, 16
    q, k, v = (_rand(rng, B, N, H, d) for _ in range(3))
    idx = np.stack([np.sort(rng.choice(N, 13, replace=False)) for _ in range(B)]).astype(np.int32)
    o_all, lse_all, _ = oracle.sparse_attn(q, k, v)
    o, lse, _ = oracle.sparse_attn(q, k, v, q_idx=idx)
    for b in range(B):
        assert np.array_equal(o[b], o_all[b, idx[b]])
        assert np.array_equal(lse[b], lse_all[b][:, idx[b]])
    # independence from the other queries: scrambling unselected q rows changes nothing
    q2 = q.copy()
    mask = np.ones((B, N), bool)
    for b in range(B):
        mask[b, idx[b]] = False
    q2[mask] = 123.0
    o2, _, _ = oracle.sparse_attn(q2, k, v, q_idx=idx)
    assert np.array_equal(o, o2)


def test_softmax_rows_sum_to_one_and_outputs_in_hull(oracle):
    rng = np.random.default_rng(3)
    B, N, H, d = 1, 64, 2, 8
    q, k, v = (3.0 * _rand(rng, B, N, H, d) for _ in range(3))
    idx = np.arange(0, N, 3, dtype=np.int32)[None]
    o, _, p = oracle.sparse_attn(q, k, v, q_idx=idx, want_probs=True)
    assert np.abs(p.sum(-1) - 1.0).max() < 1e-12
    assert (p >= 0).all()
    lo, hi = v.min(axis=1)[:, None], v.max(axis=1)[:, None]
    assert (o >= lo - 1e-12).all() and (o <= hi + 1e-12).all()


def test_zero_keys_give_mean_of_values_and_ln_n(oracle):
    rng = np.random.default_rng(4)
    B, N, H, d = 1, 33, 2, 8
    q, v = _rand(rng, B, N, H, d), _rand(rng, B, N, H, d)
    o, lse, _ = oracle.sparse_attn(q, np.zeros_like(q), v)
    assert np.abs(o - v.mean(axis=1, keepdims=True)).max() < 1e-13
    assert np.abs(lse - math.log(N)).max() < 1e-13
    o, lse, _ = oracle.sparse_attn(np.zeros_like(q), q, v)
    assert np.abs(o - v.mean(axis=1, keepdims=True)).max() < 1e-13


def test_constant_value_row_is_returned(oracle):
    rng = np.random.default_rng(5)
    B, N, H, d = 1, 20, 2, 8
    q, k = _rand(rng, B, N, H, d), _rand(rng, B, N, H, d)
    row = _rand(rng, 1, 1, H, d)
    o, _, _ = oracle.sparse_attn(q, k, np.broadcast_to(row, q.shape).copy())
    assert np.abs(o - row).max() < 1e-13


def test_dominant_key_selects_its_value(oracle):
    """One key aligned with the query and scaled up takes all the softmax mass; the
    scale is 1/sqrt(d): the logit gap is c*|q|^2/sqrt(d), which the LSE reveals."""
    rng = np.random.default_rng(6)
    B, N, H, d = 1, 16, 1, 4
    q, v = _rand(rng, B, N, H, d), _rand(rng, B, N, H, d)
    k = np.zeros_like(q)
    i, j, c = 5, 11, 40.0
    k[0, j] = c * q[0, i]
    o, lse, _ = oracle.sparse_attn(q, k, v, q_idx=np.array([[i]], np.int32))
    assert np.abs(o[0, 0] - v[0, j]).max() < 1e-9
    top = c * (q[0, i, 0] ** 2).sum() / math.sqrt(d)
    assert abs(lse[0, 0, 0] - top) < 1e-9
    # an explicit scale overrides 1/sqrt(d)
    _, lse2, _ = oracle.sparse_attn(q, k, v, q_idx=np.array([[i]], np.int32), scale=0.25)
    assert abs(lse2[0, 0, 0] - 0.25 * c * (q[0, i, 0] ** 2).sum()) < 1e-5   # the other 15 keys weigh e^-15.7 each


def test_joint_permutation_of_keys_and_values_is_invisible(oracle):
    rng = np.random.default_rng(7)
    B, N, H, d = 1, 40, 2, 8
    q, k, v = (_rand(rng, B, N, H, d) for _ in range(3))
    idx = np.array([[1, 4, 9, 30]], np.int32)
    o, lse, _ = oracle.sparse_attn(q, k, v, q_idx=idx)
    perm = rng.permutation(N)
    inv = np.argsort(perm)
    # permute tokens: query rows move with their tokens
    o2, lse2, _ = oracle.sparse_attn(q[:, perm], k[:, perm], v[:, perm],
                                     q_idx=np.sort(inv[idx[0]])[None].astype(np.int32))
    order = np.argsort(inv[idx[0]])
    assert np.abs(o2[0] - o[0, order]).max() < 1e-12
    assert np.abs(lse2[0] - lse[0][:, order]).max() < 1e-12


def test_select_q_and_k_ablation_is_attention_on_the_subset(oracle):
    rng = np.random.default_rng(8)
    B, N, H, d = 1, 24, 2, 8
    q, k, v = (_rand(rng, B, N, H, d) for _ in range(3))
    idx = np.array([[0, 3, 5, 8, 13, 21]], np.int32)
    o, _, _ = oracle.sparse_attn(q, k, v, q_idx=idx, kv_idx=idx)
    sub = lambda a: a[:, idx[0]]
    o_ref, _, _ = oracle.sparse_attn(sub(q), sub(k), sub(v))
    assert np.abs(o - o_ref).max() < 1e-13


# ------------------------------------------------------------------ reuse pins
def test_attention_over_all_keys_is_the_lse_weighted_mix_of_attentions_over_a_partition(oracle):
    """Softmax attention over a union of disjoint key sets: out = sum_i exp(lse_i - lse) out_i and lse = log sum_i
    exp(lse_i) (the identity behind every split of the keys).  Pins the LSE output together with kv_idx: a wrong sign,
    base or scale in the LSE, or keys taken from the wrong rows, breaks the identity."""
    rng = np.random.default_rng(31)
    B, N, H, d, M = 2, 90, 2, 16, 11
    q, k, v = (rng.standard_normal((B, N, H, d)) for _ in range(3))
    q_idx = np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
    o_all, lse_all, _ = oracle.sparse_attn(q, k, v, q_idx=q_idx, scale=0.3)
    perm = np.stack([rng.permutation(N) for _ in range(B)])
    cuts = [0, 17, 18, 60, N]
    outs, lses = [], []
    for a, b_ in zip(cuts[:-1], cuts[1:]):
        kv = np.sort(perm[:, a:b_], axis=1).astype(np.int32)
        o, l, _ = oracle.sparse_attn(q, k, v, q_idx=q_idx, kv_idx=kv, scale=0.3)
        outs.append(o)
        lses.append(l)
    lses = np.stack(lses)                                   # [parts, B, H, M]
    lse = np.log(np.exp(lses).sum(axis=0))
    w = np.exp(lses - lse[None])                            # [parts, B, H, M]
    mix = sum(w[i].transpose(0, 2, 1)[..., None] * outs[i] for i in range(len(outs)))
    assert np.abs(lse - lse_all).max() < 1e-12
    assert np.abs(mix - o_all).max() < 1e-12


def test_keep_ratio_zero_returns_cache_unchanged(oracle):
    rng = np.random.default_rng(9)
    B, N, H, d = 2, 12, 2, 4
    cache = _rand(rng, B, N, H, d)
    out = oracle.scatter_reuse(cache, np.empty((B, 0, H, d)), np.empty((B, 0), np.int32))
    assert np.array_equal(out, cache)
    x = _rand(rng, B, N, H * d)
    lse = _rand(rng, B, H, N)
    res = oracle.step(x, x + 0.1, lse, np.zeros((B, N), np.int32), *(_rand(rng, B, N, H, d) for _ in range(3)),
                      cache, k_keep=0)
    assert np.array_equal(res["out"], cache)
    assert np.array_equal(res["lse"], lse)
    assert (res["n_skip"] == 1).all()
    assert res["idx_sel"].shape == (B, 0) and res["idx_rem"].shape == (B, N)


def test_scatter_touches_only_selected_rows(oracle):
    rng = np.random.default_rng(10)
    B, N, R, M = 2, 17, 6, 5
    cache = _rand(rng, B, N, R)
    rows = _rand(rng, B, M, R)
    idx = np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
    out = oracle.scatter_reuse(cache, rows, idx)
    for b in range(B):
        for i in range(N):
            if i in idx[b]:
                assert np.array_equal(out[b, i], rows[b, list(idx[b]).index(i)])
            else:
                assert np.array_equal(out[b, i], cache[b, i])
    # selected rows do not depend on the prior cache contents
    out2 = oracle.scatter_reuse(np.zeros_like(cache), rows, idx)
    for b in range(B):
        assert np.array_equal(out2[b, idx[b]], out[b, idx[b]])


def test_full_step_at_keep_ratio_one_is_dense_attention(oracle):
    rng = np.random.default_rng(11)
    B, N, H, d = 1, 30, 2, 8
    x = _rand(rng, B, N, H * d)
    q, k, v, cache = (_rand(rng, B, N, H, d) for _ in range(4))
    res = oracle.step(x, x * 0.5, _rand(rng, B, H, N), np.zeros((B, N), np.int32), q, k, v, cache, k_keep=N)
    tq, tk, tv = (torch.from_numpy(a).permute(0, 2, 1, 3) for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(0, 2, 1, 3).numpy()
    assert np.abs(res["out"] - ref).max() < 1e-12
    assert (res["n_skip"] == 0).all()
    assert np.array_equal(res["x_ref"], x)


def test_scatter_lse_matches_numpy_fancy_indexing(oracle):
    """The LSE cache is [B, H, N] and its compact rows [B, H, M]: with B > 1, H > 1, M != H and N != M*H a
    transposed or mis-strided index lands somewhere numpy's own indexing does not."""
    rng = np.random.default_rng(21)
    B, H, N, M = 3, 4, 19, 7
    cache = _rand(rng, B, H, N)
    rows = _rand(rng, B, H, M)
    idx = np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
    got = oracle.scatter_lse(cache, rows, idx)
    want = cache.copy()
    for b in range(B):
        want[b][:, idx[b]] = rows[b]
    assert np.array_equal(got, want)
    assert not np.array_equal(got, cache)
    # unsorted index lists are placed the same way (the scatter does not rely on the order)
    perm = rng.permutation(M)
    assert np.array_equal(oracle.scatter_lse(cache, rows[:, :, perm], idx[:, perm]), want)
    # no rows: the cache comes back untouched
    assert np.array_equal(oracle.scatter_lse(cache, np.empty((B, H, 0)), np.empty((B, 0), np.int32)), cache)


def test_step_at_a_partial_budget_merges_computed_and_cached_state(oracle):
    """Algorithm 1 lines 6-7 and the execution flow of Section 3.2 at 0 < k < N, with always-kept tokens and
    B, H > 1: the selected tokens carry the dense library attention's rows and LSE, every other token keeps the
    cached output and LSE bit for bit; the reference inputs are refreshed at the selected tokens ONLY; the
    selection itself is the brute-force top-k of the scores, which are retyped here from the equations."""
    rng = np.random.default_rng(22)
    B, N_v, N_t, H, d = 2, 23, 3, 3, 8
    N, k_keep = N_v + N_t, 9
    x_ref = _rand(rng, B, N, H * d)
    x_cur = x_ref + 0.3 * _rand(rng, B, N, H * d)
    q, k, v, cache = (_rand(rng, B, N, H, d) for _ in range(4))
    lse_cache = 0.5 * _rand(rng, B, H, N)
    n0 = rng.integers(0, 3, (B, N_v)).astype(np.int32)
    w_a, w_b = 2.0, 0.25
    res = oracle.step(x_cur, x_ref, lse_cache, n0, q, k, v, cache, k_keep, n_always=N_t, w_alpha=w_a, w_beta=w_b)
    # scores and selection from the definitions
    s_ref = (w_a * np.exp(lse_cache).mean(1)[:, :N_v] * np.abs(x_cur - x_ref).mean(-1)[:, :N_v] + w_b * np.exp(n0))
    assert np.abs(res["score"] - s_ref).max() < 1e-12 * np.abs(s_ref).max()
    s32 = s_ref.astype(np.float32)
    tq, tk, tv = (torch.from_numpy(a).permute(0, 2, 1, 3) for a in (q, k, v))
    dense = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).permute(0, 2, 1, 3).numpy()
    dense_lse = np.log(np.exp(np.einsum("bihc,bjhc->bhij", q, k) / math.sqrt(d)).sum(-1))       # [B, H, N]
    for b in range(B):
        top, rest = _brute_select(list(map(float, s32[b])), k_keep)
        sel = top + list(range(N_v, N))
        assert list(res["idx_sel"][b]) == sel and list(res["idx_rem"][b]) == rest
        unsel = np.setdiff1d(np.arange(N), sel)
        assert len(unsel) == N_v - k_keep
        # computed rows / cached rows of the output and of the LSE cache
        assert np.abs(res["out"][b, sel] - dense[b, sel]).max() < 1e-12
        assert np.array_equal(res["out"][b, unsel], cache[b, unsel])
        assert np.abs(res["lse"][b][:, sel] - dense_lse[b][:, sel]).max() < 1e-12
        assert np.array_equal(res["lse"][b][:, unsel], lse_cache[b][:, unsel])
        # the cached values really differ from the computed ones, so the two branches cannot be confused
        assert np.abs(cache[b, unsel] - dense[b, unsel]).min() > 0 and np.abs(lse_cache[b][:, unsel] - dense_lse[b][:, unsel]).min() > 0
        # reference inputs: current inputs where computed, untouched elsewhere
        assert np.array_equal(res["x_ref"][b, sel], x_cur[b, sel])
        assert np.array_equal(res["x_ref"][b, unsel], x_ref[b, unsel])
        assert np.abs(x_cur[b, unsel] - x_ref[b, unsel]).min() > 0
        # counters
        want_n = n0[b] + 1
        want_n[top] = 0
        assert np.array_equal(res["n_skip"][b], want_n)


def test_step_with_a_forced_selection_only_swaps_the_selection(oracle):
    """forced_sel (used by the chained GPU tests at near-ties): forcing the oracle's own selection changes nothing;
    forcing another one moves exactly the rows, the remainder list and the counters that follow from it."""
    rng = np.random.default_rng(23)
    B, N, H, d, k_keep = 1, 12, 2, 4, 5
    x_ref = _rand(rng, B, N, H * d)
    x_cur = x_ref + _rand(rng, B, N, H * d)
    q, k, v, cache = (_rand(rng, B, N, H, d) for _ in range(4))
    lse = _rand(rng, B, H, N)
    n0 = rng.integers(0, 3, (B, N)).astype(np.int32)
    own = oracle.step(x_cur, x_ref, lse, n0, q, k, v, cache, k_keep)
    same = oracle.step(x_cur, x_ref, lse, n0, q, k, v, cache, k_keep, forced_sel=own["idx_sel"])
    for key in ("idx_sel", "idx_rem", "n_skip", "out", "lse", "x_ref"):
        assert np.array_equal(own[key], same[key]), key
    forced = np.array([[0, 3, 4, 7, 11]], np.int32)
    res = oracle.step(x_cur, x_ref, lse, n0, q, k, v, cache, k_keep, forced_sel=forced)
    rest = [i for i in range(N) if i not in forced[0]]
    assert list(res["idx_rem"][0]) == rest and np.array_equal(res["own_idx_sel"], own["idx_sel"])
    assert (res["n_skip"][0, forced[0]] == 0).all() and np.array_equal(res["n_skip"][0, rest], n0[0, rest] + 1)
    dense, dense_lse, _ = oracle.sparse_attn(q, k, v)
    assert np.array_equal(res["out"][0, forced[0]], dense[0, forced[0]]) and np.array_equal(res["out"][0, rest], cache[0, rest])
    assert np.array_equal(res["lse"][0][:, forced[0]], dense_lse[0][:, forced[0]]) and np.array_equal(res["lse"][0][:, rest], lse[0][:, rest])
    assert np.array_equal(res["x_ref"][0, forced[0]], x_cur[0, forced[0]]) and np.array_equal(res["x_ref"][0, rest], x_ref[0, rest])


# -------------------------------------------------------------- selection pins
def _brute_select(s, k):
    order = sorted(range(len(s)), key=lambda i: (-(s[i] if not math.isnan(s[i]) else -math.inf), i))
    return sorted(order[:k]), sorted(order[k:])


@pytest.mark.parametrize("n,levels", [(1, 2), (7, 3), (64, 4), (257, 5), (300, 1000)])
def test_select_equals_brute_force_sort(oracle, n, levels):
    for seed in range(4):
        s = synth.integer_scores(2, n, seed, levels)
        for k in sorted({0, 1, n // 3, n - 1, n} & set(range(n + 1))):
            sel, rem, _ = oracle.select(s, k)
            for b in range(2):
                bs, br = _brute_select(list(map(float, s[b])), k)
                assert list(sel[b]) == bs and list(rem[b]) == br


def test_select_ties_nan_signed_zero_and_always_kept(oracle):
    s = np.array([[1.0, 1.0, 1.0, 1.0, 1.0, 1.0]], np.float32)
    sel, rem, _ = oracle.select(s, 2)
    assert list(sel[0]) == [0, 1] and list(rem[0]) == [2, 3, 4, 5]
    s = np.array([[0.0, -0.0, np.nan, -1.0, np.inf, -0.0]], np.float32)
    sel, rem, _ = oracle.select(s, 3)          # inf, then the zeros by index (+0 == -0)
    assert list(sel[0]) == [0, 1, 4]
    sel, _, _ = oracle.select(s, 5)            # NaN ranks last
    assert list(sel[0]) == [0, 1, 3, 4, 5]
    sel, rem, n = oracle.select(np.array([[3.0, 1.0, 2.0]], np.float32), 1, n_always=2,
                                n_skip=np.array([[5, 80, 0]], np.int32))
    assert list(sel[0]) == [0, 3, 4] and list(rem[0]) == [1, 2]
    assert list(n[0]) == [0, 80, 1]           # reset, clamp, increment


def test_select_on_float_scores_matches_numpy_partition(oracle):
    rng = np.random.default_rng(12)
    s = rng.standard_normal((3, 1000)).astype(np.float32)
    k = 333
    sel, rem, _ = oracle.select(s, k)
    for b in range(3):
        ref = np.sort(np.argsort(-s[b], kind="stable")[:k])
        assert np.array_equal(sel[b], ref)
        assert np.array_equal(np.sort(np.concatenate([sel[b], rem[b]])), np.arange(1000))


def test_budget_to_k_is_floor(oracle):
    assert oracle.budget_to_k(17550, 250) == 4387       # 4387.5 floors
    assert oracle.budget_to_k(17550, 500) == 8775
    assert oracle.budget_to_k(16384, 400) == 6553
    assert oracle.budget_to_k(118800, 600) == 71280
    assert oracle.budget_to_k(100, 0) == 0 and oracle.budget_to_k(100, 1000) == 100


# ------------------------------------------------------------------ score pins
def test_score_constant_per_token_difference_closed_form(oracle):
    """x_cur = x_ref + c_i: delta is |c_i|, c_i^2, c_i for the three reductions; the
    score is w_a * mean_h exp(lse) * delta + w_b * e^{n} (selection-metric equations)."""
    rng = np.random.default_rng(13)
    B, N, D, H = 2, 9, 16, 3
    x_ref = _rand(rng, B, N, D)
    c = rng.choice([-0.5, 0.25, 0.125, -2.0, 1.0], size=(B, N))
    x_cur = x_ref + c[..., None]
    lse = 0.3 * _rand(rng, B, H, N)
    n = rng.integers(0, 4, size=(B, N)).astype(np.int32)
    s_lse = np.exp(lse).mean(axis=1)
    for mode, delta in ((0, np.abs(c)), (1, c * c), (2, c)):
        got = oracle.score(x_cur, x_ref, lse, n, w_alpha=0.7, w_beta=0.2, delta_mode=mode)
        want = 0.7 * s_lse * delta + 0.2 * np.exp(n)
        assert np.abs(got - want).max() < 1e-12
    got = oracle.score(x_cur, x_ref, lse, n, w_alpha=1.0, w_beta=0.0, lse_mode=1)
    assert np.abs(got - lse.mean(axis=1) * np.abs(c)).max() < 1e-12
    # no LSE, no counters: S_LSE = 1, e^0 = 1
    got = oracle.score(x_cur, x_ref, None, None, H=H, w_alpha=1.0, w_beta=1.0)
    assert np.abs(got - (np.abs(c) + 1.0)).max() < 1e-12
    # clamp of n at 80
    big = oracle.score(x_ref, x_ref, None, np.full((B, N), 500, np.int32), w_alpha=0.0, w_beta=1.0)
    assert np.allclose(big, math.exp(80.0), rtol=1e-15)


def test_score_log_values_above_the_clamp_count_as_the_clamp(oracle):
    """The sum-of-exponentials reading keeps the fp32 scores finite: a log value above 80 counts as 80 (a reading
    of this build, stated next to the counter clamp); the log-mode score is not clamped."""
    B, N, D, H = 1, 4, 8, 2
    x_ref = np.zeros((B, N, D))
    x_cur = np.full((B, N, D), 0.5)
    lse = np.array([[[0.0, 79.0, 80.0, 1000.0], [0.0, 79.0, 85.0, 90.0]]])
    s = oracle.score(x_cur, x_ref, lse, None, w_alpha=1.0, w_beta=0.0)
    want = 0.5 * np.array([1.0, math.exp(79.0), math.exp(80.0), math.exp(80.0)])
    assert np.abs(s[0] - want).max() <= 1e-12 * want.max() and np.isfinite(s.astype(np.float32)).all()
    s1 = oracle.score(x_cur, x_ref, lse, None, w_alpha=1.0, w_beta=0.0, lse_mode=1)
    assert np.abs(s1[0] - 0.5 * np.array([0.0, 79.0, 82.5, 545.0])).max() < 1e-12


def test_score_mixed_signs_distinguish_the_three_reductions(oracle):
    x_ref = np.zeros((1, 1, 4))
    x_cur = np.array([[[1.0, -1.0, 2.0, -4.0]]])
    for mode, want in ((0, 2.0), (1, 5.5), (2, -0.5)):
        got = oracle.score(x_cur, x_ref, None, None, w_alpha=1.0, w_beta=0.0, delta_mode=mode)
        assert got[0, 0] == want


def test_score_only_covers_selectable_tokens_and_permutes_with_tokens(oracle):
    rng = np.random.default_rng(14)
    B, N, D, H, n_sel = 1, 12, 8, 2, 9
    x_ref, x_cur = _rand(rng, B, N, D), _rand(rng, B, N, D)
    lse = _rand(rng, B, H, N)
    n = rng.integers(0, 3, size=(B, n_sel)).astype(np.int32)
    s = oracle.score(x_cur, x_ref, lse, n, n_sel=n_sel)
    assert s.shape == (B, n_sel)
    perm = rng.permutation(n_sel)
    full = np.concatenate([perm, np.arange(n_sel, N)])
    s2 = oracle.score(x_cur[:, full], x_ref[:, full], lse[:, :, full], n[:, perm], n_sel=n_sel)
    assert np.array_equal(s2, s[:, perm])


def test_penalty_only_schedule_is_round_robin(oracle):
    """w_alpha = 0: scores are e^{n_i}; with ties to the lower index and n reset on selection
    the selection cycles [0,k), [k,2k), ... with period N/k."""
    N, k = 24, 6
    n = np.zeros((1, N), np.int32)
    x = np.zeros((1, N, 4))
    for t in range(3 * N // k):
        s = oracle.score(x, x, None, n, w_alpha=0.0, w_beta=1.0).astype(np.float32)
        sel, _, n = oracle.select(s, k, n_skip=n)
        start = (t * k) % N
        assert list(sel[0]) == list(range(start, start + k))


def test_drift_statistics_half_normal_mean(oracle):
    """x_cur = x_ref + sigma*eps gives E[mean|delta|] = sigma*sqrt(2/pi)."""
    rng = np.random.default_rng(15)
    N, D, sigma = 64, 4096, 0.05
    x_ref = _rand(rng, 1, N, D)
    x_cur = x_ref + sigma * _rand(rng, 1, N, D)
    s = oracle.score(x_cur, x_ref, None, None, w_alpha=1.0, w_beta=0.0)
    want = sigma * math.sqrt(2 / math.pi)
    assert abs(s.mean() - want) < 3e-4
    assert np.abs(s - want).max() < 6 * sigma * math.sqrt(1 - 2 / math.pi) / math.sqrt(D)


# -------------------------------------------------------- flop accounting pin
def test_cross_attention_of_listed_rows_matches_a_library_softmax(oracle):
    """Queries from one sequence, keys / values from another (the block's cross-attention on the selected rows):
    numpy softmax over the second sequence, rows picked by the list."""
    rng = np.random.default_rng(24)
    B, N, N_kv, H, d, M = 2, 23, 9, 2, 8, 6
    q, k, v = _rand(rng, B, N, H, d), _rand(rng, B, N_kv, H, d), _rand(rng, B, N_kv, H, d)
    idx = np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
    o, lse, p = oracle.sparse_attn(q, k, v, q_idx=idx, want_probs=True)
    s = np.einsum("bihc,bjhc->bhij", q, k) / math.sqrt(d)
    pr = np.exp(s - s.max(-1, keepdims=True))
    pr /= pr.sum(-1, keepdims=True)
    ref = np.einsum("bhij,bjhc->bihc", pr, v)
    for b in range(B):
        assert np.abs(o[b] - ref[b, idx[b]]).max() < 1e-12
        assert np.abs(lse[b] - np.log(np.exp(s[b]).sum(-1))[:, idx[b]]).max() < 1e-12
    assert p.shape == (B, H, M, N_kv) and np.abs(p.sum(-1) - 1).max() < 1e-12


# ---------------------------------------------------------------- linear layers on selected rows
def test_gathered_linear_matches_a_library_matmul_and_leaves_other_rows_alone(oracle):
    """All rows: the textbook x W^T + b (numpy matmul).  Listed rows only: those rows equal the full product,
    the others are bit-identical to the cache (Algorithm 1 lines 4-7 applied to a linear layer)."""
    rng = np.random.default_rng(21)
    B, N, K, N_out, M = 2, 29, 24, 17, 11
    x, w, bias, cache = _rand(rng, B, N, K), _rand(rng, N_out, K), _rand(rng, N_out), _rand(rng, B, N, N_out)
    full = x @ w.T + bias
    assert np.abs(oracle.gathered_linear(x, w, bias) - full).max() < 1e-12
    idx = np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
    y = oracle.gathered_linear(x, w, bias, idx, cache)
    for b in range(B):
        mask = np.zeros(N, bool)
        mask[idx[b]] = True
        assert np.abs(y[b, mask] - full[b, mask]).max() < 1e-12
        assert np.array_equal(y[b, ~mask], cache[b, ~mask])
    assert np.array_equal(oracle.gathered_linear(x, w, bias, np.zeros((B, 0), np.int32), cache), cache)


def test_gathered_linear_closed_forms_catch_a_transposed_weight_or_a_dropped_bias(oracle):
    rng = np.random.default_rng(22)
    B, N, K = 1, 7, 5
    x = _rand(rng, B, N, K)
    # a non-square one-hot weight: output feature n copies input feature sel[n] (a transposed operand cannot do this)
    sel = np.array([3, 0, 4, 4, 1, 2, 0])
    w = np.zeros((len(sel), K))
    w[np.arange(len(sel)), sel] = 1.0
    assert np.array_equal(oracle.gathered_linear(x, w), x[:, :, sel])
    # zero weight: every computed row is the bias; brute force in pure Python for a dense random case
    bias = _rand(rng, len(sel))
    assert np.array_equal(oracle.gathered_linear(x, np.zeros_like(w), bias), np.broadcast_to(bias, (B, N, len(sel))))
    w2 = _rand(rng, 3, K)
    got = oracle.gathered_linear(x, w2, bias[:3])
    for i in range(N):
        for n in range(3):
            want = bias[n] + sum(x[0, i, c] * w2[n, c] for c in range(K))
            assert abs(got[0, i, n] - want) < 1e-13


def test_gathered_linear_gelu_and_compact_input_match_library_routines(oracle):
    """The MLP of a block on the selected rows: GELU(x[idx] W1^T + b1) kept compact, then W2 applied to the compact
    rows and scattered to the tokens.  Checked against torch's fp64 gelu / linear and plain indexing."""
    rng = np.random.default_rng(23)
    B, N, K, Hd, M = 2, 19, 6, 10, 7
    x, w1, b1, w2, b2, cache = (_rand(rng, B, N, K), _rand(rng, Hd, K), _rand(rng, Hd), _rand(rng, K, Hd), _rand(rng, K),
                                _rand(rng, B, N, K))
    idx = np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
    hid_full = oracle.gathered_linear(x, w1, b1, idx, gelu=True)                    # [B, N, Hd], rows off the list are zero
    hid = np.take_along_axis(hid_full, idx[:, :, None].astype(np.int64), 1)         # compact [B, M, Hd]
    t = torch.from_numpy
    want_hid = torch.nn.functional.gelu(torch.nn.functional.linear(t(x), t(w1), t(b1))).numpy()
    assert np.abs(hid - np.take_along_axis(want_hid, idx[:, :, None].astype(np.int64), 1)).max() < 1e-12
    assert np.abs(oracle.gathered_linear(np.array([[[0.0], [1.0], [-1.0]]]), np.ones((1, 1)), gelu=True).ravel()
                  - np.array([0.0, 0.8413447460685429, -0.15865525393145707])).max() < 1e-15     # x Phi(x) at 0, 1, -1
    y = oracle.gathered_linear(hid, w2, b2, idx, cache, compact_in=True)
    want = np.array(cache)
    for b in range(B):
        want[b, idx[b]] = hid[b] @ w2.T + b2
    assert np.abs(y - want).max() < 1e-12
    mask = np.ones((B, N), bool)
    for b in range(B):
        mask[b, idx[b]] = False
    assert np.array_equal(y[mask], cache[mask])


def test_attention_flops_are_linear_in_selected_tokens_like_the_papers_tables():
    from paper_2506_05096_b200 import accounting
    path = os.path.join(os.path.dirname(__file__), "golden", "flops_tables.txt")
    B, H, N, d = 1, 24, 118800, 128
    full = accounting.attn_flops(B, H, N, N, d)
    assert full == 4 * B * H * N * N * d                # 4*B*N^2*(H*d): the N^2 term of the FLOPs formula
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        name, orig, *rows = line.split()
        for theta, val in zip((0.4, 0.5, 0.7), rows):
            M = int(round(theta * N))
            ratio = accounting.attn_flops(B, H, M, N, d) / full
            assert abs(ratio - float(val) / float(orig)) < 2e-4, (name, theta)


# ------------------------------------------------------------------ whole-block pins
def _block_weights(rng, B, D, hidden, modulated=True):
    lin = lambda o, i: rng.standard_normal((o, i)) / math.sqrt(i)
    w = {}
    for name, (o, i) in dict(wq=(D, D), wk=(D, D), wv=(D, D), wo=(D, D), wq2=(D, D), wo2=(D, D), w1=(hidden, D), w2=(D, hidden)).items():
        w[name] = lin(o, i)
        w["b" + name[1:]] = 0.1 * rng.standard_normal(o)
    if modulated:
        for name in ("s1", "t1", "g1", "s3", "t3", "g3"):
            w[name] = 0.3 * rng.standard_normal((B, D))
    return w


def _torch_dense_block(x, w, text_k, text_v, H, eps=1e-6):
    """The same block from torch's fp64 building blocks (layer_norm, linear, scaled_dot_product_attention, gelu)."""
    F = torch.nn.functional
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a))
    X = t(x)
    B, N, D = X.shape
    d = D // H
    mod = lambda h, s, sh: h * (1 + t(w[s])[:, None, :]) + t(w[sh])[:, None, :] if w.get(s) is not None else h
    heads = lambda a: a.reshape(B, -1, H, d).permute(0, 2, 1, 3)
    h = mod(F.layer_norm(X, (D,), eps=eps), "s1", "t1")
    q, k, v = (F.linear(h, t(w["w" + n]), t(w["b" + n])) for n in ("q", "k", "v"))
    a = F.scaled_dot_product_attention(heads(q), heads(k), heads(v)).permute(0, 2, 1, 3).reshape(B, N, D)
    o = F.linear(a, t(w["wo"]), t(w["bo"]))
    x1 = X + (o * t(w["g1"])[:, None, :] if w.get("g1") is not None else o)
    q2 = F.linear(F.layer_norm(x1, (D,), eps=eps), t(w["wq2"]), t(w["bq2"]))
    c = F.scaled_dot_product_attention(heads(q2), t(text_k).permute(0, 2, 1, 3), t(text_v).permute(0, 2, 1, 3)).permute(0, 2, 1, 3).reshape(B, N, D)
    x2 = x1 + F.linear(c, t(w["wo2"]), t(w["bo2"]))
    h3 = mod(F.layer_norm(x2, (D,), eps=eps), "s3", "t3")
    m = F.linear(F.gelu(F.linear(h3, t(w["w1"]), t(w["b1"]))), t(w["w2"]), t(w["b2"]))
    x3 = x2 + (m * t(w["g3"])[:, None, :] if w.get("g3") is not None else m)
    lse = torch.logsumexp(torch.einsum("bhic,bhjc->bhij", heads(q), heads(k)) / math.sqrt(d), -1)
    return x3.numpy(), lse.numpy()


@pytest.mark.parametrize("modulated", [True, False])
def test_block_step_at_keep_ratio_one_is_the_dense_block_of_library_modules(oracle, modulated):
    rng = np.random.default_rng(31)
    B, N, H, d, N_text, hidden = 2, 14, 2, 4, 5, 20
    D = H * d
    x = _rand(rng, B, N, D)
    w = _block_weights(rng, B, D, hidden, modulated)
    tk, tv = _rand(rng, B, N_text, H, d), _rand(rng, B, N_text, H, d)
    res = oracle.block_step(x, x + 1.0, _rand(rng, B, H, N), np.zeros((B, N), np.int32), _rand(rng, B, N, D), w, tk, tv, H, k_keep=N)
    want, want_lse = _torch_dense_block(x, w, tk, tv, H)
    assert np.abs(res["y"] - want).max() < 1e-11
    assert np.abs(res["lse"] - want_lse).max() < 1e-11
    assert np.array_equal(res["x_ref"], x) and (res["n_skip"] == 0).all()


def test_block_step_partial_budget_computes_selected_rows_and_reuses_the_rest(oracle):
    """Selected tokens carry the dense block's rows (keys and values come from all tokens, the other layers act per
    token), every other token keeps the cached block output, LSE and reference input; keep-ratio 0 changes nothing."""
    rng = np.random.default_rng(32)
    B, N_v, N_t, H, d, N_text, hidden = 2, 17, 3, 2, 4, 6, 24
    N, D, k_keep = N_v + N_t, H * d, 6
    x_ref = _rand(rng, B, N, D)
    x = x_ref + 0.4 * _rand(rng, B, N, D)
    w = _block_weights(rng, B, D, hidden)
    tk, tv = _rand(rng, B, N_text, H, d), _rand(rng, B, N_text, H, d)
    y_cache, lse_cache = _rand(rng, B, N, D), 0.3 * _rand(rng, B, H, N)
    n0 = rng.integers(0, 3, (B, N_v)).astype(np.int32)
    res = oracle.block_step(x, x_ref, lse_cache, n0, y_cache, w, tk, tv, H, k_keep, n_always=N_t)
    dense, dense_lse = _torch_dense_block(x, w, tk, tv, H)
    step = oracle.step(x, x_ref, lse_cache, n0, *(np.zeros((B, N, H, d)) for _ in range(4)), k_keep, n_always=N_t)
    assert np.array_equal(res["idx_sel"], step["idx_sel"]) and np.array_equal(res["n_skip"], step["n_skip"])   # same score / selection path
    for b in range(B):
        sel = res["idx_sel"][b]
        unsel = np.setdiff1d(np.arange(N), sel)
        assert len(sel) == k_keep + N_t and len(unsel) == N_v - k_keep
        assert np.abs(res["y"][b, sel] - dense[b, sel]).max() < 1e-11
        assert np.array_equal(res["y"][b, unsel], y_cache[b, unsel])
        assert np.abs(res["lse"][b][:, sel] - dense_lse[b][:, sel]).max() < 1e-11
        assert np.array_equal(res["lse"][b][:, unsel], lse_cache[b][:, unsel])
        assert np.array_equal(res["x_ref"][b, sel], x[b, sel]) and np.array_equal(res["x_ref"][b, unsel], x_ref[b, unsel])
    none = oracle.block_step(x, x_ref, lse_cache, n0[:, :N], y_cache, w, tk, tv, H, 0, n_always=0) if False else \
        oracle.block_step(x[:, :N_v], x_ref[:, :N_v], lse_cache[:, :, :N_v], n0, y_cache[:, :N_v], w, tk, tv, H, 0)
    assert np.array_equal(none["y"], y_cache[:, :N_v]) and np.array_equal(none["lse"], lse_cache[:, :, :N_v])
    assert np.array_equal(none["x_ref"], x_ref[:, :N_v]) and np.array_equal(none["n_skip"], n0 + 1)


def test_layernorm_modulate_matches_the_library_routine(oracle):
    rng = np.random.default_rng(33)
    B, R, D = 2, 7, 24
    x, s, t = 3.0 * _rand(rng, B, R, D) + 1.5, _rand(rng, B, D), _rand(rng, B, D)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(x), (D,), eps=1e-5).numpy()
    assert np.abs(oracle.layernorm_modulate(x, eps=1e-5) - ref).max() < 1e-13
    assert np.abs(oracle.layernorm_modulate(x, s, t, eps=1e-5) - (ref * (1 + s[:, None]) + t[:, None])).max() < 1e-13
    y = oracle.layernorm_modulate(x, eps=0.0)
    assert np.abs(y.mean(-1)).max() < 1e-13 and np.abs(y.var(-1) - 1.0).max() < 1e-12


# ------------------------------------------------------------------ variants of the ablation study, several blocks
def test_timestep_level_budgets_compute_all_or_nothing_with_the_same_total(oracle):
    for seed, T, n in ((0, 12, 100), (1, 50, 17550), (2, 7, 1)):
        rng = np.random.default_rng(seed)
        k = [n] + [int(v) for v in rng.integers(0, n + 1, T - 1)]
        out = oracle.timestep_level_budgets(k, n)
        assert out[0] == n and set(out) <= {0, n}
        assert abs(sum(out) - sum(k)) < n or sum(k) < n                  # the total budget is kept up to one step
        # a schedule that is all-or-nothing already comes back unchanged
        assert oracle.timestep_level_budgets(out, n) == out
    assert oracle.timestep_level_budgets([10, 5, 5, 0, 9, 1], 10) == [10, 0, 10, 0, 0, 10]
    assert oracle.timestep_level_budgets([3, 3, 3], 10) == [10, 0, 0]    # the first step computes everything whatever its budget


def test_select_qk_block_is_the_block_on_the_selected_tokens_alone(oracle):
    """SelectQ&K (Table 2): with keys and values restricted to the selected tokens, the selected rows of the block are
    the dense block evaluated on the sub-sequence of selected tokens."""
    rng = np.random.default_rng(41)
    B, N, H, d, N_text, hidden, k_keep = 1, 15, 2, 4, 4, 16, 6
    D = H * d
    x = _rand(rng, B, N, D)
    w = _block_weights(rng, B, D, hidden)
    tk, tv = _rand(rng, B, N_text, H, d), _rand(rng, B, N_text, H, d)
    y_cache = _rand(rng, B, N, D)
    res = oracle.block_step(x, x + 0.5 * _rand(rng, B, N, D), _rand(rng, B, H, N), np.zeros((B, N), np.int32), y_cache, w, tk, tv, H,
                            k_keep, select_qk=True)
    sel = res["idx_sel"][0]
    dense_sub, lse_sub = _torch_dense_block(x[:, sel], w, tk, tv, H)
    assert np.abs(res["y"][0, sel] - dense_sub[0]).max() < 1e-11
    assert np.abs(res["lse"][0][:, sel] - lse_sub[0]).max() < 1e-11
    unsel = np.setdiff1d(np.arange(N), sel)
    assert np.array_equal(res["y"][0, unsel], y_cache[0, unsel])


def test_model_step_chains_blocks_and_the_variants_differ_as_the_ablation_describes(oracle):
    rng = np.random.default_rng(42)
    B, N, H, d, N_text, hidden, L, k_keep = 1, 16, 2, 4, 3, 16, 3, 7
    D = H * d
    x = _rand(rng, B, N, D)
    blocks = [_block_weights(rng, B, D, hidden) for _ in range(L)]
    tks, tvs = [_rand(rng, B, N_text, H, d) for _ in range(L)], [_rand(rng, B, N_text, H, d) for _ in range(L)]
    states = [dict(x_ref=_rand(rng, B, N, D), lse=_rand(rng, B, H, N), n_skip=rng.integers(0, 3, (B, N)).astype(np.int32),
                   y=_rand(rng, B, N, D)) for _ in range(L)]
    # token-wise: the chain of single blocks, each reading the merged output of the one before
    outs = oracle.model_step(x, blocks, states, tks, tvs, H, k_keep)
    xin = x
    for l in range(L):
        r = oracle.block_step(xin, states[l]["x_ref"], states[l]["lse"], states[l]["n_skip"], states[l]["y"], blocks[l], tks[l], tvs[l], H, k_keep)
        for key in ("idx_sel", "y", "lse", "x_ref", "n_skip"):
            assert np.array_equal(outs[l][key], r[key]), (l, key)
        xin = r["y"]
    assert any(not np.array_equal(outs[0]["idx_sel"], outs[l]["idx_sel"]) for l in range(1, L))       # blocks select on their own
    # Fixed-token: every block of the step works on block 0's selection; later blocks keep counters and references
    fx = oracle.model_step(x, blocks, states, tks, tvs, H, k_keep, variant=oracle.VARIANT_FIXED_TOKEN)
    assert np.array_equal(fx[0]["y"], outs[0]["y"])
    for l in range(1, L):
        assert np.array_equal(fx[l]["idx_sel"], fx[0]["idx_sel"])
        assert np.array_equal(fx[l]["n_skip"], states[l]["n_skip"]) and np.array_equal(fx[l]["x_ref"], states[l]["x_ref"])
        unsel = np.setdiff1d(np.arange(N), fx[0]["idx_sel"][0])
        assert np.array_equal(fx[l]["y"][0, unsel], states[l]["y"][0, unsel])
    # Timestep-level: a step computes everything (the dense model) or nothing (every cache as it was)
    full = oracle.model_step(x, blocks, states, tks, tvs, H, N, variant=oracle.VARIANT_TIMESTEP)
    xin = x
    for l in range(L):
        xin, _ = _torch_dense_block(xin, blocks[l], tks[l], tvs[l], H)
        assert np.abs(full[l]["y"] - xin).max() < 1e-10
    none = oracle.model_step(x, blocks, states, tks, tvs, H, 0, variant=oracle.VARIANT_TIMESTEP)
    for l in range(L):
        assert np.array_equal(none[l]["y"], states[l]["y"]) and np.array_equal(none[l]["lse"], states[l]["lse"])
    with pytest.raises(AssertionError):
        oracle.model_step(x, blocks, states, tks, tvs, H, 5, variant=oracle.VARIANT_TIMESTEP)


def test_partial_scores_of_head_shards_add_up_to_the_score(oracle):
    """Head-sharded form: the selection metric from partial sums over contiguous head ranges equals the unsharded one."""
    rng = np.random.default_rng(51)
    B, N, N_sel, H, d = 2, 21, 18, 6, 4
    D = H * d
    x_ref = _rand(rng, B, N, D)
    x_cur = x_ref + 0.3 * _rand(rng, B, N, D)
    lse = _rand(rng, B, H, N)
    lse[0, 2, 5] = 95.0                                   # above the clamp
    n = rng.integers(0, 4, (B, N_sel)).astype(np.int32)
    for delta_mode in (0, 1, 2):
        for lse_mode in (0, 1):
            want = oracle.score(x_cur, x_ref, lse, n, n_sel=N_sel, w_alpha=0.7, w_beta=0.2, delta_mode=delta_mode, lse_mode=lse_mode)
            for bounds in ([0, 6], [0, 2, 6], [0, 1, 3, 4, 6]):
                part = sum(oracle.score_partial(x_cur[:, :, h0 * d:h1 * d], x_ref[:, :, h0 * d:h1 * d], lse[:, h0:h1], N_sel, delta_mode, lse_mode)
                           for h0, h1 in zip(bounds[:-1], bounds[1:]))
                got = oracle.score_combine(part, n, D, H, True, 0.7, 0.2)
                assert np.abs(got - want).max() <= 1e-12 * np.abs(want).max()
    got = oracle.score_combine(oracle.score_partial(x_cur, x_ref, None, N_sel), None, D, H, False)
    assert np.abs(got - oracle.score(x_cur, x_ref, None, None, n_sel=N_sel)).max() < 1e-12
