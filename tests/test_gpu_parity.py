"""Parity of the CUDA library (through its C ABI) with the CPU oracle, element by element,
on the same seeded inputs.  Integer / index results must be bit-exact; floating-point
results within the stated tolerances (attention: max-abs 2e-2, mean-abs 2e-3 against the
fp64 oracle on the bf16-rounded inputs; LSE 1e-3; scores 1e-5 relative)."""
import math

import numpy as np
import pytest
import torch

from paper_2506_05096_b200 import binding as A
from paper_2506_05096_b200 import synth
from helpers import Guarded, assert_attn_close, bf16_dev_to_f64, check_step_against_oracle, dev, device_state, f64, to_dev_bf16

pytestmark = pytest.mark.gpu

ATTN_MAX_ABS, ATTN_MEAN_ABS, LSE_ABS, SCORE_RTOL = 2e-2, 2e-3, 1e-3, 1e-5


# ---------------------------------------------------------------------- score
def _score_case(oracle, w, seed, n_sel, delta_mode, lse_mode, use_lse=True, use_n=True, w_alpha=1.0, w_beta=1.0):
    inp = synth.make_step_inputs(w, seed, parts=("x_ref", "x_cur"))
    B, N, D, H = w.B, w.N, w.D, w.H
    lse = inp["lse"] if use_lse else None
    if lse is not None and lse_mode == A.LSE_SUM_EXP:
        lse = (lse - np.float32(math.log(N))).astype(np.float32)      # keep exp() moderate for any N
    n_skip = inp["n_skip"][:, :n_sel].copy() if use_n else None
    want = oracle.score(f64(inp["x_cur"]), f64(inp["x_ref"]), lse, n_skip, n_sel=n_sel, H=H, w_alpha=w_alpha,
                        w_beta=w_beta, delta_mode=delta_mode, lse_mode=lse_mode)
    out = torch.full((B, n_sel), float("nan"), device="cuda")
    A.astraea_score(to_dev_bf16(inp["x_cur"]), to_dev_bf16(inp["x_ref"]),
                    None if lse is None else dev(lse), None if n_skip is None else dev(n_skip), out,
                    B, N, n_sel, D, H, w_alpha, w_beta, delta_mode, lse_mode)
    torch.cuda.synchronize()
    got = out.cpu().numpy().astype(np.float64)
    err = np.abs(got - want) / np.maximum(np.abs(want), 1e-30)
    assert err.max() < SCORE_RTOL, err.max()
    return got, want


@pytest.mark.parametrize("delta_mode", [A.DELTA_MEAN_ABS, A.DELTA_MEAN_SQ, A.DELTA_MEAN_SIGNED])
@pytest.mark.parametrize("lse_mode", [A.LSE_SUM_EXP, A.LSE_LOG])
def test_score_tiny_all_modes(oracle, delta_mode, lse_mode):
    w = synth.scaled(synth.WORKLOADS["tiny"], n_skip_max=5)
    # the signed mean cancels to ~0: compare it in absolute terms through a w_beta = 1 offset
    _score_case(oracle, w, 0, w.N_v, delta_mode, lse_mode, w_alpha=0.5, w_beta=1.0)


@pytest.mark.parametrize("name,N_v,N_t", [("cogvideox", 1013, 26), ("opensora", 777, 0), ("hunyuan", 530, 0)])
def test_score_workload_shapes_ragged(oracle, name, N_v, N_t):
    w = synth.scaled(synth.WORKLOADS[name], N_v=N_v, N_t=N_t)
    _score_case(oracle, w, 1, N_v, A.DELTA_MEAN_ABS, A.LSE_SUM_EXP)


def test_score_without_lse_and_counters_and_odd_width(oracle):
    w = synth.Workload("odd", B=2, H=3, d=24, N_v=70, N_t=3)      # D = 72: 9 vectors per row, a ragged tail
    _score_case(oracle, w, 2, 70, A.DELTA_MEAN_ABS, A.LSE_SUM_EXP, use_lse=False, use_n=False)
    w = synth.Workload("wide", B=1, H=5, d=200, N_v=33, N_t=0)    # D = 1000: 125 vectors, unrolled body + tail
    _score_case(oracle, w, 3, 33, A.DELTA_MEAN_SQ, A.LSE_LOG)


def test_score_counter_clamp(oracle):
    B, N, D = 1, 8, 64
    x = torch.zeros(B, N, D, dtype=torch.bfloat16, device="cuda")
    n = torch.tensor([[0, 1, 2, 79, 80, 81, 1000, 2 ** 30]], dtype=torch.int32, device="cuda")
    out = torch.empty(B, N, device="cuda")
    A.astraea_score(x, x, None, n, out, B, N, N, D, 1, 1.0, 1.0)
    want = np.exp(np.minimum(n.cpu().numpy().astype(np.float64), 80.0))
    got = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert (np.abs(got - want) / want).max() < 1e-5


def test_score_lse_clamp_keeps_fp32_scores_finite(oracle):
    """Log values above 80 (a row with one logit of that size, as sharpened attention leaves behind) count as 80 in
    the sum-of-exponentials mode, on the device as in the oracle; the scores stay finite and ordered."""
    B, N, D, H = 1, 16, 64, 2
    rng = np.random.default_rng(3)
    x_ref = synth.f32_to_bf16_bits(rng.standard_normal((B, N, D)).astype(np.float32))
    x_cur = synth.f32_to_bf16_bits(rng.standard_normal((B, N, D)).astype(np.float32))
    lse = rng.uniform(-5, 5, (B, H, N)).astype(np.float32)
    lse[0, 0, 3], lse[0, 1, 5], lse[0, :, 7], lse[0, 0, 9] = 79.5, 80.0, 95.0, 3.0e4
    want = oracle.score(f64(x_cur), f64(x_ref), lse, None, H=H, w_alpha=1e-3, w_beta=0.0)
    out = torch.empty(B, N, device="cuda")
    A.astraea_score(to_dev_bf16(x_cur), to_dev_bf16(x_ref), dev(lse), None, out, B, N, N, D, H, 1e-3, 0.0)
    got = out.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert (np.abs(got - want) / np.abs(want)).max() < SCORE_RTOL


# --------------------------------------------------------------------- select
def _select_case(oracle, s, k, n_always=0, with_n=True, with_rem=True, seed=0):
    B, n_sel = s.shape
    rng = np.random.default_rng(seed)
    n0 = rng.integers(0, 85, size=(B, n_sel)).astype(np.int32) if with_n else None
    want_sel, want_rem, want_n = oracle.select(s, k, n_always, n0)
    # every output sits between guard bands: a write one past either end is caught
    g_sel = Guarded((B, k + n_always), torch.int32)
    g_rem = Guarded((B, n_sel - k), torch.int32) if with_rem else None
    g_n = Guarded((B, n_sel), torch.int32, init=dev(n0)) if with_n else None
    idx_sel, idx_rem, n_dev = g_sel.t, (g_rem.t if with_rem else None), (g_n.t if with_n else None)
    ws = A.new_workspace(A.OP_SELECT, B, 0, n_sel, k, 0)
    A.astraea_select(dev(s), B, n_sel, k, n_always, idx_sel, idx_rem, n_dev, ws)
    for g in (g_sel, g_rem, g_n):
        if g is not None:
            g.check(("select", B, n_sel, k, n_always))
    assert np.array_equal(idx_sel.cpu().numpy(), want_sel)
    if with_rem:
        assert np.array_equal(idx_rem.cpu().numpy(), want_rem)
    if with_n:
        assert np.array_equal(n_dev.cpu().numpy(), want_n)


@pytest.mark.parametrize("n_sel", [1, 5, 256, 1000, 4096, 4097, 9000])
def test_select_integer_scores_bit_exact(oracle, n_sel):
    for seed, levels in ((0, 2), (1, 7), (2, 64), (3, 100000)):
        s = synth.integer_scores(2, n_sel, seed, levels)
        for k in sorted({0, 1, n_sel // 4, n_sel // 2, n_sel - 1, n_sel}):
            if 0 <= k <= n_sel:
                _select_case(oracle, s, k, seed=seed)


def test_select_all_equal_and_special_values(oracle):
    _select_case(oracle, np.ones((2, 5000), np.float32), 1234)
    s = np.random.default_rng(4).standard_normal((1, 3000)).astype(np.float32)
    s[0, ::7] = 0.0
    s[0, 3::7] = -0.0
    s[0, 5::97] = np.nan
    s[0, 11::101] = np.inf
    s[0, 13::103] = -np.inf
    s[0, 17::89] = 1e-42           # denormal
    for k in (0, 10, 100, 1500, 2900, 2999, 3000):
        _select_case(oracle, s, k)


def test_select_rows_longer_than_a_cluster_holds(oracle):
    """Rows above 131072 tokens take the one-CTA path that re-reads the row in every pass."""
    s = np.random.default_rng(9).standard_normal((2, 140001)).astype(np.float32)
    s[:, ::5] = 0.25                     # plenty of ties
    for k in (0, 1, 70000, 140001):
        _select_case(oracle, s, k, n_always=3)


def test_select_always_kept_span_and_optional_outputs(oracle):
    s = synth.integer_scores(2, 700, 5, 9)
    _select_case(oracle, s, 300, n_always=26)
    _select_case(oracle, s, 0, n_always=26)
    _select_case(oracle, s, 300, n_always=26, with_n=False, with_rem=False)


@pytest.mark.parametrize("name", ["cogvideox", "opensora", "hunyuan", "sweep"])
def test_select_full_size_float_scores(oracle, name):
    w = synth.WORKLOADS[name]
    rng = np.random.default_rng(6)
    s = np.exp(rng.standard_normal((w.B, w.N_v))).astype(np.float32) * 8000 + np.exp(rng.integers(0, 4, (w.B, w.N_v))).astype(np.float32)
    for th in w.thetas_permille[:3]:
        _select_case(oracle, s, w.k_of(th), n_always=w.N_t)
    _select_case(oracle, synth.integer_scores(w.B, w.N_v, 7, 50), w.k_of(w.thetas_permille[0]), n_always=w.N_t)


# -------------------------------------------------------------------- scatter
@pytest.mark.parametrize("B,N,M,R", [(1, 256, 128, 128), (2, 301, 77, 3072), (1, 64, 64, 72), (2, 50, 1, 1152)])
def test_scatter_reuse_bit_exact(oracle, B, N, M, R):
    rng = np.random.default_rng(8)
    cache = synth.f32_to_bf16_bits(rng.standard_normal((B, N, R)).astype(np.float32))
    rows = synth.f32_to_bf16_bits(rng.standard_normal((B, M, R)).astype(np.float32))
    full = synth.f32_to_bf16_bits(rng.standard_normal((B, N, R)).astype(np.float32))
    idx = np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    g = Guarded((B, N, R), torch.bfloat16, init=to_dev_bf16(cache))
    A.astraea_scatter_reuse(g.t, to_dev_bf16(rows), dev(idx), B, N, M, R, workspace=ws)
    want = oracle.scatter_reuse(f64(cache), f64(rows), idx)
    g.check("scatter")
    assert np.array_equal(bf16_dev_to_f64(g.t), want)
    g = Guarded((B, N, R), torch.bfloat16, init=to_dev_bf16(cache))
    A.astraea_scatter_reuse(g.t, to_dev_bf16(full), dev(idx), B, N, M, R, A.SCATTER_SRC_FULL, workspace=ws)
    want = oracle.scatter_reuse(f64(cache), np.take_along_axis(f64(full), idx[:, :, None].astype(np.int64), 1), idx)
    g.check("scatter, full-layout source")
    assert np.array_equal(bf16_dev_to_f64(g.t), want)
    A.astraea_poll_error(ws)                     # nothing to report


def test_scatter_reports_and_skips_bad_index_entries():
    """Out of range, duplicate and descending entries: each is skipped (no write outside the cache, no row written
    twice), the rest of the list is applied, and the error word says BAD_INDEX when a workspace is given."""
    B, N, M, R = 1, 32, 7, 64
    cache = torch.zeros(B, N, R, dtype=torch.bfloat16, device="cuda")
    rows = (torch.arange(1, M + 1, device="cuda").float()[None, :, None].expand(B, M, R)).bfloat16().contiguous()
    idx = torch.tensor([[3, 5, 5, 4, 9, 31, 32]], dtype=torch.int32, device="cuda")     # dup 5, descending 4, 32 out of range
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    g = Guarded((B, N, R), torch.bfloat16, init=cache)
    A.astraea_scatter_reuse(g.t, rows, idx, B, N, M, R, workspace=ws)
    with pytest.raises(A.AstraeaError) as e:
        A.astraea_poll_error(ws)
    assert e.value.code == A.ERR_BAD_INDEX
    g.check("scatter with bad entries")
    got = g.t.float()[0, :, 0].cpu().numpy()
    want = np.zeros(N)
    want[3], want[5], want[9], want[31] = 1, 2, 5, 6          # rows 2 (the second 5), 3 (the 4) and 6 (the 32) are skipped
    assert np.array_equal(got, want)
    # without a workspace the same entries are skipped silently
    g2 = Guarded((B, N, R), torch.bfloat16, init=cache)
    A.astraea_scatter_reuse(g2.t, rows, idx, B, N, M, R)
    g2.check()
    assert torch.equal(g2.t, g.t)


def test_scatter_with_no_rows_leaves_cache_alone():
    c = torch.randn(1, 16, 64, device="cuda").bfloat16()
    before = c.clone()
    A.astraea_scatter_reuse(c, c, torch.empty(1, 0, dtype=torch.int32, device="cuda"), 1, 16, 0, 64)
    assert torch.equal(c, before)


# ------------------------------------------------------------------ attention
def _attn_case(oracle, B, H, N, d, M, seed, layout="bnhd", compact=False, dense=False, scale=0.0, amp=1.0, small_ctas=False,
               whole_keys=False, expect_split=None):
    rng = np.random.default_rng(seed)
    # amp sharpens the logits only (q, k); values and the cache stay N(0,1)
    q, k, v, cache = (synth.f32_to_bf16_bits((a * rng.standard_normal((B, N, H, d))).astype(np.float32)) for a in (amp, amp, 1.0, 1.0))
    idx = None if dense else np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
    M = N if dense else M
    want_o, want_lse, _ = oracle.sparse_attn(f64(q), f64(k), f64(v), q_idx=idx, scale=scale)

    def place(bits):
        t = to_dev_bf16(bits)
        if layout == "bhnd":
            t = t.permute(0, 2, 1, 3).contiguous()
            return t, (H * N * d, N * d, d)
        return t, A.bhnd_strides(N, H, d)

    (qd, qs), (kd, ks), (vd, vs) = place(q), place(k), place(v)
    lse_cache0 = rng.standard_normal((B, H, N)).astype(np.float32)
    if compact:
        g_out = Guarded((B, M, H, d), torch.bfloat16, init=torch.zeros(B, M, H, d, dtype=torch.bfloat16, device="cuda"))
        g_lse = Guarded((B, H, M), torch.float32, init=torch.zeros(B, H, M, device="cuda"))
    else:
        g_out = Guarded((B, N, H, d), torch.bfloat16, init=to_dev_bf16(cache))
        g_lse = Guarded((B, H, N), torch.float32, init=dev(lse_cache0))
    out, lse = g_out.t, g_lse.t
    ws = A.new_workspace(A.OP_SPARSE_ATTN, B, H, N, M, d)
    flags = (A.ATTN_COMPACT_OUT if compact else 0) | (A.ATTN_SMALL_CTAS if small_ctas else 0) | (A.ATTN_WHOLE_KEYS if whole_keys else 0)
    if expect_split is not None:
        plan = A.astraea_sparse_attn_plan(B, H, N, M, d, flags=flags, workspace_bytes=ws.numel())
        assert (plan["split"], plan["small_ctas"]) == (expect_split, False) and (plan["split_units"] > 0) == (expect_split > 1), plan
    A.astraea_sparse_attn(qd, kd, vd, qs, ks, vs, None if idx is None else dev(idx), M, out, lse, B, H, N, d,
                          scale=scale, flags=flags, workspace=ws)
    A.astraea_poll_error(ws)
    g_out.check(("attention out", B, H, N, d, M))
    g_lse.check(("attention lse", B, H, N, d, M))
    got = bf16_dev_to_f64(out)
    got_lse = lse.cpu().numpy().astype(np.float64)
    if idx is None:
        idx = np.broadcast_to(np.arange(N, dtype=np.int32), (B, N))
    if compact:
        got_rows, got_lse_rows = got, got_lse
    else:
        got_rows = np.take_along_axis(got, idx[:, :, None, None].astype(np.int64), 1)
        got_lse_rows = np.take_along_axis(got_lse, idx[:, None, :].astype(np.int64), 2)
        # rows that were not selected are bit-identical to the cache (reuse)
        mask = np.ones((B, N), bool)
        for b in range(B):
            mask[b, idx[b]] = False
        assert np.array_equal(got[mask], f64(cache)[mask])
        assert np.array_equal(got_lse.transpose(0, 2, 1)[mask], lse_cache0.astype(np.float64).transpose(0, 2, 1)[mask])
    assert_attn_close(got_rows, want_o, ATTN_MAX_ABS, ATTN_MEAN_ABS)
    # head_dim 64 takes the row sums from the tensor core, i.e. of the bf16-rounded probabilities: where one key
    # dominates a row the LSE carries that rounding (2^-8 relative at worst); elsewhere it averages out
    lse_tol = 5e-3 if (d == 64 and amp > 1.0) else LSE_ABS
    assert np.abs(got_lse_rows - want_lse).max() < lse_tol, np.abs(got_lse_rows - want_lse).max()


def test_attn_tiny_config(oracle):
    _attn_case(oracle, 1, 2, 256, 64, 128, seed=0)


@pytest.mark.parametrize("d", [64, 72, 128])
def test_attn_single_tile(oracle, d):
    _attn_case(oracle, 1, 1, 128, d, 128, seed=1, dense=True)


@pytest.mark.parametrize("d", [64, 72, 128])
@pytest.mark.parametrize("N,M", [(300, 77), (1000, 333), (129, 129), (1, 1), (127, 5), (64, 64), (65, 3)])
def test_attn_ragged_tiles(oracle, d, N, M):
    _attn_case(oracle, 2, 3, N, d, M, seed=2)


@pytest.mark.parametrize("d", [64, 72])
def test_attn_one_query_tile_per_cta_shape(oracle, d):
    """The CTA shape that the library picks for launches of a few rounds (one 128-row query tile, two CTAs per SM),
    forced here on small cases: ragged tiles, several CTAs per head, many key tiles (every stage phase), a compact
    output, and logits that make the CTAs redo their work."""
    _attn_case(oracle, 2, 3, 300, d, 77, seed=70, small_ctas=True)
    _attn_case(oracle, 2, 2, 1000, d, 333, seed=71, small_ctas=True)
    _attn_case(oracle, 1, 2, 64 * 27 + 40, d, 130, seed=72, small_ctas=True)
    _attn_case(oracle, 2, 2, 400, d, 100, seed=73, compact=True, small_ctas=True)
    _attn_case(oracle, 1, 2, 129, d, 129, seed=74, dense=True, small_ctas=True)
    _attn_case(oracle, 1, 2, 900, d, 600, seed=75, amp=12.0, small_ctas=True)
    _attn_case(oracle, 1, 1, 1, d, 1, seed=76, small_ctas=True)


@pytest.mark.parametrize("d", [64, 72, 128])
def test_attn_last_round_split_by_keys(oracle, d):
    """Launches of less than one round of CTAs and 32+ key tiles: every CTA is replaced by 2-8 CTAs with a share of the
    keys each, whose fp32 rows a second kernel merges.  Ragged last key tile, a last CTA with one query tile, shares
    of unequal length, a compact output, the head-major layout, logits that make the shares redo their work."""
    _attn_case(oracle, 1, 3, 2100, d, 700, seed=300 + d, expect_split=2)
    _attn_case(oracle, 2, 2, 64 * 53 + 7, d, 300, seed=301 + d, expect_split=3)
    _attn_case(oracle, 1, 2, 64 * 130 + 33, d, 129, seed=302 + d, expect_split=8)
    _attn_case(oracle, 1, 2, 4200, d, 520, seed=303 + d, compact=True, expect_split=4)
    _attn_case(oracle, 1, 2, 2100, d, 260, seed=304 + d, layout="bhnd", expect_split=2)
    _attn_case(oracle, 1, 2, 2100, d, 600, seed=305 + d, amp=12.0, expect_split=2)
    _attn_case(oracle, 1, 2, 2100, d, 2100, seed=306 + d, dense=True, expect_split=2)
    # the same launch with every CTA over all keys
    _attn_case(oracle, 1, 3, 2100, d, 700, seed=300 + d, whole_keys=True, expect_split=1)


def test_attn_many_key_tiles_exercise_every_stage_phase(oracle):
    _attn_case(oracle, 1, 2, 128 * 19 + 16, 128, 200, seed=3)
    _attn_case(oracle, 1, 2, 128 * 27 + 112, 64, 130, seed=4)
    _attn_case(oracle, 1, 2, 128 * 23 + 40, 72, 260, seed=5)


def test_attn_head_dim_72_layouts(oracle):
    _attn_case(oracle, 2, 2, 400, 72, 100, seed=11, layout="bhnd")
    _attn_case(oracle, 2, 3, 400, 72, 100, seed=12, compact=True)
    _attn_case(oracle, 1, 2, 900, 72, 128, seed=13, amp=2.5)


def test_attn_head_major_layout_compact_output_and_scale(oracle):
    _attn_case(oracle, 2, 2, 400, 64, 100, seed=5, layout="bhnd")
    _attn_case(oracle, 2, 2, 400, 128, 100, seed=6, compact=True)
    _attn_case(oracle, 1, 2, 400, 128, 100, seed=7, scale=0.05)


def test_attn_dense_equals_all_rows(oracle):
    _attn_case(oracle, 1, 2, 517, 64, 517, seed=8, dense=True)


def test_attn_peaked_softmax(oracle):
    # logits of order +-25: most of the probability mass of a row sits on a few keys
    _attn_case(oracle, 1, 2, 900, 64, 128, seed=9, amp=2.5)
    _attn_case(oracle, 1, 1, 900, 128, 128, seed=10, amp=2.0)


@pytest.mark.parametrize("d", [64, 72, 128])
def test_attn_reference_maximum_far_too_low_is_repaired_exactly(oracle, d):
    # logits of order +-600: in most rows a later key tile beats the first tile's maximum by more than 100 nats,
    # past the speculation limit of the kernel, so that the CTAs redo their work against exact row maxima;
    # three CTAs per head, the last one with a single query tile, ragged last key tile
    _attn_case(oracle, 1, 2, 900, d, 600, seed=20 + d, amp=12.0)
    # a single key tile and exactly two: the odd-tile warpgroup has nothing, or one tile, to contribute
    _attn_case(oracle, 1, 1, 40, d, 40, seed=21 + d, amp=12.0)
    _attn_case(oracle, 2, 1, 100, d, 70, seed=22 + d, amp=12.0)


@pytest.mark.parametrize("d", [64, 72, 128])
@pytest.mark.parametrize("col", [3, 12, 30, 47, 63])
def test_attn_single_overflowing_key_in_any_column_of_a_later_tile(oracle, d, col):
    """One key of the second tile beats everything in the first by 128 nats and nothing else is large: the only
    exponential that overflows sits in column `col` of its tile, whichever pipe computes that column.  The rows
    must come out as that key's value row (and the LSE as its logit)."""
    B, H, N, M = 1, 1, 129, 20
    rng = np.random.default_rng(60 + col)
    q = np.zeros((B, N, H, d), np.float32)
    k = np.zeros((B, N, H, d), np.float32)
    q[..., 0] = 32.0
    k[0, 64 + col, 0, 0] = 32.0 * math.sqrt(d) / 8.0          # logit 128 * sqrt(d) / sqrt(d) ... = 128 at that key, 0 elsewhere
    v = rng.standard_normal((B, N, H, d)).astype(np.float32)
    qb, kb, vb = (synth.f32_to_bf16_bits(a) for a in (q, k, v))
    idx = np.sort(rng.choice(N, M, replace=False)).astype(np.int32)[None]
    want_o, want_lse, _ = oracle.sparse_attn(f64(qb), f64(kb), f64(vb), q_idx=idx)
    out = torch.zeros(B, M, H, d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(B, H, M, device="cuda")
    ws = A.new_workspace(A.OP_SPARSE_ATTN, B, H, N, M, d)
    s_ = A.bhnd_strides(N, H, d)
    A.astraea_sparse_attn(to_dev_bf16(qb), to_dev_bf16(kb), to_dev_bf16(vb), s_, s_, s_, dev(idx), M, out, lse, B, H, N, d,
                          flags=A.ATTN_COMPACT_OUT, workspace=ws)
    A.astraea_poll_error(ws)
    assert np.abs(bf16_dev_to_f64(out) - want_o).max() < ATTN_MAX_ABS
    assert np.abs(lse.cpu().numpy() - want_lse).max() < 2e-2 * 1e-2 * 128          # relative 2e-4 of a logit of ~128
    assert np.abs(want_o - f64(vb)[0, 64 + col][None, None]).max() < 1e-9            # the oracle agrees: one-hot rows


@pytest.mark.parametrize("d", [64, 72, 128])
def test_attn_select_q_and_k_ablation(oracle, d):
    """kv_idx: the softmax runs over the listed keys/values only (the ablation that also masks K and V)."""
    rng = np.random.default_rng(20 + d)
    B, H, N, M, M_kv = 2, 2, 500, 90, 217
    q, k, v, cache = (synth.f32_to_bf16_bits(rng.standard_normal((B, N, H, d)).astype(np.float32)) for _ in range(4))
    q_idx = np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
    kv_idx = np.stack([np.sort(rng.choice(N, M_kv, replace=False)) for _ in range(B)]).astype(np.int32)
    want_o, want_lse, _ = oracle.sparse_attn(f64(q), f64(k), f64(v), q_idx=q_idx, kv_idx=kv_idx)
    out, lse = to_dev_bf16(cache), torch.zeros(B, H, N, device="cuda")
    ws = A.new_workspace(A.OP_SPARSE_ATTN_KV, B, H, N, M_kv, d)
    s = A.bhnd_strides(N, H, d)
    A.astraea_sparse_attn(to_dev_bf16(q), to_dev_bf16(k), to_dev_bf16(v), s, s, s, dev(q_idx), M, out, lse, B, H, N, d,
                          workspace=ws, kv_idx=dev(kv_idx), M_kv=M_kv)
    A.astraea_poll_error(ws)
    got = np.take_along_axis(bf16_dev_to_f64(out), q_idx[:, :, None, None].astype(np.int64), 1)
    assert_attn_close(got, want_o, ATTN_MAX_ABS, ATTN_MEAN_ABS)
    got_lse = np.take_along_axis(lse.cpu().numpy().astype(np.float64), q_idx[:, None, :].astype(np.int64), 2)
    assert np.abs(got_lse - want_lse).max() < LSE_ABS
    mask = np.ones((B, N), bool)
    for b in range(B):
        mask[b, q_idx[b]] = False
    assert np.array_equal(bf16_dev_to_f64(out)[mask], f64(cache)[mask])
    # too small a workspace for the gathered rows is refused
    with pytest.raises(A.AstraeaError) as e:
        A.astraea_sparse_attn(to_dev_bf16(q), to_dev_bf16(k), to_dev_bf16(v), s, s, s, dev(q_idx), M, out, lse, B, H, N, d,
                              workspace=A.new_workspace(A.OP_SPARSE_ATTN, B, H, N, M, d), kv_idx=dev(kv_idx), M_kv=M_kv)
    assert e.value.code == A.ERR_WORKSPACE_TOO_SMALL


def test_attn_closed_forms_on_device():
    """Zero keys: every selected output is the mean of all value rows and LSE = ln N; this
    catches phantom keys from the zero-filled tail of the last key tile."""
    B, H, N, d, M = 1, 2, 333, 64, 50
    g = torch.Generator(device="cpu").manual_seed(0)
    q = torch.randn(B, N, H, d, generator=g).bfloat16().cuda()
    v = torch.randn(B, N, H, d, generator=g).bfloat16().cuda()
    k = torch.zeros_like(q)
    idx = torch.arange(0, 2 * M, 2, dtype=torch.int32, device="cuda")[None].contiguous()
    out = torch.zeros(B, M, H, d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(B, H, M, device="cuda")
    ws = A.new_workspace(A.OP_SPARSE_ATTN, B, H, N, M, d)
    s = A.bhnd_strides(N, H, d)
    A.astraea_sparse_attn(q, k, v, s, s, s, idx, M, out, lse, B, H, N, d, flags=A.ATTN_COMPACT_OUT, workspace=ws)
    A.astraea_poll_error(ws)
    mean_v = v.double().mean(dim=1, keepdim=True)
    assert (out.double() - mean_v).abs().max().item() < 4e-3
    assert (lse.double() - math.log(N)).abs().max().item() < 1e-5


def test_attn_bad_index_is_reported_not_dereferenced():
    B, H, N, d, M = 1, 1, 64, 64, 4
    q = torch.zeros(B, N, H, d, dtype=torch.bfloat16, device="cuda")
    out = torch.ones(B, N, H, d, dtype=torch.bfloat16, device="cuda")
    idx = torch.tensor([[0, 1, 64, 2 ** 30]], dtype=torch.int32, device="cuda")
    ws = A.new_workspace(A.OP_SPARSE_ATTN, B, H, N, M, d)
    s = A.bhnd_strides(N, H, d)
    A.astraea_sparse_attn(q, q, q, s, s, s, idx, M, out, None, B, H, N, d, workspace=ws)
    with pytest.raises(A.AstraeaError) as e:
        A.astraea_poll_error(ws)
    assert e.value.code == A.ERR_BAD_INDEX
    A.astraea_poll_error(ws)                 # the word was cleared
    assert torch.equal(out[0, 2:], torch.ones_like(out[0, 2:]))


def test_bounded_wait_runs_out_reports_timeout_and_the_workspace_stays_usable(oracle):
    """Failure detection without a fault: a wait on a barrier that nothing arrives at gives up after its limit (200
    microseconds here), the error word says TIMEOUT, and the very same workspace then serves a normal attention call."""
    B, H, N, d, M = 1, 2, 300, 64, 77
    ws = A.new_workspace(A.OP_SPARSE_ATTN, B, H, N, M, d)
    gave_up = torch.zeros(1, dtype=torch.int32, device="cuda")
    A.astraea_selftest_wait(ws, 200, gave_up)
    with pytest.raises(A.AstraeaError) as e:
        A.astraea_poll_error(ws)
    assert e.value.code == A.ERR_TIMEOUT and int(gave_up.item()) == 1
    A.astraea_poll_error(ws)                 # the word was cleared
    rng = np.random.default_rng(4)
    q, k, v = (synth.f32_to_bf16_bits(rng.standard_normal((B, N, H, d)).astype(np.float32)) for _ in range(3))
    idx = np.sort(rng.choice(N, M, replace=False)).astype(np.int32)[None]
    out = torch.zeros(B, M, H, d, dtype=torch.bfloat16, device="cuda")
    s_ = A.bhnd_strides(N, H, d)
    A.astraea_sparse_attn(to_dev_bf16(q), to_dev_bf16(k), to_dev_bf16(v), s_, s_, s_, dev(idx), M, out, None, B, H, N, d,
                          flags=A.ATTN_COMPACT_OUT, workspace=ws)
    A.astraea_poll_error(ws)
    want, _, _ = oracle.sparse_attn(f64(q), f64(k), f64(v), q_idx=idx)
    assert_attn_close(bf16_dev_to_f64(out), want)


def test_attn_duplicate_and_descending_indices_are_reported_and_written_once():
    """q_idx must be strictly ascending: a duplicate would make two rows race on one output row.  The offending
    entries are skipped (their rows keep the cache), the others are computed, BAD_INDEX is reported."""
    B, H, N, d, M = 1, 2, 200, 64, 6
    g = torch.Generator(device="cpu").manual_seed(5)
    q, k, v = (torch.randn(B, N, H, d, generator=g).bfloat16().cuda() for _ in range(3))
    s = A.bhnd_strides(N, H, d)
    ws = A.new_workspace(A.OP_SPARSE_ATTN, B, H, N, M, d)
    good = torch.tensor([[2, 7, 9, 50, 120, 199]], dtype=torch.int32, device="cuda")
    want = torch.full((B, N, H, d), 3.0, dtype=torch.bfloat16, device="cuda")
    A.astraea_sparse_attn(q, k, v, s, s, s, good, M, want, None, B, H, N, d, workspace=ws)
    A.astraea_poll_error(ws)
    bad = torch.tensor([[2, 7, 7, 50, 9, 199]], dtype=torch.int32, device="cuda")       # a duplicate 7, a descending 9
    out = torch.full((B, N, H, d), 3.0, dtype=torch.bfloat16, device="cuda")
    A.astraea_sparse_attn(q, k, v, s, s, s, bad, M, out, None, B, H, N, d, workspace=ws)
    with pytest.raises(A.AstraeaError) as e:
        A.astraea_poll_error(ws)
    assert e.value.code == A.ERR_BAD_INDEX
    for tok in (2, 7, 50, 199):
        assert torch.equal(out[0, tok], want[0, tok])
    untouched = torch.ones(N, dtype=torch.bool)
    untouched[[2, 7, 50, 199]] = False
    assert bool((out[0, untouched.cuda()] == 3.0).all())


def test_attn_bad_indices_in_a_launch_that_is_split_by_keys():
    """The same rule where the CTAs take shares of the keys and a second kernel merges them: the merge skips the rows
    that the attention kernel reported, writes the others, and the rows in between keep the cache."""
    B, H, N, d, M = 1, 2, 2100, 64, 300
    g = torch.Generator(device="cpu").manual_seed(6)
    q, k, v = (torch.randn(B, N, H, d, generator=g).bfloat16().cuda() for _ in range(3))
    s = A.bhnd_strides(N, H, d)
    ws = A.new_workspace(A.OP_SPARSE_ATTN, B, H, N, M, d)
    assert A.astraea_sparse_attn_plan(B, H, N, M, d, workspace_bytes=ws.numel())["split"] == 2
    good = (torch.arange(M, dtype=torch.int32) * 7).view(1, M).cuda()
    want, want_lse = torch.full((B, N, H, d), 3.0, dtype=torch.bfloat16, device="cuda"), torch.full((B, H, N), -7.0, device="cuda")
    A.astraea_sparse_attn(q, k, v, s, s, s, good, M, want, want_lse, B, H, N, d, workspace=ws)
    A.astraea_poll_error(ws)
    bad = good.clone()
    bad[0, 10] = bad[0, 9]                       # a duplicate
    bad[0, 200] = 5                              # a descending step
    bad[0, 299] = N + 3                          # out of range
    out, lse = torch.full((B, N, H, d), 3.0, dtype=torch.bfloat16, device="cuda"), torch.full((B, H, N), -7.0, device="cuda")
    A.astraea_sparse_attn(q, k, v, s, s, s, bad, M, out, lse, B, H, N, d, workspace=ws)
    with pytest.raises(A.AstraeaError) as e:
        A.astraea_poll_error(ws)
    assert e.value.code == A.ERR_BAD_INDEX
    ok_rows = [r for r in range(M) if r not in (10, 200, 299)]
    toks = good[0, ok_rows].long()
    assert torch.equal(out[0, toks], want[0, toks]) and torch.equal(lse[0][:, toks], want_lse[0][:, toks])
    untouched = torch.ones(N, dtype=torch.bool, device="cuda")
    untouched[toks] = False
    assert bool((out[0, untouched] == 3.0).all()) and bool((lse[0][:, untouched] == -7.0).all())


# ------------------------------------------------------------- the whole step
def _step_case(oracle, w, seed, theta, steps=1):
    inp = synth.make_step_inputs(w, seed)
    B, N, H, d, D, N_sel, n_always = w.B, w.N, w.H, w.d, w.D, w.N_v, w.N_t
    k_keep = w.k_of(theta)
    M = k_keep + n_always
    # state on the device
    x_ref = to_dev_bf16(inp["x_ref"])
    lse = dev(inp["lse"] - np.float32(math.log(N)))
    n_skip = dev(inp["n_skip"])
    out = to_dev_bf16(inp["cache"])
    score = torch.empty(B, N_sel, device="cuda")
    idx_sel = torch.empty(B, M, dtype=torch.int32, device="cuda")
    idx_rem = torch.empty(B, N_sel - k_keep, dtype=torch.int32, device="cuda")
    ws = A.new_workspace(A.OP_STEP, B, H, N, M, d)
    x_bits, q_bits, k_bits, v_bits = inp["x_cur"], inp["q"], inp["k"], inp["v"]
    checked = near_ties = 0
    for t in range(steps):
        if t > 0:
            x_bits = synth.drift_step(x_bits, 100 + t, 0.05, False)
            q_bits, k_bits, v_bits = (synth.drift_step(a, 200 + 10 * t + i, 0.05, True) for i, a in enumerate((q_bits, k_bits, v_bits)))
        # teacher forcing: the oracle starts each step from the state the device had (bf16 / fp32 values)
        prev = device_state(x_ref, lse, n_skip, out)
        A.astraea_step(to_dev_bf16(x_bits), x_ref, lse, n_skip, to_dev_bf16(q_bits), to_dev_bf16(k_bits),
                       to_dev_bf16(v_bits), out, score, idx_sel, idx_rem, B, H, N, N_sel, d, k_keep, workspace=ws)
        A.astraea_poll_error(ws)
        _, tie = check_step_against_oracle(oracle, prev, x_bits, q_bits, k_bits, v_bits, k_keep, n_always,
                                           score, idx_sel, idx_rem, x_ref, lse, n_skip, out, what=(w.name, t))
        near_ties += tie
        checked += 1
    assert checked == steps                     # every step was compared in full, near-ties included
    return near_ties


def test_step_tiny_config(oracle):
    _step_case(oracle, synth.WORKLOADS["tiny"], 0, 500)


def test_step_keep_ratio_zero_and_one(oracle):
    w = synth.scaled(synth.WORKLOADS["tiny"], drift_sigma=0.05, n_skip_max=3)
    _step_case(oracle, w, 1, 0)
    _step_case(oracle, w, 1, 1000)


def test_step_with_text_tokens_and_batch(oracle):
    w = synth.Workload("mini-cog", B=2, H=4, d=64, N_v=450, N_t=26)
    _step_case(oracle, w, 2, 250)


def test_step_opensora_shaped_reduced(oracle):
    w = synth.scaled(synth.WORKLOADS["opensora"], N_v=8 * 16 * 16, H=4)
    _step_case(oracle, w, 4, 400)


def test_step_chain_of_three_steps_d128(oracle):
    w = synth.Workload("mini-hy", B=1, H=2, d=128, N_v=8 * 12 * 20, N_t=0)
    _step_case(oracle, w, 3, 600, steps=3)


def test_step_chain_of_fifty_steps_reduced_hunyuan_shape(oracle):
    """The 50-step drifting-latent workload at a reduced shape (8x12x20 tokens, 2 heads, head_dim 128):
    every step is checked against the oracle started from the device's state of the step before."""
    w = synth.Workload("mini-hy-50", B=1, H=2, d=128, N_v=8 * 12 * 20, N_t=0)
    _step_case(oracle, w, 5, 600, steps=50)
    _step_case(oracle, w, 6, 300, steps=12)



# ------------------------------------------------------------- host-buffer session
def test_session_step_host_equals_the_device_path_and_the_oracle(oracle):
    """astraea_step_host (pinned host buffers, copies overlapped with the attention by head group) against
    astraea_step on device buffers from the same initial state: bit-identical outputs over three steps; the first,
    dense step also against the oracle."""
    w = synth.Workload("mini-session", B=2, H=6, d=64, N_v=700, N_t=30)
    inp = synth.make_step_inputs(w, 11)
    B, N, H, d, N_sel, n_always = w.B, w.N, w.H, w.d, w.N_v, w.N_t
    sess = A.Session(B, H, N, N_sel, d)
    # device path, same initial state as a fresh session: zero caches and counters, x_ref = first x_cur
    x_ref = to_dev_bf16(inp["x_cur"])
    lse = torch.zeros(B, H, N, device="cuda")
    n_skip = torch.zeros(B, N_sel, dtype=torch.int32, device="cuda")
    out = torch.zeros(B, N, H, d, dtype=torch.bfloat16, device="cuda")
    score = torch.empty(B, N_sel, device="cuda")
    x_bits, q_bits, k_bits, v_bits = inp["x_cur"], inp["q"], inp["k"], inp["v"]
    host_out = torch.empty(B, N, H, d, dtype=torch.bfloat16).pin_memory()
    for t, theta in enumerate((1000, 400, 250)):
        if t > 0:
            x_bits = synth.drift_step(x_bits, 300 + t, 0.05, False)
            q_bits, k_bits, v_bits = (synth.drift_step(a, 400 + 10 * t + i, 0.05, True) for i, a in enumerate((q_bits, k_bits, v_bits)))
        k_keep = w.k_of(theta)
        M = k_keep + n_always
        host = [torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).pin_memory() for a in (x_bits, q_bits, k_bits, v_bits)]
        sess.step_host(host[0], host[1], host[2], host[3], host_out, k_keep)
        idx_sel = torch.empty(B, M, dtype=torch.int32, device="cuda")
        idx_rem = torch.empty(B, N_sel - k_keep, dtype=torch.int32, device="cuda")
        ws = A.new_workspace(A.OP_STEP, B, H, N, M, d)
        A.astraea_step(to_dev_bf16(x_bits), x_ref, lse, n_skip, to_dev_bf16(q_bits), to_dev_bf16(k_bits),
                       to_dev_bf16(v_bits), out, score, idx_sel, idx_rem, B, H, N, N_sel, d, k_keep, workspace=ws)
        A.astraea_poll_error(ws)
        assert torch.equal(host_out.view(torch.int16), out.cpu().view(torch.int16)), "step %d" % t
        if t == 0:
            want_o, _, _ = oracle.sparse_attn(f64(q_bits), f64(k_bits), f64(v_bits), q_idx=None, scale=0.0)
            err = np.abs(bf16_dev_to_f64(out) - want_o)
            assert err.max() < ATTN_MAX_ABS and err.mean() < ATTN_MEAN_ABS
    sess.close()


# ------------------------------------------------------------- linear layers on the selected rows
LINEAR_MAX_ABS = 2e-2        # one bf16 rounding of outputs of magnitude <= ~5 (2^-8 relative) on top of fp32 sums
LINEAR_MEAN_ABS = 2e-3


def _linear_case(oracle, B, N, K, N_out, M, seed, bias=True, compact=False, dense=False):
    rng = np.random.default_rng(seed)
    x = synth.f32_to_bf16_bits(rng.standard_normal((B, N, K)).astype(np.float32))
    w = synth.f32_to_bf16_bits((rng.standard_normal((N_out, K)) / math.sqrt(K)).astype(np.float32))
    bb = synth.f32_to_bf16_bits(rng.standard_normal(N_out).astype(np.float32)) if bias else None
    cache = synth.f32_to_bf16_bits(rng.standard_normal((B, N, N_out)).astype(np.float32))
    idx = None if dense else np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
    want = oracle.gathered_linear(f64(x), f64(w), None if bb is None else f64(bb), idx, f64(cache))
    g_y = (Guarded((B, M, N_out), torch.bfloat16, init=torch.zeros(B, M, N_out, dtype=torch.bfloat16, device="cuda")) if compact
           else Guarded((B, N, N_out), torch.bfloat16, init=to_dev_bf16(cache)))
    y = g_y.t
    ws = A.new_workspace(A.OP_GATHERED_LINEAR, 0, 0, 0, 0, 0)
    A.astraea_gathered_linear(to_dev_bf16(x), None if idx is None else dev(idx), M, to_dev_bf16(w),
                              None if bb is None else to_dev_bf16(bb), y, B, N, K, N_out,
                              flags=A.LINEAR_COMPACT_OUT if compact else 0, workspace=ws)
    A.astraea_poll_error(ws)
    g_y.check(("linear", B, N, K, N_out, M))
    got = bf16_dev_to_f64(y)
    if compact:
        want = np.take_along_axis(want, idx[:, :, None].astype(np.int64), 1)
    elif idx is not None:
        mask = np.ones((B, N), bool)
        for b in range(B):
            mask[b, idx[b]] = False
        assert np.array_equal(got[mask], f64(cache)[mask])          # rows that were not listed keep the cache, bit for bit
    err = np.abs(got - want)
    assert err.max() < LINEAR_MAX_ABS and err.mean() < LINEAR_MEAN_ABS, (err.max(), err.mean())


@pytest.mark.parametrize("N,K,N_out,M", [(300, 64, 256, 77), (1000, 192, 512, 333), (129, 128, 264, 129), (40, 64, 8, 1),
                                         (700, 320, 1160, 450)])
def test_gathered_linear_ragged_tiles(oracle, N, K, N_out, M):
    _linear_case(oracle, 2, N, K, N_out, M, seed=31)


def test_gathered_linear_all_rows_no_bias_compact_and_many_k_steps(oracle):
    _linear_case(oracle, 1, 260, 64, 256, 0, seed=32, dense=True)
    _linear_case(oracle, 2, 200, 128, 320, 90, seed=33, bias=False)
    _linear_case(oracle, 2, 200, 128, 320, 90, seed=34, compact=True)
    _linear_case(oracle, 1, 150, 64 * 23, 256, 100, seed=35)           # every pipeline stage several times over
    _linear_case(oracle, 1, 128 * 5 + 3, 64, 256 * 3, 128 * 5 + 3, seed=36)   # more tiles than fit one pass of two accumulators


def test_gathered_linear_bad_index_and_no_rows():
    B, N, K, N_out = 1, 64, 64, 64
    x = torch.ones(B, N, K, dtype=torch.bfloat16, device="cuda")
    w = torch.ones(N_out, K, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(B, N, N_out, dtype=torch.bfloat16, device="cuda")
    ws = A.new_workspace(A.OP_GATHERED_LINEAR, 0, 0, 0, 0, 0)
    A.astraea_gathered_linear(x, torch.empty(1, 0, dtype=torch.int32, device="cuda"), 0, w, None, y, B, N, K, N_out, workspace=ws)
    assert float(y.abs().sum()) == 0.0
    idx = torch.tensor([[1, 64, 2 ** 30]], dtype=torch.int32, device="cuda")
    A.astraea_gathered_linear(x, idx, 3, w, None, y, B, N, K, N_out, workspace=ws)
    with pytest.raises(A.AstraeaError) as e:
        A.astraea_poll_error(ws)
    assert e.value.code == A.ERR_BAD_INDEX
    assert float(y[0, 1, 0]) == 64.0 and float(y[0, 2:].abs().sum()) == 0.0
    # duplicates and descending entries: reported, and no row is written twice
    y.zero_()
    idx = torch.tensor([[1, 5, 5, 3, 9]], dtype=torch.int32, device="cuda")
    A.astraea_gathered_linear(x, idx, 5, w, None, y, B, N, K, N_out, workspace=ws)
    with pytest.raises(A.AstraeaError) as e:
        A.astraea_poll_error(ws)
    assert e.value.code == A.ERR_BAD_INDEX
    rows_written = (y[0, :, 0] != 0).nonzero().flatten().tolist()
    assert rows_written == [1, 5, 9]


# ------------------------------------------------------------- a schedule of steps as one CUDA graph
def test_schedule_graph_equals_step_by_step(oracle):
    """Four steps with budgets (all, 40 %, none, 25 %) recorded as one graph against the same four astraea_step calls:
    every piece of state ends bit-identical; and every prefix of the schedule, replayed as a graph of its own,
    against the oracle."""
    w = synth.Workload("mini-schedule", B=2, H=4, d=64, N_v=600, N_t=0)
    inp = synth.make_step_inputs(w, 17)
    B, N, H, d, N_sel = w.B, w.N, w.H, w.d, w.N_v
    budgets = [N_sel, w.k_of(400), 0, w.k_of(250)]
    xs, qs, ks, vs = [inp["x_cur"]], [inp["q"]], [inp["k"]], [inp["v"]]
    for t in range(1, len(budgets)):
        xs.append(synth.drift_step(xs[-1], 500 + t, 0.05, False))
        qs.append(synth.drift_step(qs[-1], 510 + t, 0.05, True))
        ks.append(synth.drift_step(ks[-1], 520 + t, 0.05, True))
        vs.append(synth.drift_step(vs[-1], 530 + t, 0.05, True))
    dx, dq, dk, dv = ([to_dev_bf16(a) for a in lst] for lst in (xs, qs, ks, vs))

    def fresh_state():
        return dict(x_ref=to_dev_bf16(inp["x_cur"]), lse=torch.zeros(B, H, N, device="cuda"),
                    n_skip=torch.zeros(B, N_sel, dtype=torch.int32, device="cuda"),
                    out=torch.zeros(B, N, H, d, dtype=torch.bfloat16, device="cuda"),
                    score=torch.empty(B, N_sel, device="cuda"),
                    idx_sel=torch.zeros(B, N, dtype=torch.int32, device="cuda"),
                    idx_rem=torch.zeros(B, N_sel, dtype=torch.int32, device="cuda"),
                    ws=A.new_workspace(A.OP_STEP, B, H, N, N, d))

    b0 = fresh_state()
    a, b = fresh_state(), fresh_state()
    for t, kk in enumerate(budgets):
        A.astraea_step(dx[t], a["x_ref"], a["lse"], a["n_skip"], dq[t], dk[t], dv[t], a["out"], a["score"], a["idx_sel"],
                       a["idx_rem"], B, H, N, N_sel, d, kk, workspace=a["ws"])
    A.astraea_poll_error(a["ws"])
    sched = A.Schedule(budgets, dx, dq, dk, dv, b["x_ref"], b["lse"], b["n_skip"], b["out"], b["score"], b["idx_sel"],
                       b["idx_rem"], B, H, N, N_sel, d, workspace=b["ws"])
    sched.launch()
    A.astraea_poll_error(b["ws"])
    for name in ("x_ref", "lse", "n_skip", "out", "score"):
        ta, tb = a[name], b[name]
        assert torch.equal(ta.view(torch.int16) if ta.dtype == torch.bfloat16 else ta,
                           tb.view(torch.int16) if tb.dtype == torch.bfloat16 else tb), name
    assert int((b["n_skip"] > 0).sum()) > 0 and float(b["out"].float().abs().sum()) > 0
    # Against the oracle: the graph of the first t+1 steps, replayed from a fresh state, leaves the state that
    # oracle.step produces from the state the graph of the first t steps left (teacher forcing, graph to graph).
    prev = device_state(b0["x_ref"], b0["lse"], b0["n_skip"], b0["out"])
    for t in range(len(budgets)):
        c = fresh_state()
        sc = A.Schedule(budgets[:t + 1], dx[:t + 1], dq[:t + 1], dk[:t + 1], dv[:t + 1], c["x_ref"], c["lse"], c["n_skip"],
                        c["out"], c["score"], c["idx_sel"], c["idx_rem"], B, H, N, N_sel, d, workspace=c["ws"])
        sc.launch()
        A.astraea_poll_error(c["ws"])
        prev, _ = check_step_against_oracle(oracle, prev, xs[t], qs[t], ks[t], vs[t], budgets[t], 0, c["score"], c["idx_sel"],
                                            c["idx_rem"], c["x_ref"], c["lse"], c["n_skip"], c["out"], what=("graph prefix", t))
        sc.close()
    sched.close()
    with pytest.raises(A.AstraeaError) as e:
        A.Schedule([N_sel + 1], dx[:1], dq[:1], dk[:1], dv[:1], b["x_ref"], b["lse"], b["n_skip"], b["out"], b["score"],
                   b["idx_sel"], b["idx_rem"], B, H, N, N_sel, d, workspace=b["ws"])
    assert e.value.code == A.ERR_INVALID_ARG


def test_gathered_linear_mlp_on_selected_rows_hidden_state_stays_compact(oracle):
    """The MLP of a block: GELU(x[idx] W1^T + b1) into a compact [B, M, 4K] buffer, then W2 on the compact rows with
    the result scattered over the cached output.  Both layers against the oracle (the second one fed with the
    device's bf16 hidden state, so that each layer is checked on its own)."""
    rng = np.random.default_rng(41)
    B, N, K, M = 2, 300, 128, 170
    Hd = 4 * K
    x = synth.f32_to_bf16_bits(rng.standard_normal((B, N, K)).astype(np.float32))
    w1 = synth.f32_to_bf16_bits((rng.standard_normal((Hd, K)) / math.sqrt(K)).astype(np.float32))
    b1 = synth.f32_to_bf16_bits(rng.standard_normal(Hd).astype(np.float32))
    w2 = synth.f32_to_bf16_bits((rng.standard_normal((K, Hd)) / math.sqrt(Hd)).astype(np.float32))
    b2 = synth.f32_to_bf16_bits(rng.standard_normal(K).astype(np.float32))
    cache = synth.f32_to_bf16_bits(rng.standard_normal((B, N, K)).astype(np.float32))
    idx = np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
    ws = A.new_workspace(A.OP_GATHERED_LINEAR, 0, 0, 0, 0, 0)
    hid = torch.zeros(B, M, Hd, dtype=torch.bfloat16, device="cuda")
    A.astraea_gathered_linear(to_dev_bf16(x), dev(idx), M, to_dev_bf16(w1), to_dev_bf16(b1), hid, B, N, K, Hd,
                              flags=A.LINEAR_COMPACT_OUT | A.LINEAR_GELU, workspace=ws)
    want_hid = np.take_along_axis(oracle.gathered_linear(f64(x), f64(w1), f64(b1), idx, gelu=True),
                                  idx[:, :, None].astype(np.int64), 1)
    got_hid = bf16_dev_to_f64(hid)
    err = np.abs(got_hid - want_hid)
    assert err.max() < LINEAR_MAX_ABS and err.mean() < LINEAR_MEAN_ABS, (err.max(), err.mean())
    y = to_dev_bf16(cache)
    A.astraea_gathered_linear(hid, dev(idx), M, to_dev_bf16(w2), to_dev_bf16(b2), y, B, N, Hd, K,
                              flags=A.LINEAR_COMPACT_IN, workspace=ws)
    A.astraea_poll_error(ws)
    want = oracle.gathered_linear(got_hid, f64(w2), f64(b2), idx, f64(cache), compact_in=True)
    got = bf16_dev_to_f64(y)
    err = np.abs(got - want)
    assert err.max() < LINEAR_MAX_ABS and err.mean() < LINEAR_MEAN_ABS, (err.max(), err.mean())
    mask = np.ones((B, N), bool)
    for b in range(B):
        mask[b, idx[b]] = False
    assert np.array_equal(got[mask], f64(cache)[mask])


# ------------------------------------------------------------- cross-attention of the selected rows
@pytest.mark.parametrize("d,N_kv", [(64, 226), (72, 77), (128, 300), (64, 1)])
def test_cross_attention_of_selected_rows(oracle, d, N_kv):
    rng = np.random.default_rng(50 + d)
    B, H, N, M = 2, 3, 500, 333
    q, cache = (synth.f32_to_bf16_bits(rng.standard_normal((B, N, H, d)).astype(np.float32)) for _ in range(2))
    k, v = (synth.f32_to_bf16_bits(rng.standard_normal((B, N_kv, H, d)).astype(np.float32)) for _ in range(2))
    idx = np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
    want_o, want_lse, _ = oracle.sparse_attn(f64(q), f64(k), f64(v), q_idx=idx)
    out = to_dev_bf16(cache)
    lse = torch.zeros(B, H, N, device="cuda")
    ws = A.new_workspace(A.OP_SPARSE_ATTN, B, H, N, M, d)
    A.astraea_sparse_cross_attn(to_dev_bf16(q), to_dev_bf16(k), to_dev_bf16(v), A.bhnd_strides(N, H, d),
                                A.bhnd_strides(N_kv, H, d), A.bhnd_strides(N_kv, H, d), dev(idx), M, out, lse,
                                B, H, N, N_kv, d, workspace=ws)
    A.astraea_poll_error(ws)
    got = bf16_dev_to_f64(out)
    got_rows = np.take_along_axis(got, idx[:, :, None, None].astype(np.int64), 1)
    assert_attn_close(got_rows, want_o, ATTN_MAX_ABS, ATTN_MEAN_ABS)
    got_lse = np.take_along_axis(lse.cpu().numpy().astype(np.float64), idx[:, None, :].astype(np.int64), 2)
    assert np.abs(got_lse - want_lse).max() < LSE_ABS
    mask = np.ones((B, N), bool)
    for b in range(B):
        mask[b, idx[b]] = False
    assert np.array_equal(got[mask], f64(cache)[mask])
