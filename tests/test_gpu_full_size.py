"""Parity at the full sizes of the workloads, in the launch configuration bench.py times (the four calls of a
step on one stream): scores and selection against the oracle at full size; attention on sampled selected rows
(each output row depends only on its own query and all keys/values, so a sampled row is an exact check), the
sample stratified over the CTAs of a head (first / last row of the first, a middle and the last CTA) and, on the
CogVideoX shape, over every head.  The output and LSE caches start as a NaN bit pattern that the attention cannot
produce: afterwards NO element of a selected row of ANY head may still hold it and EVERY unselected row must."""
import math

import numpy as np
import pytest
import torch

from paper_2506_05096_b200 import binding as A
from paper_2506_05096_b200 import synth
from helpers import assert_attn_close, bf16_dev_to_f64, dev, f64, to_dev_bf16

pytestmark = pytest.mark.gpu

SENTINEL_BF16 = 0x7FA5          # a quiet NaN with a payload, as int16 bits
SENTINEL_F32 = 0x7FC0A5A5


def stratified_rows(rng, sel_row, rows, cta_rows=256):
    """Token ids of selected rows: first and last row of the first, a middle and the last CTA of a head (CTAs
    take 256 consecutive entries of the index list, or 128 in the small shape), plus random ones up to `rows`."""
    M = len(sel_row)
    ranks = set()
    n_cta = (M + cta_rows - 1) // cta_rows
    for c in sorted({0, n_cta // 2, n_cta - 1}):
        lo, hi = c * cta_rows, min(M, (c + 1) * cta_rows) - 1
        ranks.update({lo, min(lo + 127, hi), min(lo + 128, hi), hi})
    extra = rng.choice(M, min(M, max(rows, len(ranks))), replace=False)
    for r in extra:
        if len(ranks) >= min(M, max(rows, len(ranks))):
            break
        ranks.add(int(r))
    return np.sort(sel_row[np.array(sorted(ranks))]).astype(np.int32)


def assert_written_exactly(out, lse, idx_sel, M):
    """On the device, by bit pattern: every element of every selected row of every head was written (attention
    of finite inputs cannot produce the sentinel NaN), every other row still holds the sentinel."""
    B, N = out.shape[:2]
    sel = torch.zeros(B, N, dtype=torch.bool, device="cuda")
    for b in range(B):
        sel[b, idx_sel[b, :M].long()] = True
    ob = out.view(torch.int16).reshape(B, N, -1)
    assert bool((ob[sel] != SENTINEL_BF16).all()), "a selected row still holds the sentinel"
    assert bool((ob[~sel] == SENTINEL_BF16).all()), "an unselected row was written"
    lb = lse.view(torch.int32).transpose(1, 2)              # [B, N, H]
    assert bool((lb[sel] != SENTINEL_F32).all()) and bool((lb[~sel] == SENTINEL_F32).all())
    assert bool(torch.isfinite(out.float().reshape(B, N, -1)[sel]).all()) and bool(torch.isfinite(lse.transpose(1, 2)[sel]).all())
    return sel


def _full_size_case(oracle, name, theta, rows=48, score_rows=4096, seed=0, all_heads=False):
    w = synth.WORKLOADS[name]
    inp = synth.make_step_inputs(w, seed, parts=("x_ref", "x_cur", "q", "k", "v"))
    B, N, H, d, D, N_sel, n_always = w.B, w.N, w.H, w.d, w.D, w.N_v, w.N_t
    k_keep = w.k_of(theta)
    M = k_keep + n_always
    lse0 = (inp["lse"] - np.float32(math.log(N))).astype(np.float32)
    x_cur, x_ref = to_dev_bf16(inp["x_cur"]), to_dev_bf16(inp["x_ref"])
    q, k, v = (to_dev_bf16(inp[n]) for n in ("q", "k", "v"))
    lse_in, n_skip = dev(lse0), dev(inp["n_skip"])
    out = torch.full((B, N, H, d), SENTINEL_BF16, dtype=torch.int16, device="cuda").view(torch.bfloat16)
    lse = torch.full((B, H, N), SENTINEL_F32, dtype=torch.int32, device="cuda").view(torch.float32)
    score = torch.empty(B, N_sel, device="cuda")
    idx_sel = torch.empty(B, M, dtype=torch.int32, device="cuda")
    idx_rem = torch.empty(B, N_sel - k_keep, dtype=torch.int32, device="cuda")
    ws = A.new_workspace(A.OP_STEP, B, H, N, M, d)
    ws_sel = A.new_workspace(A.OP_SELECT, B, 0, N_sel, k_keep, 0)
    s = A.bhnd_strides(N, H, d)
    A.astraea_score(x_cur, x_ref, lse_in, n_skip, score, B, N, N_sel, D, H, 1.0, 1.0)
    A.astraea_select(score, B, N_sel, k_keep, n_always, idx_sel, idx_rem, n_skip, ws_sel)
    A.astraea_sparse_attn(q, k, v, s, s, s, idx_sel, M, out, lse, B, H, N, d, workspace=ws)
    A.astraea_scatter_reuse(x_ref, x_cur, idx_sel, B, N, M, D, A.SCATTER_SRC_FULL)
    A.astraea_poll_error(ws)

    rng = np.random.default_rng(seed + 1)
    # scores: a sample of tokens against the oracle (rows are independent)
    got_score = score.cpu().numpy()
    pick = np.sort(rng.choice(N_sel, min(score_rows, N_sel), replace=False))
    full = np.concatenate([pick, np.arange(N_sel, N)])           # keep the [selectable | always] structure
    want = oracle.score(f64(inp["x_cur"][:, full]), f64(inp["x_ref"][:, full]), lse0[:, :, full],
                        inp["n_skip"][:, pick], n_sel=len(pick))
    rel = np.abs(got_score[:, pick].astype(np.float64) - want) / np.abs(want)
    assert rel.max() < 1e-5
    # selection: bit-exact on the scores the device produced
    want_sel, want_rem, want_n = oracle.select(got_score, k_keep, n_always, inp["n_skip"])
    got_sel = idx_sel.cpu().numpy()
    assert np.array_equal(got_sel, want_sel)
    assert np.array_equal(idx_rem.cpu().numpy(), want_rem)
    assert np.array_equal(n_skip.cpu().numpy(), want_n)
    # every selected row of every head was written, nothing else was (reuse: the rest keeps the cache bit for bit)
    sel_mask = assert_written_exactly(out, lse, idx_sel, M)
    # attention: stratified selected rows against the oracle, all keys
    heads = list(range(H)) if all_heads else sorted({0, H // 2, H - 1})
    picks = [stratified_rows(rng, got_sel[b], rows) for b in range(B)]
    r = min(len(p) for p in picks)
    rows_pick = np.stack([p[:r] for p in picks]).astype(np.int32)
    qh, kh, vh = (f64(np.ascontiguousarray(inp[n][:, :, heads])) for n in ("q", "k", "v"))
    want_o, want_l, _ = oracle.sparse_attn(qh, kh, vh, q_idx=rows_pick)
    del qh, kh, vh
    got_out = out[:, :, heads].float().cpu().numpy().astype(np.float64)
    got_rows = np.take_along_axis(got_out, rows_pick[:, :, None, None].astype(np.int64), 1)
    assert_attn_close(got_rows, want_o, what=(name, theta))
    got_l = np.take_along_axis(lse[:, heads].cpu().numpy().astype(np.float64), rows_pick[:, None, :].astype(np.int64), 2)
    assert np.abs(got_l - want_l).max() < 1e-3
    # x_ref refreshed only where selected
    x_ref0 = to_dev_bf16(inp["x_ref"])
    assert torch.equal(x_ref[~sel_mask], x_ref0[~sel_mask]) and torch.equal(x_ref[sel_mask], x_cur[sel_mask])


@pytest.mark.parametrize("theta", [500, 250])
def test_cogvideox_shaped_full_size(oracle, theta):
    _full_size_case(oracle, "cogvideox", theta, rows=24, all_heads=True)


def test_cogvideox_shaped_full_size_dense(oracle):
    _full_size_case(oracle, "cogvideox", 1000, rows=16, all_heads=True)


def test_opensora_shaped_full_size(oracle):
    _full_size_case(oracle, "opensora", 400)


def test_sweep_shaped_full_size(oracle):
    _full_size_case(oracle, "sweep", 300, rows=32)


def test_hunyuan_shaped_full_size(oracle):
    _full_size_case(oracle, "hunyuan", 600, rows=24, score_rows=2048)


def test_cogvideox_shaped_projection_and_cross_attention_full_size(oracle):
    """The layers next to the self-attention at the CogVideoX shape, keep-ratio 0.5: the query projection of the
    9001 selected rows (K = N_out = 3072) and their cross-attention against 226 keys; sampled rows against the oracle,
    all rows that were not listed bit-identical to what they held."""
    w = synth.WORKLOADS["cogvideox"]
    rng = np.random.default_rng(9)
    B, N, H, d, D = w.B, w.N, w.H, w.d, w.D
    M = w.k_of(500) + w.N_t
    idx = np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
    x = synth.f32_to_bf16_bits(rng.standard_normal((B, N, D)).astype(np.float32))
    wq = synth.f32_to_bf16_bits((rng.standard_normal((D, D)) / math.sqrt(D)).astype(np.float32))
    bq = synth.f32_to_bf16_bits(rng.standard_normal(D).astype(np.float32))
    cache = synth.f32_to_bf16_bits(rng.standard_normal((B, N, D)).astype(np.float32))
    y = to_dev_bf16(cache)
    ws = A.new_workspace(A.OP_GATHERED_LINEAR, 0, 0, 0, 0, 0)
    A.astraea_gathered_linear(to_dev_bf16(x), dev(idx), M, to_dev_bf16(wq), to_dev_bf16(bq), y, B, N, D, D, workspace=ws)
    A.astraea_poll_error(ws)
    pick = np.stack([np.sort(rng.choice(idx[b], 96, replace=False)) for b in range(B)]).astype(np.int32)
    want = oracle.gathered_linear(f64(x), f64(wq), f64(bq), pick)
    got = bf16_dev_to_f64(y)
    err = np.abs(np.take_along_axis(got, pick[:, :, None].astype(np.int64), 1) - np.take_along_axis(want, pick[:, :, None].astype(np.int64), 1))
    assert err.max() < 2e-2 and err.mean() < 2e-3, (err.max(), err.mean())
    unsel = np.ones((B, N), bool)
    for b in range(B):
        unsel[b, idx[b]] = False
    assert np.array_equal(got[unsel], f64(cache)[unsel])
    # cross-attention of the same rows (as heads of the projected queries) against N_kv = 226 other tokens
    N_kv = w.N_t
    kx, vx = (synth.f32_to_bf16_bits(rng.standard_normal((B, N_kv, H, d)).astype(np.float32)) for _ in range(2))
    q_bits = synth.f32_to_bf16_bits(got.astype(np.float32)).reshape(B, N, H, d)
    out = to_dev_bf16(cache.reshape(B, N, H, d))
    ws2 = A.new_workspace(A.OP_SPARSE_ATTN, B, H, N, M, d)
    A.astraea_sparse_cross_attn(to_dev_bf16(q_bits), to_dev_bf16(kx), to_dev_bf16(vx), A.bhnd_strides(N, H, d),
                                A.bhnd_strides(N_kv, H, d), A.bhnd_strides(N_kv, H, d), dev(idx), M, out, None,
                                B, H, N, N_kv, d, workspace=ws2)
    A.astraea_poll_error(ws2)
    heads = [0, H // 2, H - 1]
    want_o, _, _ = oracle.sparse_attn(f64(np.ascontiguousarray(q_bits[:, :, heads])), f64(np.ascontiguousarray(kx[:, :, heads])),
                                      f64(np.ascontiguousarray(vx[:, :, heads])), q_idx=pick)
    got_o = np.take_along_axis(bf16_dev_to_f64(out)[:, :, heads], pick[:, :, None, None].astype(np.int64), 1)
    assert_attn_close(got_o, want_o)
    assert np.array_equal(bf16_dev_to_f64(out)[unsel], f64(cache.reshape(B, N, H, d))[unsel])


def test_hunyuan_shaped_consecutive_steps_full_size(oracle):
    """Steps 0 and 1 of the drifting-latent workload at the full HunyuanVideo shape: step 0 computes every token and
    fills the output and LSE caches from real data; step 1 (keep-ratio 0.6) is checked with the oracle started from the
    device's state after step 0 (scores from the device's LSE cache, selection on the device's scores, sampled
    attention rows, reuse of step 0's outputs bit for bit, refresh of x_ref where selected)."""
    w = synth.WORKLOADS["hunyuan"]
    inp = synth.make_step_inputs(w, 3)
    B, N, H, d, D, N_sel = w.B, w.N, w.H, w.d, w.D, w.N_v
    rng = np.random.default_rng(4)
    x0, q0, k0, v0 = inp["x_cur"], inp["q"], inp["k"], inp["v"]
    x1 = synth.drift_step(x0, 901, 0.05, False)
    q1, k1, v1 = (synth.drift_step(a, 902 + i, 0.05, True) for i, a in enumerate((q0, k0, v0)))
    x_ref = to_dev_bf16(x0)                                   # no earlier step: the reference inputs are the first ones
    out = torch.zeros(B, N, H, d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(B, H, N, device="cuda")
    n_skip = torch.zeros(B, N_sel, dtype=torch.int32, device="cuda")
    score = torch.empty(B, N_sel, device="cuda")
    idx_sel = torch.empty(B, N, dtype=torch.int32, device="cuda")
    idx_rem = torch.empty(B, N_sel, dtype=torch.int32, device="cuda")
    ws = A.new_workspace(A.OP_STEP, B, H, N, N, d)
    w_alpha = 1.0 / N
    A.astraea_step(to_dev_bf16(x0), x_ref, lse, n_skip, to_dev_bf16(q0), to_dev_bf16(k0), to_dev_bf16(v0), out, score,
                   idx_sel, idx_rem, B, H, N, N_sel, d, N_sel, w_alpha=w_alpha, workspace=ws)
    A.astraea_poll_error(ws)
    out0, lse0 = out.clone(), lse.clone()
    # step 0, sampled: dense attention rows and their LSE
    heads = [0, H - 1]
    pick0 = np.sort(rng.choice(N, 16, replace=False)).astype(np.int32)[None]
    want_o, want_l, _ = oracle.sparse_attn(*(f64(np.ascontiguousarray(a[:, :, heads])) for a in (q0, k0, v0)), q_idx=pick0)
    got = np.take_along_axis(out0[:, :, heads].float().cpu().numpy().astype(np.float64), pick0[:, :, None, None].astype(np.int64), 1)
    assert_attn_close(got, want_o)
    assert np.abs(np.take_along_axis(lse0[:, heads].cpu().numpy().astype(np.float64), pick0[:, None, :].astype(np.int64), 2) - want_l).max() < 1e-3
    # step 1
    k_keep = w.k_of(600)
    A.astraea_step(to_dev_bf16(x1), x_ref, lse, n_skip, to_dev_bf16(q1), to_dev_bf16(k1), to_dev_bf16(v1), out, score,
                   idx_sel, idx_rem, B, H, N, N_sel, d, k_keep, w_alpha=w_alpha, workspace=ws)
    A.astraea_poll_error(ws)
    got_score = score.cpu().numpy()
    pick = np.sort(rng.choice(N_sel, 2048, replace=False))
    want_s = oracle.score(f64(x1[:, pick]), f64(x0[:, pick]), lse0.cpu().numpy()[:, :, pick], np.zeros((B, len(pick)), np.int32),
                          n_sel=len(pick), w_alpha=w_alpha)
    assert (np.abs(got_score[:, pick].astype(np.float64) - want_s) / np.abs(want_s)).max() < 1e-5
    want_sel, want_rem, want_n = oracle.select(got_score, k_keep, 0, np.zeros((B, N_sel), np.int32))
    got_sel = idx_sel.cpu().numpy()[:, :k_keep] if B == 1 else None
    assert np.array_equal(got_sel, want_sel)
    assert np.array_equal(n_skip.cpu().numpy(), want_n)
    rows = np.sort(rng.choice(want_sel[0], 16, replace=False)).astype(np.int32)[None]
    want_o, want_l, _ = oracle.sparse_attn(*(f64(np.ascontiguousarray(a[:, :, heads])) for a in (q1, k1, v1)), q_idx=rows)
    got = np.take_along_axis(out[:, :, heads].float().cpu().numpy().astype(np.float64), rows[:, :, None, None].astype(np.int64), 1)
    assert_attn_close(got, want_o)
    unsel = torch.ones(B, N, dtype=torch.bool, device="cuda")
    unsel[0, idx_sel[0, :k_keep].long()] = False
    assert torch.equal(out[unsel], out0[unsel]) and torch.equal(lse.transpose(1, 2)[unsel], lse0.transpose(1, 2)[unsel])
    x1d, x0d = to_dev_bf16(x1), to_dev_bf16(x0)
    assert torch.equal(x_ref[unsel], x0d[unsel]) and torch.equal(x_ref[~unsel], x1d[~unsel])


def test_hunyuan_shaped_fifty_consecutive_steps_full_size(oracle):
    """The 50-step drifting-latent workload at the full HunyuanVideo shape (118800 tokens, 24 heads of 128): a dense
    step 0 from empty caches, then 49 steps at keep-ratio 0.6 with the real LSE / x_ref / counter chain.  The latents
    drift on the device (seeded generator: inputs, not arithmetic of the method).  At steps 0, 1, 25 and 49 the step is
    checked with the oracle started from the device's state before it: sampled scores, the whole selection and the
    counters bit for bit on the device's scores, sampled attention rows, reuse and refresh bit for bit.  At the end the
    penalty term must have kept every token from being skipped for longer than its bound."""
    w = synth.WORKLOADS["hunyuan"]
    B, N, H, d, D, N_sel = w.B, w.N, w.H, w.d, w.D, w.N_v
    T, theta, checks = 50, 600, (0, 1, 25, 49)
    g = torch.Generator(device="cuda").manual_seed(11)
    rng = np.random.default_rng(12)

    def drift(t, sigma, preserve):
        inv = 1.0 / math.sqrt(1.0 + sigma * sigma) if preserve else 1.0
        flat = t.view(-1, D)
        for r0 in range(0, flat.shape[0], 16384):
            r1 = min(flat.shape[0], r0 + 16384)
            eps = torch.randn(r1 - r0, D, device="cuda", generator=g)
            flat[r0:r1] = ((flat[r0:r1].float() + sigma * eps) * inv).to(torch.bfloat16)

    x, q, k, v = (torch.randn(B, N, D, device="cuda", generator=g, dtype=torch.bfloat16) for _ in range(4))
    x_ref = x.clone()
    out = torch.zeros(B, N, H, d, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(B, H, N, device="cuda")
    n_skip = torch.zeros(B, N_sel, dtype=torch.int32, device="cuda")
    score = torch.empty(B, N_sel, device="cuda")
    idx_sel = torch.empty(B, N, dtype=torch.int32, device="cuda")
    idx_rem = torch.empty(B, N_sel, dtype=torch.int32, device="cuda")
    ws = A.new_workspace(A.OP_STEP, B, H, N, N, d)
    w_alpha = 1.0 / N
    heads = [0, H - 1]
    f = lambda t: t.float().cpu().numpy().astype(np.float64)
    max_sig = 0.0
    for t in range(T):
        if t > 0:
            drift(x, 0.05, False)
            for a in (q, k, v):
                drift(a, 0.05, True)
        k_keep = N_sel if t == 0 else w.k_of(theta)
        check = t in checks
        if check:
            x_ref0, out0, lse0, n0 = x_ref.clone(), out.clone(), lse.clone(), n_skip.clone()
        A.astraea_step(x, x_ref, lse, n_skip, q, k, v, out, score, idx_sel, idx_rem, B, H, N, N_sel, d, k_keep,
                       w_alpha=w_alpha, workspace=ws)
        if not check:
            continue
        A.astraea_poll_error(ws)
        # scores on sampled tokens, from the device's state before the step
        pick = np.sort(rng.choice(N_sel, 1024, replace=False))
        pk = torch.from_numpy(pick).cuda()
        want_s = oracle.score(f(x[:, pk]), f(x_ref0[:, pk]), f(lse0[:, :, pk]), n0[:, pk].cpu().numpy(), n_sel=len(pick), w_alpha=w_alpha)
        got_score = score.cpu().numpy()
        assert (np.abs(got_score[:, pick].astype(np.float64) - want_s) / np.abs(want_s)).max() < 1e-5, t
        n0_h = n0.cpu().numpy()
        max_sig = max(max_sig, float((got_score.astype(np.float64) - np.exp(np.minimum(n0_h, 80))).max()))
        # the whole selection and the counters, bit for bit on the device's scores
        want_sel, want_rem, want_n = oracle.select(got_score, k_keep, 0, n0_h)
        got_sel = idx_sel.cpu().numpy()[:, :k_keep]
        assert np.array_equal(got_sel, want_sel) and np.array_equal(n_skip.cpu().numpy(), want_n), t
        assert np.array_equal(idx_rem.cpu().numpy()[:, :N_sel - k_keep], want_rem), t
        # sampled attention rows (first and last rows of the first, a middle and the last CTA, and random ones)
        rows = stratified_rows(rng, got_sel[0], 16)[None]
        rw = torch.from_numpy(rows[0]).long().cuda()
        qh, kh, vh = (f(a.view(B, N, H, d)[:, :, heads]) for a in (q, k, v))
        want_o, want_l, _ = oracle.sparse_attn(qh, kh, vh, q_idx=rows)
        del qh, kh, vh
        assert_attn_close(f(out[:, rw][:, :, heads]), want_o, what=("step", t))
        assert np.abs(f(lse[:, heads][:, :, rw]) - want_l).max() < 1e-3, t
        # reuse and refresh, bit for bit, over the whole tensors
        sel = torch.zeros(B, N, dtype=torch.bool, device="cuda")
        sel[0, idx_sel[0, :k_keep].long()] = True
        assert torch.equal(out[~sel], out0[~sel]) and torch.equal(lse.transpose(1, 2)[~sel], lse0.transpose(1, 2)[~sel]), t
        assert torch.equal(x_ref[~sel], x_ref0[~sel]) and torch.equal(x_ref[sel], x[sel]), t
        if t > 0:
            assert not torch.equal(out[sel][:4096], out0[sel][:4096]), t              # the selected rows were recomputed
        del x_ref0, out0, lse0, n0
    A.astraea_poll_error(ws)
    # Penalty term (Section 3.2, S_penalty = e^n with w_beta = 1): at a keep-ratio of one half or more the tokens that
    # were skipped (at most 40 % of them) outrank every token that was just computed as soon as e^n exceeds the largest
    # significance term + 1, so no counter can pass that n
    bound = max(1, int(math.ceil(math.log(1.0 + max(max_sig, 0.0)))))
    assert int(n_skip.max().item()) <= bound, (int(n_skip.max().item()), bound, max_sig)
