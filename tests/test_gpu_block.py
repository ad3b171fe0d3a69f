"""A whole compute block with token-wise reuse (astraea_block_step) and its element-wise / residual pieces against the
CPU oracle.  Every layer is checked on its own with the tight per-layer tolerances, fed with the device's bf16 output
of the layer before (teacher forcing, so that one layer's rounding cannot hide another's error); the chain of single
calls must then equal astraea_block_step bit for bit; and the block as a whole is compared with the oracle's block."""
import math

import numpy as np
import pytest
import torch

from paper_2506_05096_b200 import binding as A
from paper_2506_05096_b200 import synth
from helpers import Guarded, assert_attn_close, bf16_dev_to_f64, dev, f64, to_dev_bf16

pytestmark = pytest.mark.gpu

# one bf16 rounding of values of magnitude up to ~8 on top of fp32 sums: 2^-8 relative, absolute below one
ROW_MAX, ROW_MEAN = 2e-2, 2e-3


def _bits(rng, *shape, scale=1.0):
    return synth.f32_to_bf16_bits((scale * rng.standard_normal(shape)).astype(np.float32))


def _close(got, want, what=""):
    err = np.abs(got - want) / np.maximum(1.0, np.abs(want))
    assert err.max() < ROW_MAX and err.mean() < ROW_MEAN, (what, err.max(), err.mean())


def _sorted_idx(rng, B, N, M):
    return np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)


# ------------------------------------------------------------------ layer norm + modulation
@pytest.mark.parametrize("D", [128, 1152, 3072, 4096, 72])
@pytest.mark.parametrize("mode", ["all", "full", "compact_out", "compact_in_out"])
def test_layernorm_modulate(oracle, D, mode):
    rng = np.random.default_rng(D)
    B, N, M = 2, 37, 11
    x = _bits(rng, B, N, D, scale=2.0)
    x = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(x) + np.float32(0.75))        # a mean that is not zero
    sc, sh = _bits(rng, B, D, scale=0.3), _bits(rng, B, D, scale=0.3)
    idx = None if mode == "all" else _sorted_idx(rng, B, N, M)
    cache = _bits(rng, B, N, D)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    want_rows = oracle.layernorm_modulate(f64(x) if idx is None else oracle.take_rows(f64(x), idx), f64(sc), f64(sh), 1e-6)
    if mode == "all":
        g = Guarded((B, N, D), torch.bfloat16, init=to_dev_bf16(cache))
        A.astraea_layernorm_modulate(to_dev_bf16(x), None, 0, to_dev_bf16(sc), to_dev_bf16(sh), g.t, B, N, D, workspace=ws)
        got = bf16_dev_to_f64(g.t)
    elif mode == "full":
        g = Guarded((B, N, D), torch.bfloat16, init=to_dev_bf16(cache))
        A.astraea_layernorm_modulate(to_dev_bf16(x), dev(idx), M, to_dev_bf16(sc), to_dev_bf16(sh), g.t, B, N, D, workspace=ws)
        full = bf16_dev_to_f64(g.t)
        got = oracle.take_rows(full, idx)
        mask = np.ones((B, N), bool)
        for b in range(B):
            mask[b, idx[b]] = False
        assert np.array_equal(full[mask], f64(cache)[mask])
    else:
        g = Guarded((B, M, D), torch.bfloat16, init=torch.zeros(B, M, D, dtype=torch.bfloat16, device="cuda"))
        src = to_dev_bf16(x) if mode == "compact_out" else to_dev_bf16(np.ascontiguousarray(np.take_along_axis(x, idx[:, :, None].astype(np.int64), 1)))
        A.astraea_layernorm_modulate(src, dev(idx), M, to_dev_bf16(sc), to_dev_bf16(sh), g.t, B, N, D,
                                     flags=A.LN_COMPACT_OUT | (A.LN_COMPACT_IN if mode == "compact_in_out" else 0), workspace=ws)
        got = bf16_dev_to_f64(g.t)
    g.check(("layernorm", D, mode))
    A.astraea_poll_error(ws)
    _close(got, want_rows, ("layernorm", D, mode))


def test_layernorm_plain_and_bad_index(oracle):
    rng = np.random.default_rng(5)
    B, N, D = 1, 20, 256
    x = _bits(rng, B, N, D, scale=3.0)
    y = torch.zeros(B, N, D, dtype=torch.bfloat16, device="cuda")
    A.astraea_layernorm_modulate(to_dev_bf16(x), None, 0, None, None, y, B, N, D, eps=1e-5)
    _close(bf16_dev_to_f64(y), oracle.layernorm_modulate(f64(x), eps=1e-5))
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    y.zero_()
    idx = torch.tensor([[1, 4, 4, 3, 9, 25]], dtype=torch.int32, device="cuda")
    A.astraea_layernorm_modulate(to_dev_bf16(x), idx, 6, None, None, y, B, N, D, workspace=ws)
    with pytest.raises(A.AstraeaError) as e:
        A.astraea_poll_error(ws)
    assert e.value.code == A.ERR_BAD_INDEX
    assert (y[0].float().abs().sum(-1) != 0).nonzero().flatten().tolist() == [1, 4, 9]
    with pytest.raises(A.AstraeaError) as e:
        A.astraea_layernorm_modulate(to_dev_bf16(x), None, 0, None, None, y, B, N, 8192)
    assert e.value.code == A.ERR_UNSUPPORTED


# ------------------------------------------------------------------ linear layer with a gated residual
@pytest.mark.parametrize("res_compact,out_compact,in_compact,gelu", [(False, False, False, False), (False, True, False, False),
                                                                     (True, True, True, False), (True, False, True, True)])
def test_gathered_linear_residual(oracle, res_compact, out_compact, in_compact, gelu):
    rng = np.random.default_rng(77)
    B, N, K, N_out, M = 2, 300, 192, 328, 131
    idx = _sorted_idx(rng, B, N, M)
    x_full = _bits(rng, B, N, K)
    x_in = np.ascontiguousarray(np.take_along_axis(x_full, idx[:, :, None].astype(np.int64), 1)) if in_compact else x_full
    w, bias, gate = _bits(rng, N_out, K, scale=1 / math.sqrt(K)), _bits(rng, N_out), _bits(rng, B, N_out)
    res_full = _bits(rng, B, N, N_out)
    res_in = np.ascontiguousarray(np.take_along_axis(res_full, idx[:, :, None].astype(np.int64), 1)) if res_compact else res_full
    cache = _bits(rng, B, N, N_out)
    lin = oracle.take_rows(oracle.gathered_linear(f64(x_full), f64(w), f64(bias), idx, gelu=gelu), idx)
    want = oracle.take_rows(f64(res_full), idx) + f64(gate)[:, None, :] * lin
    g = (Guarded((B, M, N_out), torch.bfloat16, init=torch.zeros(B, M, N_out, dtype=torch.bfloat16, device="cuda")) if out_compact
         else Guarded((B, N, N_out), torch.bfloat16, init=to_dev_bf16(cache)))
    ws = A.new_workspace(A.OP_GATHERED_LINEAR, 0, 0, 0, 0, 0)
    flags = ((A.LINEAR_COMPACT_RES if res_compact else 0) | (A.LINEAR_COMPACT_OUT if out_compact else 0) |
             (A.LINEAR_COMPACT_IN if in_compact else 0) | (A.LINEAR_GELU if gelu else 0))
    A.astraea_gathered_linear_residual(to_dev_bf16(x_in), dev(idx), M, to_dev_bf16(w), to_dev_bf16(bias), to_dev_bf16(res_in),
                                       to_dev_bf16(gate), g.t, B, N, K, N_out, flags=flags, workspace=ws)
    A.astraea_poll_error(ws)
    g.check("linear + residual")
    got = bf16_dev_to_f64(g.t)
    if not out_compact:
        mask = np.ones((B, N), bool)
        for b in range(B):
            mask[b, idx[b]] = False
        assert np.array_equal(got[mask], f64(cache)[mask])
        got = oracle.take_rows(got, idx)
    _close(got, want, "linear + residual")
    # no gate, no residual: the plain layer, bit for bit
    y1 = torch.zeros(B, M, N_out, dtype=torch.bfloat16, device="cuda")
    y2 = torch.zeros_like(y1)
    f2 = (A.LINEAR_COMPACT_IN if in_compact else 0) | A.LINEAR_COMPACT_OUT
    A.astraea_gathered_linear_residual(to_dev_bf16(x_in), dev(idx), M, to_dev_bf16(w), to_dev_bf16(bias), None, None, y1, B, N, K, N_out, flags=f2, workspace=ws)
    A.astraea_gathered_linear(to_dev_bf16(x_in), dev(idx), M, to_dev_bf16(w), to_dev_bf16(bias), y2, B, N, K, N_out, flags=f2, workspace=ws)
    assert torch.equal(y1.view(torch.int16), y2.view(torch.int16))


# ------------------------------------------------------------------ the whole block
def make_block(rng, B, H, d, hidden, N_text, modulated=True):
    D = H * d
    bits = {}
    for name, (o, i) in dict(wq=(D, D), wk=(D, D), wv=(D, D), wo=(D, D), wq2=(D, D), wo2=(D, D), w1=(hidden, D), w2=(D, hidden)).items():
        bits[name] = _bits(rng, o, i, scale=1 / math.sqrt(i))
        bits["b" + name[1:]] = _bits(rng, o, scale=0.1)
    if modulated:
        for name in ("s1", "t1", "g1", "s3", "t3", "g3"):
            bits[name] = _bits(rng, B, D, scale=0.3)
            if name[0] == "g":
                bits[name] = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(bits[name]) + np.float32(1.0))
    text_k, text_v = _bits(rng, B, N_text, H, d), _bits(rng, B, N_text, H, d)
    return bits, text_k, text_v


def device_chain(Wd, x, idx, M, tk, tv, N_text, y_cache, lse, B, H, N, d, hidden, eps=1e-6):
    """The layers of astraea_block_step as single calls on buffers of their own (nothing aliased), so that every
    intermediate can be read back.  Returns the dict of device tensors."""
    D = H * d
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device="cuda")
    ws = A.new_workspace(A.OP_GATHERED_LINEAR, 0, 0, 0, 0, 0)
    s, ts = A.bhnd_strides(N, H, d), A.bhnd_strides(N_text, H, d)
    t = dict(h=z(B, N, D), k=z(B, N, D), v=z(B, N, D), q=z(B, N, D), a=z(B, N, D), x1=z(B, M, D), h2=z(B, M, D), q2=z(B, N, D),
             c=z(B, M, D), x2=z(B, M, D), h3=z(B, M, D), u=z(B, M, hidden))
    g = Wd.get
    A.astraea_layernorm_modulate(x, None, 0, g("s1"), g("t1"), t["h"], B, N, D, eps, workspace=ws)
    A.astraea_gathered_linear(t["h"], None, 0, Wd["wk"], g("bk"), t["k"], B, N, D, D, workspace=ws)
    A.astraea_gathered_linear(t["h"], None, 0, Wd["wv"], g("bv"), t["v"], B, N, D, D, workspace=ws)
    A.astraea_gathered_linear(t["h"], idx, M, Wd["wq"], g("bq"), t["q"], B, N, D, D, workspace=ws)
    A.astraea_sparse_attn(t["q"], t["k"], t["v"], s, s, s, idx, M, t["a"], lse, B, H, N, d, workspace=ws)
    A.astraea_gathered_linear_residual(t["a"], idx, M, Wd["wo"], g("bo"), x, g("g1"), t["x1"], B, N, D, D, flags=A.LINEAR_COMPACT_OUT, workspace=ws)
    A.astraea_layernorm_modulate(t["x1"], idx, M, None, None, t["h2"], B, N, D, eps, flags=A.LN_COMPACT_IN | A.LN_COMPACT_OUT, workspace=ws)
    A.astraea_gathered_linear(t["h2"], idx, M, Wd["wq2"], g("bq2"), t["q2"], B, N, D, D, flags=A.LINEAR_COMPACT_IN, workspace=ws)
    A.astraea_sparse_cross_attn(t["q2"], tk, tv, s, ts, ts, idx, M, t["c"], None, B, H, N, N_text, d, flags=A.ATTN_COMPACT_OUT, workspace=ws)
    A.astraea_gathered_linear_residual(t["c"], idx, M, Wd["wo2"], g("bo2"), t["x1"], None, t["x2"], B, N, D, D,
                                       flags=A.LINEAR_COMPACT_IN | A.LINEAR_COMPACT_OUT | A.LINEAR_COMPACT_RES, workspace=ws)
    A.astraea_layernorm_modulate(t["x2"], idx, M, g("s3"), g("t3"), t["h3"], B, N, D, eps, flags=A.LN_COMPACT_IN | A.LN_COMPACT_OUT, workspace=ws)
    A.astraea_gathered_linear(t["h3"], idx, M, Wd["w1"], g("b1"), t["u"], B, N, D, hidden,
                              flags=A.LINEAR_COMPACT_IN | A.LINEAR_COMPACT_OUT | A.LINEAR_GELU, workspace=ws)
    A.astraea_gathered_linear_residual(t["u"], idx, M, Wd["w2"], g("b2"), t["x2"], g("g3"), y_cache, B, N, hidden, D,
                                       flags=A.LINEAR_COMPACT_IN | A.LINEAR_COMPACT_RES, workspace=ws)
    A.astraea_poll_error(ws)
    return t


def check_layers(oracle, bits, t, x_bits, idx, tk_bits, tv_bits, B, H, N, d, rows=None, heads=None):
    """Every layer of the chain against the oracle, each fed with the device's output of the layer before.
    rows: sampled positions in the index list (all if None); heads: sampled heads for the attention checks."""
    D = H * d
    Wf = {n: f64(a) for n, a in bits.items()}
    g = Wf.get
    M = idx.shape[1]
    pos = np.arange(M) if rows is None else np.asarray(rows)
    tok = np.stack([idx[b][pos] for b in range(B)]).astype(np.int32)           # the sampled tokens
    take = lambda full: oracle.take_rows(full, tok)
    cpu = {n: bf16_dev_to_f64(a) for n, a in t.items()}
    crow = lambda name: cpu[name][:, pos]                                       # sampled rows of a compact tensor
    hs = list(range(H)) if heads is None else list(heads)
    x = f64(x_bits)
    # h = LN(x)(1 + s1) + t1 on the sampled tokens; k, v, q from the DEVICE's h
    _close(take(cpu["h"]), oracle.layernorm_modulate(take(x), g("s1"), g("t1")), "h")
    h_rows = take(cpu["h"])
    for name in ("k", "v", "q"):
        _close(take(cpu[name]), oracle.gathered_linear(h_rows, Wf["w" + name], g("b" + name)), name)
    # self-attention rows from the DEVICE's q, k, v (sampled heads)
    dq, dk, dv = (bf16_dev_to_f64(t[n].view(B, N, H, d)[:, :, hs]) for n in ("q", "k", "v"))
    want_a, _, _ = oracle.sparse_attn(dq, dk, dv, q_idx=tok)
    assert_attn_close(take(cpu["a"]).reshape(B, len(pos), H, d)[:, :, hs], want_a, what="attention rows")
    del dq, dk, dv
    # x1 = x[I] + g1 * (a Wo^T + bo) from the DEVICE's a
    o = oracle.gathered_linear(take(cpu["a"]), Wf["wo"], g("bo"))
    o = o * g("g1")[:, None, :] if g("g1") is not None else o
    _close(crow("x1"), take(x) + o, "x1")
    _close(crow("h2"), oracle.layernorm_modulate(crow("x1")), "h2")
    _close(take(cpu["q2"]), oracle.gathered_linear(crow("h2"), Wf["wq2"], g("bq2")), "q2")
    want_c, _, _ = oracle.sparse_attn(take(cpu["q2"]).reshape(B, len(pos), H, d)[:, :, hs], f64(tk_bits)[:, :, hs], f64(tv_bits)[:, :, hs])
    assert_attn_close(crow("c").reshape(B, len(pos), H, d)[:, :, hs], want_c, what="cross-attention rows")
    _close(crow("x2"), crow("x1") + oracle.gathered_linear(crow("c"), Wf["wo2"], g("bo2")), "x2")
    _close(crow("h3"), oracle.layernorm_modulate(crow("x2"), g("s3"), g("t3")), "h3")
    _close(crow("u"), oracle.gathered_linear(crow("h3"), Wf["w1"], g("b1"), gelu=True), "u")
    m = oracle.gathered_linear(crow("u"), Wf["w2"], g("b2"))
    m = m * g("g3")[:, None, :] if g("g3") is not None else m
    return tok, crow("x2") + m


@pytest.mark.parametrize("modulated", [True, False])
def test_block_step_reduced_shape_layer_by_layer_and_as_a_whole(oracle, modulated):
    rng = np.random.default_rng(91)
    B, H, d, N_v, N_t, N_text, hidden = 2, 4, 64, 450, 26, 40, 1024
    N, D = N_v + N_t, H * d
    bits, tk_bits, tv_bits = make_block(rng, B, H, d, hidden, N_text, modulated)
    Wd = {n: to_dev_bf16(a) for n, a in bits.items()}
    tk, tv = to_dev_bf16(tk_bits), to_dev_bf16(tv_bits)
    x_ref_bits = _bits(rng, B, N, D)
    x_bits = synth.f32_to_bf16_bits(synth.bf16_bits_to_f32(x_ref_bits) + np.float32(0.1) * rng.standard_normal((B, N, D)).astype(np.float32))
    cache_bits = _bits(rng, B, N, D)
    lse0 = (0.3 * rng.standard_normal((B, H, N))).astype(np.float32)
    n0 = rng.integers(0, 3, (B, N_v)).astype(np.int32)
    k_keep = 180
    M = k_keep + N_t
    # the block in one call
    x = to_dev_bf16(x_bits)
    x_ref, lse, n_skip = to_dev_bf16(x_ref_bits), dev(lse0), dev(n0)
    g_y = Guarded((B, N, D), torch.bfloat16, init=to_dev_bf16(cache_bits))
    score = torch.empty(B, N_v, device="cuda")
    idx_sel = torch.empty(B, M, dtype=torch.int32, device="cuda")
    idx_rem = torch.empty(B, N_v - k_keep, dtype=torch.int32, device="cuda")
    ws = torch.zeros(A.astraea_block_workspace_bytes(B, H, N, d, hidden), dtype=torch.uint8, device="cuda")
    A.astraea_block_step(x, A.block_weights(Wd, hidden), x_ref, lse, n_skip, g_y.t, tk, tv, N_text, score, idx_sel, idx_rem,
                         B, H, N, N_v, d, k_keep, workspace=ws)
    A.astraea_poll_error(ws)
    g_y.check("block output cache")
    # score / selection / counters / reference refresh: as in astraea_step
    want_s = oracle.score(f64(x_bits), f64(x_ref_bits), lse0, n0, n_sel=N_v)
    assert (np.abs(score.cpu().numpy() - want_s) / np.abs(want_s)).max() < 1e-5
    want_sel, want_rem, want_n = oracle.select(score.cpu().numpy(), k_keep, N_t, n0)
    idx = idx_sel.cpu().numpy()
    assert np.array_equal(idx, want_sel) and np.array_equal(idx_rem.cpu().numpy(), want_rem) and np.array_equal(n_skip.cpu().numpy(), want_n)
    assert np.array_equal(bf16_dev_to_f64(x_ref), oracle.scatter_reuse(f64(x_ref_bits), oracle.take_rows(f64(x_bits), idx), idx))
    # the same layers as single calls: identical bits, and every layer against the oracle
    y2, lse2 = to_dev_bf16(cache_bits), dev(lse0)
    t = device_chain(Wd, x, idx_sel, M, tk, tv, N_text, y2, lse2, B, H, N, d, hidden)
    assert torch.equal(y2.view(torch.int16), g_y.t.view(torch.int16)) and torch.equal(lse2, lse)
    tok, want_y_rows = check_layers(oracle, bits, t, x_bits, idx, tk_bits, tv_bits, B, H, N, d)
    got_y = bf16_dev_to_f64(g_y.t)
    _close(oracle.take_rows(got_y, idx), want_y_rows, "y")
    mask = np.ones((B, N), bool)
    for b in range(B):
        mask[b, idx[b]] = False
    assert np.array_equal(got_y[mask], f64(cache_bits)[mask])                       # reuse: bit for bit
    assert np.array_equal(lse.cpu().numpy().transpose(0, 2, 1)[mask], lse0.transpose(0, 2, 1)[mask])
    # the block as a whole against the oracle's block (fp64 throughout, intermediates rounded to bf16 where the device
    # stores them): eight roundings of values of order 1-4 accumulate
    Wf = {n: f64(a) for n, a in bits.items()}
    rd = lambda a: synth.bf16_to_f64(synth.f32_to_bf16_bits(a.astype(np.float32)))
    res = oracle.block_step(f64(x_bits), f64(x_ref_bits), lse0.astype(np.float64), n0, f64(cache_bits), Wf, f64(tk_bits), f64(tv_bits), H,
                            k_keep, n_always=N_t, forced_sel=idx, rounder=rd)
    err = np.abs(got_y - res["y"]) / np.maximum(1.0, np.abs(res["y"]))
    assert err.max() < 6e-2 and err.mean() < 4e-3, (err.max(), err.mean())
    assert np.abs(lse.cpu().numpy() - res["lse"]).max() < 2e-2                      # the LSE follows bf16-rounded q and k
    # the pure fp64 block, no rounding anywhere: the end-to-end error of the bf16 pipeline
    pure = oracle.block_step(f64(x_bits), f64(x_ref_bits), lse0.astype(np.float64), n0, f64(cache_bits), Wf, f64(tk_bits), f64(tv_bits), H,
                             k_keep, n_always=N_t, forced_sel=idx)
    err = np.abs(got_y - pure["y"]) / np.maximum(1.0, np.abs(pure["y"]))
    assert err.max() < 1e-1 and err.mean() < 8e-3, (err.max(), err.mean())


def test_block_step_keep_ratio_zero_one_and_shared_selection(oracle):
    rng = np.random.default_rng(92)
    B, H, d, N, N_text, hidden = 1, 2, 64, 200, 9, 256
    D = H * d
    bits, tk_bits, tv_bits = make_block(rng, B, H, d, hidden, N_text)
    Wd = {n: to_dev_bf16(a) for n, a in bits.items()}
    W = A.block_weights(Wd, hidden)
    tk, tv = to_dev_bf16(tk_bits), to_dev_bf16(tv_bits)
    x_bits, x_ref_bits, cache_bits = _bits(rng, B, N, D), _bits(rng, B, N, D), _bits(rng, B, N, D)
    ws = torch.zeros(A.astraea_block_workspace_bytes(B, H, N, d, hidden), dtype=torch.uint8, device="cuda")
    score = torch.empty(B, N, device="cuda")
    idx_sel = torch.zeros(B, N, dtype=torch.int32, device="cuda")
    idx_rem = torch.zeros(B, N, dtype=torch.int32, device="cuda")

    def state():
        return to_dev_bf16(x_ref_bits), torch.zeros(B, H, N, device="cuda"), torch.zeros(B, N, dtype=torch.int32, device="cuda"), to_dev_bf16(cache_bits)

    # keep-ratio 0: only the counters move
    x_ref, lse, n_skip, y = state()
    A.astraea_block_step(to_dev_bf16(x_bits), W, x_ref, lse, n_skip, y, tk, tv, N_text, score, idx_sel, idx_rem, B, H, N, N, d, 0, workspace=ws)
    A.astraea_poll_error(ws)
    assert torch.equal(y, to_dev_bf16(cache_bits)) and torch.equal(x_ref, to_dev_bf16(x_ref_bits)) and float(lse.abs().sum()) == 0
    assert bool((n_skip == 1).all())
    # keep-ratio 1: the dense block (the oracle's, pinned against library modules on the CPU side)
    x_ref, lse, n_skip, y = state()
    A.astraea_block_step(to_dev_bf16(x_bits), W, x_ref, lse, n_skip, y, tk, tv, N_text, score, idx_sel, idx_rem, B, H, N, N, d, N, workspace=ws)
    A.astraea_poll_error(ws)
    Wf = {n: f64(a) for n, a in bits.items()}
    rd = lambda a: synth.bf16_to_f64(synth.f32_to_bf16_bits(a.astype(np.float32)))
    res = oracle.block_step(f64(x_bits), f64(x_ref_bits), np.zeros((B, H, N)), np.zeros((B, N), np.int32), f64(cache_bits), Wf,
                            f64(tk_bits), f64(tv_bits), H, N, rounder=rd)
    err = np.abs(bf16_dev_to_f64(y) - res["y"]) / np.maximum(1.0, np.abs(res["y"]))
    assert err.max() < 6e-2 and err.mean() < 4e-3, (err.max(), err.mean())
    assert torch.equal(x_ref, to_dev_bf16(x_bits)) and bool((n_skip == 0).all())
    # a selection made elsewhere and shared (the Fixed-token variant): no scoring, counters and x_ref untouched
    x_ref, lse, n_skip, y = state()
    sel = np.sort(rng.choice(N, 77, replace=False)).astype(np.int32)[None]
    idx_sel[:, :77] = dev(sel)
    score.fill_(-5.0)
    A.astraea_block_step(to_dev_bf16(x_bits), W, x_ref, lse, n_skip, y, tk, tv, N_text, score, idx_sel, idx_rem, B, H, N, N, d, 77,
                         flags=A.BLOCK_REUSE_SELECTION, workspace=ws)
    A.astraea_poll_error(ws)
    assert bool((score == -5.0).all()) and bool((n_skip == 0).all()) and torch.equal(x_ref, to_dev_bf16(x_ref_bits))
    res = oracle.block_step(f64(x_bits), f64(x_ref_bits), np.zeros((B, H, N)), np.zeros((B, N), np.int32), f64(cache_bits), Wf,
                            f64(tk_bits), f64(tv_bits), H, 77, forced_sel=sel, rounder=rd)
    err = np.abs(bf16_dev_to_f64(y) - res["y"]) / np.maximum(1.0, np.abs(res["y"]))
    assert err.max() < 6e-2 and err.mean() < 4e-3, (err.max(), err.mean())
    mask = np.ones(N, bool)
    mask[sel[0]] = False
    assert np.array_equal(bf16_dev_to_f64(y)[0, mask], f64(cache_bits)[0, mask])


def test_block_step_cogvideox_shape_sampled_rows_layer_by_layer(oracle):
    """The block at the full CogVideoX shape (17776 tokens, 48 heads of 64, MLP width 12288, 226 text keys), keep-ratio
    0.5: astraea_block_step equals the chain of single calls bit for bit, and every layer of that chain is checked on
    sampled selected rows (and three heads for the two attentions) against the oracle."""
    w = synth.WORKLOADS["cogvideox"]
    rng = np.random.default_rng(93)
    B, H, d, N, N_v, N_t, hidden, N_text = w.B, w.H, w.d, w.N, w.N_v, w.N_t, 4 * w.D, 226
    D = H * d
    bits, tk_bits, tv_bits = make_block(rng, B, H, d, hidden, N_text)
    Wd = {n: to_dev_bf16(a) for n, a in bits.items()}
    tk, tv = to_dev_bf16(tk_bits), to_dev_bf16(tv_bits)
    x_ref_bits = _bits(rng, B, N, D)
    x_bits = synth.drift_step(x_ref_bits, 7, 0.05, False)
    x = to_dev_bf16(x_bits)
    x_ref, lse = to_dev_bf16(x_ref_bits), torch.zeros(B, H, N, device="cuda")
    n_skip = torch.zeros(B, N_v, dtype=torch.int32, device="cuda")
    sentinel = torch.full((B, N, D), 0x7FA5, dtype=torch.int16, device="cuda").view(torch.bfloat16)
    y = sentinel.clone()
    k_keep = w.k_of(500)
    M = k_keep + N_t
    score = torch.empty(B, N_v, device="cuda")
    idx_sel = torch.empty(B, M, dtype=torch.int32, device="cuda")
    ws = torch.zeros(A.astraea_block_workspace_bytes(B, H, N, d, hidden), dtype=torch.uint8, device="cuda")
    A.astraea_block_step(x, A.block_weights(Wd, hidden), x_ref, lse, n_skip, y, tk, tv, N_text, score, idx_sel, None,
                         B, H, N, N_v, d, k_keep, workspace=ws)
    A.astraea_poll_error(ws)
    del ws
    idx = idx_sel.cpu().numpy()
    want_sel, _, _ = oracle.select(score.cpu().numpy(), k_keep, N_t, None)
    assert np.array_equal(idx, want_sel)
    sel_mask = torch.zeros(B, N, dtype=torch.bool, device="cuda")
    sel_mask[0, idx_sel[0].long()] = True
    yb = y.view(torch.int16)
    assert bool((yb[sel_mask] != 0x7FA5).all()) and bool((yb[~sel_mask] == 0x7FA5).all())      # every selected row written, nothing else
    y2, lse2 = sentinel.clone(), torch.zeros(B, H, N, device="cuda")
    t = device_chain(Wd, x, idx_sel, M, tk, tv, N_text, y2, lse2, B, H, N, d, hidden)
    assert torch.equal(y2.view(torch.int16), yb) and torch.equal(lse2, lse)
    rows = np.unique(np.concatenate([[0, 127, 128, 255, 256, M // 2, M - 257, M - 256, M - 1], rng.choice(M, 23, replace=False)]))
    tok, want_y_rows = check_layers(oracle, bits, t, x_bits, idx, tk_bits, tv_bits, B, H, N, d, rows=rows, heads=[0, H // 2, H - 1])
    _close(oracle.take_rows(bf16_dev_to_f64(y), tok), want_y_rows, "y")


# ------------------------------------------------------------------ a generation of T steps x L blocks as one graph
@pytest.mark.parametrize("variant", [A.VARIANT_TOKEN_WISE, A.VARIANT_SELECT_QK, A.VARIANT_TIMESTEP, A.VARIANT_FIXED_TOKEN])
def test_model_schedule_two_blocks_six_steps_against_the_oracle(oracle, variant):
    """The four rows of the ablation study (Table 2) as scheduled runs of 2 blocks x 6 steps.  The graph of the first
    t+1 steps, replayed from fresh state, must leave in every block the state that the oracle's block produces from the
    state the graph of the first t steps left (teacher forcing from graph to graph, block by block: block 1 is fed the
    device's output of block 0 of the same step)."""
    rng = np.random.default_rng(200 + variant)
    B, H, d, N_v, N_t, N_text, hidden, L, T = 1, 2, 64, 300, 12, 20, 256, 2, 6
    N, D = N_v + N_t, H * d
    budgets = [N_v, N_v * 40 // 100, N_v * 25 // 100, 0, N_v * 60 // 100, N_v * 30 // 100]
    if variant == A.VARIANT_TIMESTEP:
        budgets = A.astraea_timestep_level_budgets([N_v, 120, 100, 90, 200, 130], N_v)
        assert budgets == oracle.timestep_level_budgets([N_v, 120, 100, 90, 200, 130], N_v) and 0 in budgets and budgets.count(N_v) >= 2
    blocks = [make_block(rng, B, H, d, hidden, N_text) for _ in range(L)]
    Wd = [({n: to_dev_bf16(a) for n, a in bits.items()}, hidden) for bits, _, _ in blocks]
    Wf = [{n: f64(a) for n, a in bits.items()} for bits, _, _ in blocks]
    tk, tv = [to_dev_bf16(b[1]) for b in blocks], [to_dev_bf16(b[2]) for b in blocks]
    tkf, tvf = [f64(b[1]) for b in blocks], [f64(b[2]) for b in blocks]
    xs = [_bits(rng, B, N, D)]
    for t in range(1, T):
        xs.append(synth.drift_step(xs[-1], 700 + t, 0.1, False))
    dx = [to_dev_bf16(a) for a in xs]
    cache0 = [_bits(rng, B, N, D) for _ in range(L)]
    rd = lambda a: synth.bf16_to_f64(synth.f32_to_bf16_bits(a.astype(np.float32)))

    def fresh():
        return [dict(x_ref=to_dev_bf16(xs[0]), lse_cache=torch.zeros(B, H, N, device="cuda"),
                     n_skip=torch.zeros(B, N_v, dtype=torch.int32, device="cuda"), y_cache=to_dev_bf16(cache0[l]),
                     score=torch.zeros(B, N_v, device="cuda"), idx_sel=torch.zeros(B, N, dtype=torch.int32, device="cuda"),
                     idx_rem=torch.zeros(B, N_v, dtype=torch.int32, device="cuda")) for l in range(L)]

    def host(states):
        return [dict(x_ref=bf16_dev_to_f64(s["x_ref"]), lse=s["lse_cache"].cpu().numpy().astype(np.float64),
                     n_skip=s["n_skip"].cpu().numpy().copy(), y=bf16_dev_to_f64(s["y_cache"]),
                     score=s["score"].cpu().numpy().astype(np.float64), idx_sel=s["idx_sel"].cpu().numpy().copy()) for s in states]

    ws = torch.zeros(A.astraea_block_workspace_bytes(B, H, N, d, hidden), dtype=torch.uint8, device="cuda")
    prev = host(fresh())
    for t in range(T):
        st = fresh()
        sched = A.ModelSchedule(budgets[:t + 1], dx[:t + 1], Wd, st, tk, tv, N_text, B, H, N, N_v, d, variant=variant, workspace=ws)
        sched.launch()
        A.astraea_poll_error(ws)
        sched.close()
        now = host(st)
        k_keep = budgets[t]
        M = k_keep + N_t
        x_in = f64(xs[t])
        shared = None
        for l in range(L):
            what = (variant, t, l)
            fixed_later = variant == A.VARIANT_FIXED_TOKEN and l > 0
            got_sel = (now[0] if fixed_later else now[l])["idx_sel"].reshape(-1)[:B * M].reshape(B, M)
            res = oracle.block_step(x_in, prev[l]["x_ref"], prev[l]["lse"], prev[l]["n_skip"], prev[l]["y"], Wf[l], tkf[l], tvf[l], H, k_keep,
                                    n_always=N_t, rounder=rd, select_qk=(variant == A.VARIANT_SELECT_QK), shared_sel=shared if fixed_later else None)
            if not fixed_later:
                rel = np.abs(now[l]["score"] - res["score"]) / np.abs(res["score"])
                assert rel.max() < 1e-5, what
                if not np.array_equal(got_sel, res["idx_sel"]):
                    # near-ties of the k-th score only; then the oracle adopts the device's (valid) selection
                    for b in range(B):
                        assert (np.diff(got_sel[b]) > 0).all() and np.array_equal(got_sel[b][k_keep:], np.arange(N_v, N)), what
                        kth = np.sort(res["score"][b])[::-1][k_keep - 1]
                        diff = np.setxor1d(got_sel[b], res["idx_sel"][b])
                        assert (np.abs(res["score"][b][diff] - kth) <= 1e-6 * abs(kth)).all(), what
                    res = oracle.block_step(x_in, prev[l]["x_ref"], prev[l]["lse"], prev[l]["n_skip"], prev[l]["y"], Wf[l], tkf[l], tvf[l], H,
                                            k_keep, n_always=N_t, rounder=rd, select_qk=(variant == A.VARIANT_SELECT_QK), forced_sel=got_sel)
                assert np.array_equal(now[l]["n_skip"], res["n_skip"]), what
            else:
                assert np.array_equal(now[l]["n_skip"], prev[l]["n_skip"]), what             # a later block of a Fixed-token step
            assert np.array_equal(now[l]["x_ref"], res["x_ref"]), what
            sel_mask = np.zeros((B, N), bool)
            for b in range(B):
                sel_mask[b, got_sel[b]] = True
            err = np.abs(now[l]["y"] - res["y"]) / np.maximum(1.0, np.abs(res["y"]))
            assert err.max() < 6e-2 and err.mean() < 4e-3, (what, err.max(), err.mean())
            assert np.array_equal(now[l]["y"][~sel_mask], prev[l]["y"][~sel_mask]), what     # reuse: bit for bit
            assert np.abs(now[l]["lse"] - res["lse"]).max() < 2e-2, what
            assert np.array_equal(now[l]["lse"].transpose(0, 2, 1)[~sel_mask], prev[l]["lse"].transpose(0, 2, 1)[~sel_mask]), what
            if M:
                assert np.abs(now[l]["y"][sel_mask] - prev[l]["y"][sel_mask]).max() > 1e-3, what    # the selected rows did change
            if variant == A.VARIANT_FIXED_TOKEN and l == 0:
                shared = got_sel
            x_in = now[l]["y"]                       # block l + 1 reads the device's merged output of block l
        prev = now
    # a Timestep-level schedule refuses partial budgets
    if variant == A.VARIANT_TIMESTEP:
        with pytest.raises(A.AstraeaError) as e:
            A.ModelSchedule([N_v, 7], dx[:2], Wd, fresh(), tk, tv, N_text, B, H, N, N_v, d, variant=variant, workspace=ws)
        assert e.value.code == A.ERR_INVALID_ARG
