"""Seeded random shapes, layouts and logit scales through every entry point, each case against the oracle.  The fixed
cases of test_gpu_parity.py pick the tile boundaries by hand; these walk over what lies between them."""
import math
import random

import numpy as np
import pytest
import torch

from paper_2506_05096_b200 import binding as A
from paper_2506_05096_b200 import synth
from helpers import assert_attn_close, bf16_dev_to_f64, dev, f64, to_dev_bf16

pytestmark = pytest.mark.gpu


def _bits(rng, *shape, scale=1.0):
    return synth.f32_to_bf16_bits((scale * rng.standard_normal(shape)).astype(np.float32))


@pytest.mark.parametrize("seed", range(6))
def test_random_attention_cases(oracle, seed):
    rnd = random.Random(1000 + seed)
    rng = np.random.default_rng(1000 + seed)
    for _ in range(8):
        d = rnd.choice([64, 72, 128])
        B, H = rnd.choice([1, 2]), rnd.choice([1, 2, 3])
        N = rnd.choice([1, 2, 63, 64, 65, 127, 128, 129, 191, 192, 193, 255, 257, 300, 640, 777, 1100, 2150])   # 1024+ keys: the launch may split them
        M = rnd.randint(1, N)
        mode = rnd.choice(["self", "self", "cross", "kv"])
        N_kv = rnd.choice([1, 5, 64, 100, 226, 300, 1300]) if mode == "cross" else N
        fl = A.ATTN_SMALL_CTAS if (d != 128 and rnd.random() < 0.4) else 0   # the other CTA shape of head_dim 64 / 72
        sig = rnd.choice([0.0, 0.0, 0.5, 1.0])                       # per-token lognormal norms: heavy-tailed logits
        amp = rnd.choice([1.0, 1.0, 2.0, 12.0])                      # 12: the speculation limit is passed, the CTAs redo
        sq, sk = np.exp(sig * rng.standard_normal((B, N, 1, 1))), np.exp(sig * rng.standard_normal((B, N_kv, 1, 1)))
        q = synth.f32_to_bf16_bits((amp * sq * rng.standard_normal((B, N, H, d))).astype(np.float32))
        k = synth.f32_to_bf16_bits((amp * sk * rng.standard_normal((B, N_kv, H, d))).astype(np.float32))
        v, cache = _bits(rng, B, N_kv, H, d), _bits(rng, B, N, H, d)
        idx = np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
        kv = None
        if mode == "kv":
            M_kv = rnd.randint(1, N)
            kv = np.stack([np.sort(rng.choice(N, M_kv, replace=False)) for _ in range(B)]).astype(np.int32)
        want_o, want_lse, _ = oracle.sparse_attn(f64(q), f64(k), f64(v), q_idx=idx, kv_idx=kv)
        out, lse = to_dev_bf16(cache), torch.zeros(B, H, N, device="cuda")
        sq_, sk_ = A.bhnd_strides(N, H, d), A.bhnd_strides(N_kv, H, d)
        if mode == "cross":
            ws = A.new_workspace(A.OP_SPARSE_ATTN, B, H, max(N, N_kv), M, d)     # room for a split over the N_kv keys
            A.astraea_sparse_cross_attn(to_dev_bf16(q), to_dev_bf16(k), to_dev_bf16(v), sq_, sk_, sk_, dev(idx), M, out, lse,
                                        B, H, N, N_kv, d, flags=fl, workspace=ws)
        elif mode == "kv":
            ws = A.new_workspace(A.OP_SPARSE_ATTN_KV, B, H, N, kv.shape[1], d)
            A.astraea_sparse_attn(to_dev_bf16(q), to_dev_bf16(k), to_dev_bf16(v), sq_, sq_, sq_, dev(idx), M, out, lse, B, H, N, d,
                                  flags=fl, workspace=ws, kv_idx=dev(kv), M_kv=kv.shape[1])
        else:
            ws = A.new_workspace(A.OP_SPARSE_ATTN, B, H, N, M, d)
            A.astraea_sparse_attn(to_dev_bf16(q), to_dev_bf16(k), to_dev_bf16(v), sq_, sq_, sq_, dev(idx), M, out, lse, B, H, N, d,
                                  flags=fl, workspace=ws)
        A.astraea_poll_error(ws)
        got = bf16_dev_to_f64(out)
        rows = np.take_along_axis(got, idx[:, :, None, None].astype(np.int64), 1)
        case = (d, B, H, N, M, mode, N_kv, sig, amp, fl)
        # one bf16 rounding of the output and of P: absolute for values of order one, relative beyond
        assert_attn_close(rows, want_o, what=case)
        got_lse = np.take_along_axis(lse.cpu().numpy().astype(np.float64), idx[:, None, :].astype(np.int64), 2)
        # head_dim 64 sums the bf16-rounded probabilities on the tensor core: 2^-8 relative at worst, where one key
        # dominates a row (sharpened or heavy-tailed logits only); everything else keeps the 1e-3 bound
        lse_tol = 5e-3 if (d == 64 and (amp > 1.0 or sig > 0.0)) else 1e-3
        assert (np.abs(got_lse - want_lse) / np.maximum(1.0, np.abs(want_lse))).max() < lse_tol, case
        mask = np.ones((B, N), bool)
        for b in range(B):
            mask[b, idx[b]] = False
        assert np.array_equal(got[mask], f64(cache)[mask]), case


@pytest.mark.parametrize("seed", range(3))
def test_random_linear_cases(oracle, seed):
    rnd = random.Random(2000 + seed)
    rng = np.random.default_rng(2000 + seed)
    for _ in range(8):
        B, N = rnd.choice([1, 2]), rnd.choice([1, 5, 127, 128, 129, 255, 256, 257, 400, 700])
        M = rnd.randint(1, N)
        K, N_out = 64 * rnd.choice([1, 2, 3, 7]), 8 * rnd.choice([1, 5, 31, 32, 33, 64, 70])
        gelu, compact, dense = rnd.random() < 0.3, rnd.random() < 0.3, rnd.random() < 0.2
        x, w, bias = _bits(rng, B, N, K), _bits(rng, N_out, K, scale=1 / math.sqrt(K)), _bits(rng, N_out)
        cache = _bits(rng, B, N, N_out)
        idx = None if dense else np.stack([np.sort(rng.choice(N, M, replace=False)) for _ in range(B)]).astype(np.int32)
        compact = compact and idx is not None
        want = oracle.gathered_linear(f64(x), f64(w), f64(bias), idx, f64(cache), gelu=gelu)
        y = torch.zeros(B, M, N_out, dtype=torch.bfloat16, device="cuda") if compact else to_dev_bf16(cache)
        ws = A.new_workspace(A.OP_GATHERED_LINEAR, 0, 0, 0, 0, 0)
        A.astraea_gathered_linear(to_dev_bf16(x), None if idx is None else dev(idx), M, to_dev_bf16(w), to_dev_bf16(bias), y,
                                  B, N, K, N_out, flags=(A.LINEAR_GELU if gelu else 0) | (A.LINEAR_COMPACT_OUT if compact else 0),
                                  workspace=ws)
        A.astraea_poll_error(ws)
        got = bf16_dev_to_f64(y)
        if compact:
            want = np.take_along_axis(want, idx[:, :, None].astype(np.int64), 1)
        err = np.abs(got - want) / np.maximum(1.0, np.abs(want))
        assert err.max() < 2e-2 and err.mean() < 2e-3, ((B, N, M, K, N_out, gelu, compact, dense), err.max(), err.mean())


@pytest.mark.parametrize("seed", range(3))
def test_random_select_cases(oracle, seed):
    rnd = random.Random(3000 + seed)
    rng = np.random.default_rng(3000 + seed)
    for _ in range(10):
        B = rnd.choice([1, 2, 3])
        N = rnd.choice([1, 2, 31, 33, 1000, 4096, 4097, 9000, 17550, 40000])
        k = rnd.choice([0, 1, N // 2, N - 1, N, rnd.randint(0, N)])
        n_always = rnd.choice([0, 0, 7])
        kind = rnd.choice(["float", "ints", "few", "special"])
        if kind == "float":
            s = rng.standard_normal((B, N)).astype(np.float32)
        elif kind == "ints":
            s = rng.integers(-50, 50, (B, N)).astype(np.float32)
        elif kind == "few":
            s = rng.integers(0, 3, (B, N)).astype(np.float32)
        else:
            s = rng.standard_normal((B, N)).astype(np.float32)
            m = rng.random((B, N))
            s[m < 0.05] = np.inf
            s[(m >= 0.05) & (m < 0.1)] = -0.0
            s[(m >= 0.1) & (m < 0.15)] = 0.0
            s[(m >= 0.15) & (m < 0.2)] = -np.inf
        n0 = rng.integers(0, 85, (B, N)).astype(np.int32)
        want_sel, want_rem, want_n = oracle.select(s, k, n_always, n0)
        sel = torch.full((B, k + n_always), -1, dtype=torch.int32, device="cuda")
        rem = torch.full((B, max(N - k, 1)), -1, dtype=torch.int32, device="cuda")
        ns = dev(n0)
        A.astraea_select(dev(s), B, N, k, n_always, sel, rem, ns, A.new_workspace(A.OP_SELECT, B, 0, N, k, 0))
        case = (B, N, k, n_always, kind)
        assert np.array_equal(sel.cpu().numpy(), want_sel), case
        assert np.array_equal(rem.cpu().numpy()[:, :N - k], want_rem), case
        assert np.array_equal(ns.cpu().numpy(), want_n), case
