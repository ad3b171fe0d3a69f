"""ctypes front end of the CPU oracle (astraea_oracle.c).

TEST INFRASTRUCTURE ONLY.  Importers: tests/, the smoke check and the CPU-baseline
leg of the benchmark.  The CUDA library and its Python binding never import this
module, and this module imports nothing from them.

All floating-point arrays are float64 numpy arrays; bf16 inputs are upcast
exactly by the caller before they get here.  `step()` chains the four stages in
the order of Algorithm 1.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "astraea_oracle.c")
_LIB = os.path.join(_HERE, "libastraea_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2 -fopenmp).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_select.restype = ctypes.c_int
        _lib.oracle_budget_to_k.restype = ctypes.c_int
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def _i32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.int32)


def num_threads() -> int:
    """Threads the OpenMP loops will use (OMP_NUM_THREADS or all cores)."""
    v = os.environ.get("OMP_NUM_THREADS")
    return int(v) if v else (os.cpu_count() or 1)


def budget_to_k(n_sel: int, theta_permille: int) -> int:
    return int(_load().oracle_budget_to_k(int(n_sel), int(theta_permille)))


def score(x_cur, x_ref, lse=None, n_skip=None, n_sel=None, H=1, w_alpha=1.0, w_beta=1.0,
          delta_mode=0, lse_mode=0):
    """S_token for tokens [0, n_sel) of every batch row; returns float64 [B, n_sel]."""
    x_cur, x_ref, lse, n_skip = _f64(x_cur), _f64(x_ref), _f64(lse), _i32(n_skip)
    B, N, D = x_cur.shape
    n_sel = N if n_sel is None else n_sel
    if lse is not None:
        H = lse.shape[1]
        assert lse.shape == (B, H, N)
    out = np.empty((B, n_sel), dtype=np.float64)
    _load().oracle_score(_p(x_cur), _p(x_ref), _p(lse), _p(n_skip), _p(out),
                         B, N, n_sel, D, H, ctypes.c_double(w_alpha), ctypes.c_double(w_beta),
                         int(delta_mode), int(lse_mode))
    return out


def score_partial(x_cur, x_ref, lse=None, n_sel=None, delta_mode=0, lse_mode=0):
    """The two sums behind the selection metric over a shard of the channels / heads (head-sharded multi-GPU form):
    (sum over the given channels of the difference term, sum over the given heads of exp(min(lse, 80)) or of lse).
    Plain numpy; float64 [2, B, n_sel]."""
    x_cur, x_ref = _f64(x_cur), _f64(x_ref)
    B, N, D = x_cur.shape
    n_sel = N if n_sel is None else n_sel
    diff = (x_cur - x_ref)[:, :n_sel]
    a = np.abs(diff).sum(-1) if delta_mode == 0 else (diff * diff).sum(-1) if delta_mode == 1 else diff.sum(-1)
    if lse is None:
        b = np.zeros((B, n_sel))
    else:
        l = _f64(lse)[:, :, :n_sel]
        b = np.exp(np.minimum(l, 80.0)).sum(1) if lse_mode == 0 else l.sum(1)
    return np.stack([a, b])


def score_combine(part, n_skip, D, H, has_lse=True, w_alpha=1.0, w_beta=1.0):
    """S_token from the partial sums added up over all shards: w_alpha (part[1]/H)(part[0]/D) + w_beta e^min(n, 80)."""
    part = _f64(part)
    n = np.zeros(part.shape[1:], dtype=np.int64) if n_skip is None else np.minimum(np.asarray(n_skip, dtype=np.int64), 80)
    s_lse = part[1] / H if has_lse else 1.0
    return w_alpha * s_lse * (part[0] / D) + w_beta * np.exp(n.astype(np.float64))


def select(score_f32, k, n_always=0, n_skip=None):
    """Top-k per batch row on float32 scores.  Returns (idx_sel, idx_rem, n_skip_new)."""
    s = np.ascontiguousarray(score_f32, dtype=np.float32)
    B, n_sel = s.shape
    idx_sel = np.empty((B, k + n_always), dtype=np.int32)
    idx_rem = np.empty((B, n_sel - k), dtype=np.int32)
    n_new = None if n_skip is None else np.array(n_skip, dtype=np.int32, copy=True, order="C")
    rc = _load().oracle_select(_p(s), B, n_sel, int(k), int(n_always), _p(idx_sel), _p(idx_rem), _p(n_new))
    if rc != 0:
        raise ValueError("oracle_select: bad k")
    return idx_sel, idx_rem, n_new


def sparse_attn(q, k, v, q_idx=None, kv_idx=None, scale=0.0, want_probs=False):
    """Attention rows for the listed queries against all keys (or kv_idx).

    q: [B, N, H, d]; k, v: [B, N_kv, H, d] (N_kv = N for self-attention; another length for the cross-attention
    of the listed rows against a second sequence).  Returns (o [B, M, H, d], lse [B, H, M], probs or None).
    """
    q, k, v = _f64(q), _f64(k), _f64(v)
    B, N, H, d = q.shape
    N_kv = k.shape[1]
    assert k.shape == v.shape == (B, N_kv, H, d)
    q_idx = _i32(q_idx)
    kv_idx = _i32(kv_idx)
    M = N if q_idx is None else q_idx.shape[1]
    M_kv = 0 if kv_idx is None else kv_idx.shape[1]
    Nk = N_kv if kv_idx is None else M_kv
    o = np.empty((B, M, H, d), dtype=np.float64)
    lse = np.empty((B, H, M), dtype=np.float64)
    probs = np.empty((B, H, M, Nk), dtype=np.float64) if want_probs else None
    _load().oracle_sparse_attn(_p(q), _p(k), _p(v), _p(q_idx), M, _p(kv_idx), M_kv,
                               _p(o), _p(lse), _p(probs), B, H, N, N_kv, d, ctypes.c_double(scale))
    return o, lse, probs


def scatter_reuse(cache, rows, idx):
    """Copy of `cache` [B, N, ...] with rows idx[b, r] replaced by rows[b, r]."""
    out = np.array(cache, dtype=np.float64, copy=True, order="C")
    rows = _f64(rows)
    idx = _i32(idx)
    B, N = out.shape[:2]
    R = int(np.prod(out.shape[2:]))
    M = idx.shape[1]
    if M:
        _load().oracle_scatter_reuse(_p(out), _p(rows), _p(idx), B, N, M, R)
    return out


def gathered_linear(x, w, bias=None, idx=None, y_cache=None, compact_in=False, gelu=False, N=None):
    """y = copy of y_cache [B, N, N_out] (zeros if None) with rows idx[b, r] (all rows if idx is None)
    replaced by act(x[b, i, :] @ w.T + bias); w is [N_out, K].  compact_in: x is [B, M, K], row r belongs to
    token idx[b, r] (pass N, the number of tokens, or y_cache).  gelu: act = exact GELU, else identity."""
    x, w = _f64(x), _f64(w)
    B, rows_x, K = x.shape
    if compact_in:
        assert idx is not None and (y_cache is not None or N is not None)
        N = N if y_cache is None else np.asarray(y_cache).shape[1]
    else:
        N = rows_x
    N_out = w.shape[0]
    assert w.shape == (N_out, K)
    y = np.zeros((B, N, N_out)) if y_cache is None else np.array(y_cache, dtype=np.float64, copy=True, order="C")
    assert y.shape == (B, N, N_out)
    bias = None if bias is None else _f64(bias)
    M = 0
    if idx is not None:
        idx = _i32(idx)
        M = idx.shape[1]
        if M == 0:
            return y
    assert not compact_in or x.shape[1] == M
    _load().oracle_gathered_linear(_p(x), _p(idx), M, _p(w), _p(bias), _p(y), B, N, K, N_out, int(compact_in), int(gelu))
    return y


def layernorm_modulate(x, scale=None, shift=None, eps=1e-6):
    """y = LayerNorm(x) * (1 + scale[b]) + shift[b] over the last axis (no learned affine); x: [B, R, D]."""
    x = _f64(x)
    B, R, D = x.shape
    y = np.empty_like(x)
    _load().oracle_layernorm_modulate(_p(x), _p(_f64(scale)), _p(_f64(shift)), _p(y), B, R, D, ctypes.c_double(eps))
    return y


def scatter_lse(lse_cache, lse_rows, idx):
    out = np.array(lse_cache, dtype=np.float64, copy=True, order="C")
    lse_rows, idx = _f64(lse_rows), _i32(idx)
    B, H, N = out.shape
    M = idx.shape[1]
    if M:
        _load().oracle_scatter_lse(_p(out), _p(lse_rows), _p(idx), B, H, N, M)
    return out


def step(x_cur, x_ref, lse_cache, n_skip, q, k, v, cache, k_keep, n_always=0,
         w_alpha=1.0, w_beta=1.0, delta_mode=0, lse_mode=0, scale=0.0, forced_sel=None):
    """One attention block at one denoising step (Algorithm 1), all in fp64.

    Returns a dict with score (fp64), score_f32, idx_sel, idx_rem, n_skip (new),
    out (new cache, [B,N,H,d]), lse (new lse cache, [B,H,N]), x_ref (refreshed at
    the selected tokens: the "last computed" reference).

    forced_sel [B, k_keep + n_always] (ascending; tests only): the rest of the step runs on this selection
    instead of the oracle's own (a chained test hands over a selection that differs from the oracle's only at
    exact near-ties of the k-th score, after having checked that); `own_idx_sel` then holds the oracle's.
    """
    B, N = x_cur.shape[:2]
    n_sel = N - n_always
    s64 = score(x_cur, x_ref, lse_cache, n_skip, n_sel=n_sel, w_alpha=w_alpha, w_beta=w_beta,
                delta_mode=delta_mode, lse_mode=lse_mode)
    s32 = s64.astype(np.float32)
    idx_sel, idx_rem, n_new = select(s32, k_keep, n_always, n_skip)
    own = idx_sel
    if forced_sel is not None:
        idx_sel = _i32(forced_sel)
        assert idx_sel.shape == own.shape
        chosen = np.zeros((B, N), dtype=bool)
        for b in range(B):
            chosen[b, idx_sel[b]] = True
        idx_rem = np.stack([np.flatnonzero(~chosen[b, :n_sel]) for b in range(B)]).astype(np.int32)
        if n_skip is not None:
            n_old = np.asarray(n_skip, dtype=np.int64)
            n_new = np.where(chosen[:, :n_sel], 0, np.minimum(n_old + 1, 80)).astype(np.int32)
    if idx_sel.shape[1]:
        o, l, _ = sparse_attn(q, k, v, q_idx=idx_sel, scale=scale)
        out = scatter_reuse(cache, o, idx_sel)
        lse_new = scatter_lse(lse_cache, l, idx_sel)
        xr = scatter_reuse(x_ref, np.take_along_axis(_f64(x_cur), idx_sel[:, :, None].astype(np.int64), axis=1), idx_sel)
    else:
        out = np.array(cache, dtype=np.float64, copy=True)
        lse_new = np.array(lse_cache, dtype=np.float64, copy=True)
        xr = np.array(x_ref, dtype=np.float64, copy=True)
    return dict(score=s64, score_f32=s32, idx_sel=idx_sel, idx_rem=idx_rem, n_skip=n_new,
                out=out, lse=lse_new, x_ref=xr, own_idx_sel=own)


def take_rows(a, idx):
    """Rows idx[b, r] of a [B, N, ...] array as [B, M, ...]."""
    a = np.asarray(a)
    ix = np.asarray(idx, dtype=np.int64).reshape(idx.shape + (1,) * (a.ndim - 2))
    return np.take_along_axis(a, ix, axis=1)


def block_step(x, x_ref, lse_cache, n_skip, y_cache, weights, text_k, text_v, H, k_keep, n_always=0,
               w_alpha=1.0, w_beta=1.0, delta_mode=0, lse_mode=0, eps=1e-6, forced_sel=None, rounder=None,
               select_qk=False, shared_sel=None):
    """One transformer block at one denoising step with token-wise reuse (Algorithm 1 and the execution flow of
    Section 3.2 applied to a whole compute block): the tokens are scored on the block's input and selected;
    keys and values come from ALL tokens of the current step; the query projection, the self-attention rows, the
    output projection, the cross-attention against the text keys / values and the MLP are evaluated for the selected
    tokens only; every other token keeps the block's cached output.  Pre-norm block with residuals:

        h  = LN(x) (1 + s1) + t1                      all tokens (keys / values need them)
        K, V = h Wk^T + bk, h Wv^T + bv               all tokens;   Q = h[sel] Wq^T + bq
        x1 = x[sel] + g1 * (Attn(Q, K, V) Wo^T + bo)
        x2 = x1 + Attn(LN(x1) Wq2^T + bq2, text_k, text_v) Wo2^T + bo2
        x3 = x2 + g3 * (GELU((LN(x2) (1 + s3) + t3) W1^T + b1) W2^T + b2)
        y_cache[sel] = x3;  lse_cache[:, sel] = LSE of the self-attention rows;  x_ref[sel] = x[sel]

    weights: dict of float64 arrays wq, bq, wk, bk, wv, bv, wo, bo, wq2, bq2, wo2, bo2, w1, b1, w2, b2 ([out, in] /
    [out]) and the modulation vectors s1, t1, g1, s3, t3, g3 ([B, D], any of them None).  text_k, text_v: [B, N_text, H, d].
    rounder: None, or a function applied to every intermediate tensor that the device stores as bf16 (the parity
    tests pass the bf16 rounding there, so that the oracle follows the device's storage precision layer by layer).
    select_qk: the SelectQ&K variant of the ablation study (Table 2): the self-attention's keys and values are
    restricted to the selected tokens as well.  shared_sel [B, M]: the Fixed-token variant: the selection was made by
    another block of this step; nothing is scored here, counters and reference inputs stay as they are.
    Returns a dict: idx_sel, idx_rem, n_skip, score, y (new cache), lse, x_ref, and the intermediates.
    """
    rd = (lambda a: a) if rounder is None else rounder
    x = _f64(x)
    B, N, D = x.shape
    d = D // H
    n_sel = N - n_always
    w = weights
    if shared_sel is not None:
        idx_sel = own = _i32(shared_sel)
        s64, idx_rem, forced_sel = None, None, None
        n_new = None if n_skip is None else np.array(n_skip, dtype=np.int32, copy=True)
    else:
        s64 = score(x, x_ref, lse_cache, n_skip, n_sel=n_sel, w_alpha=w_alpha, w_beta=w_beta, delta_mode=delta_mode, lse_mode=lse_mode)
        idx_sel, idx_rem, n_new = select(s64.astype(np.float32), k_keep, n_always, n_skip)
        own = idx_sel
    if forced_sel is not None:
        idx_sel = _i32(forced_sel)
        chosen = np.zeros((B, N), dtype=bool)
        for b in range(B):
            chosen[b, idx_sel[b]] = True
        idx_rem = np.stack([np.flatnonzero(~chosen[b, :n_sel]) for b in range(B)]).astype(np.int32)
        if n_skip is not None:
            n_new = np.where(chosen[:, :n_sel], 0, np.minimum(np.asarray(n_skip, dtype=np.int64) + 1, 80)).astype(np.int32)
    res = dict(score=s64, idx_sel=idx_sel, idx_rem=idx_rem, n_skip=n_new, own_idx_sel=own)
    M = idx_sel.shape[1]
    if M == 0:
        res.update(y=np.array(y_cache, dtype=np.float64, copy=True), lse=np.array(lse_cache, dtype=np.float64, copy=True),
                   x_ref=np.array(x_ref, dtype=np.float64, copy=True))
        return res
    h = rd(layernorm_modulate(x, w.get("s1"), w.get("t1"), eps))
    kv_rows = idx_sel if select_qk else None                                      # rows outside a list stay zero and are never read
    k = rd(gathered_linear(h, w["wk"], w.get("bk"), kv_rows))
    v = rd(gathered_linear(h, w["wv"], w.get("bv"), kv_rows))
    q = rd(gathered_linear(h, w["wq"], w.get("bq"), idx_sel))
    a, l, _ = sparse_attn(q.reshape(B, N, H, d), k.reshape(B, N, H, d), v.reshape(B, N, H, d), q_idx=idx_sel, kv_idx=kv_rows)
    a = rd(a.reshape(B, M, D))
    o = gathered_linear(a, w["wo"], w.get("bo"))
    if w.get("g1") is not None:
        o = o * _f64(w["g1"])[:, None, :]
    x1 = rd(take_rows(x, idx_sel) + o)
    h2 = rd(layernorm_modulate(x1, None, None, eps))
    q2 = rd(gathered_linear(h2, w["wq2"], w.get("bq2")))
    c, _, _ = sparse_attn(q2.reshape(B, M, H, d), text_k, text_v)
    c = rd(c.reshape(B, M, D))
    x2 = rd(x1 + gathered_linear(c, w["wo2"], w.get("bo2")))
    h3 = rd(layernorm_modulate(x2, w.get("s3"), w.get("t3"), eps))
    u = rd(gathered_linear(h3, w["w1"], w.get("b1"), gelu=True))
    m = gathered_linear(u, w["w2"], w.get("b2"))
    if w.get("g3") is not None:
        m = m * _f64(w["g3"])[:, None, :]
    x3 = rd(x2 + m)
    res.update(h=h, k=k, v=v, q_rows=take_rows(q, idx_sel), attn_rows=a, x1=x1, h2=h2, q2=q2, cross_rows=c, x2=x2, h3=h3, u=u, x3=x3,
               y=scatter_reuse(y_cache, x3, idx_sel), lse=scatter_lse(lse_cache, l, idx_sel),
               x_ref=(np.array(x_ref, dtype=np.float64, copy=True) if shared_sel is not None
                      else scatter_reuse(x_ref, take_rows(x, idx_sel), idx_sel)))
    return res


def timestep_level_budgets(k_keep, n_sel):
    """Host policy of the Timestep-level variant (ablation study, Table 2): every step computes all tokens or none.
    The token-wise budgets are accumulated; a step computes everything once the accumulated budget covers all n_sel
    tokens, and the first step always does."""
    out, carry = [], 0
    for t, k in enumerate(k_keep):
        carry += int(k)
        if t == 0 or (n_sel > 0 and carry >= n_sel):
            out.append(n_sel)
            carry = max(0, carry - n_sel)
        else:
            out.append(0)
    return out


VARIANT_TOKEN_WISE, VARIANT_SELECT_QK, VARIANT_TIMESTEP, VARIANT_FIXED_TOKEN = 0, 1, 2, 3


def model_step(x_in, blocks, states, text_k, text_v, H, k_keep, n_always=0, variant=0, forced_sels=None, rounder=None, **kw):
    """One denoising step through L compute blocks (execution flow of Section 3.2): block 0 reads x_in, block l > 0
    the merged output (computed + reused rows) of block l-1.  blocks: list of weight dicts; states: list of dicts
    with x_ref, lse, n_skip, y.  variant: the rows of the ablation study (Table 2): 0 token-wise (every block scores and
    selects), 1 SelectQ&K, 2 Timestep-level (k_keep must be 0 or all), 3 Fixed-token (block 0's selection is shared by
    the other blocks of the step).  forced_sels: per block, a selection to adopt (tests, near-ties).  Returns the list
    of per-block result dicts; `states` is not modified."""
    n_sel = np.asarray(x_in).shape[1] - n_always
    if variant == VARIANT_TIMESTEP:
        assert k_keep in (0, n_sel), "the Timestep-level variant computes all tokens or none"
    outs, x = [], x_in
    for l, (w, st) in enumerate(zip(blocks, states)):
        shared = outs[0]["idx_sel"] if (variant == VARIANT_FIXED_TOKEN and l > 0) else None
        forced = None if forced_sels is None else forced_sels[l]
        r = block_step(x, st["x_ref"], st["lse"], st["n_skip"], st["y"], w, text_k[l], text_v[l], H, k_keep, n_always,
                       forced_sel=None if shared is not None else forced, rounder=rounder,
                       select_qk=(variant == VARIANT_SELECT_QK), shared_sel=shared, **kw)
        outs.append(r)
        x = r["y"] if rounder is None else rounder(r["y"])
    return outs
