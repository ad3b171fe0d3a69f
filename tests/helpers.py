"""Shared helpers of the GPU parity tests: move seeded inputs to the device, run the
oracle on the exact values the GPU sees (bf16 upcast to fp64)."""
import numpy as np
import torch

from paper_2506_05096_b200 import synth


def to_dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16).cuda()


def bf16_dev_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def f64(bits: np.ndarray) -> np.ndarray:
    return synth.bf16_to_f64(bits)


def assert_attn_close(got, want, max_abs=2e-2, mean_abs=2e-3, what=""):
    """Attention rows [..., d] against the fp64 oracle: the stated absolute tolerances (max-abs 2e-2, mean-abs
    2e-3, relative beyond magnitude one), and a bound that scales with each row's own magnitude, because at the
    workloads' sizes an output row of N(0,1) values is only ~0.01 large and the absolute tolerances alone would
    accept a row that belongs to another query.  Per row the error is one bf16 rounding of the output (2^-9 of
    its magnitude) plus the independent bf16 roundings of the probabilities (2^-9 relative each, i.e. of the
    same order after the weighted sum); 2^-6 of the row's largest element leaves a factor of four."""
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    err = np.abs(got - want)
    rel1 = err / np.maximum(1.0, np.abs(want))
    assert rel1.max() < max_abs and rel1.mean() < mean_abs, (what, rel1.max(), rel1.mean())
    row_scale = np.abs(want).max(axis=-1, keepdims=True)
    excess = err - (2.0 ** -6 * row_scale + 2e-5)
    assert excess.max() <= 0.0, (what, "row-scaled bound", float((err / (row_scale + 1e-30)).max()))


def device_state(x_ref, lse, n_skip, out):
    """The cross-step state of one attention block as the oracle takes it (exact upcasts of the device's values)."""
    return dict(x_ref=bf16_dev_to_f64(x_ref), lse=lse.cpu().numpy().astype(np.float64),
                n_skip=n_skip.cpu().numpy().copy(), out=bf16_dev_to_f64(out))


def check_step_against_oracle(oracle, prev, x_bits, q_bits, k_bits, v_bits, k_keep, n_always,
                              score, idx_sel, idx_rem, x_ref, lse, n_skip, out,
                              w_alpha=1.0, w_beta=1.0, delta_mode=0, lse_mode=0, what=""):
    """One step of the device (its tensors after the step) against oracle.step started from `prev`, the
    device's state before the step (teacher forcing).  Scores within 1e-5 relative; the selection bit-exact, or
    - only where scores lie within 1e-6 relative of the k-th - a valid selection that differs at such near-ties,
    which the oracle then adopts for the rest of the step; remainder list and counters bit-exact; computed rows
    within the attention tolerances; reused rows, the LSE cache elsewhere and x_ref bit-exact.
    Returns (state after the step, whether a near-tie was met)."""
    B, N = x_bits.shape[:2]
    N_sel, M = N - n_always, k_keep + n_always
    args = (f64(x_bits), prev["x_ref"], prev["lse"], prev["n_skip"], f64(q_bits), f64(k_bits), f64(v_bits), prev["out"],
            k_keep, n_always)
    kw = dict(w_alpha=w_alpha, w_beta=w_beta, delta_mode=delta_mode, lse_mode=lse_mode)
    res = oracle.step(*args, **kw)
    got_score = score.cpu().numpy().astype(np.float64)[:, :N_sel]
    rel = np.abs(got_score - res["score"]) / np.maximum(np.abs(res["score"]), 1e-300)
    assert rel.max() < 1e-5, (what, rel.max())
    got_sel = idx_sel.cpu().numpy().reshape(-1)[:B * M].reshape(B, M)
    near_tie = False
    if not np.array_equal(got_sel, res["idx_sel"]):
        for b in range(B):
            assert (np.diff(got_sel[b]) > 0).all(), what                      # ascending, hence duplicate-free
            assert (got_sel[b][:k_keep] >= 0).all() and (got_sel[b][:k_keep] < N_sel).all(), what
            assert np.array_equal(got_sel[b][k_keep:], np.arange(N_sel, N)), what
            kth = np.sort(res["score"][b])[::-1][k_keep - 1]
            diff = np.setxor1d(got_sel[b], res["idx_sel"][b])
            assert (np.abs(res["score"][b][diff] - kth) <= 1e-6 * abs(kth)).all(), what
        res = oracle.step(*args, forced_sel=got_sel, **kw)
        near_tie = True
    if idx_rem is not None:
        got_rem = idx_rem.cpu().numpy().reshape(-1)[:B * (N_sel - k_keep)].reshape(B, N_sel - k_keep)
        assert np.array_equal(got_rem, res["idx_rem"]), what
    assert np.array_equal(n_skip.cpu().numpy(), res["n_skip"]), what
    got_out = bf16_dev_to_f64(out)
    sel_mask = np.zeros((B, N), bool)
    for b in range(B):
        sel_mask[b, res["idx_sel"][b]] = True
    if M:
        assert_attn_close(got_out[sel_mask], res["out"][sel_mask], what=what)
    assert np.array_equal(got_out[~sel_mask], prev["out"][~sel_mask]), what           # reuse is bit-exact
    got_lse = lse.cpu().numpy().astype(np.float64)
    assert np.abs(got_lse - res["lse"]).max() < 1e-3, what
    assert np.array_equal(got_lse.transpose(0, 2, 1)[~sel_mask], prev["lse"].transpose(0, 2, 1)[~sel_mask]), what
    assert np.array_equal(bf16_dev_to_f64(x_ref), res["x_ref"]), what
    return dict(x_ref=res["x_ref"], lse=got_lse, n_skip=res["n_skip"], out=got_out), near_tie


GUARD_ELEMS = 64


class Guarded:
    """An output tensor carved out of a larger allocation with 64 sentinel elements (bytes 0xA5) before and after
    it: a write one past either end of the tensor shows in `check()`.  The stand-in for a memory checker."""

    def __init__(self, shape, dtype, init=None):
        self.n = int(np.prod(shape))
        item = torch.empty(0, dtype=dtype).element_size()
        self.pad = GUARD_ELEMS * item
        self.raw = torch.full((self.n * item + 2 * self.pad,), 0xA5, dtype=torch.uint8, device="cuda")
        self.t = self.raw[self.pad:self.pad + self.n * item].view(dtype).view(*shape)
        if init is not None:
            self.t.copy_(init)

    def check(self, what=""):
        torch.cuda.synchronize()
        lo, hi = self.raw[:self.pad], self.raw[self.raw.numel() - self.pad:]
        assert bool((lo == 0xA5).all()), ("write before the start of an output", what)
        assert bool((hi == 0xA5).all()), ("write past the end of an output", what)
