"""The head-sharded step (paper_2506_05096_b200.head_parallel) on ONE GPU: the ranks are emulated one after the other
(no kernel waits for another rank), the all-reduce is the sum of the ranks' partial-sum buffers.  The assembled result
must be what the oracle's unsharded step gives, and all ranks must arrive at the same selection."""
import math

import numpy as np
import pytest
import torch

from paper_2506_05096_b200 import binding as A
from paper_2506_05096_b200 import synth
from paper_2506_05096_b200.head_parallel import HeadShard, head_range
from helpers import assert_attn_close, bf16_dev_to_f64, dev, f64, to_dev_bf16

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world,d,H", [(2, 64, 4), (3, 128, 7), (4, 72, 4)])
def test_head_sharded_step_equals_the_unsharded_oracle(oracle, world, d, H):
    w = synth.Workload("hp", B=2, H=H, d=d, N_v=500, N_t=20)
    inp = synth.make_step_inputs(w, 5)
    B, N, N_sel, D = w.B, w.N, w.N_v, w.D
    k_keep = 170
    M = k_keep + w.N_t
    lse0 = (inp["lse"] - np.float32(math.log(N))).astype(np.float32)
    col = lambda bits, h0, h1: np.ascontiguousarray(bits.reshape(B, N, H, d)[:, :, h0:h1]).reshape(B, N, (h1 - h0) * d)
    shards, local = [], []
    for r in range(world):
        h0, h1 = head_range(H, world, r)
        loc = dict(x_cur=to_dev_bf16(col(inp["x_cur"], h0, h1)), q=to_dev_bf16(col(inp["q"], h0, h1)), k=to_dev_bf16(col(inp["k"], h0, h1)),
                   v=to_dev_bf16(col(inp["v"], h0, h1)))
        sh = HeadShard(A, B, H, N, N_sel, d, world, r, x_ref=to_dev_bf16(col(inp["x_ref"], h0, h1)), lse_cache=dev(lse0[:, h0:h1]),
                       n_skip=dev(inp["n_skip"]), out_cache=to_dev_bf16(col(inp["cache"], h0, h1)).view(B, N, h1 - h0, d),
                       reduce_sum=lambda t: None)
        shards.append(sh)
        local.append(loc)
    # the step, rank by rank: partial sums, the "all-reduce" (sum over the ranks, the same total for everyone), the rest
    for sh, loc in zip(shards, local):
        sh.partial_scores(loc["x_cur"])
    total = torch.stack([sh.part for sh in shards]).sum(0)
    for sh, loc in zip(shards, local):
        sh.part.copy_(total)
        sh.finish(loc["x_cur"], loc["q"], loc["k"], loc["v"], k_keep)
        A.astraea_poll_error(sh.ws)
    res = oracle.step(f64(inp["x_cur"]), f64(inp["x_ref"]), lse0, inp["n_skip"], f64(inp["q"]), f64(inp["k"]), f64(inp["v"]),
                      f64(inp["cache"]), k_keep, w.N_t)
    got_score = shards[0].score.cpu().numpy().astype(np.float64)
    assert (np.abs(got_score - res["score"]) / np.abs(res["score"])).max() < 1e-5
    sel0 = shards[0].idx_sel.cpu().numpy().reshape(-1)[:B * M].reshape(B, M)
    for sh in shards[1:]:
        assert torch.equal(sh.score, shards[0].score) and torch.equal(sh.idx_sel.view(-1)[:B * M], shards[0].idx_sel.view(-1)[:B * M])
        assert torch.equal(sh.n_skip, shards[0].n_skip)
    if not np.array_equal(sel0, res["idx_sel"]):            # near-ties of the k-th score only; the oracle then adopts the device's list
        for b in range(B):
            kth = np.sort(res["score"][b])[::-1][k_keep - 1]
            diff = np.setxor1d(sel0[b], res["idx_sel"][b])
            assert (np.abs(res["score"][b][diff] - kth) <= 1e-6 * abs(kth)).all()
        res = oracle.step(f64(inp["x_cur"]), f64(inp["x_ref"]), lse0, inp["n_skip"], f64(inp["q"]), f64(inp["k"]), f64(inp["v"]),
                          f64(inp["cache"]), k_keep, w.N_t, forced_sel=sel0)
    assert np.array_equal(shards[0].n_skip.cpu().numpy(), res["n_skip"])
    sel_mask = np.zeros((B, N), bool)
    for b in range(B):
        sel_mask[b, sel0[b]] = True
    for r, sh in enumerate(shards):
        h0, h1 = sh.h0, sh.h1
        got = bf16_dev_to_f64(sh.out_cache)
        assert_attn_close(got[sel_mask], res["out"][:, :, h0:h1][sel_mask], what=("rank", r))
        assert np.array_equal(got[~sel_mask], f64(inp["cache"])[:, :, h0:h1][~sel_mask])
        assert np.abs(sh.lse_cache.cpu().numpy() - res["lse"][:, h0:h1]).max() < 1e-3
        assert np.array_equal(bf16_dev_to_f64(sh.x_ref), res["x_ref"].reshape(B, N, H, d)[:, :, h0:h1].reshape(B, N, -1))
