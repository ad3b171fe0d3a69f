"""Host logic of the head-sharded multi-GPU step on CPU: the partition of the heads, and two gloo ranks that each
hold a shard, exchange their partial sums with ONE all-reduce and arrive at the same scores and the same selection as
the unsharded oracle.  (The kernels themselves are covered on the GPU, with the ranks emulated one after the other.)"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2506_05096_b200.head_parallel import all_reduce_sum, head_range


def test_head_range_is_a_contiguous_balanced_partition():
    for H in (1, 2, 3, 16, 24, 48):
        for world in range(1, min(H, 9) + 1):
            spans = [head_range(H, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == H
            assert all(a[1] == b[0] for a, b in zip(spans[:-1], spans[1:]))
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        head_range(4, 5, 0)
    with pytest.raises(ValueError):
        head_range(4, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import astraea_oracle as oracle
    rng = np.random.default_rng(77)                       # the same full problem on every rank; each takes its shard
    B, N, N_sel, H, d, k_keep = 2, 40, 36, 6, 4, 13
    D = H * d
    x_ref = rng.standard_normal((B, N, D))
    x_cur = x_ref + 0.2 * rng.standard_normal((B, N, D))
    lse = rng.standard_normal((B, H, N))
    n = rng.integers(0, 3, (B, N_sel)).astype(np.int32)
    h0, h1 = head_range(H, world, rank)
    part = torch.from_numpy(oracle.score_partial(x_cur[:, :, h0 * d:h1 * d], x_ref[:, :, h0 * d:h1 * d], lse[:, h0:h1], N_sel))
    all_reduce_sum(part)                                  # the one exchange of the step
    score = oracle.score_combine(part.numpy(), n, D, H)
    sel, rem, n_new = oracle.select(score.astype(np.float32), k_keep, N - N_sel, n)
    want = oracle.score(x_cur, x_ref, lse, n, n_sel=N_sel)
    want_sel, _, want_n = oracle.select(want.astype(np.float32), k_keep, N - N_sel, n)
    assert np.abs(score - want).max() <= 1e-12 * np.abs(want).max()
    assert np.array_equal(sel, want_sel) and np.array_equal(n_new, want_n)
    # every rank ends with bitwise the same totals, hence the same selection, without exchanging it
    gathered = [torch.zeros_like(part) for _ in range(world)]
    dist.all_gather(gathered, part)
    assert all(torch.equal(g, part) for g in gathered)
    np.save(os.path.join(out_dir, "sel%d.npy" % rank), sel)
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_scores_and_selection(tmp_path):
    from oracle import astraea_oracle
    astraea_oracle.build()
    world, port = 2, _free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    sels = [np.load(tmp_path / ("sel%d.npy" % r)) for r in range(world)]
    assert np.array_equal(sels[0], sels[1])
