"""astraea_sparse_attn_noalloc, the entry point for callers that cannot allocate device memory (their
allocator is locked, or they run where cudaMalloc would stall the device): it must give what
astraea_sparse_attn gives while taking its scratch from a fixed array inside the library.  Two calls in
a row share that array, so the second call also checks that nothing stale from the first one leaks in.
This file sorts last on purpose: a run that stops at the first failure has then run everything else."""
import numpy as np
import pytest
import torch

from paper_2506_05096_b200 import binding as A
from helpers import assert_attn_close

pytestmark = pytest.mark.gpu


def _inputs(seed, B, H, N, d, M):
    g = torch.Generator(device="cpu").manual_seed(seed)
    q, k, v, cache = (torch.randn(B, N, H, d, generator=g).bfloat16().cuda() for _ in range(4))
    idx = torch.stack([torch.sort(torch.randperm(N, generator=g)[:M])[0] for _ in range(B)]).int().cuda()
    return q, k, v, cache, idx


def test_noalloc_entry_matches_the_workspace_entry_on_two_calls_in_a_row(oracle):
    for call, (seed, B, H, N, d, M) in enumerate([(1, 2, 3, 700, 64, 300), (2, 1, 2, 1500, 128, 260)]):
        q, k, v, cache, idx = _inputs(seed, B, H, N, d, M)
        s = A.bhnd_strides(N, H, d)
        want, want_lse = cache.clone(), torch.zeros(B, H, N, device="cuda")
        ws = A.new_workspace(A.OP_SPARSE_ATTN, B, H, N, M, d)
        A.astraea_sparse_attn(q, k, v, s, s, s, idx, M, want, want_lse, B, H, N, d, workspace=ws)
        A.astraea_poll_error(ws)
        got, got_lse = cache.clone(), torch.zeros(B, H, N, device="cuda")
        A.astraea_sparse_attn_noalloc(q, k, v, s, s, s, idx, M, got, got_lse, B, H, N, d)
        torch.cuda.synchronize()
        # the same deterministic kernel ran twice: the two entry points agree bit for bit
        assert torch.equal(got.view(torch.int16), want.view(torch.int16)), call
        assert torch.equal(got_lse, want_lse), call
        # and the result is the attention the CPU oracle computes for the listed rows
        f = lambda t: t.float().cpu().numpy().astype(np.float64)
        want_o, want_l, _ = oracle.sparse_attn(f(q), f(k), f(v), q_idx=idx.cpu().numpy())
        rows = np.take_along_axis(f(got), idx.cpu().numpy()[:, :, None, None].astype(np.int64), 1)
        assert_attn_close(rows, want_o, what=("noalloc", call))
        got_l = np.take_along_axis(got_lse.cpu().numpy().astype(np.float64), idx.cpu().numpy()[:, None, :].astype(np.int64), 2)
        assert np.abs(got_l - want_l).max() < 1e-3
        # rows that were not selected keep the cache, exactly as with the workspace entry
        mask = torch.ones(B, N, dtype=torch.bool, device="cuda")
        for b in range(B):
            mask[b, idx[b].long()] = False
        assert torch.equal(got[mask], cache[mask])


def test_noalloc_entry_takes_the_same_flags_and_refuses_what_does_not_fit_its_scratch():
    """The two entry points share one validation and launch path: the CTA-shape flag is accepted, and a kv_idx
    problem whose gathered key / value rows do not fit the built-in scratch is refused with WORKSPACE_TOO_SMALL."""
    B, H, N, d, M = 1, 2, 400, 64, 100
    q, k, v, cache, idx = _inputs(3, B, H, N, d, M)
    s = A.bhnd_strides(N, H, d)
    want, got = cache.clone(), cache.clone()
    ws = A.new_workspace(A.OP_SPARSE_ATTN, B, H, N, M, d)
    A.astraea_sparse_attn(q, k, v, s, s, s, idx, M, want, None, B, H, N, d, flags=A.ATTN_SMALL_CTAS, workspace=ws)
    A.astraea_sparse_attn_noalloc(q, k, v, s, s, s, idx, M, got, None, B, H, N, d, flags=A.ATTN_SMALL_CTAS)
    torch.cuda.synchronize()
    assert torch.equal(got.view(torch.int16), want.view(torch.int16))
    with pytest.raises(A.AstraeaError) as e:
        A.astraea_sparse_attn_noalloc(q, k, v, s, s, s, idx, M, got, None, B, H, N, d, kv_idx=idx, M_kv=M)
    assert e.value.code == A.ERR_WORKSPACE_TOO_SMALL
    assert A.astraea_workspace_bytes(A.OP_SPARSE_ATTN_KV, B, H, N, M, d) > A.NOALLOC_SCRATCH_BYTES


def test_noalloc_entry_rejects_bad_arguments_like_the_workspace_entry():
    z = torch.zeros(1, 64, 1, 64, dtype=torch.bfloat16, device="cuda")
    s = A.bhnd_strides(64, 1, 64)
    with pytest.raises(A.AstraeaError) as e:
        A.astraea_sparse_attn_noalloc(z, z, z, s, s, s, None, 65, z, None, 1, 1, 64, 64)
    assert e.value.code == A.ERR_INVALID_ARG
    with pytest.raises(A.AstraeaError) as e:
        A.astraea_sparse_attn_noalloc(z, z, z, s, s, s, None, 64, z, None, 1, 1, 64, 96)
    assert e.value.code == A.ERR_UNSUPPORTED
