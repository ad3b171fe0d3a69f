"""Head-sharded multi-GPU form of one step of the path (the paper's multi-GPU scalability experiment, Section 4; the
paper does not name its scheme).  Every rank owns a contiguous range of heads: the columns of the hidden states that
belong to them, their full-length queries / keys / values, their slice of the output cache and of the LSE cache.
Attention, scatter and the refresh of the reference inputs need no communication (heads are independent).  The selection
metric is a product of a sum over ALL channels and a sum over ALL heads, so each rank computes raw partial sums
(astraea_score_partial), ONE all-reduce adds the 2*B*N_sel floats up (NCCL over NVLink: at most ~1 MB, bitwise identical
on every rank afterwards), astraea_score_combine turns the totals into scores, and the deterministic selection then
comes out identical on every rank without being exchanged.  Keys and values never leave their GPU.

Host logic only: every step of the arithmetic runs in the library's kernels.  `reduce_sum` is the collective: by default
torch.distributed.all_reduce on the default process group; tests on one GPU pass a function that adds the ranks' buffers.
"""
from __future__ import annotations

from typing import Callable, Optional, Tuple


def head_range(H: int, world: int, rank: int) -> Tuple[int, int]:
    """Heads [h0, h1) of `rank`: contiguous, sizes differing by at most one, the larger shards first."""
    if not (world >= 1 and 0 <= rank < world and H >= world):
        raise ValueError("need 1 <= world <= H and 0 <= rank < world (H=%d, world=%d, rank=%d)" % (H, world, rank))
    base, extra = divmod(H, world)
    h0 = rank * base + min(rank, extra)
    return h0, h0 + base + (1 if rank < extra else 0)


def all_reduce_sum(t) -> None:
    """The default collective: in-place sum over the default process group (NCCL on GPUs, gloo in the CPU tests)."""
    import torch.distributed as dist
    dist.all_reduce(t, op=dist.ReduceOp.SUM)


class HeadShard:
    """One rank's share of an attention block's tensors and the step over them.

    Local tensors (this rank's heads h0..h1, D_local = (h1 - h0) * d): x_ref [B,N,D_local], lse_cache [B,H_local,N],
    out_cache [B,N,H_local,d]; n_skip [B,N_sel], score [B,N_sel], idx_sel [B,N], idx_rem [B,N_sel] are replicated.
    """

    def __init__(self, A, B: int, H: int, N: int, N_sel: int, d: int, world: int, rank: int, x_ref, lse_cache, n_skip, out_cache,
                 reduce_sum: Optional[Callable] = None, device="cuda"):
        import torch
        self.A, self.B, self.H, self.N, self.N_sel, self.d = A, B, H, N, N_sel, d
        self.h0, self.h1 = head_range(H, world, rank)
        self.H_local = self.h1 - self.h0
        self.D_local = self.H_local * d
        self.x_ref, self.lse_cache, self.n_skip, self.out_cache = x_ref, lse_cache, n_skip, out_cache
        self.reduce_sum = reduce_sum or all_reduce_sum
        self.part = torch.zeros(2, B, N_sel, device=device)
        self.score = torch.empty(B, N_sel, device=device)
        self.idx_sel = torch.empty(B, N, dtype=torch.int32, device=device)
        self.idx_rem = torch.empty(B, max(N_sel, 1), dtype=torch.int32, device=device)
        self.ws = A.new_workspace(A.OP_STEP, B, self.H_local, N, N, d, device=device)
        self.ws_sel = A.new_workspace(A.OP_SELECT, B, 0, N_sel, 0, 0, device=device)

    def partial_scores(self, x_cur, delta_mode=0, lse_mode=0) -> None:
        A = self.A
        A.astraea_score_partial(x_cur, self.x_ref, self.lse_cache, self.part, self.B, self.N, self.N_sel, self.D_local, self.H_local,
                                delta_mode, lse_mode)

    def finish(self, x_cur, q, k, v, k_keep: int, w_alpha=1.0, w_beta=1.0) -> None:
        """Everything after the all-reduce: combine, select (replicated), attention and refresh on the local heads."""
        A, B, N, N_sel, d = self.A, self.B, self.N, self.N_sel, self.d
        M = k_keep + (N - N_sel)
        A.astraea_score_combine(self.part, self.n_skip, self.score, B, N_sel, self.H * d, self.H, True, w_alpha, w_beta)
        A.astraea_select(self.score, B, N_sel, k_keep, N - N_sel, self.idx_sel, self.idx_rem, self.n_skip, self.ws_sel)
        s = A.bhnd_strides(N, self.H_local, d)
        A.astraea_sparse_attn(q, k, v, s, s, s, self.idx_sel, M, self.out_cache, self.lse_cache, B, self.H_local, N, d, workspace=self.ws)
        A.astraea_scatter_reuse(self.x_ref, x_cur, self.idx_sel, B, N, M, self.D_local, A.SCATTER_SRC_FULL, workspace=self.ws)

    def step(self, x_cur, q, k, v, k_keep: int, w_alpha=1.0, w_beta=1.0, delta_mode=0, lse_mode=0) -> None:
        """One step on this rank: x_cur [B,N,D_local], q / k / v [B,N,H_local,d] are the local slices of the step's inputs."""
        self.partial_scores(x_cur, delta_mode, lse_mode)
        self.reduce_sum(self.part)                     # the one exchange of the step
        self.finish(x_cur, q, k, v, k_keep, w_alpha, w_beta)
