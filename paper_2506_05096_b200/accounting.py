"""Algorithmic work of each call of the hot path (bytes moved / flops), used for the
roofline figures.  Host arithmetic only."""
from __future__ import annotations


def attn_flops(B: int, H: int, M: int, N: int, d: int) -> int:
    """QK^T and PV for M selected queries against N keys: 2*M*N*d each per head.
    The paper's self-attention count 4*B*N^2*(H*d) with the query count replaced by M
    (its cross-attention form 4*B*N_q*N_kv*H); softmax is excluded as in the paper."""
    return 4 * B * H * M * N * d


def attn_min_bytes(B: int, H: int, M: int, N: int, d: int) -> int:
    """Compulsory traffic: read M query rows, N key and N value rows, write M output rows (bf16)."""
    return B * H * (2 * M + 2 * N) * d * 2


def score_bytes(B: int, N: int, N_sel: int, D: int, H: int) -> int:
    """Read x_cur and x_ref rows of the scored tokens (bf16), their per-head LSE (fp32) and
    counters (int32); write one fp32 score per token."""
    return B * (2 * N_sel * D * 2 + 4 * H * N_sel + 4 * N_sel + 4 * N_sel)


def select_bytes(B: int, N_sel: int, k: int, with_counters: bool = True) -> int:
    """Read scores once, write both index lists, read+write the counters."""
    return B * (4 * N_sel + 4 * k + 4 * (N_sel - k) + (8 * N_sel if with_counters else 0))


def scatter_bytes(B: int, M: int, row_elems: int) -> int:
    """Read M compact rows and write them into the cache (bf16), plus the index list."""
    return B * M * (2 * row_elems * 2 + 4)
