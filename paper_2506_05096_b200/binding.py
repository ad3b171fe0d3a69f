"""ctypes binding of libastraea.so: same names as include/astraea.h, argument marshalling only.

Tensors are torch CUDA tensors (torch is used for device memory and streams, nothing else);
every step of the path runs in the library's kernels.  Loading fails loudly if the library
has not been built (python -m paper_2506_05096_b200.build): there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libastraea.so")

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, ERR_TIMEOUT, ERR_BAD_INDEX = -1, -2, -3, -4, -5, -6
DELTA_MEAN_ABS, DELTA_MEAN_SQ, DELTA_MEAN_SIGNED = 0, 1, 2
LSE_SUM_EXP, LSE_LOG = 0, 1
ATTN_COMPACT_OUT = 1
ATTN_SMALL_CTAS = 2
ATTN_WHOLE_KEYS = 4
SCATTER_SRC_FULL = 1
LINEAR_COMPACT_OUT, LINEAR_COMPACT_IN, LINEAR_GELU, LINEAR_COMPACT_RES = 1, 2, 4, 8
LN_COMPACT_IN, LN_COMPACT_OUT = 1, 2
BLOCK_REUSE_SELECTION, BLOCK_SELECT_QK = 1, 2
VARIANT_TOKEN_WISE, VARIANT_SELECT_QK, VARIANT_TIMESTEP, VARIANT_FIXED_TOKEN = 0, 1, 2, 3
OP_SELECT, OP_SPARSE_ATTN, OP_STEP, OP_SPARSE_ATTN_KV, OP_GATHERED_LINEAR, OP_LAYERNORM = 1, 2, 3, 4, 5, 6
N_SKIP_CLAMP = 80
NOALLOC_SCRATCH_BYTES = 4096

EXPORTS = [
    "astraea_score", "astraea_score_partial", "astraea_score_combine", "astraea_select", "astraea_sparse_attn", "astraea_sparse_attn_plan", "astraea_sparse_cross_attn", "astraea_sparse_attn_noalloc", "astraea_scatter_reuse", "astraea_step",
    "astraea_gathered_linear", "astraea_gathered_linear_residual", "astraea_layernorm_modulate",
    "astraea_block_step", "astraea_block_workspace_bytes", "astraea_model_schedule_create", "astraea_model_schedule_launch",
    "astraea_model_schedule_destroy", "astraea_timestep_level_budgets", "astraea_schedule_create", "astraea_schedule_launch", "astraea_schedule_destroy",
    "astraea_session_create", "astraea_session_destroy", "astraea_step_host", "astraea_session_last_h2d_bytes",
    "astraea_workspace_bytes", "astraea_budget_to_k", "astraea_poll_error", "astraea_selftest_wait",
    "astraea_last_error", "astraea_version",
]


class BlockWeights(ctypes.Structure):
    """struct astraea_block_weights: device pointers of one compute block's parameters."""
    NAMES = ("wq", "bq", "wk", "bk", "wv", "bv", "wo", "bo", "wq2", "bq2", "wo2", "bo2", "w1", "b1", "w2", "b2",
             "s1", "t1", "g1", "s3", "t3", "g3")
    _fields_ = [(n, ctypes.c_void_p) for n in NAMES] + [("hidden", ctypes.c_int32)]


class BlockState(ctypes.Structure):
    """struct astraea_block_state: the cross-step state of one compute block."""
    _fields_ = [("x_ref", ctypes.c_void_p), ("lse_cache", ctypes.c_void_p), ("n_skip", ctypes.c_void_p), ("y_cache", ctypes.c_void_p)]


class AstraeaError(RuntimeError):
    def __init__(self, code: int, text: str):
        super().__init__("astraea error %d: %s" % (code, text))
        self.code = code


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libastraea.so is not built; run `python -m paper_2506_05096_b200.build` "
                              "(the CUDA library is the only implementation: there is no fallback)")
        L = ctypes.CDLL(LIB_PATH)
        c_i, c_f, c_p, c_sz, c_i64, c_u = (ctypes.c_int, ctypes.c_float, ctypes.c_void_p, ctypes.c_size_t,
                                           ctypes.c_int64, ctypes.c_uint32)
        L.astraea_score.argtypes = [c_p, c_p, c_p, c_p, c_p, c_i, c_i, c_i, c_i, c_i, c_f, c_f, c_i, c_i, c_p]
        L.astraea_score_partial.argtypes = [c_p, c_p, c_p, c_p, c_i, c_i, c_i, c_i, c_i, c_i, c_i, c_p]
        L.astraea_score_combine.argtypes = [c_p, c_p, c_p, c_i, c_i, c_i, c_i, c_i, c_f, c_f, c_p]
        L.astraea_score_partial.restype = L.astraea_score_combine.restype = ctypes.c_int32
        L.astraea_select.argtypes = [c_p, c_i, c_i, c_i, c_i, c_p, c_p, c_p, c_p, c_sz, c_p]
        L.astraea_sparse_attn.argtypes = [c_p, c_p, c_p] + [c_i64] * 9 + [c_p, c_i, c_p, c_i, c_p, c_p,
                                                                         c_i, c_i, c_i, c_i, c_f, c_u, c_p, c_sz, c_p]
        L.astraea_sparse_cross_attn.argtypes = [c_p, c_p, c_p] + [c_i64] * 9 + [c_p, c_i, c_p, c_p,
                                                                               c_i, c_i, c_i, c_i, c_i, c_f, c_u, c_p, c_sz, c_p]
        L.astraea_sparse_attn_noalloc.argtypes = [c_p, c_p, c_p] + [c_i64] * 9 + [c_p, c_i, c_p, c_i, c_p, c_p,
                                                                                 c_i, c_i, c_i, c_i, c_f, c_u, c_p]
        L.astraea_sparse_attn_plan.argtypes = [c_i, c_i, c_i, c_i, c_i, c_u, c_sz, c_p, c_p, c_p]
        L.astraea_sparse_attn_plan.restype = ctypes.c_int32
        L.astraea_scatter_reuse.argtypes = [c_p, c_p, c_p, c_i, c_i, c_i, c_i, c_u, c_p, c_p]
        L.astraea_gathered_linear.argtypes = [c_p, c_p, c_i, c_p, c_p, c_p, c_i, c_i, c_i, c_i, c_u, c_p, c_sz, c_p]
        L.astraea_gathered_linear_residual.argtypes = [c_p, c_p, c_i, c_p, c_p, c_p, c_p, c_p, c_i, c_i, c_i, c_i, c_u, c_p, c_sz, c_p]
        L.astraea_layernorm_modulate.argtypes = [c_p, c_p, c_i, c_p, c_p, c_p, c_i, c_i, c_i, c_f, c_u, c_p, c_p]
        L.astraea_block_step.argtypes = [c_p, ctypes.POINTER(BlockWeights), ctypes.POINTER(BlockState), c_p, c_p, c_i, c_p, c_p, c_p,
                                         c_i, c_i, c_i, c_i, c_i, c_i, c_f, c_f, c_i, c_i, c_f, c_u, c_p, c_sz, c_p]
        L.astraea_model_schedule_create.argtypes = [ctypes.POINTER(c_p), c_i, c_i, c_p, c_p, ctypes.POINTER(BlockWeights),
                                                    ctypes.POINTER(BlockState), c_p, c_p, c_i, c_p, c_p, c_p,
                                                    c_i, c_i, c_i, c_i, c_i, c_f, c_f, c_i, c_i, c_f, c_i, c_p, c_sz]
        L.astraea_model_schedule_launch.argtypes = [c_p, c_p]
        L.astraea_model_schedule_destroy.argtypes = [c_p]
        L.astraea_model_schedule_destroy.restype = None
        L.astraea_timestep_level_budgets.argtypes = [c_p, c_i, c_i, c_p]
        L.astraea_block_workspace_bytes.argtypes = [c_i] * 5
        L.astraea_block_workspace_bytes.restype = c_sz
        L.astraea_step.argtypes = [c_p] * 11 + [c_i] * 6 + [c_f, c_f, c_i, c_i, c_p, c_sz, c_p]
        L.astraea_schedule_create.argtypes = [ctypes.POINTER(c_p), c_i, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p, c_p,
                                              c_i, c_i, c_i, c_i, c_i, c_f, c_f, c_i, c_i, c_p, c_sz]
        L.astraea_schedule_launch.argtypes = [c_p, c_p]
        L.astraea_schedule_destroy.argtypes = [c_p]
        L.astraea_schedule_destroy.restype = None
        L.astraea_session_create.argtypes = [ctypes.POINTER(c_p), c_i, c_i, c_i, c_i, c_i]
        L.astraea_session_destroy.argtypes = [c_p]
        L.astraea_session_destroy.restype = None
        L.astraea_step_host.argtypes = [c_p, c_p, c_p, c_p, c_p, c_p, c_i, c_f, c_f, c_i, c_i]
        L.astraea_session_last_h2d_bytes.argtypes = [c_p]
        L.astraea_session_last_h2d_bytes.restype = c_sz
        L.astraea_workspace_bytes.argtypes = [c_i] * 6
        L.astraea_workspace_bytes.restype = c_sz
        L.astraea_budget_to_k.argtypes = [c_i, c_i]
        L.astraea_poll_error.argtypes = [c_p, c_p]
        L.astraea_selftest_wait.argtypes = [c_p, c_i, c_p, c_p]
        L.astraea_selftest_wait.restype = ctypes.c_int32
        L.astraea_last_error.restype = ctypes.c_char_p
        L.astraea_version.restype = ctypes.c_char_p
        for name in ("astraea_score", "astraea_select", "astraea_sparse_attn", "astraea_sparse_cross_attn", "astraea_sparse_attn_noalloc", "astraea_scatter_reuse",
                     "astraea_step", "astraea_gathered_linear", "astraea_gathered_linear_residual", "astraea_layernorm_modulate", "astraea_block_step", "astraea_model_schedule_create", "astraea_model_schedule_launch",
                     "astraea_timestep_level_budgets", "astraea_schedule_create", "astraea_schedule_launch",
                     "astraea_session_create", "astraea_step_host", "astraea_budget_to_k",
                     "astraea_poll_error"):
            getattr(L, name).restype = ctypes.c_int32
        _lib = L
    return _lib


def _check(rc: int) -> None:
    if rc != OK:
        raise AstraeaError(rc, lib().astraea_last_error().decode())


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def astraea_version() -> str:
    return lib().astraea_version().decode()


def astraea_last_error() -> str:
    return lib().astraea_last_error().decode()


def astraea_budget_to_k(n_sel: int, theta_permille: int) -> int:
    k = lib().astraea_budget_to_k(n_sel, theta_permille)
    if k < 0:
        raise AstraeaError(k, "bad budget")
    return k


def astraea_workspace_bytes(op: int, B: int, H: int, N: int, M: int, d: int) -> int:
    return int(lib().astraea_workspace_bytes(op, B, H, N, M, d))


def new_workspace(op: int, B: int, H: int, N: int, M: int, d: int, device="cuda") -> torch.Tensor:
    """A zeroed workspace of the size the op asks for (caller-owned device memory)."""
    return torch.zeros(max(256, astraea_workspace_bytes(op, B, H, N, M, d)), dtype=torch.uint8, device=device)


def astraea_score(x_cur, x_ref, lse, n_skip, score, B, N, N_sel, D, H, w_alpha=1.0, w_beta=1.0,
                  delta_mode=DELTA_MEAN_ABS, lse_mode=LSE_SUM_EXP, stream=None) -> None:
    _check(lib().astraea_score(_ptr(x_cur), _ptr(x_ref), _ptr(lse), _ptr(n_skip), _ptr(score),
                               B, N, N_sel, D, H, w_alpha, w_beta, delta_mode, lse_mode, _stream(stream)))


def astraea_score_partial(x_cur, x_ref, lse, part, B, N, N_sel, D_local, H_local, delta_mode=DELTA_MEAN_ABS, lse_mode=LSE_SUM_EXP,
                          stream=None) -> None:
    """Raw partial sums of the selection metric over a shard of the channels / heads: part is fp32 [2, B, N_sel]."""
    _check(lib().astraea_score_partial(_ptr(x_cur), _ptr(x_ref), _ptr(lse), _ptr(part), B, N, N_sel, D_local, H_local,
                                       delta_mode, lse_mode, _stream(stream)))


def astraea_score_combine(part, n_skip, score, B, N_sel, D, H, has_lse=True, w_alpha=1.0, w_beta=1.0, stream=None) -> None:
    """S_token from the partial sums added up over all shards (D, H: total channel and head counts)."""
    _check(lib().astraea_score_combine(_ptr(part), _ptr(n_skip), _ptr(score), B, N_sel, D, H, 1 if has_lse else 0,
                                       w_alpha, w_beta, _stream(stream)))


def astraea_select(score, B, N_sel, k, n_always, idx_sel, idx_rem, n_skip, workspace, stream=None) -> None:
    _check(lib().astraea_select(_ptr(score), B, N_sel, k, n_always, _ptr(idx_sel), _ptr(idx_rem), _ptr(n_skip),
                                _ptr(workspace), workspace.numel() if workspace is not None else 0, _stream(stream)))


def astraea_sparse_attn(q, k, v, q_strides, k_strides, v_strides, q_idx, M, out, lse_out, B, H, N, d,
                        scale=0.0, flags=0, workspace=None, kv_idx=None, M_kv=0, stream=None) -> None:
    """q_strides etc. are (batch, head, token) element strides."""
    _check(lib().astraea_sparse_attn(_ptr(q), _ptr(k), _ptr(v), *q_strides, *k_strides, *v_strides,
                                     _ptr(q_idx), M, _ptr(kv_idx), M_kv, _ptr(out), _ptr(lse_out),
                                     B, H, N, d, scale, flags, _ptr(workspace),
                                     workspace.numel() if workspace is not None else 0, _stream(stream)))


def astraea_sparse_attn_plan(B, H, N, M, d, flags=0, workspace_bytes=None) -> dict:
    """The launch schedule astraea_sparse_attn would pick (host logic only).  workspace_bytes None: the full size."""
    if workspace_bytes is None:
        workspace_bytes = astraea_workspace_bytes(OP_SPARSE_ATTN, B, H, N, M, d)
    r = (ctypes.c_int32 * 3)()
    _check(lib().astraea_sparse_attn_plan(B, H, N, M, d, flags, workspace_bytes, ctypes.byref(r, 0), ctypes.byref(r, 4), ctypes.byref(r, 8)))
    return {"small_ctas": bool(r[0]), "split_units": int(r[1]), "split": int(r[2])}


def astraea_sparse_attn_noalloc(q, k, v, q_strides, k_strides, v_strides, q_idx, M, out, lse_out, B, H, N, d,
                                scale=0.0, flags=0, kv_idx=None, M_kv=0, stream=None) -> None:
    """astraea_sparse_attn for callers that cannot allocate: the scratch is a fixed array inside the
    library (NOALLOC_SCRATCH_BYTES per GPU), shared by all calls on the device, so overlapping calls race."""
    _check(lib().astraea_sparse_attn_noalloc(_ptr(q), _ptr(k), _ptr(v), *q_strides, *k_strides, *v_strides,
                                             _ptr(q_idx), M, _ptr(kv_idx), M_kv, _ptr(out), _ptr(lse_out),
                                             B, H, N, d, scale, flags, _stream(stream)))


def astraea_sparse_cross_attn(q, k, v, q_strides, k_strides, v_strides, q_idx, M, out, lse_out, B, H, N, N_kv, d,
                              scale=0.0, flags=0, workspace=None, stream=None) -> None:
    """As astraea_sparse_attn with keys / values of another sequence (N_kv tokens)."""
    _check(lib().astraea_sparse_cross_attn(_ptr(q), _ptr(k), _ptr(v), *q_strides, *k_strides, *v_strides,
                                           _ptr(q_idx), M, _ptr(out), _ptr(lse_out), B, H, N, N_kv, d, scale, flags,
                                           _ptr(workspace), workspace.numel() if workspace is not None else 0, _stream(stream)))


def astraea_scatter_reuse(cache, rows, idx, B, N, M, row_elems, flags=0, workspace=None, stream=None) -> None:
    """workspace (optional): any workspace tensor; bad index entries are then reported by astraea_poll_error."""
    _check(lib().astraea_scatter_reuse(_ptr(cache), _ptr(rows), _ptr(idx), B, N, M, row_elems, flags,
                                       _ptr(workspace), _stream(stream)))


def astraea_gathered_linear(x, idx, M, w, bias, y, B, N, K, N_out, flags=0, workspace=None, stream=None) -> None:
    """y[b, idx[b,r], :] = x[b, idx[b,r], :] @ w.T + bias (idx None: all rows); other rows of y are left alone."""
    if idx is not None and M == 0:
        return          # an empty index tensor has a null data pointer, which the C ABI reads as "all rows"
    _check(lib().astraea_gathered_linear(_ptr(x), _ptr(idx), M, _ptr(w), _ptr(bias), _ptr(y), B, N, K, N_out, flags,
                                         _ptr(workspace), workspace.numel() if workspace is not None else 0, _stream(stream)))


def astraea_gathered_linear_residual(x, idx, M, w, bias, residual, gate, y, B, N, K, N_out, flags=0, workspace=None, stream=None) -> None:
    """y[rows] = residual[rows] + gate[b] * act(x[rows] @ w.T + bias): astraea_gathered_linear with a gated residual."""
    if idx is not None and M == 0:
        return
    _check(lib().astraea_gathered_linear_residual(_ptr(x), _ptr(idx), M, _ptr(w), _ptr(bias), _ptr(residual), _ptr(gate), _ptr(y),
                                                  B, N, K, N_out, flags, _ptr(workspace),
                                                  workspace.numel() if workspace is not None else 0, _stream(stream)))


def astraea_layernorm_modulate(x, idx, M, scale, shift, y, B, N, D, eps=1e-6, flags=0, workspace=None, stream=None) -> None:
    """y[rows] = LayerNorm(x[rows]) * (1 + scale[b]) + shift[b] (idx None: all rows)."""
    if idx is not None and M == 0:
        return
    _check(lib().astraea_layernorm_modulate(_ptr(x), _ptr(idx), M, _ptr(scale), _ptr(shift), _ptr(y), B, N, D, eps, flags,
                                            _ptr(workspace), _stream(stream)))


def astraea_block_workspace_bytes(B: int, H: int, N: int, d: int, hidden: int) -> int:
    return int(lib().astraea_block_workspace_bytes(B, H, N, d, hidden))


def block_weights(tensors: dict, hidden: int) -> BlockWeights:
    """A BlockWeights struct from a dict of device tensors (missing / None entries become NULL).  The caller keeps the
    tensors alive."""
    w = BlockWeights()
    for n in BlockWeights.NAMES:
        t = tensors.get(n)
        setattr(w, n, None if t is None else t.data_ptr())
    w.hidden = hidden
    return w


def astraea_block_step(x, weights: BlockWeights, x_ref, lse_cache, n_skip, y_cache, text_k, text_v, N_text,
                       score, idx_sel, idx_rem, B, H, N, N_sel, d, k_keep, w_alpha=1.0, w_beta=1.0,
                       delta_mode=DELTA_MEAN_ABS, lse_mode=LSE_SUM_EXP, eps=1e-6, flags=0, workspace=None, stream=None) -> None:
    st = BlockState(x_ref.data_ptr(), lse_cache.data_ptr(), None if n_skip is None else n_skip.data_ptr(), y_cache.data_ptr())
    _check(lib().astraea_block_step(_ptr(x), ctypes.byref(weights), ctypes.byref(st), _ptr(text_k), _ptr(text_v), N_text,
                                    _ptr(score), _ptr(idx_sel), _ptr(idx_rem), B, H, N, N_sel, d, k_keep, w_alpha, w_beta,
                                    delta_mode, lse_mode, eps, flags, _ptr(workspace),
                                    workspace.numel() if workspace is not None else 0, _stream(stream)))


def astraea_step(x_cur, x_ref, lse_cache, n_skip, q, k, v, out_cache, score, idx_sel, idx_rem,
                 B, H, N, N_sel, d, k_keep, w_alpha=1.0, w_beta=1.0, delta_mode=DELTA_MEAN_ABS,
                 lse_mode=LSE_SUM_EXP, workspace=None, stream=None) -> None:
    _check(lib().astraea_step(_ptr(x_cur), _ptr(x_ref), _ptr(lse_cache), _ptr(n_skip), _ptr(q), _ptr(k), _ptr(v),
                              _ptr(out_cache), _ptr(score), _ptr(idx_sel), _ptr(idx_rem),
                              B, H, N, N_sel, d, k_keep, w_alpha, w_beta, delta_mode, lse_mode,
                              _ptr(workspace), workspace.numel() if workspace is not None else 0, _stream(stream)))


def astraea_selftest_wait(workspace, limit_us=200, gave_up=None, stream=None) -> None:
    """Runs the give-up path of the bounded device-side waits in isolation (see include/astraea.h)."""
    _check(lib().astraea_selftest_wait(_ptr(workspace), limit_us, _ptr(gave_up), _stream(stream)))


def astraea_poll_error(workspace, stream=None) -> None:
    _check(lib().astraea_poll_error(_ptr(workspace), _stream(stream)))


def astraea_timestep_level_budgets(k_keep, N_sel: int):
    """The all-or-nothing schedule of the Timestep-level variant made from a token-wise one (host policy)."""
    T = len(k_keep)
    src = (ctypes.c_int32 * T)(*[int(a) for a in k_keep])
    out = (ctypes.c_int32 * T)()
    rc = lib().astraea_timestep_level_budgets(src, T, N_sel, out)
    if rc < 0:
        raise AstraeaError(rc, lib().astraea_last_error().decode())
    return list(out)


class ModelSchedule:
    """A generation of T steps x L compute blocks as one CUDA graph (astraea_model_schedule_*).
    x_in: list of T device tensors; weights: list of L (dict of device tensors, hidden); states: list of L dicts with
    x_ref, lse_cache, n_skip, y_cache, score, idx_sel, idx_rem (idx_rem may be None); text_k / text_v: lists of L tensors."""

    def __init__(self, k_keep, x_in, weights, states, text_k, text_v, N_text, B, H, N, N_sel, d, w_alpha=1.0, w_beta=1.0,
                 delta_mode=DELTA_MEAN_ABS, lse_mode=LSE_SUM_EXP, eps=1e-6, variant=VARIANT_TOKEN_WISE, workspace=None):
        T, L = len(k_keep), len(weights)
        assert len(x_in) == T and len(states) == L and len(text_k) == L and len(text_v) == L
        self._keep = (list(x_in), weights, states, list(text_k), list(text_v), workspace)   # the graph keeps pointers
        kk = (ctypes.c_int32 * T)(*[int(a) for a in k_keep])
        xs = (ctypes.c_void_p * T)(*[t.data_ptr() for t in x_in])
        W = (BlockWeights * L)(*[block_weights(w, hidden) for (w, hidden) in weights])
        S = (BlockState * L)(*[BlockState(s["x_ref"].data_ptr(), s["lse_cache"].data_ptr(), s["n_skip"].data_ptr(), s["y_cache"].data_ptr())
                               for s in states])
        ptrs = lambda lst: (ctypes.c_void_p * L)(*[None if t is None else t.data_ptr() for t in lst])
        rem = None if all(s.get("idx_rem") is None for s in states) else ptrs([s.get("idx_rem") for s in states])
        self._h = ctypes.c_void_p()
        _check(lib().astraea_model_schedule_create(ctypes.byref(self._h), L, T, kk, xs, W, S, ptrs(text_k), ptrs(text_v), N_text,
                                                   ptrs([s["score"] for s in states]), ptrs([s["idx_sel"] for s in states]), rem,
                                                   B, H, N, N_sel, d, w_alpha, w_beta, delta_mode, lse_mode, eps, variant,
                                                   _ptr(workspace), workspace.numel() if workspace is not None else 0))

    def launch(self, stream=None) -> None:
        _check(lib().astraea_model_schedule_launch(self._h, _stream(stream)))

    def close(self) -> None:
        if getattr(self, "_h", None):
            lib().astraea_model_schedule_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Schedule:
    """T steps of one attention block as one CUDA graph (astraea_schedule_create / _launch / _destroy).
    x_cur, q, k, v are lists of T device tensors; the state tensors are those of astraea_step."""

    def __init__(self, k_keep, x_cur, q, k, v, x_ref, lse_cache, n_skip, out_cache, score, idx_sel, idx_rem,
                 B, H, N, N_sel, d, w_alpha=1.0, w_beta=1.0, delta_mode=DELTA_MEAN_ABS, lse_mode=LSE_SUM_EXP,
                 workspace=None):
        T = len(k_keep)
        assert len(x_cur) == len(q) == len(k) == len(v) == T
        # the graph keeps pointers: hold on to the tensors for as long as the schedule lives
        self._keep = (list(x_cur), list(q), list(k), list(v), x_ref, lse_cache, n_skip, out_cache, score, idx_sel, idx_rem, workspace)
        kk = (ctypes.c_int32 * T)(*[int(a) for a in k_keep])
        arrs = [(ctypes.c_void_p * T)(*[t.data_ptr() for t in lst]) for lst in (x_cur, q, k, v)]
        self._h = ctypes.c_void_p()
        _check(lib().astraea_schedule_create(ctypes.byref(self._h), T, kk, *arrs, _ptr(x_ref), _ptr(lse_cache), _ptr(n_skip),
                                             _ptr(out_cache), _ptr(score), _ptr(idx_sel), _ptr(idx_rem), B, H, N, N_sel, d,
                                             w_alpha, w_beta, delta_mode, lse_mode, _ptr(workspace),
                                             workspace.numel() if workspace is not None else 0))

    def launch(self, stream=None) -> None:
        _check(lib().astraea_schedule_launch(self._h, _stream(stream)))

    def close(self) -> None:
        if getattr(self, "_h", None):
            lib().astraea_schedule_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Session:
    """Host-buffer session (astraea_session_create / astraea_step_host / astraea_session_destroy)."""

    def __init__(self, B: int, H: int, N: int, N_sel: int, d: int):
        self._h = ctypes.c_void_p()
        _check(lib().astraea_session_create(ctypes.byref(self._h), B, H, N, N_sel, d))
        self.shape = (B, N, H, d)

    def step_host(self, x_cur, q, k, v, out, k_keep, w_alpha=1.0, w_beta=1.0,
                  delta_mode=DELTA_MEAN_ABS, lse_mode=LSE_SUM_EXP) -> None:
        """All five tensors are HOST (ideally pinned) bf16 tensors of shape [B,N,H*d]."""
        for t in (x_cur, q, k, v, out):
            assert not t.is_cuda and t.is_contiguous()
        _check(lib().astraea_step_host(self._h, _ptr(x_cur), _ptr(q), _ptr(k), _ptr(v), _ptr(out), k_keep,
                                       w_alpha, w_beta, delta_mode, lse_mode))

    def last_h2d_bytes(self) -> int:
        """Host-to-device bytes of the last step (a pinned q contributes only its selected rows)."""
        return int(lib().astraea_session_last_h2d_bytes(self._h))

    def close(self) -> None:
        if self._h:
            lib().astraea_session_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def bhnd_strides(N: int, H: int, d: int):
    """(batch, head, token) element strides of a contiguous [B, N, H, d] tensor."""
    return (N * H * d, d, H * d)
