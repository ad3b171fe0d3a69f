"""The C-ABI library loads and exports every symbol include/astraea.h declares; host-side
argument validation answers before anything is launched (no GPU needed)."""
import ctypes
import os
import re

import pytest

from paper_2506_05096_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    build.build_library()
    return binding.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "astraea.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(astraea_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = _declared()
    assert len(names) >= 13
    for n in names:
        assert hasattr(L, n), n
    assert sorted(binding.EXPORTS) == names


def test_version_and_budget(L):
    assert b"sm_100a" in L.astraea_version()
    assert binding.astraea_budget_to_k(17550, 250) == 4387
    assert binding.astraea_budget_to_k(118800, 600) == 71280
    assert L.astraea_budget_to_k(10, 1001) == binding.ERR_INVALID_ARG
    assert L.astraea_workspace_bytes(99, 1, 1, 1, 1, 64) == 0
    assert L.astraea_workspace_bytes(binding.OP_STEP, 1, 24, 118800, 71280, 128) >= 512


def test_argument_errors_are_reported_before_any_launch(L):
    p = ctypes.c_void_p(0x1000)          # never dereferenced: validation fails first
    rc = L.astraea_score(p, p, None, None, p, 1, 16, 17, 64, 1, 1.0, 1.0, 0, 0, None)
    assert rc == binding.ERR_INVALID_ARG and b"N_sel" in L.astraea_last_error()
    rc = L.astraea_score(p, p, None, None, p, 1, 16, 16, 60, 1, 1.0, 1.0, 0, 0, None)
    assert rc == binding.ERR_INVALID_ARG
    rc = L.astraea_score(p, p, None, None, p, 1, 16, 16, 64, 1, 1.0, 1.0, 7, 0, None)
    assert rc == binding.ERR_UNSUPPORTED
    rc = L.astraea_score(None, p, None, None, p, 1, 16, 16, 64, 1, 1.0, 1.0, 0, 0, None)
    assert rc == binding.ERR_INVALID_ARG
    rc = L.astraea_select(p, 1, 16, 17, 0, p, None, None, p, 1024, None)
    assert rc == binding.ERR_INVALID_ARG and b"k=17" in L.astraea_last_error()
    rc = L.astraea_select(p, 1, 16, 4, 0, p, None, None, None, 0, None)
    assert rc == binding.ERR_WORKSPACE_TOO_SMALL
    s = (64 * 16, 64, 64)
    args = lambda d, kv=None, ws=p, wsb=4096, flags=0, qsn=64: (p, p, p, s[0], s[1], qsn, *s, *s, None, 16, kv, 0, p, None,
                                                               1, 1, 16, d, 0.0, flags, ws, wsb, None)
    assert L.astraea_sparse_attn(*args(96)) == binding.ERR_UNSUPPORTED
    assert L.astraea_sparse_attn(*args(64, kv=p)) == binding.ERR_INVALID_ARG      # kv_idx with M_kv = 0
    assert L.astraea_sparse_attn(*args(64, flags=8)) == binding.ERR_UNSUPPORTED
    assert L.astraea_sparse_attn(*args(64, wsb=8)) == binding.ERR_WORKSPACE_TOO_SMALL
    assert L.astraea_sparse_attn(*args(64, qsn=60)) == binding.ERR_INVALID_ARG
    assert L.astraea_sparse_attn(*args(64, ws=ctypes.c_void_p(0x1010))) == binding.ERR_INVALID_ARG
    assert L.astraea_scatter_reuse(p, p, p, 1, 16, 4, 12, 0, None, None) == binding.ERR_INVALID_ARG
    assert L.astraea_scatter_reuse(p, p, p, 1, 16, 17, 16, 0, None, None) == binding.ERR_INVALID_ARG
    assert L.astraea_scatter_reuse(p, p, p, 1, 16, 0, 16, 0, None, None) == binding.OK     # M = 0: nothing to do
    assert L.astraea_poll_error(None, None) == binding.ERR_INVALID_ARG


def test_argument_errors_of_the_next_layer_entry_points(L):
    p = ctypes.c_void_p(0x1000)
    lin = lambda K=64, N_out=64, M=4, flags=0, ws=p, wsb=4096, idx=p, x=p: L.astraea_gathered_linear(
        x, idx, M, p, None, p, 1, 16, K, N_out, flags, ws, wsb, None)
    assert lin(K=60) == binding.ERR_INVALID_ARG and b"multiple of 64" in L.astraea_last_error()
    assert lin(N_out=12) == binding.ERR_INVALID_ARG
    assert lin(M=17) == binding.ERR_INVALID_ARG
    assert lin(flags=64) == binding.ERR_UNSUPPORTED
    assert lin(flags=binding.LINEAR_COMPACT_OUT, idx=None) == binding.ERR_INVALID_ARG     # compact rows need a list
    assert lin(wsb=8) == binding.ERR_WORKSPACE_TOO_SMALL
    assert lin(ws=ctypes.c_void_p(0x1010)) == binding.ERR_INVALID_ARG
    assert lin(x=None) == binding.ERR_INVALID_ARG
    assert lin(M=0) == binding.OK                                                         # an empty list: nothing to do
    s = (64 * 16, 64, 64)
    cross = lambda N_kv=8, d=64: L.astraea_sparse_cross_attn(p, p, p, *s, *s, *s, None, 16, p, None, 1, 1, 16, N_kv, d, 0.0, 0,
                                                             p, 4096, None)
    assert cross(N_kv=0) == binding.ERR_INVALID_ARG and b"N_kv" in L.astraea_last_error()
    assert cross(d=80) == binding.ERR_UNSUPPORTED and b"astraea_sparse_cross_attn" in L.astraea_last_error()
    h = ctypes.c_void_p()
    kk = (ctypes.c_int32 * 2)(4, 99)
    arr = (ctypes.c_void_p * 2)(0x1000, 0x1000)
    sched = lambda T=2, keep=kk, wsb=1 << 20: L.astraea_schedule_create(ctypes.byref(h), T, keep, arr, arr, arr, arr, p, p, p, p, p, p, None,
                                                                         1, 1, 16, 16, 64, 1.0, 1.0, 0, 0, p, wsb)
    assert sched() == binding.ERR_INVALID_ARG and b"k_keep[1]=99" in L.astraea_last_error() and not h.value
    assert sched(T=0) == binding.ERR_INVALID_ARG
    assert sched(keep=(ctypes.c_int32 * 2)(4, 4), wsb=8) == binding.ERR_WORKSPACE_TOO_SMALL
    assert L.astraea_schedule_launch(None, None) == binding.ERR_INVALID_ARG
    L.astraea_schedule_destroy(None)                                                       # a null handle is ignored


def test_timestep_level_policy_matches_the_oracles(L, oracle):
    import numpy as np
    for seed, T, n in ((0, 12, 100), (1, 50, 17550), (2, 7, 1), (3, 30, 118800)):
        rng = np.random.default_rng(seed)
        k = [n] + [int(v) for v in rng.integers(0, n + 1, T - 1)]
        assert binding.astraea_timestep_level_budgets(k, n) == oracle.timestep_level_budgets(k, n)
    with pytest.raises(binding.AstraeaError):
        binding.astraea_timestep_level_budgets([5, 11], 10)
