"""Host logic of the attention launch schedule (astraea_sparse_attn_plan): no GPU needed, the SM count falls back to 148."""
import pytest

from paper_2506_05096_b200 import binding as A, synth


def _plan(B, H, N, M, d, **kw):
    return A.astraea_sparse_attn_plan(B, H, N, M, d, **kw)


def test_plans_of_the_workloads():
    w = synth.WORKLOADS
    cog, osr, sw, hy = w["cogvideox"], w["opensora"], w["sweep"], w["hunyuan"]
    # 832 units = 5.6 rounds: the last 92 are split three ways
    assert _plan(osr.B, osr.H, osr.N, osr.M_of(400), osr.d) == {"small_ctas": False, "split_units": 92, "split": 3}
    # 912 units = 6.2 rounds: the last 24, eight ways
    assert _plan(cog.B, cog.H, cog.N, cog.M_of(250), cog.d) == {"small_ctas": False, "split_units": 24, "split": 8}
    # many rounds: whole
    for ww, th in ((cog, 1000), (sw, 500), (sw, 1000), (hy, 600), (hy, 300)):
        assert _plan(ww.B, ww.H, ww.N, ww.M_of(th), ww.d) == {"small_ctas": False, "split_units": 0, "split": 1}, (ww.name, th)
    # the tiny config has four key tiles: nothing to split
    t = w["tiny"]
    assert _plan(t.B, t.H, t.N, t.M_of(500), t.d)["split"] == 1


@pytest.mark.parametrize("d", [64, 72, 128])
def test_plan_invariants(d):
    for (B, H, N) in [(1, 3, 2100), (2, 16, 16384), (1, 48, 17776), (1, 24, 65536), (1, 2, 1023), (1, 1, 4096)]:
        ws_full = A.astraea_workspace_bytes(A.OP_SPARSE_ATTN, B, H, N, N, d)
        key_tiles = (N + 63) // 64
        for M in sorted({1, 127, 128, 129, 255, 257, N // 7, N // 3, N // 2, N - 1, N}):
            if M <= 0:
                continue
            p = _plan(B, H, N, M, d)
            units = B * H * ((M + 255) // 256)
            assert 0 <= p["split_units"] <= min(units, 147) and 1 <= p["split"] <= 8
            assert (p["split"] == 1) == (p["split_units"] == 0)
            if p["split"] > 1:
                assert not p["small_ctas"]
                assert key_tiles // p["split"] >= 16                           # a share keeps at least 16 key tiles
                assert p["split_units"] * p["split"] <= 296
                assert p["split_units"] == units % 148
            # the size for the largest M serves every smaller M
            assert A.astraea_workspace_bytes(A.OP_SPARSE_ATTN, B, H, N, M, d) <= ws_full
            assert _plan(B, H, N, M, d, workspace_bytes=ws_full) == p
            # no room, or the flag: every CTA runs over all keys
            assert _plan(B, H, N, M, d, workspace_bytes=256)["split"] == 1
            assert _plan(B, H, N, M, d, flags=A.ATTN_WHOLE_KEYS)["split"] == 1
            assert _plan(B, H, N, M, d, flags=A.ATTN_SMALL_CTAS)["small_ctas"] == (d != 128)


def test_plan_rejects_bad_arguments():
    with pytest.raises(A.AstraeaError) as e:
        _plan(1, 2, 100, 101, 64)
    assert e.value.code == A.ERR_INVALID_ARG
    with pytest.raises(A.AstraeaError) as e:
        _plan(1, 2, 100, 10, 96)
    assert e.value.code == A.ERR_UNSUPPORTED
