"""Seeded synthetic inputs shaped like the paper's video workloads.

This module only draws random numbers and rounds them to bf16.  It holds none of
the method's arithmetic (no score, no selection, no attention), so both the CUDA
path's tests and the CPU oracle's tests can take their inputs from here without
sharing any of the computation under test.

Token order is [video tokens 0..N_v) | always-kept text tokens N_v..N).
Hidden states and the cached attention output are [B, N, D] row-major with
D = H*d and head h in columns [h*d, (h+1)*d), i.e. [B, N, H, d].  bf16 tensors
are carried as uint16 bit patterns so that numpy (which has no bf16) can hold
them; `bf16_to_f64` upcasts them exactly.

Draw order for one step (fixed, so a seed names one input set):
    norms (only when `lognormal_sigma` > 0), x_ref, eps, q, k, v, cache, lse_z, n_skip
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np


# --------------------------------------------------------------------------- bf16
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns uint16 bits."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    rounding = ((u >> 16) & 1) + np.uint32(0x7FFF)
    out = ((u + rounding) >> 16).astype(np.uint16)
    nan = np.isnan(a)
    if nan.any():
        out[nan] = 0x7FC0
    return out


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact upcast of bf16 bit patterns to float64."""
    return bf16_bits_to_f32(np.ascontiguousarray(bits)).astype(np.float64)


def _normal_bf16(rng: np.random.Generator, shape, scale=None, chunk_rows=4096) -> np.ndarray:
    """N(0,1) samples (optionally scaled per leading-row) rounded to bf16 bits,
    drawn in row chunks to bound the float32 transient."""
    out = np.empty(shape, dtype=np.uint16)
    flat = out.reshape(-1, shape[-1]) if len(shape) > 1 else out.reshape(1, -1)
    rows = flat.shape[0]
    sc = None if scale is None else np.asarray(scale, dtype=np.float32).reshape(-1, 1)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        blk = rng.standard_normal((r1 - r0, flat.shape[1]), dtype=np.float32)
        if sc is not None:
            blk *= sc[r0:r1]
        flat[r0:r1] = f32_to_bf16_bits(blk)
    return out


# --------------------------------------------------------------------- workloads
@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    d: int
    N_v: int            # selectable (video) tokens
    N_t: int = 0        # always-kept (text) tokens appended after the video tokens
    thetas_permille: tuple = (500,)
    drift_sigma: float = 0.05      # x_cur = x_ref + drift_sigma * eps  (0 => x_cur independent N(0,1))
    lognormal_sigma: float = 0.0   # per-token norm ~ LogNormal(0, sigma) applied to x_ref, eps, q, k, v rows
    n_skip_max: int = 3            # n_skip ~ U{0..n_skip_max}
    grid: tuple = field(default=())

    @property
    def N(self) -> int:
        return self.N_v + self.N_t

    @property
    def D(self) -> int:
        return self.H * self.d

    def k_of(self, theta_permille: int) -> int:
        return (self.N_v * int(theta_permille)) // 1000

    def M_of(self, theta_permille: int) -> int:
        return self.k_of(theta_permille) + self.N_t


WORKLOADS = {
    "tiny": Workload("tiny", B=1, H=2, d=64, N_v=256, N_t=0, thetas_permille=(500,),
                     drift_sigma=0.0, n_skip_max=0, grid=(4, 8, 8)),
    "cogvideox": Workload("cogvideox", B=1, H=48, d=64, N_v=17550, N_t=226,
                          thetas_permille=(1000, 500, 250), grid=(13, 30, 45)),
    "opensora": Workload("opensora", B=2, H=16, d=72, N_v=16384, N_t=0,
                         thetas_permille=(400,), lognormal_sigma=0.5, grid=(16, 32, 32)),
    "hunyuan": Workload("hunyuan", B=1, H=24, d=128, N_v=118800, N_t=0,
                        thetas_permille=(600, 300), grid=(33, 45, 80)),
    "sweep": Workload("sweep", B=1, H=24, d=128, N_v=65536, N_t=0,
                      thetas_permille=tuple(range(50, 1001, 50))),
}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some sizes replaced (reduced shapes for tests)."""
    d = {f: getattr(w, f) for f in w.__dataclass_fields__}
    d.update(kw)
    return Workload(**d)


def make_step_inputs(w: Workload, seed: int = 0, parts=None) -> dict:
    """One denoising step's inputs for one attention block.

    Returns uint16 (bf16 bits) arrays x_ref, x_cur [B,N,D]; q, k, v, cache [B,N,H,d];
    float32 lse [B,H,N] (log domain, the value an attention pass over N(0,1) logits
    would leave: ln N + 0.5 + 0.25 z); int32 n_skip [B,N_v].
    `parts` restricts which tensors are materialised (the draws still happen in
    the fixed order so that the others keep their values).
    """
    rng = np.random.default_rng(seed)
    B, N, H, d, D = w.B, w.N, w.H, w.d, w.D
    want = (lambda name: parts is None or name in parts)
    out = {}
    norms = None
    if w.lognormal_sigma > 0:
        norms = rng.lognormal(0.0, w.lognormal_sigma, size=(B * N,)).astype(np.float32)
        out["norms"] = norms.reshape(B, N)

    def draw(shape, scale):
        return _normal_bf16(rng, shape, scale)

    # x_ref, eps
    x_ref = draw((B * N, D), norms)
    if w.drift_sigma > 0:
        x_cur = np.empty_like(x_ref)
        sig = np.float32(w.drift_sigma)
        for r0 in range(0, B * N, 4096):
            r1 = min(B * N, r0 + 4096)
            eps = rng.standard_normal((r1 - r0, D), dtype=np.float32)
            if norms is not None:
                eps *= norms[r0:r1, None]
            x_cur[r0:r1] = f32_to_bf16_bits(bf16_bits_to_f32(x_ref[r0:r1]) + sig * eps)
    else:
        x_cur = draw((B * N, D), norms)
    if want("x_ref"):
        out["x_ref"] = x_ref.reshape(B, N, D)
    if want("x_cur"):
        out["x_cur"] = x_cur.reshape(B, N, D)
    del x_ref, x_cur
    for name in ("q", "k", "v"):
        t = draw((B * N, D), norms)
        if want(name):
            out[name] = t.reshape(B, N, H, d)
        del t
    t = draw((B * N, D), None)
    if want("cache"):
        out["cache"] = t.reshape(B, N, H, d)
    del t
    z = rng.standard_normal((B, H, N), dtype=np.float32)
    out["lse"] = (np.float32(math.log(N) + 0.5) + np.float32(0.25) * z).astype(np.float32)
    if w.n_skip_max > 0:
        out["n_skip"] = rng.integers(0, w.n_skip_max + 1, size=(B, w.N_v), dtype=np.int32)
    else:
        out["n_skip"] = np.zeros((B, w.N_v), dtype=np.int32)
    return out


def drift_step(prev_bits: np.ndarray, seed: int, sigma: float, preserve_variance: bool) -> np.ndarray:
    """Next-step latent: prev + sigma*eps (optionally rescaled to keep unit variance), bf16 bits."""
    rng = np.random.default_rng(seed)
    flat = prev_bits.reshape(-1, prev_bits.shape[-1])
    out = np.empty_like(flat)
    s = np.float32(sigma)
    inv = np.float32(1.0 / math.sqrt(1.0 + sigma * sigma)) if preserve_variance else np.float32(1.0)
    for r0 in range(0, flat.shape[0], 4096):
        r1 = min(flat.shape[0], r0 + 4096)
        eps = rng.standard_normal((r1 - r0, flat.shape[1]), dtype=np.float32)
        out[r0:r1] = f32_to_bf16_bits((bf16_bits_to_f32(flat[r0:r1]) + s * eps) * inv)
    return out.reshape(prev_bits.shape)


def integer_scores(B: int, n: int, seed: int, levels: int = 64) -> np.ndarray:
    """Integer-valued float32 scores with many exact ties (for bit-exact selection tests)."""
    rng = np.random.default_rng(seed)
    return rng.integers(0, levels, size=(B, n)).astype(np.float32)
