#!/usr/bin/env python
"""Benchmark of the hot path (score -> select -> sparse attention with fused scatter ->
reference refresh) on synthetic latents shaped like the paper's video workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W]
    python bench.py --impl reference ...       # the CPU oracle, timed on the host cores

One "step" is one pass of the whole path for one attention block at one keep-ratio.  The headline
(`value`, `ms_per_step`, `roofline`, `e2e`, `cpu_baseline`) is the keep-ratio-sweep workload (24 heads,
head_dim 128, 65536 tokens) at keep-ratio 0.5: `value` is the attention's algorithmic FLOPs (4*B*H*M*N*d)
per second of whole-step time with the inputs resident in HBM; `e2e` is the same through astraea_step_host
with pinned HOST buffers (host<->device copies inside the timed region).  The same line also carries
`keep_ratio_sweep` (all twenty keep-ratios 0.05 .. 1.0 over ten seeds) and `workloads`: the CogVideoX-, Open-Sora-
and HunyuanVideo-shaped configurations (the last one as 50 consecutive steps of a drifting latent after a dense
step 0) and the tiny one, each with per-kernel times and roofline fractions, and `worst_attn_frac` /
`worst_hbm_frac` over all of them.  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2506_05096_b200 import accounting, replicas, synth  # noqa: E402

METRIC = "sparse_attn_effective_tflops"
UNIT = "TFLOP/s"
HEADLINE, HEADLINE_THETA = "sweep", 500

NOMINAL_BF16_TFLOPS, NOMINAL_HBM_GBS = 2250.0, 8000.0     # the part's nominal dense bf16 and HBM3e figures, for context
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the attention kernel, from the ncu captures summarised
# in profiles/ (workload -> theta_permille -> (bytes, file)); None where not captured at that size.
NCU_TRAFFIC = {
    "cogvideox": {500: (276493056 + 47539200, "profiles/sparse_attn_d64_cogvideox.md")},
    "opensora": {400: (183320320 + 24948736, "profiles/sparse_attn_d72_opensora.md")},
    "sweep": {250: (1142801000 + 112186368, "profiles/sparse_attn_d128_sweep.md")},
}
# The headline launch (sweep shape, keep-ratio 0.5) holds too much for a multi-pass capture: its traffic is the
# keep-ratio-0.25 capture scaled by the compulsory bytes (the traffic is Q and output rows of M tokens plus K and V of
# N tokens, each read through L2 at the same hit rate)
NCU_TRAFFIC_SCALED_FROM = {"sweep": 250}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def mark(self) -> int:
        return len(self.rows)

    def summary(self, lo: int = 0, hi=None) -> dict:
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows[lo:hi]:
            try:
                sm.append(float(r[0]))
                mx = float(r[1])
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}

    def stop(self):
        if self.proc:
            self.proc.terminate()
            self.t.join(timeout=2)


# ------------------------------------------------------------------ the oracle legs
class OracleSample:
    """The CPU oracle on a bounded sample of a workload: score and select at full size, attention for `rows`
    sampled selected queries x `heads` heads against all keys.  The inputs are drawn once."""

    def __init__(self, w, theta, heads=None, seed=0):
        from oracle import astraea_oracle as oracle
        oracle.build()
        self.oracle, self.w, self.theta = oracle, w, theta
        inp = synth.make_step_inputs(w, seed, parts=("x_ref", "x_cur", "q", "k", "v"))
        f = synth.bf16_to_f64
        self.hs = w.H if heads is None else min(heads, w.H)
        self.x_cur, self.x_ref = f(inp["x_cur"]), f(inp["x_ref"])
        self.lse = (inp["lse"] - np.float32(math.log(w.N))).astype(np.float64)
        self.n_skip = inp["n_skip"]
        self.q, self.k, self.v = (f(np.ascontiguousarray(inp[n][:, :, :self.hs])) for n in ("q", "k", "v"))

    def run(self, rows, seed=0):
        """Returns (effective TFLOP/s of the attention sample, seconds, threads, description)."""
        w, o = self.w, self.oracle
        k_keep = w.k_of(self.theta)
        t0 = time.perf_counter()
        s = o.score(self.x_cur, self.x_ref, self.lse, self.n_skip, n_sel=w.N_v)
        sel, _, _ = o.select(s.astype(np.float32), k_keep, w.N_t, self.n_skip)
        t1 = time.perf_counter()
        rng = np.random.default_rng(seed)
        r = min(rows, sel.shape[1])
        pick = np.stack([np.sort(rng.choice(sel[b], r, replace=False)) for b in range(w.B)]).astype(np.int32)
        o.sparse_attn(self.q, self.k, self.v, q_idx=pick)
        t2 = time.perf_counter()
        flops = accounting.attn_flops(w.B, self.hs, r, w.N, w.d)
        desc = ("oracle fp64: score+select at full size (%.2f s, not in the rate); attention of %d sampled selected "
                "rows x %d of %d heads x all %d keys (%.2f s)" % (t1 - t0, r, self.hs, w.H, w.N, t2 - t1))
        return flops / (t2 - t1) / 1e12, (t2 - t1), o.num_threads(), desc


def config_of(w, theta, world):
    """The `config` object of the line: identical keys and values in both arms."""
    k_keep = w.k_of(theta)
    return {"workload": w.name, "theta_permille": theta, "B": w.B, "H": w.H, "d": w.d, "N": w.N, "N_sel": w.N_v,
            "k_keep": k_keep, "M": k_keep + w.N_t, "parallelism": "replicas only (%d)" % world,
            "l2": "two alternating input sets, %.0f MB touched per step > 126 MB L2" % ((6 * w.B * w.N * w.D * 2) / 1e6)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = synth.WORKLOADS[args.workload]
    theta = args.theta
    sample = OracleSample(w, theta, heads=args.ref_heads)
    vals, secs = [], []
    desc, threads = "", 1
    for i in range(args.warmup + args.steps):
        v, s, threads, desc = sample.run(args.ref_rows, seed=i)
        if i >= args.warmup:
            vals.append(v)
            secs.append(s)
    value = float(np.mean(vals))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(secs)),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(w, theta, int(os.environ.get("WORLD_SIZE", "1"))),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------- the CUDA leg
class Block:
    """Device-resident inputs and state of one attention block of a workload, generated on the device with a seeded
    torch generator (inputs only: no arithmetic of the method), and the four calls of a step."""

    def __init__(self, torch, A, w, seed, sets=2):
        self.torch, self.A, self.w = torch, A, w
        B, N, D, H = w.B, w.N, w.D, w.H
        g = torch.Generator(device="cuda").manual_seed(1234 + seed)
        norms = None
        if w.lognormal_sigma > 0:
            norms = torch.exp(w.lognormal_sigma * torch.randn(B, N, 1, device="cuda", generator=g))

        def normal(scale=True):
            t = torch.randn(B, N, D, device="cuda", generator=g, dtype=torch.bfloat16)
            if norms is not None and scale:
                t = (t.float() * norms).to(torch.bfloat16)
            return t

        self.g = g
        self.x_ref = normal()
        self.sets = []
        prev = None
        for _ in range(sets):
            base = self.x_ref if prev is None else prev["x_cur"]
            s = {"x_cur": self.drift(base, w.drift_sigma if w.drift_sigma > 0 else 1.0, False, norms)}
            for n in ("q", "k", "v"):
                s[n] = normal() if prev is None else self.drift(prev[n], 0.05, True, None)
            self.sets.append(s)
            prev = s
        self.out = normal(scale=False)
        self.lse = (math.log(N) + 0.5 + 0.25 * torch.randn(B, H, N, device="cuda", generator=g)).float()
        self.n_skip = torch.randint(0, w.n_skip_max + 1, (B, w.N_v), device="cuda", generator=g, dtype=torch.int32)
        self.score = torch.empty(B, w.N_v, device="cuda")
        self.idx_sel = torch.empty(B, N, dtype=torch.int32, device="cuda")
        self.idx_rem = torch.empty(B, w.N_v + 1, dtype=torch.int32, device="cuda")
        self.ws = A.new_workspace(A.OP_STEP, B, H, N, N, w.d)
        self.ws_sel = A.new_workspace(A.OP_SELECT, B, 0, w.N_v, 0, 0)
        self.strides = A.bhnd_strides(N, H, w.d)
        # the scale of exp(lse) ~ N does not matter for timing; keep the scores of order one
        self.w_alpha = float(1.0 / N)

    def drift(self, t, sigma, preserve, norms):
        """t + sigma * eps (variance-preserving for q, k, v), in row chunks to bound the fp32 transient."""
        torch = self.torch
        out = torch.empty_like(t)
        flat_in, flat_out = t.view(-1, t.shape[-1]), out.view(-1, t.shape[-1])
        nf = None if norms is None else norms.view(-1, 1)
        inv = 1.0 / math.sqrt(1.0 + sigma * sigma) if preserve else 1.0
        for r0 in range(0, flat_in.shape[0], 16384):
            r1 = min(flat_in.shape[0], r0 + 16384)
            eps = torch.randn(r1 - r0, t.shape[-1], device="cuda", generator=self.g)
            if nf is not None:
                eps *= nf[r0:r1]
            flat_out[r0:r1] = ((flat_in[r0:r1].float() + sigma * eps) * inv).to(torch.bfloat16)
        return out

    def step(self, t, k_keep, ev=None, pair_ev=None):
        """The four calls of a step.  ev: five events recorded around every call; pair_ev: two events recorded before
        the score and after the selection only (the selection is launched as a programmatic dependent of the
        kernel before it, which an event record between the two would undo)."""
        A, w = self.A, self.w
        s = self.sets[t % len(self.sets)]
        B, N, H, d, D, N_sel, n_always = w.B, w.N, w.H, w.d, w.D, w.N_v, w.N_t
        M = k_keep + n_always
        if ev:
            ev[0].record()
        if pair_ev:
            pair_ev[0].record()
        A.astraea_score(s["x_cur"], self.x_ref, self.lse, self.n_skip, self.score, B, N, N_sel, D, H, self.w_alpha, 1.0)
        if ev:
            ev[1].record()
        A.astraea_select(self.score, B, N_sel, k_keep, n_always, self.idx_sel, self.idx_rem, self.n_skip, self.ws_sel)
        if ev:
            ev[2].record()
        if pair_ev:
            pair_ev[1].record()
        A.astraea_sparse_attn(s["q"], s["k"], s["v"], self.strides, self.strides, self.strides, self.idx_sel, M, self.out,
                              self.lse, B, H, N, d, workspace=self.ws)
        if ev:
            ev[3].record()
        A.astraea_scatter_reuse(self.x_ref, s["x_cur"], self.idx_sel, B, N, M, D, A.SCATTER_SRC_FULL, workspace=self.ws)
        if ev:
            ev[4].record()

    def timed(self, k_keep, steps, warmup, barrier, t_base=1):
        """`steps` consecutive steps after `warmup` untimed ones; returns (total ms, median ms of each of the four calls
        over the steps, all the per-step times)."""
        torch = self.torch
        for t in range(warmup):
            self.step(t_base + t, k_keep)
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(steps)]
        barrier()
        for t in range(steps):
            self.step(t_base + warmup + t, k_keep, evs[t])
        barrier()
        total_ms = evs[0][0].elapsed_time(evs[-1][4])
        parts = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(4)] for e in evs])
        return total_ms, np.median(parts, axis=0), parts

    def timed_plain_copy(self, k_keep, steps=10, t_base=1):
        """The yardstick for the refresh of x_ref on the small shapes: torch's contiguous device-to-device copy of as
        many bytes (M rows of the OTHER input set, which the step has not just read), launched right behind the step's
        own calls and timed the same way."""
        torch, w = self.torch, self.w
        M = k_keep + w.N_t
        if M == 0:
            return None
        n = w.B * M * w.D
        dst = torch.empty(n, dtype=torch.bfloat16, device="cuda")
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps)]
        self.step(t_base, k_keep)
        for t in range(steps):
            self.step(t_base + 1 + t, k_keep)
            src = self.sets[(t_base + 2 + t) % len(self.sets)]["x_cur"].view(-1)[:n]
            evs[t][0].record()
            dst.copy_(src)
            evs[t][1].record()
        torch.cuda.synchronize()
        return float(np.mean([e[0].elapsed_time(e[1]) for e in evs]))

    def timed_pair(self, k_keep, steps=10, t_base=1):
        """Median time of score + select launched back to back (whole steps run; events around the pair only)."""
        torch = self.torch
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(steps)]
        self.step(t_base, k_keep)
        for t in range(steps):
            self.step(t_base + 1 + t, k_keep, pair_ev=evs[t])
        torch.cuda.synchronize()
        return float(np.median([e[0].elapsed_time(e[1]) for e in evs]))


def add_copy_yardstick(kernels, copy_ms):
    """Next to the refresh of x_ref: what torch's plain copy of as many bytes takes in the same place."""
    if copy_ms:
        e = kernels["scatter_reuse(x_ref)"]
        e["torch_copy_of_as_many_bytes_ms"] = copy_ms
        e["time_vs_torch_copy"] = e["ms"] / copy_ms


def cool_down(torch, seconds=0.5):
    """A pause between independent short measurements, so that each starts from the same power state (the power cap
    averages over a window: a leg measured right behind another one inherits its lowered clock)."""
    torch.cuda.synchronize()
    time.sleep(seconds)


def attn_schedule(w, theta):
    """What the attention launch of this workload looks like (astraea_sparse_attn_plan): CTA shape, and how many CTAs
    of the last, partial round were replaced by how many key shares each (merged by one more kernel launch)."""
    from paper_2506_05096_b200 import binding as A
    M = w.k_of(theta) + w.N_t
    plan = A.astraea_sparse_attn_plan(w.B, w.H, w.N, M, w.d) if M > 0 else {"small_ctas": False, "split_units": 0, "split": 1}
    plan["launches"] = 2 if plan["split"] > 1 else 1
    return plan


def kernel_report(w, theta, parts, peaks, long_region=False, pair_ms=None, all_parts=None, stat="median"):
    """Per-kernel figures of one step: times (the median over the timed steps; with all_parts also the minimum and the
    number of launches), achieved rates and fractions of the measured and nominal peaks."""
    B, N, H, d, D, N_sel = w.B, w.N, w.H, w.d, w.D, w.N_v
    k_keep = w.k_of(theta)
    M = k_keep + w.N_t
    hbm = peaks["hbm_gbs"]
    sb = accounting.score_bytes(B, N, N_sel, D, H)
    cb = accounting.scatter_bytes(B, M, D)
    selb = accounting.select_bytes(B, N_sel, k_keep)
    flops = accounting.attn_flops(B, H, M, N, d)
    attn_ms = float(parts[2])
    achieved = flops / (attn_ms * 1e-3) / 1e12 if attn_ms > 0 else 0.0

    def hbm_entry(nbytes, ms):
        gbs = nbytes / ms / 1e6 if ms > 0 else 0.0
        return {"ms": float(ms), "GB/s": gbs, "frac_hbm": gbs / hbm, "frac_hbm_nominal": gbs / NOMINAL_HBM_GBS}

    traffic = NCU_TRAFFIC.get(w.name, {}).get(theta)
    if traffic is None and w.name in NCU_TRAFFIC_SCALED_FROM:
        th0 = NCU_TRAFFIC_SCALED_FROM[w.name]
        b0, src = NCU_TRAFFIC[w.name][th0]
        ratio = accounting.attn_min_bytes(B, H, M, N, d) / accounting.attn_min_bytes(B, H, w.M_of(th0), N, d)
        traffic = (int(b0 * ratio), "%s (keep-ratio %.2f capture x %.3f = ratio of the compulsory bytes)" % (src, th0 / 1000, ratio))
    roofline = {"bound": "tensor", "kernel": "sparse_attn_kernel<%d>" % d, "achieved": achieved,
                "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                "peak_kind": "%s burst bf16" % peaks["source"],
                "frac_nominal": achieved / NOMINAL_BF16_TFLOPS,
                "traffic": traffic[0] if traffic else None, "traffic_from": traffic[1] if traffic else None,
                "kernel_ms": attn_ms, "min_bytes": accounting.attn_min_bytes(B, H, M, N, d),
                "dense_equivalent_tflops(speed-up credit, not a roofline figure)":
                    accounting.attn_flops(B, H, N, N, d) / (attn_ms * 1e-3) / 1e12 if attn_ms > 0 else None}
    if long_region and peaks.get("bf16_tflops_sustained"):
        roofline["frac_of_sustained_peak"] = achieved / peaks["bf16_tflops_sustained"]
    kernels = {"score": hbm_entry(sb, parts[0]),
               "select": {"ms": float(parts[1]), "GB/s": selb / parts[1] / 1e6 if parts[1] > 0 else 0.0, "note": "latency-bound"},
               # as a pair: the two calls back to back, events around the pair only (the figure the 70 % target is read on);
               # "sum of the two alone" adds the two isolated times, each with its own launch latency
               "score+select": {**hbm_entry(sb + selb, pair_ms if pair_ms is not None else parts[0] + parts[1]),
                                "how": "pair, back to back" if pair_ms is not None else "sum of the two alone",
                                "sum_of_the_two_alone_ms": float(parts[0] + parts[1])},
               "sparse_attn": {"ms": attn_ms, "TFLOP/s": achieved, "schedule": attn_schedule(w, theta)},
               "scatter_reuse(x_ref)": hbm_entry(cb, parts[3])}
    if all_parts is not None:
        for i, n in enumerate(("score", "select", "sparse_attn", "scatter_reuse(x_ref)")):
            kernels[n]["min_ms"] = float(np.min(all_parts[:, i]))
            kernels[n]["launches_timed"] = int(all_parts.shape[0])
            kernels[n]["of"] = stat
    return roofline, kernels


def block_leg(torch, A, w, thetas, peaks, sampler, hidden_mult=4, N_text=226, reps=5):
    """The whole compute block (astraea_block_step: score, select, K/V projections of all rows, query projection,
    self-attention, output projection, cross-attention and MLP on the selected rows) at several keep-ratios, and its
    layers one by one at the first of them.  Keep-ratio 1000 is the dense block."""
    B, N, H, d, D, N_sel, n_always = w.B, w.N, w.H, w.d, w.D, w.N_v, w.N_t
    hidden = hidden_mult * D
    g = torch.Generator(device="cuda").manual_seed(99)
    rn = lambda *s, scale=1.0: (scale * torch.randn(*s, device="cuda", generator=g)).to(torch.bfloat16)
    W = {}
    for name, (o, i) in dict(wq=(D, D), wk=(D, D), wv=(D, D), wo=(D, D), wq2=(D, D), wo2=(D, D), w1=(hidden, D), w2=(D, hidden)).items():
        W[name] = rn(o, i, scale=1 / math.sqrt(i))
        W["b" + name[1:]] = rn(o, scale=0.1)
    for name in ("s1", "t1", "g1", "s3", "t3", "g3"):
        W[name] = rn(B, D, scale=0.3)
    tk, tv = rn(B, N_text, H, d), rn(B, N_text, H, d)
    xs = [rn(B, N, D), None]
    xs[1] = (xs[0].float() + 0.05 * torch.randn(B, N, D, device="cuda", generator=g)).to(torch.bfloat16)
    x_ref = xs[0].clone()
    lse = torch.zeros(B, H, N, device="cuda")
    n_skip = torch.zeros(B, N_sel, dtype=torch.int32, device="cuda")
    y = torch.zeros(B, N, D, dtype=torch.bfloat16, device="cuda")
    score = torch.empty(B, N_sel, device="cuda")
    idx_sel = torch.empty(B, N, dtype=torch.int32, device="cuda")
    ws = torch.zeros(A.astraea_block_workspace_bytes(B, H, N, d, hidden), dtype=torch.uint8, device="cuda")
    bw = A.block_weights(W, hidden)
    w_alpha = float(1.0 / N)

    def run(t, k_keep):
        A.astraea_block_step(xs[t & 1], bw, x_ref, lse, n_skip, y, tk, tv, N_text, score, idx_sel, None, B, H, N, N_sel, d, k_keep,
                             w_alpha=w_alpha, workspace=ws)

    run(0, N_sel)                                  # dense first step fills the caches
    A.astraea_poll_error(ws)
    out = {"shape": {"B": B, "N": N, "D": D, "H": H, "d": d, "hidden": hidden, "N_text": N_text}, "keep_ratios": {}}
    for th in thetas:
        k_keep = w.k_of(th)
        M = k_keep + n_always
        cool_down(torch)
        for t in range(2):
            run(t + 1, k_keep)
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        torch.cuda.synchronize()
        m0 = sampler.mark()
        evs[0].record()
        for t in range(reps):
            run(t + 1, k_keep)
            evs[t + 1].record()
        torch.cuda.synchronize()
        m1 = sampler.mark()
        A.astraea_poll_error(ws)
        ms = float(np.median([evs[i].elapsed_time(evs[i + 1]) for i in range(reps)]))
        # algorithmic flops of the block as built: K/V projections of all rows, the rest on M rows
        fl = (2 * 2 * B * N * D * D                                    # K, V
              + 2 * B * M * D * D * 4                                  # Q, out-projection, cross-attention query and output projection
              + 2 * 2 * B * M * D * hidden                             # MLP
              + accounting.attn_flops(B, H, M, N, d) + accounting.attn_flops(B, H, M, N_text, d))
        out["keep_ratios"][str(th)] = {"ms": ms, "M": M, "TFLOP/s": fl / (ms * 1e-3) / 1e12,
                                       "frac_bf16_peak": fl / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"], "flops": fl,
                                       "clocks": sampler.summary(m0, m1) if m1 > m0 else None}
    dense = out["keep_ratios"].get("1000")
    if dense:
        for th, e in out["keep_ratios"].items():
            e["speedup_vs_dense_block"] = dense["ms"] / e["ms"]
            e["flops_vs_dense_block"] = e["flops"] / dense["flops"]
    # the layers one by one at the middle keep-ratio (the same calls astraea_block_step makes, buffers of their own)
    th = thetas[len(thetas) // 2]
    k_keep = w.k_of(th)
    M = k_keep + n_always
    run(1, k_keep)
    idx = idx_sel.view(-1)[:B * M].view(B, M)
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device="cuda")
    h, kk, vv, qq, a = z(B, N, D), z(B, N, D), z(B, N, D), z(B, N, D), z(B, N, D)
    x1, h2, c, x2, u = z(B, M, D), z(B, M, D), z(B, M, D), z(B, M, D), z(B, M, hidden)
    st, ts = A.bhnd_strides(N, H, d), A.bhnd_strides(N_text, H, d)
    x = xs[0]
    CI, CO, CR = A.LINEAR_COMPACT_IN, A.LINEAR_COMPACT_OUT, A.LINEAR_COMPACT_RES
    layers = [
        ("layernorm+modulate (all rows)", 2 * B * N * D * 2, None, lambda: A.astraea_layernorm_modulate(x, None, 0, W["s1"], W["t1"], h, B, N, D, workspace=ws)),
        ("K projection (all rows)", None, 2 * B * N * D * D, lambda: A.astraea_gathered_linear(h, None, 0, W["wk"], W["bk"], kk, B, N, D, D, workspace=ws)),
        ("V projection (all rows)", None, 2 * B * N * D * D, lambda: A.astraea_gathered_linear(h, None, 0, W["wv"], W["bv"], vv, B, N, D, D, workspace=ws)),
        ("Q projection (selected rows)", None, 2 * B * M * D * D, lambda: A.astraea_gathered_linear(h, idx, M, W["wq"], W["bq"], qq, B, N, D, D, workspace=ws)),
        ("self-attention (selected rows x all keys)", None, accounting.attn_flops(B, H, M, N, d),
         lambda: A.astraea_sparse_attn(qq, kk, vv, st, st, st, idx, M, a, lse, B, H, N, d, workspace=ws)),
        ("output projection + gated residual", None, 2 * B * M * D * D,
         lambda: A.astraea_gathered_linear_residual(a, idx, M, W["wo"], W["bo"], x, W["g1"], x1, B, N, D, D, flags=CO, workspace=ws)),
        ("layernorm (selected rows)", 2 * B * M * D * 2, None,
         lambda: A.astraea_layernorm_modulate(x1, idx, M, None, None, h2, B, N, D, flags=A.LN_COMPACT_IN | A.LN_COMPACT_OUT, workspace=ws)),
        ("cross-attention query projection", None, 2 * B * M * D * D, lambda: A.astraea_gathered_linear(h2, idx, M, W["wq2"], W["bq2"], qq, B, N, D, D, flags=CI, workspace=ws)),
        ("cross-attention (selected rows x text keys)", None, accounting.attn_flops(B, H, M, N_text, d),
         lambda: A.astraea_sparse_cross_attn(qq, tk, tv, st, ts, ts, idx, M, c, None, B, H, N, N_text, d, flags=A.ATTN_COMPACT_OUT, workspace=ws)),
        ("cross-attention output projection + residual", None, 2 * B * M * D * D,
         lambda: A.astraea_gathered_linear_residual(c, idx, M, W["wo2"], W["bo2"], x1, None, x2, B, N, D, D, flags=CI | CO | CR, workspace=ws)),
        ("layernorm+modulate (selected rows)", 2 * B * M * D * 2, None,
         lambda: A.astraea_layernorm_modulate(x2, idx, M, W["s3"], W["t3"], h2, B, N, D, flags=A.LN_COMPACT_IN | A.LN_COMPACT_OUT, workspace=ws)),
        ("MLP up-projection + GELU", None, 2 * B * M * D * hidden,
         lambda: A.astraea_gathered_linear(h2, idx, M, W["w1"], W["b1"], u, B, N, D, hidden, flags=CI | CO | A.LINEAR_GELU, workspace=ws)),
        ("MLP down-projection + gated residual + scatter", None, 2 * B * M * D * hidden,
         lambda: A.astraea_gathered_linear_residual(u, idx, M, W["w2"], W["b2"], x2, W["g3"], y, B, N, hidden, D, flags=CI | CR, workspace=ws)),
    ]
    per = {}
    for name, nbytes, fl, fn in layers:
        for _ in range(2):
            fn()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        torch.cuda.synchronize()
        evs[0].record()
        for i in range(reps):
            fn()
            evs[i + 1].record()
        torch.cuda.synchronize()
        ms = float(np.median([evs[i].elapsed_time(evs[i + 1]) for i in range(reps)]))
        e = {"ms": ms}
        if fl:
            e["TFLOP/s"] = fl / (ms * 1e-3) / 1e12
            e["frac_bf16_peak"] = e["TFLOP/s"] / peaks["bf16_tflops"]
        if nbytes:
            e["GB/s"] = nbytes / ms / 1e6
            e["frac_hbm"] = e["GB/s"] / peaks["hbm_gbs"]
        per[name] = e
    A.astraea_poll_error(ws)
    out["layers_at_keep_ratio_%d" % th] = per
    out["layers_note"] = ("each layer timed alone in a loop over one buffer set (inputs of the small layers stay in L2); the block "
                          "figures above are whole astraea_block_step calls on alternating inputs")
    return out


def model_leg(torch, A, w, theta, sampler, L=2, T=8, hidden_mult=4, N_text=226, reps=3):
    """A generation of T steps x L compute blocks as ONE CUDA graph (astraea_model_schedule_*), for the four rows of the
    ablation study (Table 2): token-wise selection, SelectQ&K, Timestep-level and Fixed-token, all made from the same
    budget schedule (dense step 0, then keep-ratio theta), next to the all-dense schedule of the same size."""
    B, N, H, d, D, N_sel, n_always = w.B, w.N, w.H, w.d, w.D, w.N_v, w.N_t
    hidden = hidden_mult * D
    g = torch.Generator(device="cuda").manual_seed(123)
    rn = lambda *s, scale=1.0: (scale * torch.randn(*s, device="cuda", generator=g)).to(torch.bfloat16)
    Ws = []
    for _ in range(L):
        W = {}
        for name, (o, i) in dict(wq=(D, D), wk=(D, D), wv=(D, D), wo=(D, D), wq2=(D, D), wo2=(D, D), w1=(hidden, D), w2=(D, hidden)).items():
            W[name] = rn(o, i, scale=1 / math.sqrt(i))
            W["b" + name[1:]] = rn(o, scale=0.1)
        for name in ("s1", "t1", "g1", "s3", "t3", "g3"):
            W[name] = rn(B, D, scale=0.3)
        Ws.append((W, hidden))
    tk, tv = [rn(B, N_text, H, d) for _ in range(L)], [rn(B, N_text, H, d) for _ in range(L)]
    x0 = rn(B, N, D)
    x1 = (x0.float() + 0.05 * torch.randn(B, N, D, device="cuda", generator=g)).to(torch.bfloat16)
    x_in = [x0 if t % 2 == 0 else x1 for t in range(T)]
    states = [dict(x_ref=x0.clone(), lse_cache=torch.zeros(B, H, N, device="cuda"),
                   n_skip=torch.zeros(B, N_sel, dtype=torch.int32, device="cuda"),
                   y_cache=torch.zeros(B, N, D, dtype=torch.bfloat16, device="cuda"),
                   score=torch.zeros(B, N_sel, device="cuda"), idx_sel=torch.zeros(B, N, dtype=torch.int32, device="cuda"),
                   idx_rem=None) for _ in range(L)]
    ws = torch.zeros(A.astraea_block_workspace_bytes(B, H, N, d, hidden), dtype=torch.uint8, device="cuda")
    k_keep = w.k_of(theta)
    token_wise = [N_sel] + [k_keep] * (T - 1)
    schedules = [("dense", A.VARIANT_TOKEN_WISE, [N_sel] * T),
                 ("token-wise (Astraea)", A.VARIANT_TOKEN_WISE, token_wise),
                 ("SelectQ&K", A.VARIANT_SELECT_QK, token_wise),
                 ("Timestep-level", A.VARIANT_TIMESTEP, A.astraea_timestep_level_budgets(token_wise, N_sel)),
                 ("Fixed-token", A.VARIANT_FIXED_TOKEN, token_wise)]
    out = {"shape": {"B": B, "N": N, "D": D, "H": H, "d": d, "hidden": hidden, "N_text": N_text, "blocks": L, "steps": T},
           "keep_ratio_permille": theta, "schedules": {}}
    for name, variant, budgets in schedules:
        sched = A.ModelSchedule(budgets, x_in, Ws, states, tk, tv, N_text, B, H, N, N_sel, d, w_alpha=float(1.0 / N),
                                variant=variant, workspace=ws)
        cool_down(torch)
        sched.launch()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        torch.cuda.synchronize()
        m0 = sampler.mark()
        evs[0].record()
        for i in range(reps):
            sched.launch()
            evs[i + 1].record()
        torch.cuda.synchronize()
        m1 = sampler.mark()
        A.astraea_poll_error(ws)
        sched.close()
        ms = float(np.median([evs[i].elapsed_time(evs[i + 1]) for i in range(reps)]))
        out["schedules"][name] = {"ms_per_generation": ms, "ms_per_step_and_block": ms / (T * L),
                                  "tokens_computed_fraction": float(sum(b + n_always for b in budgets)) / (T * N),
                                  "budgets": [int(b) for b in budgets], "clocks": sampler.summary(m0, m1) if m1 > m0 else None}
    dense = out["schedules"]["dense"]["ms_per_generation"]
    for e in out["schedules"].values():
        e["speedup_vs_dense"] = dense / e["ms_per_generation"]
    out["note"] = ("one graph launch per generation; SelectQ&K gathers the selected K / V rows in a pass of its own before the "
                   "attention (twice the K / V bytes of those rows through HBM); Fixed-token scores and selects in block 0 only")
    return out


def e2e_leg(torch, A, w, theta, steps, barrier):
    """The same step through astraea_step_host: pinned host buffers in, merged output back, every step."""
    B, N, D = w.B, w.N, w.D
    k_keep = w.k_of(theta)
    tb = B * N * D * 2
    # host-side N(0,1) values: one block of 2^24 draws, laid out with a different offset per tensor (the period is no
    # multiple of the row length, so no two rows are equal); the values do not matter for the timing
    g = torch.Generator().manual_seed(7)
    block = torch.randn((1 << 24) + 4096, generator=g).to(torch.bfloat16)
    host = {}
    for i, n in enumerate(("x_cur", "q", "k", "v")):
        t = torch.empty(B, N, D, dtype=torch.bfloat16).pin_memory()
        flat = t.view(-1)
        for r0 in range(0, flat.numel(), 1 << 24):
            r1 = min(flat.numel(), r0 + (1 << 24))
            flat[r0:r1] = block[1024 * i:1024 * i + (r1 - r0)]
        host[n] = t
    host_out = torch.empty(B, N, D, dtype=torch.bfloat16).pin_memory()
    sess = A.Session(B, w.H, N, w.N_v, w.d)
    w_alpha = float(1.0 / N)
    sess.step_host(host["x_cur"], host["q"], host["k"], host["v"], host_out, w.N_v, w_alpha, 1.0)   # dense first step
    for _ in range(2):
        sess.step_host(host["x_cur"], host["q"], host["k"], host["v"], host_out, k_keep, w_alpha, 1.0)
    barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        sess.step_host(host["x_cur"], host["q"], host["k"], host["v"], host_out, k_keep, w_alpha, 1.0)
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    h2d = sess.last_h2d_bytes()             # x_cur, k, v in full; of the pinned q only the selected rows
    sess.close()
    flops = accounting.attn_flops(B, w.H, k_keep + w.N_t, N, w.d)
    return dt, flops * steps, {"h2d_bytes_per_step": h2d, "d2h_bytes_per_step": tb, "steps": steps,
                               "api": "astraea_step_host (pinned host buffers)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="astraea", choices=["astraea", "reference"])
    ap.add_argument("--workload", default=HEADLINE, choices=sorted(synth.WORKLOADS), help="workload of the headline")
    ap.add_argument("--theta", type=int, default=HEADLINE_THETA, help="keep-ratio of the headline in permille")
    ap.add_argument("--ref-rows", type=int, default=64, help="sampled query rows per step of the reference arm")
    ap.add_argument("--ref-heads", type=int, default=8)
    ap.add_argument("--cpu-rows", type=int, default=256, help="sampled query rows of the cpu_baseline leg (all heads)")
    ap.add_argument("--seeds", type=int, default=10, help="seeds of the keep-ratio sweep")
    ap.add_argument("--chain-steps", type=int, default=50, help="consecutive steps of the HunyuanVideo-shaped chain")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-workloads", action="store_true", help="headline only")
    ap.add_argument("--no-next", action="store_true", help="skip the query projection of the selected rows (astraea_gathered_linear)")
    ap.add_argument("--no-model", action="store_true", help="skip the scheduled generations (astraea_model_schedule_*: 2 blocks x 8 steps, four variants); --no-block skips them too")
    ap.add_argument("--no-block", action="store_true", help="skip the whole-block leg (astraea_block_step on the CogVideoX shape)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.warmup < 3:
        args.warmup = 3
    w = synth.WORKLOADS[args.workload]
    theta = args.theta

    import torch
    import torch.distributed as dist
    from paper_2506_05096_b200 import binding as A

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    A.lib()
    peaks = measured_peaks()
    extras = rank == 0 and world == 1

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    t_start = time.perf_counter()

    # ------------------------------------------------------------ the short workloads first
    # (each is 20 steps of 1-4 ms, i.e. a burst like the one the burst peak was measured in; behind the seconds of
    # head_dim-128 work further down the power cap holds the SM clock near 1500 MHz and the same launches run ~10 % slower:
    # `clocks` of every entry says what it ran at)
    workloads, attn_fracs, hbm_fracs = {}, {}, {}
    if not args.no_workloads and extras:
        for name, thetas in (("cogvideox", (1000, 500, 250)), ("opensora", (400,)), ("tiny", (500,))):
            ww = synth.WORKLOADS[name]
            b2 = Block(torch, A, ww, seed=0)
            b2.step(0, ww.N_v)
            workloads[name] = {}
            for th in thetas:
                n_st = 20                     # 80 ms at most: with 50 steps (0.2 s) the power cap already pulls the clock down inside the leg
                cool_down(torch)
                m0 = sampler.mark()
                tot, pp, allp = b2.timed(ww.k_of(th), n_st, 3, barrier)
                m1 = sampler.mark()
                A.astraea_poll_error(b2.ws)
                rl, kn = kernel_report(ww, th, pp, peaks, pair_ms=b2.timed_pair(ww.k_of(th), steps=20), all_parts=allp)
                add_copy_yardstick(kn, b2.timed_plain_copy(ww.k_of(th)))
                entry = {"config": config_of(ww, th, world), "ms_per_step": tot / n_st, "steps": n_st,
                         "step_tflops": accounting.attn_flops(ww.B, ww.H, ww.M_of(th), ww.N, ww.d) / (tot / n_st * 1e-3) / 1e12,
                         "roofline": rl, "kernels": kn, "clocks": sampler.summary(m0, m1)}
                workloads[name][str(th)] = entry
                if name != "tiny":           # the tiny configuration is a parity case: 17 MFLOP, all launch latency
                    attn_fracs["%s@%d" % (name, th)] = rl["frac"]
                    for n in ("score", "score+select", "scatter_reuse(x_ref)"):
                        hbm_fracs["%s@%d:%s" % (name, th, n)] = kn[n]["frac_hbm"]
            del b2
            torch.cuda.empty_cache()
            if not args.no_e2e:
                th = thetas[len(thetas) // 2] if name == "cogvideox" else thetas[0]
                dt, fl, info = e2e_leg(torch, A, ww, th, 5, barrier)
                workloads[name][str(th)]["e2e"] = {"value": fl / dt / 1e12, "unit": UNIT, **info, "ms_per_step": 1e3 * dt / 5}
    # the whole compute block on the CogVideoX shape (head_dim 64 as well: before the long legs for the same reason)
    block = None
    if not args.no_block and extras:
        block = block_leg(torch, A, synth.WORKLOADS["cogvideox"], (1000, 500, 250), peaks, sampler)
        torch.cuda.empty_cache()
    model = None
    if not args.no_model and not args.no_block and extras:
        model = model_leg(torch, A, synth.WORKLOADS["cogvideox"], 500, sampler)
        torch.cuda.empty_cache()

    # ------------------------------------------------------------ headline: K consecutive steps, device-resident inputs
    blk = Block(torch, A, w, seed=replicas.rank_seed(0, rank))
    B, N, H, d, D, N_sel, n_always = w.B, w.N, w.H, w.d, w.D, w.N_v, w.N_t
    blk.step(0, N_sel)                       # step 0 of a generation computes every token: fills the output and LSE caches
    A.astraea_poll_error(blk.ws)
    k_keep = w.k_of(theta)
    M = k_keep + n_always
    c0 = sampler.mark()
    total_ms, parts, all_parts = blk.timed(k_keep, args.steps, args.warmup, barrier)
    c1 = sampler.mark()
    A.astraea_poll_error(blk.ws)
    flops = accounting.attn_flops(B, H, M, N, d)
    total_ms, job_flops = replicas.aggregate(total_ms, flops * args.steps, device="cuda")
    ms_per_step = total_ms / args.steps
    value = replicas.throughput(job_flops, total_ms) / 1e12
    pair_ms = blk.timed_pair(k_keep) if extras else None
    # the headline's roofline divides by the kernel's AVERAGE launch duration over the timed steps
    roofline, kernels = kernel_report(w, theta, all_parts.mean(axis=0), peaks, pair_ms=pair_ms, all_parts=all_parts, stat="mean")
    if extras:
        add_copy_yardstick(kernels, blk.timed_plain_copy(k_keep))
    kernels["hbm_peaks_gbs"] = {"measured": peaks["hbm_gbs"], "nominal": NOMINAL_HBM_GBS}
    clocks = sampler.summary(c0, c1) if c1 > c0 else sampler.summary()
    attn_fracs["%s@%d" % (w.name, theta)] = roofline["frac"]
    hbm_fracs.update({"%s@%d:%s" % (w.name, theta, n): kernels[n]["frac_hbm"] for n in ("score", "score+select", "scatter_reuse(x_ref)")})

    # ------------------------------------------------------------ the next layer of the block and the graph replay
    nxt = None
    if not args.no_next and extras and M > 0:
        g = torch.Generator(device="cuda").manual_seed(7)
        w_q = (torch.randn(D, D, device="cuda", generator=g) / math.sqrt(D)).to(torch.bfloat16)
        ys = [torch.zeros(B, N, D, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
        ws_lin = A.new_workspace(A.OP_GATHERED_LINEAR, 0, 0, 0, 0, 0)
        idx_now = blk.idx_sel.view(-1)[:B * M].view(B, M)
        reps = 10
        for t in range(3):
            A.astraea_gathered_linear(blk.sets[t & 1]["x_cur"], idx_now, M, w_q, None, ys[t & 1], B, N, D, D, workspace=ws_lin)
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        torch.cuda.synchronize()
        evs[0].record()
        for t in range(reps):     # two alternating x / y sets: 2 x (M rows of x and y) + W > 126 MB L2 on every workload but tiny
            A.astraea_gathered_linear(blk.sets[t & 1]["x_cur"], idx_now, M, w_q, None, ys[t & 1], B, N, D, D, workspace=ws_lin)
            evs[t + 1].record()
        torch.cuda.synchronize()
        A.astraea_poll_error(ws_lin)
        lin_ms = float(np.median([evs[i].elapsed_time(evs[i + 1]) for i in range(reps)]))
        lin_flops = 2.0 * B * M * D * D
        nxt = {"gathered_linear(q projection of the selected rows)": {
            "ms": lin_ms, "TFLOP/s": lin_flops / (lin_ms * 1e-3) / 1e12,
            "frac_bf16_peak": lin_flops / (lin_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "shape": {"rows": B * M, "K": D, "N_out": D}}}
        del ys, w_q
        T = 10
        sets = blk.sets
        sched = A.Schedule([k_keep] * T, [sets[t & 1]["x_cur"] for t in range(T)], [sets[t & 1]["q"] for t in range(T)],
                           [sets[t & 1]["k"] for t in range(T)], [sets[t & 1]["v"] for t in range(T)], blk.x_ref, blk.lse,
                           blk.n_skip, blk.out, blk.score, blk.idx_sel, blk.idx_rem, B, H, N, N_sel, d, blk.w_alpha, 1.0,
                           workspace=blk.ws)
        sched.launch()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        sched.launch()
        e1.record()
        torch.cuda.synchronize()
        A.astraea_poll_error(blk.ws)
        nxt["schedule_graph(%d steps, one launch)" % T] = {"ms_per_step": e0.elapsed_time(e1) / T,
                                                          "ms_per_step_separate_launches": ms_per_step}
        sched.close()

    # ------------------------------------------------------------ keep-ratio sweep: twenty ratios x seeds
    sweep = {}
    if not args.no_sweep and extras:
        sw = synth.WORKLOADS["sweep"]
        per = {th: {"attn": [], "step": []} for th in sw.thetas_permille}
        for seed in range(args.seeds):
            b2 = blk if (seed == 0 and w.name == "sweep") else Block(torch, A, sw, seed=seed, sets=1)
            b2.step(0, sw.N_v)
            for th in sw.thetas_permille:
                tot, pp, _ = b2.timed(sw.k_of(th), 2, 1, barrier)
                per[th]["attn"].append(float(pp[2]))
                per[th]["step"].append(tot / 2)
            A.astraea_poll_error(b2.ws)
            if b2 is not blk:
                del b2
                torch.cuda.empty_cache()
        for th in sw.thetas_permille:
            f = accounting.attn_flops(sw.B, sw.H, sw.M_of(th), sw.N, sw.d)
            a, s = np.array(per[th]["attn"]), np.array(per[th]["step"])
            tf = f / (a * 1e-3) / 1e12
            sweep[str(th)] = {"attn_ms": float(a.mean()), "attn_ms_min": float(a.min()), "attn_ms_max": float(a.max()),
                              "ms_per_step": float(s.mean()), "attn_tflops": float(tf.mean()), "attn_tflops_min": float(tf.min()),
                              "attn_tflops_max": float(tf.max()), "step_tflops": float((f / (s * 1e-3) / 1e12).mean()),
                              "frac_bf16_peak": float(tf.mean() / peaks["bf16_tflops"]), "seeds": len(a)}
            if th >= 250:
                attn_fracs["sweep@%d" % th] = float(tf.mean() / peaks["bf16_tflops"])
        sweep["note"] = ("B1 H24 d128 N=65536; per ratio and seed 1 warm-up + 2 timed steps after a dense step 0; ratio 1000 is "
                         "the dense reference point; ratios below 250 are outside the stated 0.25-1.0 target range")

    # ------------------------------------------------------------ e2e of the headline
    e2e = None
    if not args.no_e2e:
        del blk.sets[1:]
        torch.cuda.empty_cache()
        n_e2e = max(3, min(args.steps, 5))
        dt, fl, info = e2e_leg(torch, A, w, theta, n_e2e, barrier)
        dt_ms, e2e_flops = replicas.aggregate(dt * 1e3, fl, device="cuda")
        e2e = {"value": replicas.throughput(e2e_flops, dt_ms) / 1e12, "unit": UNIT, **info, "ms_per_step": dt_ms / n_e2e}
    del blk
    torch.cuda.empty_cache()

    # ------------------------------------------------------------ the HunyuanVideo-shaped chain
    if not args.no_workloads and extras:
        # HunyuanVideo shape: a dense step 0 from empty caches, then `chain_steps` consecutive steps of a latent that
        # drifts by sigma = 0.05 per step (real LSE / x_ref / counter chain).  The drift is applied on the device
        # between the steps and is outside the per-step event pairs.
        hw = synth.WORKLOADS["hunyuan"]
        workloads["hunyuan"] = {}
        for th in (600, 300):
            b2 = Block(torch, A, hw, seed=0, sets=1)
            b2.out.zero_(); b2.lse.zero_(); b2.n_skip.zero_()
            b2.x_ref.copy_(b2.sets[0]["x_cur"])
            ev0 = [torch.cuda.Event(enable_timing=True) for _ in range(5)]
            barrier()
            b2.step(0, hw.N_v, ev0)
            barrier()
            dense_parts = np.array([ev0[i].elapsed_time(ev0[i + 1]) for i in range(4)])
            evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.chain_steps)]
            m0 = sampler.mark()
            t0 = time.perf_counter()
            for t in range(args.chain_steps):
                s = b2.sets[0]
                s["x_cur"] = b2.drift(s["x_cur"], 0.05, False, None)
                for n in ("q", "k", "v"):
                    s[n] = b2.drift(s[n], 0.05, True, None)
                b2.step(0, hw.k_of(th), evs[t])
            barrier()
            wall = time.perf_counter() - t0
            m1 = sampler.mark()
            A.astraea_poll_error(b2.ws)
            allp = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(4)] for e in evs])
            pp = np.median(allp, axis=0)
            rl, kn = kernel_report(hw, th, pp, peaks, long_region=True, pair_ms=b2.timed_pair(hw.k_of(th), steps=3, t_base=0), all_parts=allp)
            step_ms = allp.sum(axis=1)
            n_max = int(b2.n_skip.max().item())
            workloads["hunyuan"][str(th)] = {
                "config": config_of(hw, th, world), "chain_steps": args.chain_steps,
                "ms_per_step": float(step_ms.mean()), "ms_per_step_min": float(step_ms.min()), "ms_per_step_max": float(step_ms.max()),
                "chain_ms": float(step_ms.sum()), "wall_ms_including_the_drift_of_the_inputs": 1e3 * wall,
                "step_tflops": accounting.attn_flops(hw.B, hw.H, hw.M_of(th), hw.N, hw.d) / (float(step_ms.mean()) * 1e-3) / 1e12,
                "dense_step0": {"ms": float(dense_parts.sum()), "attn_ms": float(dense_parts[2]),
                                "attn_tflops": accounting.attn_flops(hw.B, hw.H, hw.N, hw.N, hw.d) / (dense_parts[2] * 1e-3) / 1e12},
                "max_skip_counter_after_the_chain": n_max, "roofline": rl, "kernels": kn, "clocks": sampler.summary(m0, m1)}
            attn_fracs["hunyuan@%d" % th] = rl["frac"]
            for n in ("score", "score+select", "scatter_reuse(x_ref)"):
                hbm_fracs["hunyuan@%d:%s" % (th, n)] = kn[n]["frac_hbm"]
            del b2
            torch.cuda.empty_cache()
        if not args.no_e2e:
            dt, fl, info = e2e_leg(torch, A, hw, 600, 3, barrier)
            workloads["hunyuan"]["600"]["e2e"] = {"value": fl / dt / 1e12, "unit": UNIT, **info, "ms_per_step": 1e3 * dt / 3}
    sampler.stop()

    cpu = None
    if extras and not args.no_cpu_baseline:
        v, s, threads, desc = OracleSample(w, theta).run(args.cpu_rows)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}

    if rank == 0:
        worst_a = min(attn_fracs, key=attn_fracs.get)
        worst_h = min(hbm_fracs, key=hbm_fracs.get)
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": config_of(w, theta, world),
                "gpu_launches": (3 + kernels["sparse_attn"]["schedule"]["launches"]) * args.steps, "clocks": clocks, "roofline": roofline, "kernels": kernels,
                "worst_attn_frac": {"value": attn_fracs[worst_a], "where": worst_a, "of": "measured burst bf16",
                                    "of_nominal_2250": attn_fracs[worst_a] * peaks["bf16_tflops"] / NOMINAL_BF16_TFLOPS,
                                    "all": attn_fracs},
                "worst_hbm_frac": {"value": hbm_fracs[worst_h], "where": worst_h, "of": "measured copy bandwidth",
                                   "of_nominal_8000": hbm_fracs[worst_h] * peaks["hbm_gbs"] / NOMINAL_HBM_GBS, "all": hbm_fracs},
                "keep_ratio_sweep": sweep, "workloads": workloads, "next": nxt, "block": block, "model_schedules": model, "e2e": e2e, "cpu_baseline": cpu,
                "bench_seconds": time.perf_counter() - t_start}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
