#!/usr/bin/env python
"""Benchmark of the hot path (score -> select -> sparse attention with fused scatter ->
reference refresh) on synthetic latents shaped like the paper's video workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cogvideox] [--theta 500]
    python bench.py --impl reference ...       # the CPU oracle, timed on the host cores

One "step" is one pass of the whole path for one attention block at keep-ratio theta.
`value` is the attention's algorithmic FLOPs (4*B*H*M*N*d) per second of whole-step time,
inputs resident in HBM; `e2e` is the same through astraea_step_host with pinned HOST buffers
(host<->device copies inside the timed region).  Prints ONE JSON line on rank 0.
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

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the attention kernel, from the ncu
# capture summarised in profiles/ (workload -> theta_permille -> bytes); None where not captured.
NOMINAL_BF16_TFLOPS, NOMINAL_HBM_GBS = 2250.0, 8000.0     # the part's nominal dense bf16 and HBM3e figures, for context
NCU_TRAFFIC_BYTES = {"cogvideox": {500: 324246784}, "sweep": {250: 1285133616}}


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

    def stop(self) -> dict:
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.t.join(timeout=2)
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
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


# ------------------------------------------------------------------ the oracle legs
def oracle_sample(w, theta, rows=2048, heads=None, seed=0):
    """Times the CPU oracle on a bounded sample of the workload: score and select at full size,
    attention for `rows` sampled selected queries x `heads` heads against all keys.  Returns
    (effective TFLOP/s of the attention sample, seconds, threads, description)."""
    from oracle import astraea_oracle as oracle
    oracle.build()
    inp = synth.make_step_inputs(w, seed)
    f = synth.bf16_to_f64
    k_keep = w.k_of(theta)
    x_cur, x_ref = f(inp["x_cur"]), f(inp["x_ref"])
    lse = (inp["lse"] - np.float32(math.log(w.N))).astype(np.float64)
    hs = w.H if heads is None else min(heads, w.H)
    q, k, v = (f(np.ascontiguousarray(inp[n][:, :, :hs])) for n in ("q", "k", "v"))
    t0 = time.perf_counter()
    s = oracle.score(x_cur, x_ref, lse, inp["n_skip"], n_sel=w.N_v)
    sel, _, _ = oracle.select(s.astype(np.float32), k_keep, w.N_t, inp["n_skip"])
    t1 = time.perf_counter()
    rng = np.random.default_rng(seed)
    r = min(rows, sel.shape[1])
    pick = np.stack([np.sort(rng.choice(sel[b], r, replace=False)) for b in range(w.B)]).astype(np.int32)
    o, l, _ = oracle.sparse_attn(q, k, v, q_idx=pick)
    t2 = time.perf_counter()
    flops = accounting.attn_flops(w.B, hs, r, w.N, w.d)
    desc = ("oracle fp64: score+select at full size (%.2f s, not in the rate); attention of %d sampled selected "
            "rows x %d of %d heads x all %d keys (%.2f s)" % (t1 - t0, r, hs, w.H, w.N, t2 - t1))
    return flops / (t2 - t1) / 1e12, (t2 - t1), oracle.num_threads(), desc


def run_reference(args, w, theta):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals, secs = [], []
    desc, threads = "", 1
    for i in range(args.warmup + args.steps):
        v, s, threads, desc = oracle_sample(w, theta, rows=args.ref_rows, heads=args.ref_heads, seed=i)
        if i >= args.warmup:
            vals.append(v)
            secs.append(s)
    value = float(np.mean(vals))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(secs)),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "theta_permille": theta, "B": w.B, "H": w.H, "d": w.d, "N": w.N},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------- the CUDA leg
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="astraea", choices=["astraea", "reference"])
    ap.add_argument("--workload", default="cogvideox", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--theta", type=int, default=500, help="keep-ratio in permille")
    ap.add_argument("--ref-rows", type=int, default=256, help="sampled query rows per step of the reference arm")
    ap.add_argument("--ref-heads", type=int, default=8)
    ap.add_argument("--cpu-rows", type=int, default=1024, help="sampled query rows of the cpu_baseline leg (all heads)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-next", action="store_true", help="skip the query projection of the selected rows (astraea_gathered_linear)")
    args = ap.parse_args()
    w = synth.WORKLOADS[args.workload]
    theta = args.theta
    if args.impl == "reference":
        run_reference(args, w, theta)
        return
    if args.warmup < 3:
        args.warmup = 3

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

    B, N, H, d, D, N_sel, n_always = w.B, w.N, w.H, w.d, w.D, w.N_v, w.N_t

    def bf(bits):
        return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()

    # two input sets (step t and t+1 of a drifting latent), alternated so that the reference
    # inputs keep differing from the current ones; replicas use different seeds
    inp = synth.make_step_inputs(w, seed=replicas.rank_seed(0, rank))
    sets = [{n: bf(inp[n]) for n in ("x_cur", "q", "k", "v")}]
    sets.append({"x_cur": bf(synth.drift_step(inp["x_cur"], 1000 + rank, 0.05, False)),
                 **{n: bf(synth.drift_step(inp[n], 1001 + i + rank, 0.05, True)) for i, n in enumerate(("q", "k", "v"))}})
    x_ref = bf(inp["x_ref"])
    out = bf(inp["cache"])
    lse = torch.from_numpy(inp["lse"]).cuda()
    n_skip = torch.from_numpy(inp["n_skip"]).cuda()
    score = torch.empty(B, N_sel, device="cuda")
    idx_sel = torch.empty(B, N, dtype=torch.int32, device="cuda")
    idx_rem = torch.empty(B, N_sel + 1, dtype=torch.int32, device="cuda")
    ws = A.new_workspace(A.OP_STEP, B, H, N, N, d)
    ws_sel = A.new_workspace(A.OP_SELECT, B, 0, N_sel, 0, 0)
    strides = A.bhnd_strides(N, H, d)
    # the drifting scale of exp(lse) does not matter for timing; keep the scores finite
    w_alpha = float(1.0 / N)

    def step(t, k_keep, ev=None):
        s = sets[t & 1]
        M = k_keep + n_always
        if ev:
            ev[0].record()
        A.astraea_score(s["x_cur"], x_ref, lse, n_skip, score, B, N, N_sel, D, H, w_alpha, 1.0)
        if ev:
            ev[1].record()
        A.astraea_select(score, B, N_sel, k_keep, n_always, idx_sel, idx_rem, n_skip, ws_sel)
        if ev:
            ev[2].record()
        A.astraea_sparse_attn(s["q"], s["k"], s["v"], strides, strides, strides, idx_sel, M, out, lse,
                              B, H, N, d, workspace=ws)
        if ev:
            ev[3].record()
        A.astraea_scatter_reuse(x_ref, s["x_cur"], idx_sel, B, N, M, D, A.SCATTER_SRC_FULL)
        if ev:
            ev[4].record()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(k_keep, steps, warmup, t_base):
        for t in range(warmup):
            step(t_base + t, k_keep)
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(steps)]
        barrier()
        for t in range(steps):
            step(t_base + warmup + t, k_keep, evs[t])
        barrier()
        total_ms = evs[0][0].elapsed_time(evs[-1][4])
        parts = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(4)] for e in evs])
        return total_ms, parts.mean(axis=0)

    sampler = ClockSampler(local)
    sampler.start()
    # step 0 of a generation computes every token: fills the output and LSE caches
    step(0, N_sel)
    A.astraea_poll_error(ws)

    k_keep = w.k_of(theta)
    M = k_keep + n_always
    total_ms, parts = timed(k_keep, args.steps, args.warmup, 1)
    A.astraea_poll_error(ws)
    flops = accounting.attn_flops(B, H, M, N, d)
    total_ms, job_flops = replicas.aggregate(total_ms, flops * args.steps, device="cuda")
    ms_per_step = total_ms / args.steps
    value = replicas.throughput(job_flops, total_ms) / 1e12

    peaks = measured_peaks()
    attn_ms = float(parts[2])
    achieved = flops / (attn_ms * 1e-3) / 1e12
    traffic = NCU_TRAFFIC_BYTES.get(w.name, {}).get(theta)
    roofline = {"bound": "tensor", "kernel": "sparse_attn_kernel<%d>" % d, "achieved": achieved,
                "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                "peak_kind": "%s burst bf16 (MEASURED_PEAKS.json)" % peaks["source"] if peaks["source"] == "measured"
                else "fallback burst bf16", "traffic": traffic, "kernel_ms": attn_ms,
                "min_bytes": accounting.attn_min_bytes(B, H, M, N, d),
                # for context only: the nominal dense bf16 figure of the part, and the credit for the rows that were skipped
                "frac_of_nominal_2250_tflops": achieved / NOMINAL_BF16_TFLOPS,
                "dense_equivalent_tflops(speed-up credit, not a roofline figure)":
                    accounting.attn_flops(B, H, N, N, d) / (attn_ms * 1e-3) / 1e12}
    hbm = peaks["hbm_gbs"]
    sb = accounting.score_bytes(B, N, N_sel, D, H)
    cb = accounting.scatter_bytes(B, M, D)
    selb = accounting.select_bytes(B, N_sel, k_keep)
    kernels = {
        "hbm_peaks_gbs": {"measured": hbm, "nominal": NOMINAL_HBM_GBS},
        "score": {"ms": float(parts[0]), "GB/s": sb / parts[0] / 1e6, "frac_hbm": sb / parts[0] / 1e6 / hbm,
                  "frac_hbm_nominal": sb / parts[0] / 1e6 / NOMINAL_HBM_GBS},
        "select": {"ms": float(parts[1]), "GB/s": selb / parts[1] / 1e6, "note": "latency-bound"},
        "score+select": {"ms": float(parts[0] + parts[1]), "GB/s": (sb + selb) / (parts[0] + parts[1]) / 1e6,
                         "frac_hbm": (sb + selb) / (parts[0] + parts[1]) / 1e6 / hbm,
                         "frac_hbm_nominal": (sb + selb) / (parts[0] + parts[1]) / 1e6 / NOMINAL_HBM_GBS},
        "sparse_attn": {"ms": attn_ms, "TFLOP/s": achieved},
        "scatter_reuse(x_ref)": {"ms": float(parts[3]), "GB/s": cb / parts[3] / 1e6, "frac_hbm": cb / parts[3] / 1e6 / hbm,
                                 "frac_hbm_nominal": cb / parts[3] / 1e6 / NOMINAL_HBM_GBS},
    }

    sweep = {}
    if not args.no_sweep and rank == 0 and world == 1:
        for th in w.thetas_permille:
            if th == theta:
                sweep[str(th)] = {"ms_per_step": ms_per_step, "attn_ms": attn_ms, "tflops": value}
                continue
            kk = w.k_of(th)
            tot, pp = timed(kk, max(5, args.steps // 2), 3, 1)
            f = accounting.attn_flops(B, H, kk + n_always, N, d)
            n_st = max(5, args.steps // 2)
            sweep[str(th)] = {"ms_per_step": tot / n_st, "attn_ms": float(pp[2]), "tflops": f / (tot / n_st * 1e-3) / 1e12,
                              "attn_tflops": f / (pp[2] * 1e-3) / 1e12}
        A.astraea_poll_error(ws)
    # ---- the next layer of the block on the same selection: query projection of the selected rows
    nxt = None
    if not args.no_next and rank == 0 and world == 1 and M > 0:
        g = torch.Generator(device="cuda").manual_seed(7)
        w_q = (torch.randn(D, D, device="cuda", generator=g) / math.sqrt(D)).to(torch.bfloat16)
        ys = [torch.zeros(B, N, D, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
        ws_lin = A.new_workspace(A.OP_GATHERED_LINEAR, 0, 0, 0, 0, 0)
        step(0, k_keep)          # the selection of the timed keep-ratio (the sweep left another one behind)
        idx_now = idx_sel[:, :M] if B == 1 else idx_sel.view(-1)[:B * M].view(B, M)
        reps = 10
        for t in range(3):
            A.astraea_gathered_linear(sets[t & 1]["x_cur"], idx_now, M, w_q, None, ys[t & 1], B, N, D, D, workspace=ws_lin)
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
        torch.cuda.synchronize()
        evs[0].record()
        for t in range(reps):     # two alternating x / y sets: 2 x (M rows of x and y) + W > 126 MB L2 on every workload but tiny
            A.astraea_gathered_linear(sets[t & 1]["x_cur"], idx_now, M, w_q, None, ys[t & 1], B, N, D, D, workspace=ws_lin)
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
        # the same steps recorded once as a CUDA graph (a fixed budget schedule) and replayed with one launch
        T = 10
        sched = A.Schedule([k_keep] * T, [sets[t & 1]["x_cur"] for t in range(T)], [sets[t & 1]["q"] for t in range(T)],
                           [sets[t & 1]["k"] for t in range(T)], [sets[t & 1]["v"] for t in range(T)], x_ref, lse, n_skip,
                           out, score, idx_sel, idx_rem, B, H, N, N_sel, d, w_alpha, 1.0, workspace=ws)
        sched.launch()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        sched.launch()
        e1.record()
        torch.cuda.synchronize()
        A.astraea_poll_error(ws)
        nxt["schedule_graph(%d steps, one launch)" % T] = {"ms_per_step": e0.elapsed_time(e1) / T,
                                                          "ms_per_step_separate_launches": ms_per_step}
        sched.close()
    clocks = sampler.stop()      # covers warm-up, the timed steps, the keep-ratio sweep and the projection

    # ---- end to end through the host-buffer session
    e2e = None
    if not args.no_e2e:
        del sets[1]
        tb = B * N * D * 2
        host = {n: torch.from_numpy(inp[n].view(np.int16).reshape(B, N, D)).view(torch.bfloat16).pin_memory()
                for n in ("x_cur", "q", "k", "v")}
        host_out = torch.empty(B, N, D, dtype=torch.bfloat16).pin_memory()
        sess = A.Session(B, H, N, N_sel, d)
        sess.step_host(host["x_cur"], host["q"], host["k"], host["v"], host_out, N_sel, w_alpha, 1.0)   # dense first step
        for _ in range(2):
            sess.step_host(host["x_cur"], host["q"], host["k"], host["v"], host_out, k_keep, w_alpha, 1.0)
        n_e2e = max(3, min(args.steps, 10))
        barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            sess.step_host(host["x_cur"], host["q"], host["k"], host["v"], host_out, k_keep, w_alpha, 1.0)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt_ms, e2e_flops = replicas.aggregate(dt * 1e3, flops * n_e2e, device="cuda")
        dt = dt_ms * 1e-3
        sess.close()
        e2e = {"value": replicas.throughput(e2e_flops, dt_ms) / 1e12, "unit": UNIT, "h2d_bytes_per_step": 4 * tb,
               "d2h_bytes_per_step": tb, "ms_per_step": 1e3 * dt / n_e2e, "steps": n_e2e,
               "api": "astraea_step_host (pinned host buffers)"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, s, threads, desc = oracle_sample(w, theta, rows=args.cpu_rows, heads=None, seed=0)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": {"workload": w.name, "theta_permille": theta, "B": B, "H": H, "d": d, "N": N,
                           "N_sel": N_sel, "k_keep": k_keep, "M": M,
                           "parallelism": "replicas only (%d)" % world,
                           "l2": "two alternating input sets, %.0f MB touched per step > 126 MB L2"
                                 % ((6 * B * N * D * 2) / 1e6)},
                "gpu_launches": 4 * args.steps, "clocks": clocks, "roofline": roofline, "kernels": kernels,
                "keep_ratio_sweep": sweep, "next": nxt, "e2e": e2e, "cpu_baseline": cpu}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
