#!/usr/bin/env python
"""Benchmark of the VC-Attention hot path (prep + quantized attention forward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3] [--bits 8]
    python bench.py --impl reference ...      # the CPU oracle on the host cores

One step = one pass of the whole hot path (vc_attn: preprocessing pass + attention
forward) over one synthetic batch shaped like the named workload, inputs resident in HBM.
Metric: attention TFLOP/s = 4 B H N^2 d / time.  Prints ONE JSON line on rank 0.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

import vc_inputs  # noqa: E402
import vc_kmeans_harness  # noqa: E402

METRIC = "quantized attn fwd TFLOPS (hot path: prep + attention forward)"
UNIT = "TFLOP/s"


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"], "bf16_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is not None and self.proc.poll() is None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def window(self, t0=None, t1=None):
        """Median SM clock and the throttle reasons seen between wall-clock times t0 and t1
        (the sampler keeps running: one process serves every window of the run)."""
        import datetime
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)                      # let the sample that covers t1 arrive
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = []
        for line in list(self.lines):
            f = [x.strip() for x in line.split(",")]
            if len(f) < 8:
                continue
            try:
                ts = datetime.datetime.strptime(f[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(f[1]), float(f[2]), float(f[3]), [n for n, v in zip(names, f[4:8]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        inside = [r for r in rows if t0 is not None and t0 - 0.02 <= r[0] <= t1 + 0.02]
        window = "timed region"
        if not inside:      # region shorter than the sampling period: fall back to the samples under load
            inside = [r for r in rows if r[3] > 300.0] or rows
            window = "whole run (timed region shorter than the sampling period)"
        sm = [r[1] for r in inside]
        reasons = sorted({n for r in inside for n in r[4]})
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max((r[2] for r in inside), default=None),
                "power_w_max": max((r[3] for r in inside), default=None), "reasons": reasons, "samples": len(sm),
                "window": window}


def max_over_ranks(value, device=None):
    """Max of a per-rank scalar over the process group (the identity without one)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(flops_per_rank, ms_per_step_this_rank, world, device=None):
    """Whole-job TFLOP/s: every rank processes its own copy of the workload (weak scaling, no
    collective on the data path); the step time is the slowest rank's."""
    ms = max_over_ranks(ms_per_step_this_rank, device)
    return world * flops_per_rank / (ms * 1e-3) / 1e12, ms


def _oracle_cfg(w, bits, hybrid):
    """(PrepConfig, probability format) of the oracle for the arrangement the bench runs."""
    from oracle import attention as OA
    from oracle import prep as OP
    if hybrid:
        return OP.PrepConfig(N=w.N, d=w.d, grid=w.grid, bits=4, v_format="mxfp4"), OA.P_EXPCAST
    return OP.PrepConfig(N=w.N, d=w.d, grid=w.grid, bits=bits), None


def run_reference(args, w, bits):
    """The oracle as it stands, timed on the host cores on a bounded sample of the workload."""
    import numpy as np
    from oracle import attention as OA
    from oracle import prep as OP
    rows_per_step = args.ref_rows
    q, k, v = [t[0, 0].float().numpy() for t in vc_inputs.make_qkv(w, heads=[0])]
    cfg, pf = _oracle_cfg(w, bits, bits == 4 and args.p_format == "expcast")
    rows = np.linspace(0, w.N - 1, rows_per_step).astype(np.int64)

    def step():
        bundle = OP.prep_head(q, k, v, None, cfg)
        OA.emulate_head(bundle, cfg, rows=rows, p_format=pf)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    flops = 4.0 * rows_per_step * w.N * w.d            # the sampled rows against all keys
    value = flops / dt / 1e12
    sample = f"per step: preprocessing of 1 head in full + {rows_per_step} query rows x all {w.N} keys of that head"
    return {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "impl": "reference",
            "config": {"workload": w.name, "B": w.B, "H": w.H, "N": w.N, "d": w.d, "bits": bits, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def cpu_baseline(w, bits, hybrid=False, budget_rows=4096, heads=2):
    """The oracle as it stands on a bounded sample (about 10-30 s of CPU work)."""
    import numpy as np
    from oracle import attention as OA
    from oracle import prep as OP
    cfg, pf = _oracle_cfg(w, bits, hybrid)
    rows = np.linspace(0, w.N - 1, min(budget_rows, w.N)).astype(np.int64)
    tp = ta = 0.0
    for h in range(heads):
        q, k, v = [t[0, 0].float().numpy() for t in vc_inputs.make_qkv(w, heads=[h])]
        t0 = time.perf_counter()
        bundle = OP.prep_head(q, k, v, None, cfg)
        t1 = time.perf_counter()
        OA.emulate_head(bundle, cfg, rows=rows, p_format=pf)
        t2 = time.perf_counter()
        tp += t1 - t0
        ta += t2 - t1
    flops = 4.0 * heads * len(rows) * w.N * w.d
    # what the synthetic inputs look like to the softmax (not timed): spread of the exact scores
    # and the effective number of keys 1 / sum p^2 per row, on 64 rows of the last sampled head
    rs = np.linspace(0, w.N - 1, 64).astype(np.int64)
    cos, sin = OP.rope_tables(cfg)
    qr, kr = OP.rope_apply(q, cos, sin).astype(np.float64), OP.rope_apply(k, cos, sin).astype(np.float64)
    sc = (qr[rs] @ kr.T) / np.sqrt(w.d)
    pr_ = np.exp(sc - sc.max(axis=1, keepdims=True))
    pr_ /= pr_.sum(axis=1, keepdims=True)
    stats = {"score_std": float(sc.std(axis=1).mean()), "effective_keys": float((1.0 / (pr_ ** 2).sum(axis=1)).mean()),
             "rows": int(len(rs))}
    return {"value": flops / (tp + ta) / 1e12, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle", "input_statistics": stats,
            "sample": f"{heads} of {w.B * w.H} heads: preprocessing in full ({tp:.1f} s) + {len(rows)} of {w.N} query rows x "
                      f"all keys per head ({ta:.1f} s); NumPy, threads as its BLAS picks"}


def parity_report(w, p, q, k, v, perm, o, quant, work, bits, hybrid, int8_qk, n_rows=256):
    """The GPU output of one head on sampled query rows against the oracle's emulation of the same
    arrangement (the parity target) and against exact fp64 attention (accuracy), same buffers,
    same permutation.  Not timed."""
    import numpy as np
    import paper_2609_15810_b200 as vc
    from oracle import attention as OA
    from oracle import compare as CMP
    from oracle import prep as OP
    vc.vc_attn(p, q, k, v, perm, o, quant, work)          # the arrangement asked for, once more
    vc.vc_poll_status(work)
    h = w.H - 1
    f = lambda t: t[0, h].float().cpu().numpy()
    qh, kh, vh = f(q), f(k), f(v)
    pm = None if perm is None else perm[0, h].cpu().numpy().astype(np.int64)
    cfg, pf = _oracle_cfg(w, bits, hybrid)
    if int8_qk:
        cfg.qk_format = "int8"
    nb = (w.N + 127) // 128
    tiles = sorted({nb // 2, nb - 1})                      # a full tile and the ragged last one
    rows = np.concatenate([np.arange(128 * t, min(128 * (t + 1), w.N)) for t in tiles])[:n_rows]
    bundle = OP.prep_head(qh, kh, vh, pm, cfg)
    emu = OA.emulate_head(bundle, cfg, rows=rows, p_format=pf).astype(np.float64)
    exact = OA.reference_head(qh, kh, vh, cfg, rows=rows)
    got = o[0, h].float().cpu().numpy()[rows].astype(np.float64)
    vmax = float(np.abs(vh).max())
    pick = lambda m: {"max_err_over_vmax": m["max_err_over_vmax"], "cos": m["cos"], "psnr_db": float(m["psnr_db"])}
    return {"head": [0, h], "rows": int(len(rows)), "tolerance": "|delta| <= 2e-2 max|V| and cos >= 0.999 against the emulation",
            "gpu_vs_emulation": pick(CMP.output_metrics(got, emu, vmax)),
            "gpu_vs_exact_fp64": pick(CMP.output_metrics(got, exact, vmax)),
            "emulation_vs_exact_fp64": pick(CMP.output_metrics(emu, exact, vmax))}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3")
    ap.add_argument("--bits", type=int, default=8)
    ap.add_argument("--perm", default="group", choices=["group", "kmeans", "identity", "random"],
                    help="group: vc_group on the GPU, recomputed (warm-started) every 4th step inside the timed\n"
                         "region and reused in between; kmeans: the harness's torch k-means, computed once")
    ap.add_argument("--heads-per-pass", type=int, default=0)
    ap.add_argument("--variant", type=int, default=0, help="attention kernel (vc_params.kernel_variant)")
    ap.add_argument("--p-format", default="default", choices=["default", "expcast", "exp", "exp_poly", "exp_mix"],
                    help="8-bit probability format: ExpCast-FP8 (Eq. 7, the default) or exponentiate-then-cast with 2^u on the "
                         "special-function unit (exp), on the FMA pipe (exp_poly), or one score in four there (exp_mix)")
    ap.add_argument("--int8-qk", action="store_true", help="8-bit Q/K as INT8 and an integer score product (Fig. 3)")
    ap.add_argument("--calls", type=int, default=8, help="distinct input sets (noise redrawn per call) cycled through the steps")
    ap.add_argument("--ref-rows", type=int, default=1024)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="skip the short measurement of the 4-bit arrangements")
    ap.add_argument("--no-sdpa", action="store_true")
    ap.add_argument("--data", default="workload", choices=["workload", "gauss"],
                    help="gauss: same shapes, inputs drawn with three randn calls (for profiler runs, where the\n"
                         "thousands of small generator kernels of the workload recipe would dominate the capture)")
    args = ap.parse_args()
    w = vc_inputs.WORKLOADS[args.workload]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args, w, args.bits)), flush=True)
        return

    import paper_2609_15810_b200 as vc
    from paper_2609_15810_b200.binding import Params, alloc_buffers
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    sampler = ClockSampler(local_rank)
    sampler.start()
    # every rank runs the same workload on its own GPU (heads are independent: no collective)
    # BASELINE's config 3 is a SEQUENCE of calls: the smooth field, the K offsets and the V block
    # shifts stay, the noise is redrawn per call, and the permutation is recomputed every 4th call
    # and reused (stale) in between.  n_calls input sets are cycled through the timed steps.
    if args.data == "gauss":
        g = torch.Generator(device=dev).manual_seed(w.seed)
        inputs = [[torch.randn(w.B, w.H, w.N, w.d, generator=g, device=dev).to(torch.bfloat16) for _ in range(3)]]
    else:
        inputs = vc_inputs.make_qkv_calls(w, max(1, min(args.calls, args.steps)), device=dev)
    n_calls = len(inputs)
    q, k, v = inputs[0]
    p = Params.make(w.B, w.H, w.N, w.d, w.grid, bits=args.bits, heads_per_pass=args.heads_per_pass,
                    kernel_variant=args.variant, flags=15 | (16 if args.int8_qk else 0),
                    p_format={"default": 0, "expcast": 1, "exp": 2, "exp_poly": 4, "exp_mix": 5}[args.p_format])
    group_k, group_every = 64, 4
    if args.perm == "group":
        gwork = torch.empty(vc.vc_group_workspace_bytes(p), dtype=torch.uint8, device=dev)
        centroids = torch.zeros(w.B, w.H, group_k, w.d, dtype=torch.float32, device=dev)
        perm = torch.empty(w.B, w.H, w.N, dtype=torch.int32, device=dev)
        vc.vc_group(p, v, group_k, 4, False, centroids, perm, gwork)      # cold start: 4 Lloyd iterations
    elif args.perm == "kmeans":
        perm = vc_kmeans_harness.kmeans_perm_all(v)
    elif args.perm == "random":
        perm = vc_inputs.random_perm(w.B, w.H, w.N, w.seed, device=dev)
    else:
        perm = None
    quant, work = alloc_buffers(p, device=dev)
    o = torch.empty(w.B, w.H, w.N, w.d, dtype=torch.bfloat16, device=dev)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(args.warmup, 3)):
        qi, ki, vi = inputs[i % n_calls]
        vc.vc_attn(p, qi, ki, vi, perm, o, quant, work)
    vc.vc_poll_status(work)

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    launches0 = vc.vc_launch_count()
    barrier()
    wall0 = time.time()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record(stream)
    for s in range(args.steps):
        qi, ki, vi = inputs[s % n_calls]
        ev[s][3].record(stream)
        if args.perm == "group" and s % group_every == 0:     # a grouping step: one warm-started iteration
            vc.vc_group(p, vi, group_k, 1, True, centroids, perm, gwork)
        ev[s][0].record(stream)
        vc.vc_prep(p, qi, ki, vi, perm, quant, work)
        ev[s][1].record(stream)
        vc.vc_attn_fwd(p, quant, o, work)
        ev[s][2].record(stream)
    t_end.record(stream)
    barrier()
    wall1 = time.time()
    launches = vc.vc_launch_count() - launches0
    clocks = sampler.window(wall0, wall1)
    vc.vc_poll_status(work)
    if args.perm == "group":
        vc.vc_poll_status(gwork)
    ms_total = t_start.elapsed_time(t_end)
    prep_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in ev)
    attn_all = [e[1].elapsed_time(e[2]) for e in ev]
    prep_all = [e[0].elapsed_time(e[1]) for e in ev]
    attn_ms = statistics.mean(attn_all)
    group = None
    if args.perm == "group":
        calls = [e[3].elapsed_time(e[0]) for i, e in enumerate(ev) if i % group_every == 0]
        group = {"ms_per_call": statistics.mean(calls), "calls": len(calls), "every": group_every, "k": group_k,
                 "iters": {"cold": 4, "warm": 1}, "ms_amortized_per_step": sum(calls) / args.steps,
                 "share_of_attention_on_a_grouping_step": statistics.mean(calls) / attn_ms}
    value, ms_step = job_throughput(w.flops, ms_total / args.steps, world, dev)

    # end to end through the host-buffer entry point: H2D of Q, K, V, pi and D2H of O inside the timer
    e2e = None
    if not args.no_e2e:
        hq, hk, hv = [t.cpu().pin_memory() for t in (q, k, v)]
        hperm = perm.cpu().pin_memory() if perm is not None else None
        ho = torch.empty(o.shape, dtype=o.dtype).pin_memory()
        n_e2e = max(2, min(args.steps, 5))
        vc.vc_attn_host(p, hq, hk, hv, hperm, ho, q, k, v, perm, o, quant, work)
        barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            vc.vc_attn_host(p, hq, hk, hv, hperm, ho, q, k, v, perm, o, quant, work)
        barrier()
        e2e_value, e2e_ms = job_throughput(w.flops, (time.perf_counter() - t0) * 1e3 / n_e2e, world, dev)
        nbytes = q.numel() * 2
        e2e = {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": 3 * nbytes + (perm.numel() * 4 if perm is not None else 0),
               "d2h_bytes_per_step": nbytes, "steps": n_e2e}

    # the 4-bit arrangements on the same inputs and permutation, for the record (the metric names
    # both widths); the headline numbers above stay those of the arrangement asked for
    others = None
    if (world == 1 and not args.no_others and args.bits == 8 and args.p_format == "default" and not args.int8_qk
            and args.variant == 0):
        others = []
        for name, kw in (("4-bit: NVFP4 Q, K, V and P", dict(bits=4)),
                         ("4-bit hybrid: NVFP4 QK^T, ExpCast-FP8 P, FP8 x FP4 PV", dict(bits=4, p_format=1))):
            p2 = Params.make(w.B, w.H, w.N, w.d, w.grid, **kw)
            quant2, work2 = alloc_buffers(p2, device=dev)
            for i in range(3):
                qi, ki, vi = inputs[i % n_calls]
                vc.vc_attn(p2, qi, ki, vi, perm, o, quant2, work2)
            n2 = max(3, min(args.steps, 10))
            ev2 = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n2)]
            torch.cuda.synchronize()
            w0 = time.time()
            for s in range(n2):
                qi, ki, vi = inputs[s % n_calls]
                ev2[s][0].record(stream)
                vc.vc_prep(p2, qi, ki, vi, perm, quant2, work2)
                ev2[s][1].record(stream)
                vc.vc_attn_fwd(p2, quant2, o, work2)
                ev2[s][2].record(stream)
            torch.cuda.synchronize()
            w1 = time.time()
            vc.vc_poll_status(work2)
            pm = statistics.mean(e[0].elapsed_time(e[1]) for e in ev2)
            am = statistics.mean(e[1].elapsed_time(e[2]) for e in ev2)
            others.append({"arrangement": name, "hybrid": "p_format" in kw, "steps": n2, "prep_ms": pm, "attn_ms": am,
                           "attn_ms_min": min(e[1].elapsed_time(e[2]) for e in ev2),
                           "attn_tflops": w.flops / (am * 1e-3) / 1e12, "step_tflops": w.flops / ((pm + am) * 1e-3) / 1e12,
                           "clocks": sampler.window(w0, w1)})
            del quant2, work2

    # the pass with the statistics handed in (App. B: from the producer of K and V): K and V read once
    prep_stats_ms = None
    if world == 1 and args.bits == 8:
        try:
            qi, ki, vi = inputs[0]
            vc.vc_prep(p, qi, ki, vi, perm, quant, work)
            st = [t.clone() for t in vc.vc_prep_stats_view(p, quant, work)]
            for _ in range(3):
                vc.vc_prep_with_stats(p, qi, ki, vi, perm, st[0], st[1], st[2], quant, work)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(10):
                vc.vc_prep_with_stats(p, qi, ki, vi, perm, st[0], st[1], st[2], quant, work)
            e1.record(stream)
            torch.cuda.synchronize()
            prep_stats_ms = e0.elapsed_time(e1) / 10
        except Exception as exc:  # pragma: no cover
            prep_stats_ms = None

    # the tensor-core rate of this GPU for the products' MMAs alone (own microbenchmark, sub-second)
    mma_peak = None
    if world == 1:
        try:
            time.sleep(0.5)
            w0 = time.time()
            tf8, mac8 = vc.vc_mma_peak(8, 8192)
            tf4, mac4 = vc.vc_mma_peak(4, 8192)
            mma_peak = {"fp8_tflops": tf8, "fp8_mac_per_clk_sm": mac8, "fp4_tflops": tf4, "fp4_mac_per_clk_sm": mac4,
                        "what": "back-to-back tcgen05.mma on resident tiles, all SMs, 2 x 8192 products of 128^3 per SM and kind "
                                "(kind::f8f6f4 E4M3; kind::mxf4nvf4 block16), CUDA events",
                        "clocks": sampler.window(w0, time.time())}
        except Exception as exc:  # pragma: no cover
            mma_peak = {"error": str(exc)[:200]}
    sampler.stop()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = _peaks()
    # Dominant kernel: the attention forward, a dense contraction on the tensor cores.  Its peak is
    # the measured bf16 figure x the nominal ratio of its own format (FP8 : bf16 = 2, FP4 : bf16 = 4;
    # the hybrid arrangement runs half of its FLOPs at each rate: 1/4 + 1/2 of a bf16 pass = 8/3).
    # `frac` is taken against the BURST figure: the timed region is a fraction of a second and the
    # sampled SM clocks sit near the maximum, which is the state the burst figure was measured in;
    # the fraction of the sustained figure (measured minutes-long under the power cap at a much lower
    # clock) is kept beside it, as are the fractions of the nominal peak and of this GPU's own
    # MMA-only rate.
    hybrid = args.bits == 4 and args.p_format == "expcast"

    def roofline_of(ms, ms_all, bits, hyb, clk):
        ratio = 2.0 if bits == 8 else (8.0 / 3.0 if hyb else 4.0)
        nominal = 4500.0 if bits == 8 else (6000.0 if hyb else 9000.0)
        ach = w.flops / (ms * 1e-3) / 1e12
        r = {"bound": "tensor", "kernel": "vc_attn_fwd", "achieved": ach, "peak": peaks["bf16_burst"] * ratio, "unit": UNIT,
             "frac": ach / (peaks["bf16_burst"] * ratio),
             "peak_source": f"{peaks['source']}: bf16 burst {peaks['bf16_burst']} TF/s x {ratio:.4g} (nominal ratio of the format to bf16)",
             "frac_of_sustained": ach / (peaks["bf16_sustained"] * ratio),
             "sustained_peak": peaks["bf16_sustained"] * ratio,
             "frac_of_nominal": ach / nominal, "nominal_peak": nominal,
             "ms": ms}
        if ms_all:
            r.update({"ms_median": statistics.median(ms_all), "ms_min": min(ms_all)})
        if mma_peak and "fp8_tflops" in mma_peak:
            own = mma_peak["fp8_tflops"] if bits == 8 else (1.0 / (0.5 / mma_peak["fp4_tflops"] + 0.5 / mma_peak["fp8_tflops"]) if hyb
                                                            else mma_peak["fp4_tflops"])
            r.update({"mma_only_peak": own, "frac_of_mma_only_peak": ach / own})
        if clk and clk.get("sm_mhz"):
            # time x clock: cycles per step, the figure to compare across boxes that settle at different clocks
            r["ms_x_sm_mhz"] = ms * clk["sm_mhz"]
        return r

    achieved = w.flops / (attn_ms * 1e-3) / 1e12
    # DRAM traffic of one attention launch: measured once under ncu on a smaller case of the same
    # kernel (the headline launch is too long to capture) and proportional to B*H*N (codes in,
    # bf16 out; key/value re-reads are L2 hits)
    per_ht = {8: 322.2e6, 4: 219.2e6}[args.bits] / (32 * 16384) * (w.d / 128.0)
    traffic = per_ht * w.B * w.H * w.N
    n_pad = 128 * ((w.N + 127) // 128)
    prep_bytes = w.B * w.H * (3 * w.N * w.d * 2 + 2 * w.N * 4 + 3 * n_pad * w.d * (1 if args.bits == 8 else 0.5625)
                              + (2 * (n_pad // 128) * 4 + w.d * 4) + (n_pad // 128) * w.d * 2)
    prep_gbs = prep_bytes / (prep_ms * 1e-3) / 1e9
    roof = roofline_of(attn_ms, attn_all, args.bits, hybrid, clocks)
    roof.update({"traffic": traffic,
                 "traffic_source": "ncu dram__bytes_read+write of this kernel on B2 H16 N16384 d128, scaled by "
                                   "head-tokens: %.0f B per (head, token)" % per_ht})
    if others:
        for oth in others:
            oth["roofline"] = roofline_of(oth["attn_ms"], None, 4, oth["hybrid"], oth["clocks"])
            oth["roofline"]["ms_min"] = oth["attn_ms_min"]
    targets = {"attention_frac_of_nominal_fp8_peak": {"target": 0.60, "measured": roof["frac_of_nominal"] if args.bits == 8 else None},
               "prep_frac_of_8tbs": {"target": 0.70, "measured": prep_gbs / 8000.0},
               "met": bool(args.bits == 8 and roof["frac_of_nominal"] >= 0.60 and prep_gbs / 8000.0 >= 0.70)}
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": ("int8 QK / e4m3 PV" if args.int8_qk else "e4m3") if args.bits == 8 else ("nvfp4 QK / e4m3 x e2m1 PV" if hybrid else "nvfp4"), "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "N": w.N, "d": w.d, "grid": list(w.grid),
                   "bits": args.bits, "p_format": args.p_format, "perm": args.perm, "data": args.data, "calls": n_calls, "l2": "inputs larger than L2 (Q+K+V = %.0f MB)" % (3 * q.numel() * 2 / 1e6),
                   "step": "vc_prep + vc_attn_fwd" + (" (+ vc_group every 4th step)" if args.perm == "group" else "")
                           + (f"; {n_calls} input sets cycled (noise redrawn per call, permutation stale between regroupings)" if n_calls > 1 else "")},
        "clocks": clocks, "gpu_launches": launches, "e2e": e2e, "other_arrangements": others,
        "roofline": roof, "mma_only_peak": mma_peak, "targets": targets,
        "group": group,
        "prep": {"ms": prep_ms, "ms_median": statistics.median(prep_all), "ms_min": min(prep_all), "algorithmic_gb": prep_bytes / 1e9, "gbs": prep_gbs,
                 "frac_of_measured_hbm": prep_gbs / peaks["hbm_gbs"], "frac_of_8tbs": prep_gbs / 8000.0,
                 "with_supplied_statistics": None if prep_stats_ms is None else
                 {"ms": prep_stats_ms, "gbs": prep_bytes / (prep_stats_ms * 1e-3) / 1e9,
                  "frac_of_measured_hbm": prep_bytes / (prep_stats_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                  "what": "vc_prep_with_stats: K mean, V block means and residual maxima from the caller, no statistics launches"}},
    }
    if not args.no_sdpa:
        try:    # context only: a library bf16 attention on the same GPU and tensors
            import torch.nn.functional as F
            for _ in range(2):
                F.scaled_dot_product_attention(q, k, v)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(3):
                F.scaled_dot_product_attention(q, k, v)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / 3
            out["bf16_sdpa"] = {"ms": ms, "tflops": w.flops / (ms * 1e-3) / 1e12, "what": "torch SDPA bf16, default backend, no RoPE/quantization"}
        except Exception as exc:  # pragma: no cover
            out["bf16_sdpa"] = {"error": str(exc)[:200]}
    if not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(w, args.bits, hybrid)
        if args.data == "workload":
            out["parity"] = parity_report(w, p, q, k, v, perm, o, quant, work, args.bits, hybrid, args.int8_qk)
    print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
