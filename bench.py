#!/usr/bin/env python
"""Benchmark of the GELO obfuscated Q/K/V offload on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one prefill sweep over the 32 layers of a Llama-2-7B-shaped model: 32 calls of
the whole path (sample a fresh A, shield rows, mix, project, unmix) on n = 4096 token rows
with d = 4096, p = 12288, 204 shield rows, bf16 storage, mixing kind alternating between
orthogonal and non-orthogonal.  Inputs are seeded synthetic tensors (see
paper_2603_05035_b200/inputs.py).  Rank 0 prints ONE JSON line.

With N > 1 every rank runs an independent replica of the same sweep (the path has no
exchange step), and the value is the total number of token rows all ranks pushed through
the obfuscated projection divided by the slowest rank's time.

--impl reference times the fp64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

# The batched entry points keep up to 32 lane streams busy; with the default of eight hardware work queues, streams
# that share a queue wait for each other's launches (measured: 121.3 -> 118.7 ms per sweep).  The variable is read when
# the CUDA context is created, i.e. it has to be set before torch touches the GPU; a caller's own setting wins.
os.environ.setdefault("CUDA_DEVICE_MAX_CONNECTIONS", "32")

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "obfuscated-QKV tokens/s at Llama-2-7B shapes"
UNIT = "tokens/s"
WORKLOAD = "prefill_bf16"
# DRAM bytes over algorithmic bytes of the panel kernels, from one ncu capture of a panel of 3300 rows; traffic
# scales with the rows, so other panel heights use the same ratio (0.58 MB against 8 B x 4300 rows x 32 columns).
PANEL_TRAFFIC_RATIO = 0.53


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_rate(units_per_rank: float, world: int, slowest_ms: float) -> float:
    """Units all ranks processed divided by the slowest rank's time (replicas: weak scaling)."""
    return units_per_rank * world / (slowest_ms * 1e-3)


def replica_seed_base(rank: int) -> int:
    """Replicas draw different inputs and mixing seeds."""
    return rank * 1000


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "200",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------
# reference arm and CPU baseline: the oracle on the host cores
# ---------------------------------------------------------------------------------------------

def oracle_sample_step(w, n_s, k_s, call):
    """One oracle pass of the whole path on a reduced row count (same d, p, dtype, kinds)."""
    import numpy as np
    import oracle
    from paper_2603_05035_b200 import inputs
    seed = w.seed + call
    H = inputs.to_f64_numpy(inputs.make_hidden(n_s, w.d, w.dtype, seed, w.rms_norm))
    W = inputs.to_f64_numpy(inputs.make_weight(w.d, w.p, w.dtype, seed))
    t0 = time.perf_counter()
    A, X, _, _ = oracle.sample_mixing_verified(n_s + k_s, w.kind(call), seed)
    S = oracle.shield_rows(H, k_s, w.shield_scale, seed) if k_s else None
    Y = oracle.chain(A, X, H, S, W)
    dt = time.perf_counter() - t0
    assert np.isfinite(Y).all()
    return dt


def oracle_sample_desc(n_s, k_s, w):
    return (f"whole path (sample A, shields, mix, project, unmix) in fp64 on n={n_s} data rows + {k_s} "
            f"shield rows per call, d={w.d}, p={w.p}; tokens/s = {n_s} / seconds per call")


def run_reference(args):
    import oracle
    from paper_2603_05035_b200 import inputs
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    oracle.build()
    w = inputs.WORKLOADS[WORKLOAD]
    n_s, k_s = 512, 26
    for i in range(args.warmup):
        oracle_sample_step(w, 16, 1, i)
    times = [oracle_sample_step(w, n_s, k_s, i) for i in range(args.steps)]
    total = sum(times)
    value = n_s * args.steps / total
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "n": w.n, "k": w.k, "d": w.d, "p": w.p, "calls_per_step": 1,
                   "note": "CPU oracle on a bounded sample; one step = one call of the sample"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": oracle_sample_desc(n_s, k_s, w)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ---------------------------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------------------------

def run_ours(args):
    import torch
    import paper_2603_05035_b200 as gelo
    from paper_2603_05035_b200 import inputs

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus != world and world > 1:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    w = inputs.WORKLOADS[WORKLOAD]
    n, k, d, p, m = w.n, w.k, w.d, w.p, w.m
    calls = args.calls if args.calls > 0 else w.calls
    td = inputs.torch_dtype(w.dtype)
    dev = torch.device("cuda", local_rank)
    peaks = _peaks()

    ctx = gelo.Context(local_rank)
    ctx.set_lanes(args.lanes)
    ctx.set_level3(args.level3)
    ctx.set_lane_share(args.lane_share)
    ctx.ensure_batch_workspace(n, k, d, p, w.dtype, args.lanes)
    # replicas draw different inputs and mixing seeds
    base = replica_seed_base(rank)
    Hs, Ws, seeds = [], [], []
    for c in range(calls):
        h = inputs.make_hidden(n, d, w.dtype, w.seed + base + c, w.rms_norm, dev)
        wt = inputs.make_weight(d, p, w.dtype, w.seed + base + c, dev)
        Hs.append(h); Ws.append(wt); seeds.append(w.seed + base + c)
    Q = torch.empty((n, p // 3), device=dev, dtype=td); K = torch.empty_like(Q); V = torch.empty_like(Q)
    checksum = torch.zeros((), device=dev, dtype=torch.float32)

    kinds = [w.kind(c) for c in range(calls)]

    def sweep(step):
        # one batched call per sweep: the library samples the A of several calls concurrently
        ctx.qkv_offload_batch(Hs, Ws, n, k, d, p, kinds, [s_ + 100000 * step for s_ in seeds], w.shield_scale,
                              w.dtype, [Q] * calls, [K] * calls, [V] * calls)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        sweep(-1 - i)
    barrier()
    if ctx.last_status() != gelo.OK:
        raise SystemExit("device-side error during warm-up")

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    ctx.launch_count(reset=True)
    barrier()
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for s in range(args.steps):
        sweep(s)
    e1.record()
    barrier()
    ms = e0.elapsed_time(e1)
    launches = ctx.launch_count()
    clocks = sampler.stop() if rank == 0 else None
    status = ctx.last_status()
    if status != gelo.OK:
        raise SystemExit(f"device-side error {status} in the timed region")
    checksum += Q.float().abs().mean()

    if args.timed_only:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": float(n) * calls * args.steps / (ms * 1e-3), "unit": UNIT,
                              "ms_per_step": ms / args.steps, "gpu_launches": launches, "timed_only": True,
                              "config": {"workload": WORKLOAD, "calls_per_step": calls}}))
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        ctx.close()
        return 0

    # ---- per-stage device times (CUDA events on the launching stream), a few calls each ----
    stage_ms = {}
    lda = ctx.mixing_ld(m)
    A = torch.empty((m, lda), device=dev, dtype=td); X = torch.empty_like(A)
    S = torch.empty((k, d), device=dev, dtype=td)
    U = torch.empty((m, d), device=dev, dtype=td); Yp = torch.empty((m, p), device=dev, dtype=td)

    def timed(name, fn, reps):
        fn(0)
        torch.cuda.synchronize()
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record()
        for r in range(reps):
            fn(r + 1)
        b.record()
        torch.cuda.synchronize()
        stage_ms[name] = a.elapsed_time(b) / reps

    timed("sample_orthogonal", lambda r: ctx.sample_mixing(m, gelo.ORTHOGONAL, 900 + r, w.dtype, A, X, lda), 2)
    timed("sample_nonorthogonal", lambda r: ctx.sample_mixing(m, gelo.NONORTHOGONAL, 900 + r, w.dtype, A, X, lda), 2)
    timed("shield_rows", lambda r: ctx.shield_rows(Hs[r % calls], n, d, k, w.shield_scale, 5 + r, w.dtype, S), 8)
    timed("mix", lambda r: ctx.mix(A, lda, Hs[r % calls], S, n, k, d, w.dtype, U), 8)
    timed("project", lambda r: ctx.project(U, Ws[r % calls], m, d, p, w.dtype, Yp), 8)
    timed("unmix", lambda r: ctx.unmix(X, lda, Yp, n, k, p, w.dtype, Q, K, V), 8)
    timed("plain_project", lambda r: ctx.project(Hs[r % calls], Ws[r % calls], n, d, p, w.dtype, Yp), 8)
    # the same product on E4M3 operands: weights quantised once (they are resident), U quantised per call
    U8 = torch.empty((m, d), device=dev, dtype=torch.uint8); W8 = torch.empty((d, p), device=dev, dtype=torch.uint8)
    su = torch.zeros(2, device=dev); sw = torch.zeros(2, device=dev)
    ctx.quantize_e4m3(Ws[0], d, p, w.dtype, W8, sw)
    timed("quantize_u_e4m3", lambda r: ctx.quantize_e4m3(U, m, d, w.dtype, U8, su), 8)
    timed("project_e4m3", lambda r: ctx.project_e4m3(U8, su, W8, sw, m, d, p, Yp), 8)
    del U8, W8
    # the level-3 update that leads the SM time of the factorisations: C -= V W with the 512 reflectors of a superblock,
    # one tf32 product straight from the fp32 matrices (first superblock of the QR: 4300 x 3788, K = 512)
    um, un, uk = m, m - 512, 512
    uV = torch.randn((um, uk), device=dev); uW = torch.randn((uk, lda), device=dev)
    uC = [torch.randn((um, lda), device=dev) for _ in range(4)]             # 4 x 75 MB: C never waits in L2
    ctx.set_level3(3)
    timed("tf32_update", lambda r: ctx.update_f32(um, un, uk, uV, uk, uW, lda, uC[r % 4], lda), 16)
    ctx.set_level3(args.level3)
    del uV, uW, uC
    chain_ms = stage_ms["mix"] + stage_ms["project"] + stage_ms["unmix"]
    chain_flops = 2.0 * m * m * d + 2.0 * m * d * p + 2.0 * n * m * p
    plain_flops = 2.0 * n * d * p

    # ---- end to end through the host-buffer entry point (H2D of H, D2H of Q/K/V inside) ----
    Hh = [Hs[c % calls].cpu().pin_memory() for c in range(4)]
    Qh = torch.empty((n, p // 3), dtype=td).pin_memory(); Kh = torch.empty_like(Qh).pin_memory()
    Vh = torch.empty_like(Qh).pin_memory()
    e2e_calls = calls
    Hh_list = [Hh[c % 4] for c in range(calls)]
    ctx.qkv_offload_batch_host(Hh_list[:4], Ws[:4], n, k, d, p, kinds[:4], seeds[:4], w.shield_scale, w.dtype,
                               [Qh] * 4, [Kh] * 4, [Vh] * 4)
    ctx.qkv_offload_batch_host(Hh_list, Ws, n, k, d, p, kinds, [s_ + 5 for s_ in seeds], w.shield_scale, w.dtype,
                               [Qh] * calls, [Kh] * calls, [Vh] * calls)
    barrier()
    t0 = time.perf_counter()
    for s_i in range(args.steps):
        # enqueue-only variant: the sampling lanes keep running across the step boundary, as in the device-resident loop
        ctx.qkv_offload_batch_host_async(Hh_list, Ws, n, k, d, p, kinds, [s_ + 7 + s_i for s_ in seeds], w.shield_scale,
                                         w.dtype, [Qh] * calls, [Kh] * calls, [Vh] * calls)
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - t0) / args.steps
    checksum += Qh.float().abs().mean().to(dev)

    ms_max, e2e_ms_max = max_over_ranks([ms, e2e_s * 1e3], dist, dev)
    value = whole_job_rate(float(n) * calls * args.steps, world, ms_max)
    e2e_value = whole_job_rate(float(n) * e2e_calls, world, e2e_ms_max)

    # ---- per-launch device times of the main kernel classes (CUDA events on the launching stream):
    #      one orthogonal and one non-orthogonal call, sampling lanes off so that launches do not overlap ----
    ctx.set_lanes(1)
    ctx.profile_start()
    ctx.qkv_offload_batch(Hs[:2], Ws[:2], n, k, d, p, [gelo.ORTHOGONAL, gelo.NONORTHOGONAL], [s_ + 31 for s_ in seeds[:2]],
                          w.shield_scale, w.dtype, [Q] * 2, [K] * 2, [V] * 2)
    prof = ctx.profile_stop()
    ctx.set_lanes(args.lanes)
    kernels = {}
    for name, st_ in prof.items():
        if st_["launches"] == 0:
            continue
        rate = st_["work"] / (st_["ms"] * 1e-3)
        kernels[name] = {"launches": st_["launches"], "ms": round(st_["ms"], 4),
                         "avg_us": round(1e3 * st_["ms"] / st_["launches"], 3),
                         "achieved": rate / (1e12 if st_["unit"] == "flops" else 1e9),
                         "unit": "TFLOP/s" if st_["unit"] == "flops" else "GB/s"}
    dominant = max(kernels, key=lambda k_: kernels[k_]["ms"])

    # ---- structured variant (reported beside the method, never as the method): block-diagonal orthogonal A ----
    variants = {}
    if not args.no_variants:
        for block in (512, 1024):
            ctx.ensure_blockdiag_workspace(n, k, d, p, w.dtype, block, args.lanes)
            def vsweep(step):
                ctx.qkv_offload_blockdiag_batch(Hs, Ws, n, k, d, p, block, [s_ + 300000 + 1000 * step for s_ in seeds],
                                                w.shield_scale, w.dtype, [Q] * calls, [K] * calls, [V] * calls)
            for i in range(3):
                vsweep(-1 - i)
            torch.cuda.synchronize()
            a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
            a.record()
            for s_i in range(args.steps):
                vsweep(s_i)
            b.record()
            torch.cuda.synchronize()
            vms = a.elapsed_time(b) / args.steps
            variants[f"block_{block}"] = {"ms_per_step": vms, "value": float(n) * calls / (vms * 1e-3), "unit": UNIT,
                                          "groups": -(-m // block),
                                          "note": "rows mix inside groups of about `block` rows only (weaker hiding than the dense A of the method)"}
        if ctx.last_status() != gelo.OK:
            raise SystemExit("device-side error in the variant runs")

    workloads = {}
    if world == 1 and not args.no_workloads:
        # the other configurations, a few sweeps each; their numbers ride along in the main line
        ctx.set_workspace(None)
        torch.cuda.empty_cache()
        for name_ in ("tiny_f32", "layer_f32", "shield_bf16", "decode_bf16"):
            lat = args.latency_steps if name_ == "decode_bf16" else 0
            workloads[name_] = compact(measure_workload(name_, min(args.lanes, 16) if name_ != "shield_bf16" else args.lanes,
                                                        5, 3, 0, lat))

    if rank == 0:
        es = 2 if w.dtype == "bf16" else 4
        dk = kernels[dominant]
        # FP32 FMA peak of the whole GPU: 148 SMs x 128 lanes x 2 flop x 1.965 GHz (max SM clock)
        alu_peak = 148 * 128 * 2 * 1.965e9 / 1e12
        descr = {"rank_update": "rank_update_kernel: C -= A B inside the QR / LU outer blocks",
                 "vtc": "vtc_partial_kernel: V^T C inside the QR outer blocks",
                 "gemm_tc": "gemm_tc_kernel: tcgen05 GEMM (mix / project / unmix and the level-3 QR / LU updates)",
                 "qr_panel": "qr_panel_cluster_kernel: 32-column Householder panel in registers across a cluster of <= 8 CTAs",
                 "lu_panel": "lu_panel_cluster_kernel: 32-column pivoted LU panel in registers across a cluster of <= 8 CTAs"}
        roofline = {"kernel": descr[dominant], "achieved": dk["achieved"], "unit": dk["unit"],
                    "avg_launch_us": dk["avg_us"], "launches_timed": dk["launches"], "traffic": None}
        if dominant in ("qr_panel", "lu_panel"):
            per_flop = 2.0 if dominant == "qr_panel" else 1.0
            avg_rows = prof[dominant]["work"] / prof[dominant]["launches"] / (per_flop * 32 * 32)
            roofline.update({"bound": "alu", "peak": alu_peak, "frac": dk["achieved"] / alu_peak,
                             "peak_source": "derived: 148 SMs x 128 FP32 lanes x 2 x 1.965 GHz",
                             "sms_used": 8, "frac_of_sms_used": dk["achieved"] / (alu_peak * 8 / 148),
                             "note": "latency-bound by design: 33 dependent column steps per launch on one cluster; "
                                     "other lanes' kernels use the remaining SMs concurrently",
                             # ncu: 0.58 MB DRAM per launch against 1.10 MB algorithmic (8 B x rows x 32) at rows = 4300
                             "traffic": PANEL_TRAFFIC_RATIO * 8.0 * avg_rows * 32})
        elif dk["unit"] == "TFLOP/s":
            roofline.update({"bound": "tensor", "peak": peaks["bf16_tflops"], "frac": dk["achieved"] / peaks["bf16_tflops"],
                             "peak_source": peaks["source"] + " (burst bf16 GEMM)"})
        else:
            roofline.update({"bound": "hbm", "peak": peaks["hbm_gbs"], "frac": dk["achieved"] / peaks["hbm_gbs"],
                             "peak_source": peaks["source"] + " (copy bandwidth)"})
        # the projection GEMM on its own (one launch per call), the contraction the paper offloads (Eq. 2)
        proj_tflops = 2.0 * m * d * p / (stage_ms["project"] * 1e-3) / 1e12
        projection = {"kernel": "gemm_tc_kernel, Y' = U W", "bound": "tensor", "achieved": proj_tflops,
                      "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": proj_tflops / peaks["bf16_tflops"],
                      # ncu: dram read 162.6 MB + write 85.5 MB per launch (algorithmic 241.6 MB)
                      "traffic": 248.0e6}
        f8_tflops = 2.0 * m * d * p / (stage_ms["project_e4m3"] * 1e-3) / 1e12
        projection_e4m3 = {"kernel": "gemm_tc_kernel (kind::f8f6f4), Y' = (s_U s_W) U8 W8", "bound": "tensor", "achieved": f8_tflops,
                           "peak": 2.0 * peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": f8_tflops / (2.0 * peaks["bf16_tflops"]),
                           "peak_source": peaks["source"] + " bf16 GEMM x nominal fp8/bf16 ratio 2",
                           # ncu: dram read 69.9 MB + write 61.2 MB (algorithmic 173.6 MB; operands quantised just before were partly in L2)
                           "traffic": 131.1e6,
                           "note": "same product as roofline_projection_gemm on E4M3 operands; FP8-grade accuracy (see DESIGN)"}
        upd_tflops = 2.0 * um * un * uk / (stage_ms["tf32_update"] * 1e-3) / 1e12
        tf32_peak = 0.5 * peaks["bf16_tflops"]          # nominal dense tf32 : bf16 = 1.125 : 2.25
        update_roof = {"kernel": "gemm_tc_kernel (tf32, reduce-add epilogue), C -= V W, M=4300 N=3788 K=512",
                       "bound": "tensor", "achieved": upd_tflops, "peak": tf32_peak, "unit": "TFLOP/s",
                       "frac": upd_tflops / tf32_peak,
                       "peak_source": peaks["source"] + " bf16 GEMM x nominal tf32/bf16 ratio 0.5",
                       # ncu: dram read 82.1 MB + write 9.0 MB per launch (algorithmic 147 MB, half of C stays in L2)
                       "traffic": 91.1e6,
                       "note": "largest share of SM time among the sampling kernels; "
                               "510 tiles of 16 k-blocks on 148 CTAs: fp32 operands re-read from L2 for every 128 x 256 tile (8.8 TB/s L2 -> SM) "
                               "and the 3.45-wave quantisation; 630 TFLOP/s sustained at large K"}
        per_call_ms = ms_max / args.steps / calls
        chain_tflops = chain_flops / (chain_ms * 1e-3) / 1e12
        # all arithmetic of a sweep against the time the sweep takes with every lane busy: the Householder QR of every
        # call ((8/3) m^3 with the explicit Q), one Newton-Schulz step (4 m^3) per orthogonal call on the tf32 route, LU
        # and inverse (2 m^3) per non-orthogonal call, and the three products; tf32 and split-bf16 flops are counted
        # once each, so this is a lower-is-slack figure against the bf16 peak
        n_orth = sum(1 for c_ in range(calls) if kinds[c_] == gelo.ORTHOGONAL)
        sweep_flops = calls * ((8.0 / 3.0) * m ** 3 + chain_flops) + n_orth * 4.0 * m ** 3 + (calls - n_orth) * 2.0 * m ** 3
        sweep_tflops = sweep_flops / (ms_max / args.steps * 1e-3) / 1e12
        sweep_roof = {"kernel": "all kernels of one sweep, lanes saturated (SM-time-weighted)", "bound": "tensor",
                      "achieved": sweep_tflops, "unit": "TFLOP/s", "peak": peaks["bf16_tflops_sustained"],
                      "frac": sweep_tflops / peaks["bf16_tflops_sustained"],
                      "peak_source": peaks["source"] + " (sustained bf16 GEMM)", "traffic": None,
                      "algorithmic_flops_per_sweep": sweep_flops}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_max / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": WORKLOAD, "n": n, "k": k, "m": m, "d": d, "p": p, "calls_per_step": calls,
                       "mixing": "alternating orthogonal / non-orthogonal, fresh A per call",
                       "shield_scale": w.shield_scale, "l2": "inputs_larger_than_l2",
                       "api": "gelo_qkv_offload_batch", "lanes": args.lanes,
                       "replicas": world},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": calls * n * d * es,
                    "d2h_bytes_per_step": calls * n * p * es, "calls_timed": e2e_calls},
            "gpu_launches": launches,
            "roofline": roofline,
            "roofline_projection_gemm": projection,
            "roofline_level3_update": update_roof,
            "roofline_projection_e4m3": projection_e4m3,
            "kernels": kernels,
            "stage_ms": {k_: round(v, 4) for k_, v in stage_ms.items()},
            # the metric's second half: the WHOLE obfuscated call (sampling A, shields, three products) against the plain,
            # unprotected H W on the same kernel; the products alone and their arithmetic floor beside it
            "overhead_vs_plain_gemm": per_call_ms / stage_ms["plain_project"],
            "products_vs_plain_gemm": chain_ms / stage_ms["plain_project"],
            "flop_floor_vs_plain": chain_flops / plain_flops,
            "per_call_ms": per_call_ms,
            "chain": {"ms": chain_ms, "tflops": chain_tflops,
                      "products_vs_plain_gemm": chain_ms / stage_ms["plain_project"],
                      "flop_floor_vs_plain": chain_flops / plain_flops,
                      "frac_of_peak": {"measured_burst": chain_tflops / peaks["bf16_tflops"],
                                       "measured_sustained": chain_tflops / peaks["bf16_tflops_sustained"],
                                       "nominal_2250": chain_tflops / 2250.0}},
            "roofline_whole_sweep": sweep_roof,
            "checksum": float(checksum),
        }
        if workloads:
            line["workloads"] = workloads
        if variants:
            line["variants_block_diagonal_A"] = variants
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            oracle.build()
            n_s, k_s = 512, 26
            dt_s = oracle_sample_step(w, n_s, k_s, 0)
            line["cpu_baseline"] = {"value": n_s / dt_s, "unit": UNIT, "cores": oracle.num_threads(),
                                    "kind": "oracle", "sample": oracle_sample_desc(n_s, k_s, w)}
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    ctx.close()
    return 0


def measure_workload(name, lanes, steps, warmup, calls=0, latency_steps=0):
    """Whole-path rate of one of the other workloads (the parity-test configurations) through the batched entry
    point, per-stage device times, overhead against the plain H W GEMM on the same kernel.  With `latency_steps`
    (the decode-shaped workload) also the distribution of the per-call latency over that many sweeps."""
    import numpy as np
    import torch
    import paper_2603_05035_b200 as gelo
    from paper_2603_05035_b200 import inputs

    w = inputs.WORKLOADS[name]
    n, k, d, p, m = w.n, w.k, w.d, w.p, w.m
    calls = calls if calls > 0 else 32
    td = inputs.torch_dtype(w.dtype)
    dev = torch.device("cuda", torch.cuda.current_device())
    peaks = _peaks()
    ctx = gelo.Context(dev.index)
    ctx.set_lanes(lanes)
    ctx.ensure_batch_workspace(n, k, d, p, w.dtype, lanes)
    Hs = [inputs.make_hidden(n, d, w.dtype, w.seed + c, w.rms_norm, dev) for c in range(calls)]
    Ws = [inputs.make_weight(d, p, w.dtype, w.seed + c, dev) for c in range(calls)]      # 32 distinct W: larger than L2
    Q = torch.empty((n, p // 3), device=dev, dtype=td); K = torch.empty_like(Q); V = torch.empty_like(Q)
    kinds = [w.kind(c) for c in range(calls)]

    if m <= 128:
        # small batches run whole calls on concurrent lanes: every call gets its own outputs
        Qs = [torch.empty_like(Q) for _ in range(calls)]; Ks = [torch.empty_like(Q) for _ in range(calls)]
        Vs = [torch.empty_like(Q) for _ in range(calls)]
    else:
        Qs, Ks, Vs = [Q] * calls, [K] * calls, [V] * calls

    def sweep(step):
        ctx.qkv_offload_batch(Hs, Ws, n, k, d, p, kinds, [w.seed + 100000 * (step + 7) + c for c in range(calls)],
                              w.shield_scale, w.dtype, Qs, Ks, Vs)

    for i in range(max(3, warmup)):
        sweep(-1 - i)
    torch.cuda.synchronize()
    sampler = ClockSampler(dev.index)
    sampler.start()
    ctx.launch_count(reset=True)
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    e0.record()
    for s_ in range(steps):
        sweep(s_)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    launches = ctx.launch_count()
    clocks = sampler.stop()
    if ctx.last_status() != gelo.OK:
        raise SystemExit(f"device-side error in the timed region of {name}")

    stage_ms = {}
    lda = ctx.mixing_ld(m)
    A = torch.empty((m, lda), device=dev, dtype=td); X = torch.empty_like(A)
    S = torch.empty((max(k, 1), d), device=dev, dtype=td)
    U = torch.empty((m, d), device=dev, dtype=td); Yp = torch.empty((m, p), device=dev, dtype=td)

    def timed(key, fn, reps):
        fn(0)
        torch.cuda.synchronize()
        a = torch.cuda.Event(enable_timing=True); b = torch.cuda.Event(enable_timing=True)
        a.record()
        for r in range(reps):
            fn(r + 1)
        b.record()
        torch.cuda.synchronize()
        stage_ms[key] = a.elapsed_time(b) / reps

    kind0 = kinds[0]
    timed("sample", lambda r: ctx.sample_mixing(m, kind0, 900 + r, w.dtype, A, X, lda), 4)
    if k:
        timed("shield_rows", lambda r: ctx.shield_rows(Hs[r % calls], n, d, k, w.shield_scale, 5 + r, w.dtype, S), 16)
    timed("mix", lambda r: ctx.mix(A, lda, Hs[r % calls], S if k else None, n, k, d, w.dtype, U), 16)
    timed("project", lambda r: ctx.project(U, Ws[r % calls], m, d, p, w.dtype, Yp), 32)
    timed("unmix", lambda r: ctx.unmix(X, lda, Yp, n, k, p, w.dtype, Q, K, V), 16)
    if m <= 128 and w.dtype != "f32" and p % 32 == 0:
        # small batches run Eq. 2 and Eq. 3 as one kernel inside the whole call
        timed("project_unmix", lambda r: ctx.project_unmix(U, Ws[r % calls], X, lda, n, k, d, p, w.dtype, Q, K, V), 32)
    # the plain, unprotected projection through the same entry point, hence on the same kernel as the chain's products
    timed("plain_project", lambda r: ctx.project(Hs[r % calls], Ws[r % calls], n, d, p, w.dtype, Yp), 32)
    if w.dtype == "f32":
        # a context without workspace has no room for operand pairs: the same product on the FP32 FMA pipes
        bare = gelo.Context(dev.index)
        timed("plain_project_fma", lambda r: bare.project(Hs[r % calls], Ws[r % calls], n, d, p, w.dtype, Yp), 8)
        bare.close()
    per_call_ms = ms / (steps * calls)
    es = 2 if w.dtype != "f32" else 4
    proj_s = stage_ms["project"] * 1e-3
    chain_flops = 2.0 * m * m * d + 2.0 * m * d * p + 2.0 * n * m * p
    if w.dtype == "bf16" and m >= 512:
        roof = {"bound": "tensor", "achieved": 2.0 * m * d * p / proj_s / 1e12, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
    elif w.dtype == "bf16":
        # small batch: the projection is a stream of W.  Inside the call it runs fused with the unmixing (project_unmix):
        # algorithmic bytes = U + W in, Q | K | V out
        fused_s = stage_ms.get("project_unmix", stage_ms["project"]) * 1e-3
        roof = {"bound": "hbm", "achieved": es * (m * d + d * p + n * p) / fused_s / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "kernel": "project_unmix_kernel: Y' = U W streamed once, unmixed on chip",
                # ncu (n = 64, k = 4, d = 4096, p = 12288): dram read 101.3 MB + write 3.4 MB against 102.8 MB algorithmic
                "traffic_captured": 104.6e6 if (n, k, d, p) == (64, 4, 4096, 12288) else None}
    elif 2.0 * m * d * p >= 1e9 and m >= 128:
        # three tf32 products per fp32 product: the tensor cores do 3 x the algorithmic flops at the tf32 rate
        roof = {"bound": "tensor", "achieved": 2.0 * m * d * p / proj_s / 1e12, "peak": 0.5 * peaks["bf16_tflops"] / 3.0,
                "unit": "TFLOP/s", "peak_source": peaks["source"] + " bf16 GEMM x nominal tf32/bf16 ratio 0.5 / 3 products"}
    else:
        roof = {"bound": "alu", "achieved": 2.0 * m * d * p / proj_s / 1e12, "peak": 148 * 128 * 2 * 1.965e9 / 1e12,
                "unit": "TFLOP/s", "peak_source": "derived: 148 SMs x 128 FP32 lanes x 2 x 1.965 GHz"}
    roof.setdefault("peak_source", peaks["source"])
    roof.setdefault("kernel", "projection GEMM Y' = U W")
    roof.update({"frac": roof["achieved"] / roof["peak"], "traffic": roof.pop("traffic_captured", None)})
    line = {
        "metric": METRIC, "value": float(n) * calls * steps / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": steps,
        "warmup": max(3, warmup), "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "n": n, "k": k, "m": m, "d": d, "p": p, "calls_per_step": calls,
                   "mixing": ["orthogonal", "non-orthogonal"][kind0] if len(set(kinds)) == 1 else "alternating",
                   "shield_scale": w.shield_scale, "l2": "inputs_larger_than_l2" if calls * d * p * es > 126e6 else "l2_resident",
                   "api": "gelo_qkv_offload_batch", "lanes": lanes},
        "clocks": clocks, "gpu_launches": launches, "roofline": roof,
        "per_call_us": 1e3 * per_call_ms, "stage_ms": {k_: round(v, 5) for k_, v in stage_ms.items()},
        "overhead_vs_plain_gemm": per_call_ms / stage_ms["plain_project"],
        "products_vs_plain_gemm": (stage_ms["mix"] + stage_ms["project"] + stage_ms["unmix"]) / stage_ms["plain_project"],
        "flop_floor_vs_plain": chain_flops / (2.0 * n * d * p),
    }
    if "plain_project_fma" in stage_ms:
        line["overhead_vs_plain_gemm_fma"] = per_call_ms / stage_ms["plain_project_fma"]
    if latency_steps > 0:
        # per-call latency over `latency_steps` sweeps of `calls` layers: (a) sweeps through the batched entry point,
        # one event per sweep, latency = sweep time / calls; (b) single calls through gelo_qkv_offload, one event pair each
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(latency_steps + 1)]
        ev[0].record()
        for s_ in range(latency_steps):
            sweep(1000 + s_)
            ev[s_ + 1].record()
        torch.cuda.synchronize()
        per = np.array([ev[i].elapsed_time(ev[i + 1]) for i in range(latency_steps)]) * 1e3 / calls
        singles = min(2000, latency_steps * 2)
        a_ev = [torch.cuda.Event(enable_timing=True) for _ in range(singles)]
        b_ev = [torch.cuda.Event(enable_timing=True) for _ in range(singles)]
        for r in range(singles + 8):
            c_ = r % calls
            if r >= 8:
                a_ev[r - 8].record()
            ctx.qkv_offload(Hs[c_], Ws[c_], n, k, d, p, kinds[c_], 777 + r, w.shield_scale, w.dtype, Q, K, V)
            if r >= 8:
                b_ev[r - 8].record()
        torch.cuda.synchronize()
        one = np.array([a_ev[i].elapsed_time(b_ev[i]) for i in range(singles)]) * 1e3
        if ctx.last_status() != gelo.OK:
            raise SystemExit(f"device-side error in the latency run of {name}")
        line["latency_us"] = {
            "calls_timed": int(latency_steps * calls),
            "batched_per_call": {"p50": float(np.percentile(per, 50)), "p99": float(np.percentile(per, 99)),
                                 "mean": float(per.mean()), "sweeps": int(latency_steps), "calls_per_sweep": int(calls)},
            "single_call": {"p50": float(np.percentile(one, 50)), "p99": float(np.percentile(one, 99)),
                            "mean": float(one.mean()), "calls": int(singles)},
            "plain_gemm": 1e3 * stage_ms["plain_project"],
            "batched_p50_vs_plain_gemm": float(np.percentile(per, 50)) / (1e3 * stage_ms["plain_project"]),
        }
    ctx.close()
    return line


def compact(line):
    """The part of a secondary workload's line that the main line carries."""
    keep = ("per_call_us", "overhead_vs_plain_gemm", "overhead_vs_plain_gemm_fma", "products_vs_plain_gemm",
            "flop_floor_vs_plain", "value", "stage_ms", "latency_us")
    out = {k_: line[k_] for k_ in keep if k_ in line}
    out["config"] = {k_: line["config"][k_] for k_ in ("n", "k", "d", "p", "calls_per_step", "mixing", "lanes")}
    out["dtype"] = line["dtype"]
    out["projection_roofline"] = {k_: line["roofline"][k_] for k_ in ("bound", "achieved", "peak", "unit", "frac")}
    return out


def run_workload(args):
    import torch
    torch.cuda.set_device(0)
    steps = args.steps
    latency = args.latency_steps if args.workload == "decode_bf16" else 0
    print(json.dumps(measure_workload(args.workload, args.lanes, steps, args.warmup, args.calls, latency)))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-variants", action="store_true", help="skip the block-diagonal variant runs")
    ap.add_argument("--lanes", type=int, default=32, help="concurrent sampling lanes of the batched call (1..32)")
    ap.add_argument("--lane-share", type=int, default=4, help="each level-3 update uses 1/share of the SMs in batches")
    ap.add_argument("--level3", type=int, default=0, choices=[0, 1, 2, 3],
                    help="factorisation updates: 0 auto (tensor cores for bf16), 1 fp32 FMA, 2 tensor cores")
    ap.add_argument("--calls", type=int, default=0, help="projection calls per step (default: the workload's 32)")
    ap.add_argument("--latency-steps", type=int, default=1000,
                    help="decode_bf16: sweeps of 32 calls whose per-call latency distribution is reported")
    ap.add_argument("--no-workloads", action="store_true", help="skip the secondary workloads in the main line")
    ap.add_argument("--timed-only", action="store_true",
                    help="run only the warm-up and the timed sweeps (for profiler launch lists)")
    ap.add_argument("--workload", default=WORKLOAD, choices=["tiny_f32", "layer_f32", "shield_bf16", "prefill_bf16", "decode_bf16"],
                    help="prefill_bf16 is the benchmark; the others print a shorter line (one GPU)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.workload != WORKLOAD:
        return run_workload(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
