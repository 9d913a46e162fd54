#!/usr/bin/env python
"""Benchmark of the PSA forward hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one pass of the whole hot path over one synthetic attention call shaped like
Wan 2.1 14B 720p (40 heads, 21x45x80 = 75,600 tokens, head_dim 128): psa_mask_build
(block mask + index lists) followed by psa_attn_fwd (planning kernel + stripe attention
kernel).  The metric is computed TFLOP/s: 4*d FLOP per attended real (query, key) pair
divided by the time of a step.  N > 1 runs N independent replicas (the path has no
exchange step); the value is the sum over replicas divided by the slowest replica's time.
With --gpus N > 1 and no WORLD_SIZE in the environment the script starts the N ranks itself
(one process per GPU, NCCL, loopback rendezvous); under torchrun it uses the ranks it is given.
--ulysses times the head-sharded call on sequence-sharded inputs instead (two all-to-all
re-layouts around the kernel, timed separately from it).

Prints ONE JSON line (rank 0).  --impl reference times the fp64 CPU oracle on a bounded
sample of the same workload on the host cores.
"""
import argparse
import json
import math
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "psa_attn_computed_tflops_at_75600_tokens"
UNIT = "TFLOP/s"
HEAD_DIM = 128
SCALE = 1.0 / math.sqrt(128.0)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
DATASHEET_BF16_TFLOPS = 2250.0   # nominal dense bf16 figure of the part (context beside the measured peak)
# the other configurations of the benchmark set, timed at kernel level after the headline
OTHER_CONFIGS = ["tiny", "wan13b_480p", "wan13b_480p_b3x32x4", "wan13b_480p_b1x30x8", "wan13b_480p_b1x32x4", "hunyuan_720p", "sweep_00", "sweep_25", "sweep_50", "sweep_75", "sweep_90",
                 "ragged_75", "wan14b_720p_b3x8x16", "hunyuan_768p"]


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def workload_flops(w):
    return 4.0 * HEAD_DIM * w["attended_pairs"], 4.0 * HEAD_DIM * w["dense_pairs"]


def config_of(w, extra=None):
    """Names the workload; identical in both arms (--impl ours / reference)."""
    T, H, W = w["grid"]
    input_bytes = 3 * w["n_heads"] * T * H * W * HEAD_DIM * 2
    c = {"workload": w["name"], "grid": w["grid"], "tokens": T * H * W, "n_heads": w["n_heads"],
         "head_dim": HEAD_DIM, "mask_block": w["tile"], "tile_sparsity": w["tile_sparsity"],
         "step": "psa_mask_build + psa_attn_fwd", "parallelism": "replicas",
         "l2_policy": ("inputs (%.1f GB) exceed L2; no flush needed" % (input_bytes / 1e9)) if input_bytes > 2.5e8
                      else "inputs fit L2",
         "peaks": load_peaks()["_source"]}
    if extra:
        c.update(extra)
    return c


def slab_split(tile):
    """(slabs per block, keys of the last slab) of a mask block, as the attention kernel splits it:
    128-token slabs along the block's outermost axis of extent > 1, the last one possibly shorter."""
    bt, bh, bw = tile
    if bt > 1 or (bh == 1 and bw == 1):
        extent, other = bt, bh * bw
    elif bh > 1:
        extent, other = bh, bt * bw
    else:
        extent, other = bw, bt * bh
    c0 = 128 // other
    n_sub = -(-extent // c0)
    return n_sub, (extent - (n_sub - 1) * c0) * other


def issued_flops(nnz, tile):
    """FLOPs the tensor cores are asked for: every attended block pair costs (128 rows per query
    slab) x (keys of every key slab) x 4 x head_dim, padded and idle rows included."""
    n_sub, n_last = slab_split(tile)
    return 4.0 * HEAD_DIM * nnz * (128.0 * n_sub) * (128.0 * (n_sub - 1) + n_last)


# ----------------------------------------------------------------------------- CPU oracle leg
def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1


def oracle_sample(w, budget_s, rows_per_head=24, max_heads=None):
    """Runs the oracle, as it stands, on seeded sample rows of the workload until the time budget is
    spent.  Returns (attended pairs processed, seconds, rows, heads)."""
    from oracle import psa_oracle as O
    from paper_2609_37001_b200 import workloads as WL
    T, H, W = w["grid"]
    L = T * H * W
    tile = tuple(w["tile"])
    pairs, rows_done, heads_done = 0, 0, 0
    t0 = time.perf_counter()
    order = list(range(0, w["n_heads"], 7)) + [h for h in range(w["n_heads"]) if h % 7]
    for hd in order[: (max_heads or len(order))]:
        p = tuple(w["head_params"][hd])
        q, k, v = (O.bf16_bits_to_f64(WL.head_bits(w["seed"], n, hd, L)) for n in ("q", "k", "v"))
        rows = WL.sample_rows(w["seed"], hd, L, rows_per_head)
        O.attention_rows(q, k, v, rows, p, T, H, W, tile, SCALE)
        tb, sb, _ = O.token_block_coords(T, H, W, tile)
        pairs += sum(int(O.attend_row(r, p, tb, sb).sum()) for r in rows)
        rows_done += len(rows)
        heads_done += 1
        if time.perf_counter() - t0 > budget_s:
            break
    return pairs, time.perf_counter() - t0, rows_done, heads_done


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times, pairs = [], 0
    for i in range(args.warmup + args.steps):
        p, s, rows, heads = oracle_sample(w, budget_s=0.0, rows_per_head=16, max_heads=1)
        if i >= args.warmup:
            times.append(s)
            pairs += p
    total = sum(times)
    value = 4.0 * HEAD_DIM * pairs / total / 1e12
    sample = f"per step: 16 seeded query rows of 1 head against all {w['grid'][0] * w['grid'][1] * w['grid'][2]} keys (incl. input generation and bf16->fp64 conversion)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "gpus_used": 0, "ranks_that_ran": 1,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / max(len(times), 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(w),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}",
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons, pw = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.f.read().splitlines():
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); pw.append(float(parts[2]))
            except ValueError:
                continue
            for n, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update({"sm_mhz": float(np.median(sm)), "sm_max_mhz": max(mx), "power_w_max": max(pw),
                        "reasons": sorted(reasons), "samples": len(sm)})
        return out


# ----------------------------------------------------------------------------- GPU leg
def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2609_37001_b200 import build
    build.build()
    from paper_2609_37001_b200 import binding as B
    from paper_2609_37001_b200 import replicas as R
    from paper_2609_37001_b200 import workloads as WL

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    peaks = load_peaks()

    T, H, W = w["grid"]
    L, nh, tile = T * H * W, w["n_heads"], w["tile"]
    params = [tuple(p) for p in w["head_params"]]
    flops, dense_flops = workload_flops(w)

    host = {n: torch.from_numpy(WL.tensor_bits(w["seed"], n, nh, L).view(np.int16)).view(torch.bfloat16)
            for n in ("q", "k", "v")}
    q, k, v = (host[n].to(dev) for n in ("q", "k", "v"))
    out = torch.empty_like(q)
    lse = torch.empty((nh, L), dtype=torch.float32, device=dev)
    nb, nnz = B.psa_mask_sizes(params, w["grid"], tile)
    mask_out = (torch.empty((nh, nb, nb), dtype=torch.uint8, device=dev),
                torch.empty(nh * nb + 1, dtype=torch.int32, device=dev),
                torch.empty(max(nnz, 1), dtype=torch.int32, device=dev))
    stream = torch.cuda.Stream(device=dev)

    def step():
        B.psa_mask_build(params, w["grid"], tile, out=mask_out, stream=stream)
        B.psa_attn_fwd(q, k, v, params, w["grid"], tile, SCALE, out=out, lse=lse, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            step()
        st, detail = B.psa_last_device_status()
        if st != 0:
            raise SystemExit(f"device status {st} detail {hex(detail)}")

        # ---- same-process calibration (harness only, outside the timed region): a bf16 torch.matmul
        # exposes the clock state of this GPU at this moment next to the recorded peak
        calib = None
        if rank == 0 and not args.quick:
            a = torch.randn((8192, 8192), device=dev, dtype=torch.bfloat16)
            b = torch.randn((8192, 8192), device=dev, dtype=torch.bfloat16)
            c = torch.empty_like(a)
            best = float("inf")
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for _ in range(8):
                e0.record(stream)
                torch.matmul(a, b, out=c)
                e1.record(stream)
                torch.cuda.synchronize()
                best = min(best, e0.elapsed_time(e1))
            calib = {"bf16_matmul_8192_tflops_best_of_8": 2.0 * 8192 ** 3 / (best * 1e-3) / 1e12,
                     "recorded_peak_tflops": peaks["bf16_tflops"], "note": "harness only; not part of a step"}
            del a, b, c

        # ---- timed region: K back-to-back steps; kernel events rotate so every launch is measured
        kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in kev:
            a.record(stream); b.record(stream)
        sev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]   # step boundaries
        sampler = ClockSampler(local) if rank == 0 else None
        barrier()
        launches0 = B.psa_launch_count()
        sev[0].record(stream)
        for i in range(args.steps):
            B.psa_profile_events(*kev[i])
            step()
            sev[i + 1].record(stream)
        barrier()
        launches = B.psa_launch_count() - launches0
        B.psa_profile_events(None, None)
        clocks = sampler.stop() if sampler else None
        ms_step = sev[0].elapsed_time(sev[-1]) / args.steps
        step_ms = [sev[i].elapsed_time(sev[i + 1]) for i in range(args.steps)]
        kernel_ms = float(np.mean([a.elapsed_time(b) for a, b in kev]))
        st, detail = B.psa_last_device_status()
        if st != 0:
            raise SystemExit(f"device status {st} detail {hex(detail)}")

        ms_max = R.max_over_ranks(ms_step, dev)

        extra = {}
        if rank == 0 and not args.quick:
            # ---- mask build alone through the C ABI (arguments marshalled once, as a C caller would):
            # HBM-write bound on paper, launch-latency dominated in practice
            import ctypes
            mb_prob = B.make_problem(nh, tile, 1.0, 0, 128)
            mb_args = (B._params_array(params), ctypes.byref(mb_prob), T, H, W, mask_out[0].data_ptr(),
                       mask_out[1].data_ptr(), mask_out[2].data_ptr(), mask_out[2].numel(), int(stream.cuda_stream))
            mb = B.lib().psa_mask_build
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for _ in range(5):
                mb(*mb_args)
            e0.record(stream)
            for _ in range(100):
                mb(*mb_args)
            e1.record(stream)
            torch.cuda.synchronize()
            mb_us = 1e3 * e0.elapsed_time(e1) / 100
            mb_bytes = nh * (nb * nb + 4 * nb) + 4 + 4 * nnz
            # the same call captured 20 times in a CUDA graph and replayed: device-side cost per launch
            # without the host's (Python + driver) cost of issuing it
            gr = torch.cuda.CUDAGraph()
            gr.capture_begin()
            for _ in range(20):
                mb(*mb_args)
            gr.capture_end()
            gr.replay()
            torch.cuda.synchronize()
            e0.record(stream)
            gr.replay()
            e1.record(stream)
            torch.cuda.synchronize()
            mb_graph_us = 1e3 * e0.elapsed_time(e1) / 20
            extra["mask_build"] = {"us_per_call": mb_us, "us_per_launch_in_graph": mb_graph_us, "bytes": mb_bytes,
                                   "GBps": mb_bytes / (mb_graph_us * 1e-6) / 1e9, "hbm_peak_GBps": peaks["hbm_gbs"],
                                   "frac_of_hbm_peak": mb_bytes / (mb_graph_us * 1e-6) / 1e9 / peaks["hbm_gbs"],
                                   "note": "us_per_call: back-to-back C-ABI calls incl. the host's launch cost; "
                                           "us_per_launch_in_graph: 20 captured launches replayed (GB/s uses this); one kernel "
                                           "per call; the outputs stay in L2, the kernel is bound by launch latency and "
                                           "instruction issue, not by HBM"}
            # ---- the same kernel with an all-covering mask (in-house dense baseline)
            Tp, Hp, Wp = -(-T // tile[0]), -(-H // tile[1]), -(-W // tile[2])
            dense_params = [(Tp, 0, 0, Hp * Wp, 0, 0)] * nh
            for _ in range(1):
                B.psa_attn_fwd(q, k, v, dense_params, w["grid"], tile, SCALE, out=out, lse=lse, stream=stream)
            e0.record(stream)
            nd = 3
            for _ in range(nd):
                B.psa_attn_fwd(q, k, v, dense_params, w["grid"], tile, SCALE, out=out, lse=lse, stream=stream)
            e1.record(stream)
            torch.cuda.synchronize()
            dense_ms = e0.elapsed_time(e1) / nd
            extra["dense_baseline"] = {"ms": dense_ms, "tflops": dense_flops / (dense_ms * 1e-3) / 1e12,
                                       "frac_of_peak": dense_flops / (dense_ms * 1e-3) / 1e12 / peaks["bf16_tflops"]}
            extra["speedup_vs_dense"] = dense_ms / kernel_ms
            extra["dense_equiv_tflops"] = dense_flops / (kernel_ms * 1e-3) / 1e12

        # ---- end to end through the host-tensor entry point (pinned host buffers, copies timed)
        e2e = None
        if not args.quick:
            hq, hk, hv = (host[n].pin_memory() for n in ("q", "k", "v"))
            hout = torch.empty_like(hq).pin_memory()
            hlse = torch.empty((nh, L), dtype=torch.float32).pin_memory()
            staging = (q, k, v, out, lse)

            def e2e_step():
                B.psa_mask_build(params, w["grid"], tile, out=mask_out, stream=stream)
                B.psa_attn_fwd_host(hq, hk, hv, hout, hlse, staging, params, w["grid"], tile, SCALE, stream=stream)

            e2e_step()
            barrier()
            t0 = time.perf_counter()
            ne = max(2, min(args.steps, 5))
            for _ in range(ne):
                e2e_step()
            torch.cuda.synchronize()
            e2e_ms = 1e3 * (time.perf_counter() - t0) / ne
            e2e_ms = R.max_over_ranks(e2e_ms, dev)
            bytes_t = nh * L * HEAD_DIM * 2
            e2e = {"value": world * flops / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
                   "h2d_bytes_per_step": 3 * bytes_t, "d2h_bytes_per_step": bytes_t + nh * L * 4}
            if rank == 0:
                # the PCIe floor of such a step: the larger direction's bytes at the measured copy rate
                # (the two directions overlap on separate copy engines)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                q.copy_(hq, non_blocking=True)
                e1.record(stream)
                torch.cuda.synchronize()
                h2d_gbs = bytes_t / (e0.elapsed_time(e1) * 1e-3) / 1e9
                e0.record(stream)
                hout.copy_(out, non_blocking=True)
                e1.record(stream)
                torch.cuda.synchronize()
                d2h_gbs = bytes_t / (e0.elapsed_time(e1) * 1e-3) / 1e9
                floor_ms = max(3 * bytes_t / h2d_gbs, (bytes_t + nh * L * 4) / d2h_gbs) / 1e6
                e2e.update({"h2d_GBps_measured": h2d_gbs, "d2h_GBps_measured": d2h_gbs, "pcie_floor_ms": floor_ms,
                            "note": "floor = max(h2d bytes / h2d rate, d2h bytes / d2h rate); the kernel hides behind the copies"})

    if rank == 0:
        value = world * flops / (ms_max * 1e-3) / 1e12
        achieved = flops / (kernel_ms * 1e-3) / 1e12
        traffic = None   # DRAM bytes per launch from the committed ncu summary of this workload
        tp = os.path.join(ROOT, "profiles", f"attn_fwd_kernel_{w['name']}.md")
        if os.path.exists(tp):
            for ln in open(tp):
                if ln.startswith("traffic_bytes_per_launch:"):
                    traffic = int(ln.split(":")[1])
        issued = issued_flops(nnz, tile)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_max, "ms_median": float(np.median(step_ms)),
            "ms_min": float(np.min(step_ms)), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_of(w),
            "computed_flops_per_step": flops, "issued_flops_per_step": issued, "padding_ratio": issued / flops,
            "roofline": {"bound": "tensor", "kernel": "attn_fwd_kernel", "achieved": achieved,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                         "frac_of_sustained_peak": achieved / peaks["bf16_tflops_sustained"],
                         "frac_of_datasheet": achieved / DATASHEET_BF16_TFLOPS,
                         "datasheet_peak": DATASHEET_BF16_TFLOPS,
                         "datasheet_note": "nominal dense bf16 figure of the part (2.25 PFLOP/s), quoted, not measured",
                         "issued_tflops": issued / (kernel_ms * 1e-3) / 1e12,
                         "kernel_ms": kernel_ms, "algorithmic_flops_per_launch": flops, "traffic": traffic,
                         "peak_source": peaks["_source"] + " (burst cuBLAS bf16)"},
            "calibration": calib,
            "clocks": clocks, "gpu_launches": int(launches), "e2e": e2e,
            "context": {"paper_h100_psa_ms": 55.12, "paper_h100_tflops": 29.26 / 55.12e-3,
                        "note": "paper: Table 2, Wan 2.1 14B at 75.00% sparsity on one H100; unpublished per-head parameters"},
        }
        line.update(extra)
        if not args.quick:
            pairs, secs, rows, heads = oracle_sample(w, budget_s=12.0)
            line["cpu_baseline"] = {"value": 4.0 * HEAD_DIM * pairs / secs / 1e12, "unit": UNIT, "cores": blas_threads(),
                                    "kind": "oracle", "seconds": secs,
                                    "sample": f"{rows} seeded query rows over {heads} heads, each against all {L} keys, "
                                              f"incl. input generation and bf16->fp64 conversion"}
        if not args.quick and not args.no_configs:
            del host
            line["configs"] = time_other_configs(B, WL, torch, dev, peaks, skip=w["name"])
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def time_other_configs(B, WL, torch, dev, peaks, skip):
    """Kernel-level timing (back-to-back psa_attn_fwd calls, CUDA events) of the other configurations of
    the benchmark set, with inputs drawn on the device (the time does not depend on the values)."""
    res = []
    for name in OTHER_CONFIGS:
        if name == skip:
            continue
        w = WL.workload(name)
        T, H, W = w["grid"]
        L, nh, tile = T * H * W, w["n_heads"], w["tile"]
        params = [tuple(p) for p in w["head_params"]]
        g = torch.Generator(device=dev).manual_seed(w["seed"])
        q, k, v = (torch.randn((nh, L, HEAD_DIM), device=dev, generator=g).bfloat16() for _ in range(3))
        out, lse = torch.empty_like(q), torch.empty((nh, L), dtype=torch.float32, device=dev)
        flops, dflops = workload_flops(w)
        iters = 20 if flops < 1e12 else (10 if flops < 6e13 else 4)
        for _ in range(3):
            B.psa_attn_fwd(q, k, v, params, w["grid"], tile, SCALE, out=out, lse=lse)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
        ev[0].record()
        for i in range(iters):
            B.psa_attn_fwd(q, k, v, params, w["grid"], tile, SCALE, out=out, lse=lse)
            ev[i + 1].record()
        torch.cuda.synchronize()
        st, detail = B.psa_last_device_status()
        if st != 0:
            raise SystemExit(f"{name}: device status {st} {hex(detail)}")
        ms = [ev[i].elapsed_time(ev[i + 1]) for i in range(iters)]
        mean = float(np.mean(ms))
        _, nnz = B.psa_mask_sizes(params, w["grid"], tile)
        res.append({"workload": name, "grid": w["grid"], "n_heads": nh, "mask_block": tile, "tile_sparsity": w["tile_sparsity"],
                    "ms": mean, "ms_median": float(np.median(ms)), "ms_min": float(np.min(ms)),
                    "computed_tflops": flops / (mean * 1e-3) / 1e12,
                    "frac": flops / (mean * 1e-3) / 1e12 / peaks["bf16_tflops"],
                    "dense_equiv_tflops": dflops / (mean * 1e-3) / 1e12,
                    "padding_ratio": issued_flops(nnz, tile) / flops if flops else None})
        del q, k, v, out, lse
        torch.cuda.empty_cache()
    return res


def run_report(args):
    """Times every committed workload (kernel-level: planning + attention kernels through psa_attn_fwd),
    its all-covering (dense) counterpart and psa_mask_build, and writes a markdown table.  Inputs are
    seeded N(0,1) bf16 tensors drawn on the device (timing does not depend on the values)."""
    import ctypes
    import torch
    from paper_2609_37001_b200 import build
    build.build()
    from paper_2609_37001_b200 import binding as B
    from paper_2609_37001_b200 import workloads as WL
    peaks = load_peaks()
    torch.cuda.set_device(0)
    rows, dense_cache = [], {}
    names = [n for n in WL.load_workloads() if not n.startswith("tiny")]
    for name in names:
        w = WL.workload(name)
        T, H, W = w["grid"]
        L, nh, tile = T * H * W, w["n_heads"], w["tile"]
        params = [tuple(p) for p in w["head_params"]]
        g = torch.Generator(device="cuda").manual_seed(w["seed"])
        q, k, v = (torch.randn((nh, L, HEAD_DIM), device="cuda", generator=g).bfloat16() for _ in range(3))
        out, lse = torch.empty_like(q), torch.empty((nh, L), dtype=torch.float32, device="cuda")

        def timed(ps, iters):
            for _ in range(2):
                B.psa_attn_fwd(q, k, v, ps, w["grid"], tile, SCALE, out=out, lse=lse)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(iters):
                B.psa_attn_fwd(q, k, v, ps, w["grid"], tile, SCALE, out=out, lse=lse)
            e1.record()
            torch.cuda.synchronize()
            st, detail = B.psa_last_device_status()
            if st != 0:
                raise SystemExit(f"{name}: device status {st} {hex(detail)}")
            return e0.elapsed_time(e1) / iters

        flops, dflops = workload_flops(w)
        ms = timed(params, 10 if flops < 6e13 else 4)
        key = (tuple(w["grid"]), tuple(tile), nh)
        if key not in dense_cache:
            Tp, Hp, Wp = -(-T // tile[0]), -(-H // tile[1]), -(-W // tile[2])
            dense_cache[key] = timed([(Tp, 0, 0, Hp * Wp, 0, 0)] * nh, 2)
        dms = dense_cache[key]
        nb, nnz = B.psa_mask_sizes(params, w["grid"], tile)
        mo = (torch.empty((nh, nb, nb), dtype=torch.uint8, device="cuda"), torch.empty(nh * nb + 1, dtype=torch.int32, device="cuda"),
              torch.empty(max(nnz, 1), dtype=torch.int32, device="cuda"))
        prob = B.make_problem(nh, tile, 1.0, 0, 128)
        margs = (B._params_array(params), ctypes.byref(prob), T, H, W, mo[0].data_ptr(), mo[1].data_ptr(), mo[2].data_ptr(), mo[2].numel(), None)
        for _ in range(5):
            B.lib().psa_mask_build(*margs)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(100):
            B.lib().psa_mask_build(*margs)
        e1.record()
        torch.cuda.synchronize()
        mb_us = 10.0 * e0.elapsed_time(e1)
        mb_bytes = nh * (nb * nb + 4 * nb) + 4 + 4 * nnz
        rows.append((name, "x".join(map(str, w["grid"])), L, nh, "x".join(map(str, tile)), w["tile_sparsity"], ms,
                     flops / ms / 1e9, flops / ms / 1e9 / peaks["bf16_tflops"], dflops / ms / 1e9, dms, dms / ms,
                     mb_us, mb_bytes / mb_us / 1e3))
        del q, k, v, out, lse
        torch.cuda.empty_cache()
    lines = ["| workload | grid | tokens | heads | block | tile sparsity | ms/call | computed TFLOP/s | frac of measured peak | dense-equiv TFLOP/s | dense ms | speed-up vs dense | mask build us | mask build GB/s |",
             "|---|---|---|---|---|---|---|---|---|---|---|---|---|---|"]
    for r in rows:
        lines.append("| %s | %s | %d | %d | %s | %.4f | %.3f | %.1f | %.3f | %.1f | %.2f | %.2f | %.1f | %.0f |" % r)
    text = "\n".join(lines) + "\n"
    with open(args.report, "w") as f:
        f.write(text)
    sys.stderr.write(text)


def run_search(args, w):
    """PSA-Search inner loop (Algorithm 3) for ONE head of the workload's shape: psa_search_losses over
    N seeded candidates drawn from the paper's initialisation space, then psa_search_select.  Prints one
    JSON line: candidates per second, the tensor roofline of the attention launch inside it, the HBM
    roofline of the loss reduction, and the oracle timed on sampled query rows."""
    import torch
    from paper_2609_37001_b200 import build
    build.build()
    from paper_2609_37001_b200 import binding as B
    from paper_2609_37001_b200 import workloads as WL
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    peaks = load_peaks()
    T, H, W = w["grid"]
    L, tile = T * H * W, w["tile"]
    cands = WL.search_candidates(w["seed"], args.search, w["grid"], tile)
    n = len(cands)
    bits = {t: WL.head_bits(w["seed"], t, 0, L) for t in ("q", "k", "v")}
    q, k, v = (torch.from_numpy(bits[t].view(np.int16)).view(torch.bfloat16).to(dev) for t in ("q", "k", "v"))
    scratch = torch.empty(B.psa_search_scratch_bytes(n, w["grid"]), dtype=torch.uint8, device=dev)
    # attended real (query, key) pairs of every candidate from the library's own block masks
    Tp, Hp, Wp = -(-T // tile[0]), -(-H // tile[1]), -(-W // tile[2])
    real = lambda n_tok, b, nb_: torch.tensor([min(b, n_tok - i * b) for i in range(nb_)], dtype=torch.float64)
    rt, rh, rw = real(T, tile[0], Tp), real(H, tile[1], Hp), real(W, tile[2], Wp)
    real_blk = (rt[:, None, None] * rh[None, :, None] * rw[None, None, :]).reshape(-1).to(dev)
    pairs, spars = [], []
    for c0 in range(0, n, 16):
        m, _, _ = B.psa_mask_build(cands[c0:c0 + 16], w["grid"], tile)
        md = m.to(torch.float64)
        pairs += [float(x) for x in torch.einsum("hqk,q,k->h", md, real_blk, real_blk).cpu()]
        spars += [float(x) for x in (1.0 - md.mean(dim=(1, 2))).cpu()]
        del m, md
    flops = 4.0 * HEAD_DIM * (sum(pairs) + float(L) * L)
    stream = torch.cuda.Stream(device=dev)
    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            losses = B.psa_search_losses(q, k, v, cands, w["grid"], tile, SCALE, scratch=scratch, stream=stream)
        kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for a, b in kev:
            a.record(stream); b.record(stream)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler = ClockSampler(0)
        torch.cuda.synchronize()
        launches0 = B.psa_launch_count()
        ev0.record(stream)
        for i in range(args.steps):
            B.psa_profile_events(*kev[i])
            losses = B.psa_search_losses(q, k, v, cands, w["grid"], tile, SCALE, scratch=scratch, stream=stream)
        ev1.record(stream)
        torch.cuda.synchronize()
        launches = B.psa_launch_count() - launches0
        B.psa_profile_events(None, None)
        clocks = sampler.stop()
        st, detail = B.psa_last_device_status()
        if st != 0:
            raise SystemExit(f"device status {st} detail {hex(detail)}")
    ms = ev0.elapsed_time(ev1) / args.steps
    attn_ms = float(np.mean([a.elapsed_time(b) for a, b in kev]))  # the (last) attention launch of each call
    lh = losses.cpu().tolist()
    alpha = float(np.median(lh))
    chosen = B.psa_search_select(lh, spars, alpha)
    loss_bytes = (n + 1) * L * HEAD_DIM * 2   # every candidate output once + the reference once
    line = {"metric": "psa_search_candidates_per_s", "value": n / (ms * 1e-3), "unit": "candidates/s", "n_gpus": 1,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w["name"] + "_search_1head", "grid": w["grid"], "tokens": L, "mask_block": tile,
                       "n_candidates": n, "mean_candidate_tile_sparsity": float(np.mean(spars)),
                       "step": "psa_search_losses (plan + attention over candidates and full attention + loss reduction)"},
            "roofline": {"bound": "tensor", "kernel": "attn_fwd_kernel", "achieved": flops / (attn_ms * 1e-3) / 1e12,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": flops / (attn_ms * 1e-3) / 1e12 / peaks["bf16_tflops"], "kernel_ms": attn_ms,
                         "algorithmic_flops_per_launch": flops, "traffic": None,
                         "note": "valid when candidates + 1 <= 128 (one attention launch per call)"},
            "loss_reduction": {"ms": ms - attn_ms, "bytes": loss_bytes, "GBps": loss_bytes / ((ms - attn_ms) * 1e-3) / 1e9,
                               "hbm_peak_GBps": peaks["hbm_gbs"], "note": "step time minus the attention launch: plan + two reduction kernels"},
            "selection": {"alpha": alpha, "chosen": int(chosen), "chosen_params": list(cands[chosen]),
                          "chosen_sparsity": spars[chosen], "chosen_loss": lh[chosen]},
            "clocks": clocks, "gpu_launches": int(launches)}
    if not args.quick:
        from oracle import psa_oracle as O
        qf, kf, vf = (O.bf16_bits_to_f64(bits[t]) for t in ("q", "k", "v"))
        rows = WL.sample_rows(w["seed"], 0, L, 16)
        t0, done = time.perf_counter(), 0
        O.attention_rows(qf, kf, vf, rows, (Tp, 0, 0, Hp * Wp, 0, 0), T, H, W, tuple(tile), SCALE)
        for c in cands:
            O.attention_rows(qf, kf, vf, rows, tuple(c), T, H, W, tuple(tile), SCALE)
            done += 1
            if time.perf_counter() - t0 > 15.0:
                break
        secs = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": done / (secs * L / len(rows)), "unit": "candidates/s", "cores": blas_threads(),
                                "kind": "oracle", "seconds": secs,
                                "sample": f"{done} candidates + full attention on {len(rows)} seeded query rows each, "
                                          f"scaled by {L}/{len(rows)} rows"}
    print(json.dumps(line), flush=True)


def run_ulysses(args, w):
    """The head-sharded call on sequence-sharded inputs (the layout a sequence-parallel DiT keeps its
    activations in): every rank holds all heads for L / P tokens; one all-to-all per tensor gives each
    rank heads / P heads with all tokens, the single-GPU kernel runs on them, a second all-to-all
    returns out and lse.  Total work is fixed ("strong" scaling).  The three phases are timed
    separately with CUDA events; plain NCCL all-to-all, no peer pointers handed to any kernel."""
    import torch
    import torch.distributed as dist
    from paper_2609_37001_b200 import build
    build.build()
    from paper_2609_37001_b200 import binding as B
    from paper_2609_37001_b200 import replicas as R
    from paper_2609_37001_b200 import ulysses as U
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()
    T, H, W = w["grid"]
    L, nh, tile = T * H * W, w["n_heads"], w["tile"]
    if L % world or nh % world:
        raise SystemExit(f"--ulysses needs tokens ({L}) and heads ({nh}) divisible by the number of ranks ({world})")
    params = [tuple(p) for p in w["head_params"]]
    flops, _ = workload_flops(w)
    g = torch.Generator(device=dev).manual_seed(w["seed"] + rank)
    q, k, v = (torch.randn((nh, L // world, HEAD_DIM), device=dev, generator=g).bfloat16() for _ in range(3))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def phases():
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        e[0].record()
        qh, kh, vh = (U.seq_to_head_shards(t) for t in (q, k, v))
        e[1].record()
        lo, hi = U.local_heads(nh)
        oh, lh = B.psa_attn_fwd(qh, kh, vh, params[lo:hi], w["grid"], tile, SCALE)
        e[2].record()
        o = U.head_to_seq_shards(oh)
        l = U.head_to_seq_shards(lh.unsqueeze(-1).contiguous()).squeeze(-1)
        e[3].record()
        return e, o, l

    for _ in range(max(args.warmup, 3)):
        phases()
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = B.psa_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    evs = [phases()[0] for _ in range(args.steps)]
    ev1.record()
    barrier()
    launches = B.psa_launch_count() - launches0
    clocks = sampler.stop() if sampler else None
    st, detail = B.psa_last_device_status()
    if st != 0:
        raise SystemExit(f"device status {st} detail {hex(detail)}")
    ms = R.max_over_ranks(ev0.elapsed_time(ev1) / args.steps, dev)
    a2a_in = R.max_over_ranks(float(np.mean([e[0].elapsed_time(e[1]) for e in evs])), dev)
    attn = R.max_over_ranks(float(np.mean([e[1].elapsed_time(e[2]) for e in evs])), dev)
    a2a_out = R.max_over_ranks(float(np.mean([e[2].elapsed_time(e[3]) for e in evs])), dev)
    if rank == 0:
        per_rank_bytes = nh * (L // world) * HEAD_DIM * 2
        line = {"metric": METRIC, "value": flops / (ms * 1e-3) / 1e12, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "strong",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic (drawn on the device)",
                "config": config_of(w, {"parallelism": f"ulysses{world}: sequence-sharded in/out, head-sharded kernel",
                                         "step": "all_to_all(q,k,v) + psa_attn_fwd + all_to_all(out,lse)"}),
                "phases_ms": {"all_to_all_in": a2a_in, "attention": attn, "all_to_all_out": a2a_out},
                "all_to_all_bytes_per_rank": {"in": 3 * per_rank_bytes * (world - 1) // world,
                                              "out": (per_rank_bytes + nh * (L // world) * 4) * (world - 1) // world},
                "roofline": {"bound": "tensor", "kernel": "attn_fwd_kernel", "achieved": flops / world / (attn * 1e-3) / 1e12,
                             "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                             "frac": flops / world / (attn * 1e-3) / 1e12 / peaks["bf16_tflops"], "traffic": None,
                             "note": "per GPU, attention phase only (planning kernel included)"},
                "clocks": clocks, "gpu_launches": int(launches), "e2e": None}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="wan14b_720p", help="a name from workloads.json, or 'all' (= the default run: headline + configs array)")
    ap.add_argument("--quick", action="store_true", help="timed region only (no dense/e2e/CPU legs); for profiling")
    ap.add_argument("--no-configs", action="store_true", help="skip the kernel-level timing of the other configurations")
    ap.add_argument("--ulysses", action="store_true",
                    help="time the head-sharded call on sequence-sharded inputs (all-to-all, kernel, all-to-all)")
    ap.add_argument("--report", default=None, metavar="FILE.md",
                    help="time every workload (PSA, dense, mask build) on one GPU and write a markdown table; no JSON line")
    ap.add_argument("--search", type=int, default=0, metavar="N",
                    help="time the PSA-Search inner loop for one head over N seeded candidates instead of the hot path")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours" and not args.report and not args.search:
        # started without a launcher: become one (one process per GPU on this node)
        from paper_2609_37001_b200 import replicas as R
        codes = R.launch_ranks([os.path.abspath(__file__)] + sys.argv[1:], args.gpus)
        raise SystemExit(max(abs(c) for c in codes))
    if args.search:
        from paper_2609_37001_b200 import workloads as WL
        run_search(args, WL.workload(args.workload))
        return
    if args.report:
        run_report(args)
        return
    from paper_2609_37001_b200 import workloads as WL
    if args.workload == "all":      # the default run already is "all": headline line + the `configs` array
        args.workload, args.no_configs = "wan14b_720p", False
    w = WL.workload(args.workload)
    if args.impl == "reference":
        run_reference(args, w)
    elif args.ulysses:
        run_ulysses(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
