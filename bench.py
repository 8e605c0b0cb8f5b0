#!/usr/bin/env python
"""Benchmark of the QLLM quantized-linear hot path on B200.

A step = one pass of the whole path over one batch of synthetic tokens: the fused
LayerNorm + reassembly + quantization kernel, then the integer GEMM with its dequantizing
epilogue.  Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c5|c2_w4a8] [--impl reference]
"""
from __future__ import annotations

import argparse
import glob
import hashlib
import json
import math
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "W4A4 reassembled-linear tokens/s; TOPS & GB/s as % of B200 roofline"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0


def _traffic(kernel, workload, M):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of `kernel`, from the ncu summaries under
    profiles/: a line `traffic-record: kernel=.. workload=.. M=.. bytes=.. sources=a.cu,b.cuh sha256=..` holds the
    counter and the hash of the kernel's sources when it was taken.  None when there is no record for this
    workload or the sources have changed since (the counter is then stale)."""
    for path in sorted(glob.glob(os.path.join(ROOT, "profiles", "*.md"))):
        for line in open(path):
            if not line.startswith("traffic-record:"):
                continue
            kv = dict(tok.split("=", 1) for tok in line.split()[1:] if "=" in tok)
            if kv.get("kernel") != kernel or kv.get("workload") != workload or int(kv.get("M", -1)) != M:
                continue
            h = hashlib.sha256()
            for src in kv.get("sources", "").split(","):
                f = os.path.join(ROOT, "paper_2310_08041_b200", "csrc", src)
                if not os.path.exists(f):
                    return None
                h.update(open(f, "rb").read())
            return float(kv["bytes"]) if h.hexdigest().startswith(kv.get("sha256", "?")) else None
    return None


def _stats(ts):
    return dict(mean=sum(ts) / len(ts), median=statistics.median(ts), min=min(ts), n=len(ts))


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_burst=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self, t0, t1):
        if self.proc is None:
            return None
        time.sleep(0.15)
        self.proc.terminate()
        timed = [r for ts, r in self.rows if t0 <= ts <= t1]
        # a short timed region sees few 100 ms samples: then every sample since the warm-up began counts
        # (the same kernels ran throughout), and the line says so
        rows = timed if len(timed) >= 3 else [r for _, r in self.rows]
        window = "timed steps" if len(timed) >= 3 else "warm-up + timed steps + end-to-end steps"
        if not rows:
            return None
        sm = [float(r[0]) for r in rows if r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in rows if r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in rows for n, v in zip(names, r[3:7]) if v.lower().startswith("active")})
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=reasons, samples=len(rows), samples_in_timed_steps=len(timed), window=window)


def _oracle_sample(cfg, rows, L=None, parallel=False):
    """Times the oracle, as it stands, on `rows` token rows of the workload (whole path).  parallel: the same source
    built with -fopenmp, its loops over token rows on all the cores this process may use."""
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import oracle
    import parity
    from paper_2310_08041_b200 import synth
    oracle.set_parallel(False)
    if L is None:
        L = parity.oracle_layer(cfg)
    oracle.set_parallel(parallel)
    x = synth.activations(cfg, M=rows)
    t0 = time.perf_counter()
    q = oracle.reassemble_quant(x, L["gamma"], L["beta"], cfg.ln_eps, L["ptr"], L["src"], L["coef"], cfg.a_bits)
    acc = oracle.int_matmul(q["codes"], L["w_codes"])
    out = oracle.epilogue(acc, cfg.K, q["scale"], q["zero"], q["sum"], L["w_scale"], L["w_zero"], L["w_colsum"], None)
    oracle.cast_bf16(out)
    dt = time.perf_counter() - t0
    oracle.set_parallel(False)
    return rows / dt, dt, L


def _cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def _cpu_baseline(cfg, rows):
    """The oracle on the host's cores: one thread on `rows` token rows, then all cores (OpenMP over token rows) on
    as many rows per core.  The all-cores figure is the line's cpu_baseline value."""
    cores = _cores()
    v1, dt1, L = _oracle_sample(cfg, rows)
    rows_all = rows * min(cores, 16)
    os.environ["OMP_NUM_THREADS"] = str(cores)
    vN, dtN, _ = _oracle_sample(cfg, rows_all, L, parallel=True)
    return {"value": vN, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {rows_all} token rows of {cfg.name}, whole path, OpenMP over token rows, {dtN:.1f} s",
            "single_thread": {"value": v1, "cores": 1,
                              "sample": f"first {rows} token rows of {cfg.name}, whole path, {dt1:.1f} s"}}


def run_reference(args):
    from paper_2310_08041_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = synth.CONFIGS[args.workload]
    # bounded sample per step so that the whole run ends within a few minutes (~45 rows/s)
    rows = args.ref_rows or max(1, min(512, 7000 // max(1, args.steps + args.warmup)))
    L = None
    for _ in range(min(args.warmup, 1)):
        _, _, L = _oracle_sample(cfg, max(1, rows // 8), L)
    times = []
    for _ in range(args.steps):
        v, dt, L = _oracle_sample(cfg, rows, L)
        times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    val = rows / (ms / 1e3)
    sample = f"first {rows} token rows of {cfg.name} (M={cfg.M}), whole path, single thread"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: M={cfg.M} K={cfg.K} N={cfg.N} W{cfg.w_bits}A{cfg.a_bits}", "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_gpu(args):
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2310_08041_b200 import binding as B
    from paper_2310_08041_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    cfg = synth.CONFIGS[args.workload]
    M, K, N = cfg.M, cfg.K, cfg.N
    out_dtype = torch.bfloat16
    gamma, beta = synth.layernorm_params(cfg)
    # every rank holds its own batch of M tokens (token sharding; map and weights replicated)
    x_np = synth.activations(cfg, stream=100 + rank)
    to_dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    x_dev = torch.from_numpy(x_np.view(np.int16)).to(dev).view(torch.bfloat16) if x_np.dtype == np.uint16 else to_dev(x_np)
    g_d, b_d = to_dev(gamma), (None if beta is None else to_dev(beta))

    # offline side, product path only: calibration statistic on the GPU, threshold + builder on the host
    xc = synth.calibration_tokens(cfg)
    xc_d = torch.from_numpy(xc.view(np.int16)).to(dev).view(torch.bfloat16) if xc.dtype == np.uint16 else to_dev(xc)
    absmax = torch.zeros(K, dtype=torch.float32, device=dev)
    B.qllm_calib_absmax(xc_d, g_d, b_d, absmax, ln_eps=cfg.ln_eps)
    am = absmax.cpu().numpy()
    theta = B.qllm_theta_for_extra(am, 8) if cfg.theta_rule == "extra8" else B.qllm_theta_percentile(am, 0.99)
    A, Bm = synth.low_rank(cfg)
    t0 = time.perf_counter()
    h = B.qllm_build_reassembly(am, theta, synth.weights(cfg), A, Bm, cfg.w_bits)
    build_s = time.perf_counter() - t0
    stats = h.stats()
    xdt = B.QLLM_F32 if cfg.x_dtype == "f32" else B.QLLM_BF16
    # the layer object holds map, weights and workspace on the device (map compiled once for the fused kernel)
    layer = B.Layer(h, gamma, beta, cfg.ln_eps, None, cfg.a_bits, xdt, B.QLLM_BF16, max_M=M)
    row = K // 2 if cfg.a_bits == 4 else K
    out = torch.empty((M, N), dtype=out_dtype, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # > 126 MB L2
    flush_r = torch.zeros(256 << 18, dtype=torch.float32, device=dev)

    def flush_l2():
        # write a buffer larger than L2, then read another one: the cache ends up full of CLEAN lines of data
        # the step never touches (after the write alone the step's first misses would each pay for the write-back
        # of a dirty flush line)
        flush.zero_()
        flush_r.sum()

    MID_EVERY = 2

    def step(evs=None, mid=False):
        # the two calls of qllm_layer_forward.  Every MID_EVERY-th timed step records an event between them,
        # which gives the halves their times; the other steps run them back to back as a caller would (an event
        # between the calls keeps the decode GEMM, a programmatic dependent of the pre-GEMM kernel, from starting
        # its prologue under that kernel)
        if evs:
            evs[0].record()
        layer.reassemble_quant(x_dev)
        if evs and mid:
            evs[1].record()
        layer.qgemm(M, out)
        if evs:
            evs[2].record()

    sampler = ClockSampler(local) if rank == 0 else None
    for _ in range(args.warmup):
        flush_l2()
        step()
    barrier()
    assert B.qllm_poll_status() == 0, "device-side wait timed out during warm-up"
    # The timed region is K steps between a barrier + synchronize on both sides.  A region shorter than half a
    # second would see no sample of the 100 ms clock sampler, so it is repeated (same K steps, same bracketing)
    # until the rounds add up to that; every round's steps count.
    t_pre, t_gemm, t_step, t_b2b = [], [], [], []
    launches = 0
    rounds = 0
    t_start = time.time()
    while True:
        events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
        n0 = B.qllm_launch_count()
        barrier()
        for i in range(args.steps):
            flush_l2()                     # L2 flush between timed iterations (not inside the event pairs)
            step(events[i], mid=(i % MID_EVERY == 0))
        barrier()
        if rounds == 0:
            launches = B.qllm_launch_count() - n0
        rounds += 1
        for i, e in enumerate(events):
            t = e[0].elapsed_time(e[2])
            t_step.append(t)
            if i % MID_EVERY == 0:
                t_pre.append(e[0].elapsed_time(e[1]))
                t_gemm.append(e[1].elapsed_time(e[2]))
            else:
                t_b2b.append(t)
        more = time.time() - t_start < 0.6 and rounds < 5000
        if world > 1:
            flag = torch.tensor([1 if more else 0], device=dev)
            dist.broadcast(flag, 0)
            more = bool(flag.item())
        if not more:
            break
    t_end = time.time()
    assert B.qllm_poll_status() == 0, "device-side wait timed out"
    ms_step = sum(t_step) / len(t_step)
    ms_b2b = sum(t_b2b) / len(t_b2b) if t_b2b else ms_step

    # end to end through the host-buffer entry point: H2D of x and D2H of out inside the timed region
    xh = torch.from_numpy(x_np.view(np.int16) if x_np.dtype == np.uint16 else x_np).pin_memory()
    oh = torch.empty((M, N), dtype=out_dtype).pin_memory()
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(2):
        layer.forward_host(xh, oh, M)
    barrier()
    e2e_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(e2e_steps)]
    for i in range(e2e_steps):
        e2e_ev[i][0].record()
        layer.forward_host(xh, oh, M)
        e2e_ev[i][1].record()
    barrier()
    ms_e2e = sum(a.elapsed_time(b) for a, b in e2e_ev) / e2e_steps
    clocks = sampler.stop(t_start, t_end) if sampler else None
    # the same steps with nothing flushed between them (whatever of the step's 150 MB fits stays in the 126 MB L2):
    # reported beside the headline, which is the flushed figure
    n_hot = max(3, min(args.steps, 400))
    barrier()
    hot0, hot1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    hot0.record()
    for _ in range(n_hot):
        step()
    hot1.record()
    barrier()
    ms_hot = hot0.elapsed_time(hot1) / n_hot
    # the same step with the layer's opt-in resident byte copy of its 4-bit weights (memory for time: no per-call
    # widening); reported beside the headline, which keeps the 4-bit codes as the only copy
    ms_res = None
    if cfg.w_bits == 4 and M > 16:
        layer.keep_byte_weights(True)
        n_res = max(3, min(args.steps, 400))
        for _ in range(3):
            flush_l2()
            step()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n_res)]
        barrier()
        for i in range(n_res):
            flush_l2()
            step(ev[i])
        barrier()
        ms_res = sum(e[0].elapsed_time(e[2]) for e in ev) / n_res
        layer.keep_byte_weights(False)
    h2d = M * K * (2 if cfg.x_dtype == "bf16" else 4)
    d2h = M * N * 2

    def allmax(v):
        if world == 1:
            return v
        t = torch.tensor([v], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    ms_step_w, ms_e2e_w = allmax(ms_step), allmax(ms_e2e)
    ms_res_w = allmax(ms_res) if ms_res is not None else None
    ms_gemm = sum(t_gemm) / len(t_gemm)
    ms_pre = sum(t_pre) / len(t_pre)
    if rank == 0:
        peaks = _peaks()
        ops = 2.0 * M * N * K
        tops = ops / (ms_gemm * 1e-3) / 1e12
        int8_peak = 2.0 * peaks["bf16_burst"]
        pre_bytes = M * (K * (2 if cfg.x_dtype == "bf16" else 4) + row + 12)
        wrow = K // 2 if cfg.w_bits == 4 else K
        if M <= 16:
            # decode: weight-streaming kernel, HBM-bound; bytes = weights + side arrays + tokens + output
            gemm_bytes = N * wrow + 16 * N + M * row + M * N * 2
            gbs = gemm_bytes / (ms_gemm * 1e-3) / 1e9
            roofline = {"kernel": "qllm_qgemm call: qgemm_decode_kernel (weight streaming)", "bound": "hbm",
                        "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                        "peak_source": f"{peaks['source']} STREAM-style copy", "ms": ms_gemm, "bytes": gemm_bytes,
                        "frac_of_nominal_8000": gbs / NOMINAL_HBM_GBS,
                        "traffic": _traffic("qgemm_decode_kernel", cfg.name, M)}
        else:
            expand = (cfg.a_bits == 4 or cfg.w_bits == 4) and M >= 385
            roofline = {"kernel": "qllm_layer_qgemm: " + ("join of the side-stream weight expansion + " if expand and cfg.w_bits == 4 else "") +
                                  "qgemm_tc2_kernel (tcgen05 kind::i8, cta_group::2, byte lanes) + dequant epilogue",
                        "bound": "tensor", "achieved": tops, "peak": int8_peak, "unit": "TOP/s", "frac": tops / int8_peak,
                        "peak_source": f"2 x {peaks['source']} bf16 burst ({peaks['bf16_burst']} TFLOP/s); nominal int8:bf16 = 2",
                        "frac_of_nominal_4500": tops / 4500.0, "ms": ms_gemm,
                        "traffic": _traffic("qgemm_tc2_kernel", cfg.name, M)}
        line = {
            "metric": METRIC, "value": world * M / (ms_step_w * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "timed_rounds": rounds, "warmup": args.warmup, "ms_per_step": ms_step_w,
            "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u8",
            "data": "synthetic",
            "config": {"workload": f"{cfg.name}: M={M} K={K} N={N} W{cfg.w_bits}A{cfg.a_bits} x=bf16 out=bf16 per GPU",
                       "l2": "256 MB buffer written, then 256 MB read, between timed iterations", "map_extra_channels": stats["E"],
                       "merged_rows": stats["merged_rows"], "builder_s": round(build_s, 3), "parallelism": f"tokens x{world}"},
            "e2e": {"value": world * M / (ms_e2e_w * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e_w},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": roofline,
            "ms_per_step_stats": _stats(t_step),
            "ms_per_step_no_flush": ms_hot,
            "ms_x_sm_mhz": (ms_step_w * clocks["sm_mhz"]) if clocks and clocks.get("sm_mhz") else None,
            "kernels": {"reassemble_quant": {"ms": ms_pre, "ms_stats": _stats(t_pre),
                                             "GB/s": pre_bytes / (ms_pre * 1e-3) / 1e9,
                                             "frac_hbm": pre_bytes / (ms_pre * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                             "frac_of_nominal_8000": pre_bytes / (ms_pre * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
                                             "bytes": pre_bytes},
                        "qgemm": {"ms": ms_gemm, "ms_stats": _stats(t_gemm), "TOP/s": tops},
                        "timed_on": f"every {MID_EVERY}nd timed step (event between the two calls)",
                        "ms_per_step_without_that_event": ms_b2b},
        }
        if ms_res_w is not None:
            line["resident_byte_weights"] = {"ms_per_step": ms_res_w, "value": world * M / (ms_res_w * 1e-3), "unit": UNIT,
                                             "extra_device_bytes": N * K,
                                             "what": "qllm_layer_keep_byte_weights: same step, same bits, weights also held one code per byte"}
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = _cpu_baseline(cfg, args.ref_rows or 384)
        print(json.dumps(line))
    layer.destroy()
    if world > 1:
        dist.destroy_process_group()


def run_fold(args):
    """Appendix B study: with the reassembly folded into the preceding layer, the run-time stage in front of the GEMM
    is the per-token quantizer alone (qllm_quantize_rows).  Timed on 16384 token rows of the c2 shape (134 MB in:
    larger than L2) against the HBM roofline; one launch per step."""
    import numpy as np
    import torch
    from paper_2310_08041_b200 import binding as B
    from paper_2310_08041_b200 import synth
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    cfg = synth.CONFIGS["c2"].scaled(M=16384)
    M, K = cfg.M, cfg.K
    x_np = synth.activations(cfg)
    x = torch.from_numpy(x_np.view(np.int16)).to(dev).view(torch.bfloat16)
    codes = torch.empty((M, K // 2), dtype=torch.uint8, device=dev)
    sc = torch.empty(M, device=dev); ze = torch.empty(M, device=dev); rs = torch.empty(M, dtype=torch.int32, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    flush_r = torch.zeros(256 << 18, dtype=torch.float32, device=dev)

    def flush_l2():
        flush.zero_()       # write a buffer larger than L2, then read another: the cache holds clean foreign lines
        flush_r.sum()
    sampler = ClockSampler(0)
    for _ in range(args.warmup):
        flush_l2()
        B.qllm_quantize_rows(x, 4, codes, sc, ze, rs)
    torch.cuda.synchronize()
    ts = []
    n0 = B.qllm_launch_count()
    t_start = time.time()
    for _ in range(args.steps):
        flush_l2()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); B.qllm_quantize_rows(x, 4, codes, sc, ze, rs); e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    t_end = time.time()
    launches = B.qllm_launch_count() - n0
    clocks = sampler.stop(t_start, t_end)
    peaks = _peaks()
    st = _stats(ts)
    nbytes = M * (K * 2 + K // 2 + 12)
    gbs = nbytes / (st["median"] * 1e-3) / 1e9
    print(json.dumps({
        "metric": METRIC, "value": M / (st["mean"] * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": st["mean"], "ms_per_step_stats": st, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": f"c2_fold: per-token quantizer alone (Appendix B), M={M} K={K} 4-bit codes, x=bf16",
                   "l2": "256 MB buffer written, then 256 MB read, between timed iterations; 134 MB of input"},
        "gpu_launches": int(launches), "clocks": clocks,
        "roofline": {"kernel": "quantize_rows_warp", "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "frac_of_nominal_8000": gbs / NOMINAL_HBM_GBS,
                     "peak_source": f"{peaks['source']} STREAM-style copy", "bytes": nbytes,
                     "traffic": _traffic("quantize_rows_warp", "c2_fold", M)}}))


def launch_ranks(n, argv):
    """Starts n ranks of this script on this node (rank r on GPU r), as the multi-GPU contract does."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def run_stub(args):
    """The rank plumbing of run_gpu without a GPU: gloo, a stand-in step whose time depends on the rank, the
    max-over-ranks reduction and rank 0's line.  Tokens per rank are the sharding module's."""
    import torch
    import torch.distributed as dist
    from paper_2310_08041_b200 import shard
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
    M = 64
    t = []
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        time.sleep(0.001 * (rank + 1))
        if i >= args.warmup:
            t.append((time.perf_counter() - t0) * 1e3)
    ms = sum(t) / len(t)
    ms_w = shard.max_over_ranks(ms) if world > 1 else ms
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": world * M / (ms_w * 1e-3), "unit": UNIT, "n_gpus": world,
                          "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_w, "stub": True,
                          "scaling": "weak", "config": {"parallelism": f"tokens x{world}"}}))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="c2", choices=["c2", "c3", "c4", "c5", "c2_w4a8", "c2_fold"])
    ap.add_argument("--ref-rows", type=int, default=0, help="token rows of the oracle sample (0 = auto)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--stub", action="store_true",
                    help="no GPU: gloo ranks and a stand-in step, to exercise the launcher and the reduction")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    world_env = os.environ.get("WORLD_SIZE")
    if world_env is None and args.gpus > 1:
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))    # one process per GPU, this script again in each
    if int(world_env or 1) != args.gpus:
        sys.stderr.write(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world_env}: refusing to print a line\n")
        sys.exit(2)
    if args.stub:
        run_stub(args)
    elif args.workload == "c2_fold":
        run_fold(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
