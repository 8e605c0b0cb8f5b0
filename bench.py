#!/usr/bin/env python
"""Benchmark of the QLLM quantized-linear hot path on B200.

A step = one pass of the whole path over one batch of synthetic tokens: the fused
LayerNorm + reassembly + quantization kernel, then the integer GEMM with its dequantizing
epilogue.  Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c5|c2_w4a8] [--impl reference]
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "W4A4 reassembled-linear tokens/s; TOPS & GB/s as % of B200 roofline"
UNIT = "tokens/s"
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the GEMM kernel, from the ncu captures summarised
# under profiles/ (keyed by workload and tokens per GPU; absent = not captured for the current kernel)
NCU_TRAFFIC = {("c2", 2048): 79.2e6, ("c3", 16): 45.4e6}


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


def _oracle_sample(cfg, rows, L=None):
    """Times the oracle, as it stands, on `rows` token rows of the workload (whole path)."""
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import oracle
    import parity
    from paper_2310_08041_b200 import synth
    if L is None:
        L = parity.oracle_layer(cfg)
    x = synth.activations(cfg, M=rows)
    t0 = time.perf_counter()
    q = oracle.reassemble_quant(x, L["gamma"], L["beta"], cfg.ln_eps, L["ptr"], L["src"], L["coef"], cfg.a_bits)
    acc = oracle.int_matmul(q["codes"], L["w_codes"])
    out = oracle.epilogue(acc, cfg.K, q["scale"], q["zero"], q["sum"], L["w_scale"], L["w_zero"], L["w_colsum"], None)
    oracle.cast_bf16(out)
    dt = time.perf_counter() - t0
    return rows / dt, dt, L


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

    MID_EVERY = 4

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
        flush.zero_()
        step()
    barrier()
    assert B.qllm_poll_status() == 0, "device-side wait timed out during warm-up"
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    n0 = B.qllm_launch_count()
    barrier()
    t_start = time.time()
    for i in range(args.steps):
        flush.zero_()                  # L2 flush between timed iterations (not inside the event pairs)
        step(events[i], mid=(i % MID_EVERY == 0))
    barrier()
    t_end = time.time()
    launches = B.qllm_launch_count() - n0
    assert B.qllm_poll_status() == 0, "device-side wait timed out"
    halves = events[::MID_EVERY]
    t_pre = [e[0].elapsed_time(e[1]) for e in halves]
    t_gemm = [e[1].elapsed_time(e[2]) for e in halves]
    t_step = [e[0].elapsed_time(e[2]) for e in events]
    ms_step = sum(t_step) / len(t_step)
    t_b2b = [t for i, t in enumerate(t_step) if i % MID_EVERY != 0]
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
    h2d = M * K * (2 if cfg.x_dtype == "bf16" else 4)
    d2h = M * N * 2

    def allmax(v):
        if world == 1:
            return v
        t = torch.tensor([v], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    ms_step_w, ms_e2e_w = allmax(ms_step), allmax(ms_e2e)
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
                        "traffic": NCU_TRAFFIC.get((cfg.name, M))}
        else:
            expand = (cfg.a_bits == 4 or cfg.w_bits == 4) and M >= 385
            roofline = {"kernel": "qllm_layer_qgemm: " + ("join of the side-stream weight expansion + " if expand and cfg.w_bits == 4 else "") +
                                  "qgemm_tc2_kernel (tcgen05 kind::i8, cta_group::2, byte lanes) + dequant epilogue",
                        "bound": "tensor", "achieved": tops, "peak": int8_peak, "unit": "TOP/s", "frac": tops / int8_peak,
                        "peak_source": f"2 x {peaks['source']} bf16 burst ({peaks['bf16_burst']} TFLOP/s); nominal int8:bf16 = 2",
                        "frac_of_nominal_4500": tops / 4500.0, "ms": ms_gemm, "traffic": NCU_TRAFFIC.get((cfg.name, M))}
        line = {
            "metric": METRIC, "value": world * M / (ms_step_w * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step_w, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u8",
            "data": "synthetic",
            "config": {"workload": f"{cfg.name}: M={M} K={K} N={N} W{cfg.w_bits}A{cfg.a_bits} x=bf16 out=bf16 per GPU",
                       "l2": "256 MB buffer written between timed iterations", "map_extra_channels": stats["E"],
                       "merged_rows": stats["merged_rows"], "builder_s": round(build_s, 3), "parallelism": f"tokens x{world}"},
            "e2e": {"value": world * M / (ms_e2e_w * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e_w},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": roofline,
            "kernels": {"reassemble_quant": {"ms": ms_pre, "GB/s": pre_bytes / (ms_pre * 1e-3) / 1e9,
                                             "frac_hbm": pre_bytes / (ms_pre * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                             "bytes": pre_bytes},
                        "qgemm": {"ms": ms_gemm, "TOP/s": tops},
                        "timed_on": f"every {MID_EVERY}th timed step (event between the two calls)",
                        "ms_per_step_without_that_event": ms_b2b},
        }
        if world == 1 and not args.no_cpu_baseline:
            sys.path.insert(0, os.path.join(ROOT, "tests"))
            rows = args.ref_rows or 512
            v, dt, _ = _oracle_sample(cfg, rows)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": f"first {rows} token rows of {cfg.name}, whole path, {dt:.1f} s"}
        print(json.dumps(line))
    layer.destroy()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="c2", choices=["c2", "c3", "c4", "c5", "c2_w4a8"])
    ap.add_argument("--ref-rows", type=int, default=0, help="token rows of the oracle sample (0 = auto)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
