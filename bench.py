#!/usr/bin/env python
"""Benchmark of the token-adaptive quantised layer forward on B200.

One step = one pass of the whole layer path (router + selection + compaction,
gather + RMSNorm, four quantised GEMMs, rotary, attention over executed tokens,
residual scatter) over one batch of synthetic Llama-2-7B-shaped input: hidden
4096, 32 heads, FFN 11008, int4 group-128 weights, batch 4 x 2048 tokens,
top-k selection at the requested execution ratio.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--ratio R] [--impl reference]
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2602_10431_b200 import inputs  # noqa: E402

METRIC = "tokens/s per token-adaptive int4 layer (7B-shaped, prefill 4x2048) at execution ratio"
UNIT = "tokens/s"
SWEEP = [1.0, 0.9, 0.75, 0.5]
WORKLOAD = ("c2: 7B-shaped layer (hidden 4096, 32 heads, FFN 11008), int4 g128, "
            "batch 4 x seq 2048 prefill")
# DRAM traffic of the four GEMM launches of one step at ratio 0.5 (4096 executed tokens), from
# one ncu capture of the kernel as it stands; None at other ratios.
GEMM_DRAM_BYTES = 716259840
KERNELS_PER_STEP = 11  # router, gather+norm, 4 GEMMs, rotary table, rotary, tail zeroing, attention, RMSNorm


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []      # (arrival time, csv line)
        self.window = None   # (start, end) of the timed region, host clock

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [ln for (t, ln) in self.lines
                  if self.window is None or self.window[0] <= t <= self.window[1] + 0.02]
        if len(inside) < 3:  # region shorter than a few sampling periods: keep every sample
            inside = [ln for (_, ln) in self.lines]
        for ln in inside:
            f = [c.strip() for c in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
                power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons),
                    samples=len(sm), power_w_max=max(power) if power else None)


def max_over_ranks(ms: float, device=None) -> float:
    """Slowest rank's time: every rank runs its own replica of the batch, the job's
    throughput is set by the last one to finish.  No-op without a process group."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput of `world` replicas that each process tokens_per_rank per step."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def build_layer_inputs(seed, cfg_name):
    c = inputs.CONFIG_SHAPES[cfg_name]
    sh, B, S = c["shape"], c["B"], c["S"]
    w = inputs.layer_weights(seed, 0, sh)
    x = inputs.hidden_states(seed, B * S, sh.d)
    cu = inputs.cu_seqlens_uniform(B, S)
    return sh, B, S, w, x, cu


# ------------------------------------------------------------------------------------
# reference arm / CPU baseline: the oracle, as it stands, on a bounded sample
# ------------------------------------------------------------------------------------

def oracle_runner(sh, w, x, ratio, sample_tokens):
    """Returns (run, threads): run() executes the CPU oracle (router + top-k +
    layer) once on the first `sample_tokens` tokens of sequence 0."""
    import oracle
    layer = oracle.DenseLayer(sh, w)  # dequantisation of the weights is set-up, not timed

    def run():
        xs = x[:sample_tokens]
        cus = np.array([0, sample_tokens], np.int32)
        _, m = oracle.route(layer, xs, "topk", ratio=ratio)
        oracle.layer_forward(layer, xs, cus, m)

    return run, oracle.get_threads()


def sample_desc(sample, ratio):
    return ("CPU oracle on the first %d tokens of sequence 0 of the same workload (router + "
            "top-k at ratio %.2f + layer; weights dequantised beforehand); tokens/s = sample "
            "tokens / wall time" % (sample, ratio))


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return 0
    sh, B, S, w, x, cu = build_layer_inputs(0, "c2")
    sample = 256  # bounded sample per step so that K steps end within minutes
    run, threads = oracle_runner(sh, w, x, args.ratio, sample)
    warm = min(args.warmup, 1)
    for _ in range(warm):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    dt = time.perf_counter() - t0
    tps = sample * args.steps / dt
    line = dict(impl="reference", metric=METRIC, value=tps, unit=UNIT, n_gpus=args.gpus,
                steps=args.steps, warmup=warm, ms_per_step=dt / args.steps * 1e3,
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64",
                data="synthetic",
                config=dict(workload=WORKLOAD, ratio=args.ratio, select="topk"),
                cpu_baseline=dict(value=tps, unit=UNIT, cores=threads, kind="oracle",
                                  sample=sample_desc(sample, args.ratio)),
                e2e=dict(value=tps, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))
    return 0


# ------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------

def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2602_10431_b200 import api

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    api.lib()  # fail loudly if the CUDA library is missing

    sh, B, S, w, x, cu = build_layer_inputs(0, "c2")
    T = B * S
    lw = api.LayerWeights(w, dev, fuse_swiglu=True)
    cud = torch.from_numpy(cu).to(dev)
    ratio = args.ratio
    cfg = api.layer_config(sh, api.SELECT_TOPK, ratio=ratio)
    ws = torch.zeros(api.layer_workspace_bytes(cfg, T, B), dtype=torch.uint8, device=dev)
    n_buf = 4
    x_host = torch.from_numpy(x).to(torch.bfloat16).pin_memory()
    out_host = torch.empty_like(x_host).pin_memory()
    bufs = [x_host.to(dev) for _ in range(n_buf)]
    nex = torch.zeros(1, dtype=torch.int32, device=dev)

    def step(i, c=cfg):
        api.layer_forward(c, lw, bufs[i % n_buf], cud, ws, nex)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup, sampler=None, drain=None):
        for i in range(warmup):
            fn(i)
        if drain is not None:
            drain()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_start = time.time()
        e0.record()
        for i in range(steps):
            fn(i)
        if drain is not None:
            drain()  # the timed stream waits for the copies still in flight on the others
        e1.record()
        barrier()
        if sampler is not None:
            sampler.window = (t_start, time.time())
        return max_over_ranks(e0.elapsed_time(e1), dev if world > 1 else None)

    # ---- headline: device-resident inputs ----
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)  # let the first samples arrive before the timed region
    ms = timed(step, args.steps, args.warmup, sampler)
    clocks = sampler.stop()
    ms_per_step = ms / args.steps
    value = aggregate_tokens_per_s(T, world, ms_per_step)
    rc = api.device_status()
    if rc != 0:
        raise RuntimeError("device status: " + api.strerror(rc))
    n_exec = int(nex.item())

    # ---- sweep over execution ratios ----
    sweep = {}
    sw_steps = max(3, min(100, args.steps // 2))
    for r in SWEEP:
        c = api.layer_config(sh, api.SELECT_TOPK, ratio=r)
        m = timed(lambda i, c=c: step(i, c), sw_steps, 3) / sw_steps
        sweep["%.2f" % r] = dict(ms=m, tokens_per_s=world * T / (m * 1e-3))
    base = sweep["1.00"]["ms"]
    for r in sweep:
        sweep[r]["speedup_vs_ratio_1"] = base / sweep[r]["ms"]

    # ---- roofline of the dominant kernel: the four quantised GEMMs at this ratio ----
    peaks = measured_peaks()
    k = api.topk_count(ratio, T)
    m_dev = torch.tensor([k], dtype=torch.int32, device=dev)
    qd = sh.n_heads * sh.head_dim
    adt = api.act_torch_dtype(cfg.act_dtype)
    a_d = torch.randn(T, sh.d, device=dev).to(adt)
    a_q = torch.randn(T, qd, device=dev).to(adt)
    a_f = torch.randn(T, sh.ffn, device=dev).to(adt)
    y_qkv = torch.empty(T, lw.qkv.N, dtype=adt, device=dev)
    y_o = torch.empty(T, sh.d, dtype=adt, device=dev)
    y_act = torch.empty(T, sh.ffn, dtype=adt, device=dev)

    def gemms(i):
        api.wq_gemm(a_d, lw.qkv, m_dev, api.EPI_STORE_16, y=y_qkv)
        api.wq_gemm(a_q, lw.o, m_dev, api.EPI_STORE_16, y=y_o)
        api.wq_gemm(a_d, lw.gate_up, m_dev, api.EPI_SWIGLU, y=y_act)
        api.wq_gemm(a_f, lw.down, m_dev, api.EPI_STORE_16, y=y_o)

    g_steps = max(3, min(200, args.steps // 2))
    g_ms = timed(gemms, g_steps, 3) / g_steps
    flops = 2.0 * sh.linear_params() * k
    achieved = flops / (g_ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops_sustained"]
    roofline = dict(bound="tensor", kernel="wq_gemm_pair_kernel<4,1> (4 launches per step)",
                    achieved=achieved, peak=peak, unit="TFLOP/s", frac=achieved / peak,
                    peak_source="%s (sustained bf16)" % peaks["source"],
                    traffic=GEMM_DRAM_BYTES if abs(ratio - 0.5) < 1e-9 else None,
                    traffic_unit="bytes per 4 launches (dram__bytes_read.sum + dram__bytes_write.sum, "
                                 "ncu, ratio 0.5; profiles/wq_gemm_pair_layer_step_traffic.md)",
                    ms_per_4_launches=g_ms, share_of_step=g_ms / ms_per_step)

    # ---- end to end: host buffers, H2D of the inputs and D2H of the result every step ----
    # Every step copies its input from pinned host memory, runs the layer through the public
    # call and copies its result back; the copies run on two streams of their own, so step
    # i + 1's input and step i - 1's result travel while step i computes (n_buf device buffers).
    main = torch.cuda.current_stream()
    copy_in, copy_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(n_buf)]
    ev_done = [torch.cuda.Event() for _ in range(n_buf)]
    ev_out = [torch.cuda.Event() for _ in range(n_buf)]
    out_hosts = [out_host] + [torch.empty_like(x_host).pin_memory() for _ in range(n_buf - 1)]

    def e2e_step(i):
        j = i % n_buf
        buf = bufs[j]
        with torch.cuda.stream(copy_in):
            copy_in.wait_event(ev_out[j])  # the buffer's previous result has left the device
            buf.copy_(x_host, non_blocking=True)
            ev_in[j].record(copy_in)
        main.wait_event(ev_in[j])
        api.layer_forward(cfg, lw, buf, cud, ws, nex)
        ev_done[j].record(main)
        with torch.cuda.stream(copy_out):
            copy_out.wait_event(ev_done[j])
            out_hosts[j].copy_(buf, non_blocking=True)
            ev_out[j].record(copy_out)

    def e2e_drain():
        main.wait_stream(copy_in)
        main.wait_stream(copy_out)

    main.wait_stream(copy_in)
    e_steps = max(3, min(50, args.steps // 2))
    e_ms = timed(e2e_step, e_steps, 3, drain=e2e_drain) / e_steps
    nbytes = x_host.numel() * 2
    e2e = dict(value=world * T / (e_ms * 1e-3), unit=UNIT, h2d_bytes_per_step=nbytes,
               d2h_bytes_per_step=nbytes, ms_per_step=e_ms,
               note="copies on their own streams, overlapped with the neighbouring steps' compute")

    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps,
                warmup=args.warmup, ms_per_step=ms_per_step, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f16", data="synthetic",
                config=dict(workload=WORKLOAD, ratio=ratio, select="topk", executed_tokens=n_exec,
                            precision="bf16 residual stream in/out; fp16 internal activations and "
                                      "dequantised weights, fp32 accumulation",
                            tokens=T,
                            l2="inputs larger than L2 (packed weights 107 MB + more than 1 GB of "
                               "activations per step, %d rotating input buffers)" % n_buf,
                            multi_gpu="replicas only: every rank runs the same batch, no collective"),
                clocks=clocks, gpu_launches=KERNELS_PER_STEP * args.steps, sweep=sweep,
                roofline=roofline, e2e=e2e)

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample = 2048  # one whole sequence: about 10-30 s of host time
        run, threads = oracle_runner(sh, w, x, ratio, sample)
        t0 = time.perf_counter()
        run()
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = dict(value=sample / dt, unit=UNIT, cores=threads, kind="oracle",
                                    sample=sample_desc(sample, ratio) + "; one pass, %.1f s" % dt)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--ratio", type=float, default=0.5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.warmup < 3:
        args.warmup = 3
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
