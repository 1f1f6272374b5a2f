"""Times one kernel of the path in isolation through the C ABI.

    python -m paper_2602_10431_b200.kernel_probe gemm --M 4096 --N 4096 --K 4096 --epilogue store
    python -m paper_2602_10431_b200.kernel_probe router --T 8192 --d 4096 --mode topk --ratio 0.5
    python -m paper_2602_10431_b200.kernel_probe compact --T 8192 --d 4096 --ratio 0.5
    python -m paper_2602_10431_b200.kernel_probe scatter --T 8192 --d 4096 --ratio 0.5
    python -m paper_2602_10431_b200.kernel_probe layer --config c2 --ratio 0.5
    python -m paper_2602_10431_b200.kernel_probe decode --config c3_int3 --ratio 0.9 --graph

Prints one line with the mean duration (CUDA events on the launching stream, after
warm-up) and the achieved algorithmic rate: bytes the method must move (or FLOPs it must
compute) per launch divided by the duration.  Small argument values give a case that is
suitable for a profiler capture.  Inputs are synthetic (random bits are fine for timing).
"""
from __future__ import annotations

import argparse

import numpy as np
import torch

from . import api, inputs


GRAPH = False  # --graph: replay the calls from a CUDA graph, so that short kernels are not timed
               # at the rate the host can launch them


def _time(fn, iters, warmup=3):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    if GRAPH:
        side = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for _ in range(iters):
                    fn()
            g.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(side)
            for _ in range(5):
                g.replay()
            e1.record(side)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / (5 * iters) * 1e-3
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters * 1e-3


def _tiled_weight(N, K, bits, group, row_mode, dev):
    """A quantised weight built by tiling 256 real rows (generation of all rows is slow)."""
    base = inputs.quantized_weight(0, 1, 256, K, bits, group)
    rep = (N + 255) // 256
    wq = dict(packed=np.tile(base["packed"], (rep, 1))[:N], scales=np.tile(base["scales"], (rep, 1))[:N],
              zeros=np.tile(base["zeros"], (rep, 1))[:N], N=N, K=K, bits=bits, group=group)
    return api.QuantWeight(wq, dev, row_mode)


def probe_gemm(a, dev):
    T = max(a.M, a.M_cap or a.M)
    adt = torch.float16 if a.act == "f16" else torch.bfloat16
    row_mode = api.ROWS_SWIGLU if a.epilogue == "swiglu" else api.ROWS_PLAIN
    qw = _tiled_weight(a.N, a.K, a.bits, a.group, row_mode, dev)
    x = torch.randn(T, a.K, device=dev).to(adt)
    md = torch.tensor([a.M], dtype=torch.int32, device=dev)
    idx = torch.arange(T, dtype=torch.int32, device=dev)
    resid16 = torch.randn(T, a.N, device=dev).to(torch.bfloat16)
    resid32 = torch.randn(T, a.N, device=dev)
    y16 = torch.empty(T, a.N, dtype=adt, device=dev)
    y32 = torch.empty(T, a.N, dtype=torch.float32, device=dev)
    ysw = torch.empty(T, a.N // 2, dtype=adt, device=dev)
    calls = {
        "store": lambda: api.wq_gemm(x, qw, md, api.EPI_STORE_16, y=y16),
        "f32": lambda: api.wq_gemm(x, qw, md, api.EPI_STORE_F32, y=y32),
        "resid": lambda: api.wq_gemm(x, qw, md, api.EPI_RESID_F32, y=y32, idx=idx, resid=resid16),
        "scatter": lambda: api.wq_gemm(x, qw, md, api.EPI_RESID_SCATTER, idx=idx, resid=resid32, dst=resid16),
        "swiglu": lambda: api.wq_gemm(x, qw, md, api.EPI_SWIGLU, y=ysw),
    }
    sec = _time(calls[a.epilogue], a.iters)
    flops = 2.0 * a.M * a.N * a.K
    print("gemm M=%d N=%d K=%d int%d g%d %s epilogue=%s: %.1f us, %.1f TFLOP/s (status %d)" % (
        a.M, a.N, a.K, a.bits, a.group, a.act, a.epilogue, sec * 1e6, flops / sec / 1e12, api.device_status()))


def _selection(a, dev):
    T = a.T
    k = api.topk_count(a.ratio, T)
    idx = torch.sort(torch.randperm(T, device=dev)[:max(k, 1)])[0].to(torch.int32)
    idx_full = torch.zeros(T, dtype=torch.int32, device=dev)
    idx_full[:k] = idx[:k]
    return k, idx_full, torch.tensor([k], dtype=torch.int32, device=dev)


def probe_router(a, dev):
    T, d = a.T, a.d
    x = torch.randn(T, d, device=dev).to(torch.bfloat16)
    w = (torch.randn(d, device=dev) * 0.02).to(torch.bfloat16).float()
    cu = torch.tensor([0, T], dtype=torch.int32, device=dev)
    mode = api.SELECT_TOPK if a.mode == "topk" else api.SELECT_THRESHOLD
    k = api.topk_count(a.ratio, T)
    out = api.router_select(x, w, 0.0, cu, mode, theta=0.5, k=k)
    if a.select_only:  # scores supplied: times the decision + compaction alone
        sc = out["scores"].clone()
        sec = _time(lambda: api.router_select(None, None, 0.0, cu, mode, theta=0.5, k=k,
                                              scores_override=sc, out=out), a.iters)
        print("select only T=%d mode=%s: %.1f us" % (T, a.mode, sec * 1e6))
        return
    sec = _time(lambda: api.router_select(x, w, 0.0, cu, mode, theta=0.5, k=k, out=out), a.iters)
    nbytes = T * (2 * d + 4)
    print("router_select T=%d d=%d mode=%s: %.1f us, %.0f GB/s of %d algorithmic bytes (n_exec %d)" % (
        T, d, a.mode, sec * 1e6, nbytes / sec / 1e9, nbytes, int(out["n_exec"].item())))


def probe_compact(a, dev):
    T, d = a.T, a.d
    k, idx, n = _selection(a, dev)
    x = torch.randn(T, d, device=dev).to(torch.bfloat16)
    gamma = torch.ones(d, device=dev)
    xc = torch.empty_like(x)
    hn = torch.empty(T, d, dtype=torch.float16, device=dev)
    if a.norm:
        fn = lambda: api.compact(x, idx, n, gamma, 1e-5, want_xc=False, hn_out=hn, act_dtype=api.ACT_F16)
    else:
        fn = lambda: api.compact(x, idx, n, None, 1e-5, xc_out=xc)
    sec = _time(fn, a.iters)
    nbytes = k * 4 * d
    print("compact T=%d d=%d executed=%d norm=%d: %.1f us, %.0f GB/s of %d algorithmic bytes" % (
        T, d, k, int(a.norm), sec * 1e6, nbytes / sec / 1e9, nbytes))


def probe_scatter(a, dev):
    T, d = a.T, a.d
    k, idx, n = _selection(a, dev)
    x = torch.randn(T, d, device=dev).to(torch.bfloat16)
    xc = torch.randn(T, d, device=dev).to(torch.bfloat16)
    f = torch.randn(T, d, device=dev)
    sec = _time(lambda: api.scatter_add(x, xc, f, idx, n), a.iters)
    nbytes = k * 8 * d
    print("scatter_add T=%d d=%d executed=%d: %.1f us, %.0f GB/s of %d algorithmic bytes" % (
        T, d, k, sec * 1e6, nbytes / sec / 1e9, nbytes))


def probe_layer(a, dev):
    c = inputs.CONFIG_SHAPES[a.config]
    sh, B, S = c["shape"], c["B"], c["S"]
    T = B * S
    w = inputs.layer_weights(0, 0, sh)
    lw = api.LayerWeights(w, dev)
    cfg = api.layer_config(sh, api.SELECT_TOPK, ratio=a.ratio)
    ws = torch.zeros(api.layer_workspace_bytes(cfg, T, B), dtype=torch.uint8, device=dev)
    x = torch.randn(T, sh.d, device=dev).to(torch.bfloat16)
    cu = torch.from_numpy(inputs.cu_seqlens_uniform(B, S)).to(dev)
    nex = torch.zeros(1, dtype=torch.int32, device=dev)
    sec = _time(lambda: api.layer_forward(cfg, lw, x, cu, ws, nex), a.iters)
    print("layer %s ratio=%.2f: %.1f us, %.0f tokens/s (executed %d of %d, status %d)" % (
        a.config, a.ratio, sec * 1e6, T / sec, int(nex.item()), T, api.device_status()))


def probe_decode(a, dev):
    """One decode step of the layer: B sequences with one new token each, a per-layer cache of
    `--kv-len` executed tokens per sequence, router scores supplied so that round(ratio * B)
    sequences execute.  Bytes counted: packed weights once, cached K and V of the executed
    sequences once."""
    c = inputs.CONFIG_SHAPES[a.config]
    sh, B = c["shape"], c["B"]
    w = inputs.layer_weights(0, 0, sh)
    lw = api.LayerWeights(w, dev)
    k = api.topk_count(a.ratio, B)
    logits = inputs.normal(3, 77, B)
    scores = (1.0 / (1.0 + np.exp(-logits))).astype(np.float32)
    order = np.sort(scores)[::-1]
    theta = float((order[k - 1] + order[k]) / 2) if 0 < k < B else (0.0 if k == B else 2.0)
    cfg = api.layer_config(sh, api.SELECT_THRESHOLD, theta=theta)
    cap = a.kv_len + 8
    kv = api.KvCache(B, cap, sh.kv_dim, dev, act_dtype=cfg.act_dtype)
    kv.k.normal_()
    kv.v.normal_()
    ws = torch.zeros(api.layer_workspace_bytes(cfg, B, B), dtype=torch.uint8, device=dev)
    x = torch.randn(B, sh.d, device=dev).to(torch.bfloat16)
    cu = torch.arange(B + 1, dtype=torch.int32, device=dev)
    pos0 = torch.full((B,), a.kv_len, dtype=torch.int32, device=dev)
    sc = torch.from_numpy(scores).to(dev)
    nex = torch.zeros(1, dtype=torch.int32, device=dev)

    def step():
        kv.kv_len.fill_(a.kv_len)  # every step appends at the same place
        api.layer_forward(cfg, lw, x, cu, ws, nex, pos0=pos0, scores_override=sc, kv=kv,
                          phase=api.PHASE_DECODE)

    sec = _time(step, a.iters)
    wbytes = sum(q.blob.numel() for q in (lw.qkv, lw.o, lw.gate_up, lw.down))
    kvbytes = k * a.kv_len * sh.kv_dim * 2 * 2
    print("decode %s ratio=%.2f (%d of %d sequences, kv_len %d): %.1f us, %.0f GB/s of %d algorithmic "
          "bytes (weights %d + cache %d) (status %d)" % (
              a.config, a.ratio, int(nex.item()), B, a.kv_len, sec * 1e6, (wbytes + kvbytes) / sec / 1e9,
              wbytes + kvbytes, wbytes, kvbytes, api.device_status()))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("kernel", choices=["gemm", "router", "compact", "scatter", "layer", "decode"])
    ap.add_argument("--M", type=int, default=4096)
    ap.add_argument("--M_cap", type=int, default=0)
    ap.add_argument("--N", type=int, default=4096)
    ap.add_argument("--K", type=int, default=4096)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--group", type=int, default=128)
    ap.add_argument("--act", default="f16", choices=["f16", "bf16"])
    ap.add_argument("--epilogue", default="store", choices=["store", "f32", "resid", "scatter", "swiglu"])
    ap.add_argument("--T", type=int, default=8192)
    ap.add_argument("--d", type=int, default=4096)
    ap.add_argument("--ratio", type=float, default=0.5)
    ap.add_argument("--mode", default="topk", choices=["topk", "threshold"])
    ap.add_argument("--norm", action="store_true")
    ap.add_argument("--select-only", dest="select_only", action="store_true")
    ap.add_argument("--config", default="c2")
    ap.add_argument("--kv-len", dest="kv_len", type=int, default=2048)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--graph", action="store_true")
    a = ap.parse_args()
    global GRAPH
    GRAPH = a.graph
    api.lib()
    dev = torch.device("cuda", 0)
    {"gemm": probe_gemm, "router": probe_router, "compact": probe_compact, "scatter": probe_scatter,
     "layer": probe_layer, "decode": probe_decode}[a.kernel](a, dev)


if __name__ == "__main__":
    main()
