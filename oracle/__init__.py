"""ctypes front end of the CPU oracle (test infrastructure only).

The oracle is the plain C file next to this module; see its header for what
it defines and which passages of the paper each function follows.  Nothing in
the product package may import this module: only the tests, the smoke check
and the benchmark's CPU-baseline leg do.  It shares no code with the CUDA
library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qtale_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP over independent rows only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_LIB)
        _lib.orc_half_to_float.restype = C.c_float
        _lib.orc_half_to_float.argtypes = [C.c_uint16]
        _lib.orc_float_to_half.restype = C.c_uint16
        _lib.orc_float_to_half.argtypes = [C.c_float]
        _lib.orc_round_bf16.restype = C.c_float
        _lib.orc_round_bf16.argtypes = [C.c_float]
        _lib.orc_topk_count.restype = C.c_int
        _lib.orc_topk_count.argtypes = [C.c_double, C.c_int]
        _lib.orc_layer_forward.restype = C.c_int
        _lib.orc_get_threads.restype = C.c_int
        _lib.orc_row_bytes.restype = C.c_int
        _lib.orc_theta_for_ratio.restype = C.c_float
        _lib.orc_theta_for_ratio.argtypes = [C.POINTER(C.c_float), C.POINTER(C.c_uint8), C.c_long,
                                             C.c_double, C.POINTER(C.c_long)]
        set_threads(os.cpu_count() or 1)
    return _lib


def set_threads(n: int) -> None:
    lib().orc_set_threads(C.c_int(int(n)))


def get_threads() -> int:
    return int(lib().orc_get_threads())


def set_emulate_bf16(on: bool) -> None:
    lib().orc_set_emulate_bf16(C.c_int(1 if on else 0))


def _p(a, ty):
    if a is None:
        return None
    return a.ctypes.data_as(C.POINTER(ty))


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _u8(a):
    return np.ascontiguousarray(a, dtype=np.uint8)


def _u16(a):
    a = np.ascontiguousarray(a)
    if a.dtype == np.float16:
        a = a.view(np.uint16)
    return np.ascontiguousarray(a, dtype=np.uint16)


# ---- router / selection -----------------------------------------------------

def router_scores(x, w, bias, return_logits=False):
    x, w = _f32(x), _f32(w)
    T, d = x.shape
    p = np.empty(T, dtype=np.float32)
    z = np.empty(T, dtype=np.float64)
    lib().orc_router_scores(_p(x, C.c_float), T, d, _p(w, C.c_float), C.c_float(bias),
                            _p(p, C.c_float), _p(z, C.c_double))
    return (p, z) if return_logits else p


def router_mlp_scores(x, w1, b1, w2, b2, return_logits=False):
    """MLP router: w1 [h, d], b1 [h], w2 [2, h], b2 [2]; returns p0 (and g0 - g1)."""
    x, w1, b1, w2, b2 = _f32(x), _f32(w1), _f32(b1), _f32(w2), _f32(b2)
    T, d = x.shape
    h = w1.shape[0]
    assert w1.shape == (h, d) and b1.shape == (h,) and w2.shape == (2, h) and b2.shape == (2,)
    p = np.empty(T, dtype=np.float32)
    z = np.empty(T, dtype=np.float64)
    lib().orc_router_mlp_scores(_p(x, C.c_float), T, d, _p(w1, C.c_float), _p(b1, C.c_float), h,
                                _p(w2, C.c_float), _p(b2, C.c_float), _p(p, C.c_float), _p(z, C.c_double))
    return (p, z) if return_logits else p


def softmax2_p0(g0, g1):
    g0 = np.ascontiguousarray(g0, dtype=np.float64)
    g1 = np.ascontiguousarray(g1, dtype=np.float64)
    p = np.empty(g0.shape[0], dtype=np.float32)
    lib().orc_softmax2_p0(_p(g0, C.c_double), _p(g1, C.c_double), g0.shape[0], _p(p, C.c_float))
    return p


def select_threshold(p, theta, valid=None):
    p = _f32(p)
    v = None if valid is None else _u8(valid)
    m = np.empty(p.shape[0], dtype=np.uint8)
    lib().orc_select_threshold(_p(p, C.c_float), _p(v, C.c_uint8), p.shape[0], C.c_float(theta),
                               _p(m, C.c_uint8))
    return m


def topk_count(ratio, n_valid):
    return int(lib().orc_topk_count(float(ratio), int(n_valid)))


def select_topk(p, k, valid=None):
    p = _f32(p)
    v = None if valid is None else _u8(valid)
    m = np.empty(p.shape[0], dtype=np.uint8)
    lib().orc_select_topk(_p(p, C.c_float), _p(v, C.c_uint8), p.shape[0], int(k), _p(m, C.c_uint8))
    return m


def theta_for_ratio(p, ratio, valid=None):
    """Global threshold for a requested execution ratio (Sec. 3.4): returns (theta, count)."""
    p = _f32(p).reshape(-1)
    v = None if valid is None else _u8(valid).reshape(-1)
    c = C.c_long(0)
    th = lib().orc_theta_for_ratio(_p(p, C.c_float), _p(v, C.c_uint8), p.shape[0], float(ratio), C.byref(c))
    return float(th), int(c.value)


def compact_indices(mask, cu_seqlens):
    mask, cu = _u8(mask), _i32(cu_seqlens)
    T, B = mask.shape[0], cu.shape[0] - 1
    idx = np.zeros(T + 1, dtype=np.int32)
    pos = np.zeros(T + 1, dtype=np.int32)
    cu_exec = np.zeros(B + 1, dtype=np.int32)
    n = C.c_int32(0)
    lib().orc_compact_indices(_p(mask, C.c_uint8), T, _p(cu, C.c_int32), B, _p(idx, C.c_int32),
                              C.byref(n), _p(cu_exec, C.c_int32), _p(pos, C.c_int32))
    return idx[:n.value].copy(), int(n.value), cu_exec, pos[:n.value].copy()


# ---- quantised weights --------------------------------------------------------

def row_bytes(K, bits):
    return int(lib().orc_row_bytes(int(K), int(bits)))


def quantize(w, bits, group):
    w = _f32(w)
    N, K = w.shape
    ng = (K + group - 1) // group
    codes = np.empty((N, K), dtype=np.uint8)
    s = np.empty((N, ng), dtype=np.uint16)
    z = np.empty((N, ng), dtype=np.uint16)
    lib().orc_quantize(_p(w, C.c_float), N, K, bits, group, _p(codes, C.c_uint8),
                       _p(s, C.c_uint16), _p(z, C.c_uint16))
    return codes, s.view(np.float16), z.view(np.float16)


def pack_codes(codes, bits):
    codes = _u8(codes)
    N, K = codes.shape
    out = np.empty((N, row_bytes(K, bits)), dtype=np.uint8)
    lib().orc_pack_codes(_p(codes, C.c_uint8), N, K, bits, _p(out, C.c_uint8))
    return out


def unpack_codes(packed, K, bits):
    packed = _u8(packed)
    N = packed.shape[0]
    out = np.empty((N, K), dtype=np.uint8)
    lib().orc_unpack_codes(_p(packed, C.c_uint8), N, K, bits, _p(out, C.c_uint8))
    return out


def dequantize(packed, scales, zeros, K, bits, group):
    packed, s, z = _u8(packed), _u16(scales), _u16(zeros)
    N = packed.shape[0]
    out = np.empty((N, K), dtype=np.float32)
    lib().orc_dequantize(_p(packed, C.c_uint8), _p(s, C.c_uint16), _p(z, C.c_uint16), N, K, bits,
                         group, _p(out, C.c_float))
    return out


def dequantize_weight(wq):
    """wq: dict from inputs.quantized_weight."""
    return dequantize(wq["packed"], wq["scales"], wq["zeros"], wq["K"], wq["bits"], wq["group"])


def requantize_fixed(w_hat, scales, zeros, bits, group):
    w_hat, s, z = _f32(w_hat), _u16(scales), _u16(zeros)
    N, K = w_hat.shape
    out = np.empty((N, K), dtype=np.uint8)
    lib().orc_requantize_fixed(_p(w_hat, C.c_float), _p(s, C.c_uint16), _p(z, C.c_uint16), N, K,
                               bits, group, _p(out, C.c_uint8))
    return out


# ---- dense blocks ---------------------------------------------------------------

def rmsnorm(x, gamma, eps):
    x, gamma = _f32(x), _f32(gamma)
    T, d = x.shape
    y = np.empty_like(x)
    lib().orc_rmsnorm(_p(x, C.c_float), T, d, _p(gamma, C.c_float), C.c_float(eps), _p(y, C.c_float))
    return y


def linear(x, w):
    x, w = _f32(x), _f32(w)
    T, K = x.shape
    N = w.shape[0]
    assert w.shape[1] == K
    y = np.empty((T, N), dtype=np.float32)
    lib().orc_linear(_p(x, C.c_float), T, K, _p(w, C.c_float), N, _p(y, C.c_float))
    return y


def rope(v, n_heads, hd, pos, base):
    v = _f32(v).copy()
    T = v.shape[0]
    pos = _i32(pos)
    lib().orc_rope(_p(v, C.c_float), T, n_heads, hd, C.c_size_t(n_heads * hd), _p(pos, C.c_int32),
                   C.c_float(base))
    return v


def swiglu(gate, up):
    gate, up = _f32(gate), _f32(up)
    out = np.empty_like(gate)
    lib().orc_swiglu(_p(gate, C.c_float), _p(up, C.c_float), C.c_size_t(gate.size), _p(out, C.c_float))
    return out


def attention(q, k, v, H, Hkv, hd, seq_of, pos, cache_k=None, cache_v=None, kv_len=None, cap=0):
    q, k, v = _f32(q), _f32(k), _f32(v)
    Te = q.shape[0]
    seq_of, pos = _i32(seq_of), _i32(pos)
    out = np.empty((Te, H * hd), dtype=np.float32)
    ck = None if cache_k is None else _f32(cache_k)
    cv = None if cache_v is None else _f32(cache_v)
    kl = None if kv_len is None else _i32(kv_len)
    lib().orc_attention(_p(q, C.c_float), _p(k, C.c_float), _p(v, C.c_float), Te, H, Hkv, hd,
                        _p(seq_of, C.c_int32), _p(pos, C.c_int32), _p(ck, C.c_float),
                        _p(cv, C.c_float), _p(kl, C.c_int32), int(cap), _p(out, C.c_float))
    return out


def gather_rows(x, idx):
    x, idx = _f32(x), _i32(idx)
    out = np.empty((idx.shape[0], x.shape[1]), dtype=np.float32)
    lib().orc_gather_rows(_p(x, C.c_float), _p(idx, C.c_int32), idx.shape[0], x.shape[1],
                          _p(out, C.c_float))
    return out


def scatter_add(x, xc, f, idx):
    x = _f32(x).copy()
    xc, f, idx = _f32(xc), _f32(f), _i32(idx)
    lib().orc_scatter_add(_p(x, C.c_float), _p(xc, C.c_float), _p(f, C.c_float), _p(idx, C.c_int32),
                          idx.shape[0], x.shape[1])
    return x


# ---- layer ------------------------------------------------------------------------

class _Shape(C.Structure):
    _fields_ = [("d", C.c_int), ("n_heads", C.c_int), ("n_kv_heads", C.c_int),
                ("head_dim", C.c_int), ("ffn", C.c_int), ("rms_eps", C.c_float),
                ("rope_theta", C.c_float)]


class _Weights(C.Structure):
    _fields_ = [("w_qkv", C.POINTER(C.c_float)), ("w_o", C.POINTER(C.c_float)),
                ("w_gate_up", C.POINTER(C.c_float)), ("w_down", C.POINTER(C.c_float)),
                ("gamma1", C.POINTER(C.c_float)), ("gamma2", C.POINTER(C.c_float))]


class DenseLayer:
    """Dequantised fp32 weights of one layer, ready for layer_forward."""

    def __init__(self, sh, w):
        self.sh = sh
        self.w_qkv = dequantize_weight(w["qkv"])
        self.w_o = dequantize_weight(w["o"])
        self.w_gate_up = dequantize_weight(w["gate_up"])
        self.w_down = dequantize_weight(w["down"])
        self.gamma1 = _f32(w["gamma1"])
        self.gamma2 = _f32(w["gamma2"])
        self.router_w = _f32(w["router_w"])
        self.router_b = float(w["router_b"])


def layer_forward(layer: DenseLayer, x, cu_seqlens, mask, pos0=None, cache_k=None, cache_v=None,
                  kv_len=None):
    """Token-adaptive layer (Eq. 3) with a given execute mask.  Returns (x_out, n_exec).

    cache_k / cache_v ([B, cap, Hkv*hd] float32) and kv_len (int32 [B]) are
    updated IN PLACE when given.
    """
    sh = layer.sh
    x = _f32(x)
    T, d = x.shape
    cu, mask = _i32(cu_seqlens), _u8(mask)
    B = cu.shape[0] - 1
    s = _Shape(sh.d, sh.n_heads, sh.n_kv_heads, sh.head_dim, sh.ffn, sh.rms_eps, sh.rope_theta)
    w = _Weights(_p(layer.w_qkv, C.c_float), _p(layer.w_o, C.c_float),
                 _p(layer.w_gate_up, C.c_float), _p(layer.w_down, C.c_float),
                 _p(layer.gamma1, C.c_float), _p(layer.gamma2, C.c_float))
    out = np.empty_like(x)
    cap = 0
    if cache_k is not None:
        assert cache_k.dtype == np.float32 and cache_k.flags.c_contiguous
        assert cache_v.dtype == np.float32 and cache_v.flags.c_contiguous
        assert kv_len.dtype == np.int32
        cap = cache_k.shape[1]
    p0 = None if pos0 is None else _i32(pos0)
    n = lib().orc_layer_forward(C.byref(s), C.byref(w), _p(x, C.c_float), T, _p(cu, C.c_int32), B,
                                _p(mask, C.c_uint8), _p(p0, C.c_int32), _p(cache_k, C.c_float),
                                _p(cache_v, C.c_float), _p(kv_len, C.c_int32), int(cap),
                                _p(out, C.c_float))
    return out, int(n)


def route(layer: DenseLayer, x, mode, theta=0.5, ratio=None, valid=None):
    """Router + selection of one layer.  mode: 'threshold' (Eq. 9) or 'topk'."""
    p = router_scores(x, layer.router_w, layer.router_b)
    if mode == "threshold":
        return p, select_threshold(p, theta, valid)
    n_valid = int(p.shape[0] if valid is None else np.count_nonzero(valid))
    return p, select_topk(p, topk_count(ratio, n_valid), valid)


def model_prefill(layers, embed, ids, cu_seqlens, theta=None, ratios=None, final_gamma=None,
                  lm_head=None, logit_rows=None, eps=1e-5, valid=None, scores_out=None):
    """Embedding gather, L token-adaptive layers sharing one theta (or per-layer
    top-k ratios), final RMSNorm, LM head on the requested rows."""
    x = _f32(embed)[np.asarray(ids, dtype=np.int64)]
    counts = []
    for li, layer in enumerate(layers):
        if ratios is not None:
            p, m = route(layer, x, "topk", ratio=ratios[li], valid=valid)
        else:
            p, m = route(layer, x, "threshold", theta=theta, valid=valid)
        if scores_out is not None:
            scores_out.append(p)
        x, n = layer_forward(layer, x, cu_seqlens, m)
        counts.append(n)
    logits = None
    if lm_head is not None:
        rows = np.arange(x.shape[0]) if logit_rows is None else np.asarray(logit_rows)
        hn = rmsnorm(x[rows], final_gamma, eps)
        logits = linear(hn, lm_head)
    return x, logits, counts
