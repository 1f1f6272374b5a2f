"""Thin Python binding over libqtale's C ABI (argument marshalling only).

Every function here forwards to the `extern "C"` entry point of the same name
declared in include/qtale.h; all arithmetic of the path runs in the library's
CUDA kernels.  PyTorch supplies device memory and the current stream.  There
is no fallback: importing this module without the built library, or calling
it without a CUDA device, raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libqtale.so")

SELECT_THRESHOLD, SELECT_TOPK, SELECT_FORCED = 0, 1, 2
EPI_STORE_16, EPI_STORE_F32, EPI_RESID_F32, EPI_RESID_SCATTER, EPI_SWIGLU, EPI_ROPE = 0, 1, 2, 3, 4, 5
ACT_BF16, ACT_F16 = 0, 1
ROWS_PLAIN, ROWS_SWIGLU, ROWS_ROPE64, ROWS_ROPE128 = 0, 1, 2, 3
PHASE_PREFILL, PHASE_DECODE = 0, 1

EXPORTS = [
    "qtale_strerror", "qtale_device_status", "qtale_topk_count",
    "qtale_router_select_workspace_bytes", "qtale_router_select", "qtale_router_select_static",
    "qtale_index_bookkeeping",
    "qtale_compact", "qtale_scatter_add", "qtale_wq_repack", "qtale_wq_gemm",
    "qtale_wq_gemm_workspace_bytes",
    "qtale_layer_workspace_bytes", "qtale_layer_forward", "qtale_model_workspace_bytes",
    "qtale_model_prefill", "qtale_theta_workspace_bytes", "qtale_theta_for_ratio",
    "qtale_model_decode_workspace_bytes", "qtale_model_decode_step", "qtale_router_mlp_scores",
]


class QtaleError(RuntimeError):
    pass


class WqWeight(C.Structure):
    _fields_ = [("packed", C.c_void_p), ("N", C.c_int), ("K", C.c_int), ("bits", C.c_int),
                ("group", C.c_int), ("row_mode", C.c_int)]


class EpilogueArgs(C.Structure):
    _fields_ = [("idx", C.c_void_p), ("resid", C.c_void_p), ("ld_resid", C.c_int),
                ("dst", C.c_void_p), ("ld_dst", C.c_int), ("rope_cs", C.c_void_p),
                ("rope_features", C.c_int)]


class LayerConfig(C.Structure):
    _fields_ = [("d", C.c_int), ("n_heads", C.c_int), ("n_kv_heads", C.c_int),
                ("head_dim", C.c_int), ("ffn", C.c_int), ("bits", C.c_int), ("group", C.c_int),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("select_mode", C.c_int),
                ("theta", C.c_float), ("ratio", C.c_float), ("act_dtype", C.c_int)]


class LayerWeightsC(C.Structure):
    _fields_ = [("qkv", WqWeight), ("o", WqWeight), ("gate_up", WqWeight), ("down", WqWeight),
                ("gamma1", C.c_void_p), ("gamma2", C.c_void_p), ("router_w", C.c_void_p),
                ("router_b", C.c_float), ("router_h", C.c_int), ("router_w1", C.c_void_p),
                ("router_b1", C.c_void_p), ("router_w2", C.c_void_p), ("router_b2", C.c_float * 2)]


class KvCacheC(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("kv_len", C.c_void_p), ("cap", C.c_int)]


class ModelConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("vocab", C.c_int), ("layer", LayerConfig)]


class ModelWeightsC(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("layers", C.POINTER(LayerWeightsC)),
                ("final_gamma", C.c_void_p), ("lm_head", C.c_void_p)]


_lib = None


def lib():
    """Loads libqtale.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise QtaleError("libqtale.so is missing: run `python -m paper_2602_10431_b200.build`")
        L = C.CDLL(LIB_PATH)
        L.qtale_strerror.restype = C.c_char_p
        L.qtale_strerror.argtypes = [C.c_int]
        L.qtale_device_status.argtypes = [C.c_void_p]
        L.qtale_topk_count.argtypes = [C.c_double, C.c_int]
        L.qtale_router_select_workspace_bytes.restype = C.c_size_t
        L.qtale_router_select_workspace_bytes.argtypes = [C.c_int]
        L.qtale_router_select.argtypes = [
            C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_float, C.c_int, C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.qtale_router_select_static.argtypes = L.qtale_router_select.argtypes[:18] + [C.c_void_p]
        L.qtale_index_bookkeeping.argtypes = [
            C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_void_p]
        L.qtale_compact.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                    C.c_void_p, C.c_float, C.c_int, C.c_void_p, C.c_void_p,
                                    C.c_void_p]
        L.qtale_scatter_add.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_int, C.c_int, C.c_void_p]
        L.qtale_wq_repack.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                      C.c_int, C.c_int, C.c_void_p, C.POINTER(C.c_size_t)]
        L.qtale_wq_gemm.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.POINTER(WqWeight),
                                    C.c_int, C.c_int, C.POINTER(EpilogueArgs), C.c_void_p, C.c_int,
                                    C.c_void_p, C.c_size_t, C.c_void_p]
        L.qtale_attention_prefill.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                              C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_int,
                                              C.c_void_p]
        L.qtale_wq_gemm_workspace_bytes.restype = C.c_size_t
        L.qtale_wq_gemm_workspace_bytes.argtypes = []
        L.qtale_layer_workspace_bytes.restype = C.c_size_t
        L.qtale_layer_workspace_bytes.argtypes = [C.POINTER(LayerConfig), C.c_int, C.c_int]
        L.qtale_layer_forward.argtypes = [
            C.POINTER(LayerConfig), C.POINTER(LayerWeightsC), C.c_void_p, C.c_int, C.c_void_p,
            C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.POINTER(KvCacheC),
            C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.qtale_model_workspace_bytes.restype = C.c_size_t
        L.qtale_model_workspace_bytes.argtypes = [C.POINTER(ModelConfig), C.c_int, C.c_int, C.c_int]
        L.qtale_model_prefill.argtypes = [
            C.POINTER(ModelConfig), C.POINTER(ModelWeightsC), C.c_void_p, C.c_int, C.c_void_p,
            C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.qtale_model_decode_workspace_bytes.restype = C.c_size_t
        L.qtale_model_decode_workspace_bytes.argtypes = [C.POINTER(ModelConfig), C.c_int]
        L.qtale_model_decode_step.argtypes = [
            C.POINTER(ModelConfig), C.POINTER(ModelWeightsC), C.c_void_p, C.c_int, C.c_void_p,
            C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
            C.c_void_p, C.c_size_t, C.c_void_p]
        L.qtale_router_mlp_scores.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                              C.c_void_p, C.c_int, C.c_float, C.c_float, C.c_void_p,
                                              C.c_void_p]
        L.qtale_theta_workspace_bytes.restype = C.c_size_t
        L.qtale_theta_workspace_bytes.argtypes = []
        L.qtale_theta_for_ratio.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_double, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        _lib = L
    return _lib


def strerror(rc: int) -> str:
    return lib().qtale_strerror(int(rc)).decode()


def check(rc: int, what: str = "") -> None:
    if rc != 0:
        raise QtaleError("%s failed: %s (%d)" % (what or "libqtale call", strerror(rc), rc))


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def device_status() -> int:
    return int(lib().qtale_device_status(_stream()))


def topk_count(ratio: float, n_valid: int) -> int:
    return int(lib().qtale_topk_count(float(ratio), int(n_valid)))


# ---------------------------------------------------------------------------------
# selection
# ---------------------------------------------------------------------------------

ROUTER_STATIC_MAX_TOKENS = 65536


def router_select_workspace_bytes(T: int) -> int:
    return int(lib().qtale_router_select_workspace_bytes(int(T)))


def router_select(x, w_router, bias, cu_seqlens, mode, theta=0.5, k=0, scores_override=None,
                  valid=None, pos0=None, out=None):
    """qtale_router_select.  x bf16 [T, d]; w_router fp32 [d]; cu_seqlens int32 [B+1].
    Returns dict(scores, idx, n_exec, cu_exec, pos) of device tensors."""
    T = int(x.shape[0]) if x is not None else int(scores_override.shape[0])
    d = int(x.shape[1]) if x is not None else 0
    dev = (x if x is not None else scores_override).device
    B = int(cu_seqlens.shape[0]) - 1
    o = out or {}
    scores = o.get("scores", None)
    if scores is None:
        scores = torch.empty(T, dtype=torch.float32, device=dev)
    idx = o.get("idx") if "idx" in o else torch.full((T,), -1, dtype=torch.int32, device=dev)
    pos = o.get("pos") if "pos" in o else torch.full((T,), -1, dtype=torch.int32, device=dev)
    n_exec = o.get("n_exec") if "n_exec" in o else torch.zeros(1, dtype=torch.int32, device=dev)
    cu_exec = o.get("cu_exec") if "cu_exec" in o else torch.zeros(B + 1, dtype=torch.int32, device=dev)
    ws = o.get("ws") if "ws" in o else torch.empty(router_select_workspace_bytes(T), dtype=torch.uint8,
                                                   device=dev)
    check(lib().qtale_router_select(
        _ptr(x), T, d, _ptr(w_router), float(bias), _ptr(scores_override), _ptr(valid),
        _ptr(cu_seqlens), B, _ptr(pos0), int(mode), float(theta), int(k), _ptr(scores), _ptr(idx),
        _ptr(n_exec), _ptr(cu_exec), _ptr(pos), _ptr(ws), ws.numel(), _stream()),
        "qtale_router_select")
    return dict(scores=scores, idx=idx, n_exec=n_exec, cu_exec=cu_exec, pos=pos, ws=ws)


def router_select_static(x, w_router, bias, cu_seqlens, mode, out, theta=0.5, k=0,
                         scores_override=None, valid=None, pos0=None):
    """qtale_router_select_static: same as router_select but without a workspace; the
    scratch is built into the library, so this wrapper allocates nothing either --
    the caller passes every output tensor in `out` (scores, idx, n_exec, cu_exec, pos)."""
    T = int(x.shape[0]) if x is not None else int(scores_override.shape[0])
    d = int(x.shape[1]) if x is not None else 0
    B = int(cu_seqlens.shape[0]) - 1
    check(lib().qtale_router_select_static(
        _ptr(x), T, d, _ptr(w_router), float(bias), _ptr(scores_override), _ptr(valid),
        _ptr(cu_seqlens), B, _ptr(pos0), int(mode), float(theta), int(k), _ptr(out["scores"]),
        _ptr(out["idx"]), _ptr(out["n_exec"]), _ptr(out["cu_exec"]), _ptr(out["pos"]), _stream()),
        "qtale_router_select_static")
    return out


def router_mlp_scores(x, w1, b1, w2, b2, scores_out=None):
    """qtale_router_mlp_scores.  x bf16 [T, d]; w1 bf16 [h, d]; b1 fp32 [h]; w2 fp32 [2, h];
    b2 = (execute, bypass)."""
    T, d = int(x.shape[0]), int(x.shape[1])
    if scores_out is None:
        scores_out = torch.empty(T, dtype=torch.float32, device=x.device)
    check(lib().qtale_router_mlp_scores(_ptr(x), T, d, _ptr(w1), _ptr(b1), _ptr(w2), int(w1.shape[0]),
                                        float(b2[0]), float(b2[1]), _ptr(scores_out), _stream()),
          "qtale_router_mlp_scores")
    return scores_out


def theta_for_ratio(scores, ratio, valid=None, out=None):
    """qtale_theta_for_ratio on a flat fp32 device tensor of pooled router scores.
    Returns (theta, count) as one-element device tensors (no host read-back here)."""
    dev = scores.device
    o = out or {}
    theta = o.get("theta") if "theta" in o else torch.zeros(1, dtype=torch.float32, device=dev)
    count = o.get("count") if "count" in o else torch.zeros(1, dtype=torch.int32, device=dev)
    ws = o.get("ws") if "ws" in o else torch.empty(int(lib().qtale_theta_workspace_bytes()),
                                                   dtype=torch.uint8, device=dev)
    check(lib().qtale_theta_for_ratio(_ptr(scores), _ptr(valid), int(scores.numel()), float(ratio),
                                      _ptr(theta), _ptr(count), _ptr(ws), ws.numel(), _stream()),
          "qtale_theta_for_ratio")
    return theta, count


def index_bookkeeping(idx, n, T, cu_seqlens, pos0=None):
    dev = cu_seqlens.device
    B = int(cu_seqlens.shape[0]) - 1
    n_exec = torch.zeros(1, dtype=torch.int32, device=dev)
    cu_exec = torch.zeros(B + 1, dtype=torch.int32, device=dev)
    pos = torch.full((max(T, 1),), -1, dtype=torch.int32, device=dev)
    check(lib().qtale_index_bookkeeping(_ptr(idx), int(n), int(T), _ptr(cu_seqlens), B, _ptr(pos0),
                                        _ptr(n_exec), _ptr(cu_exec), _ptr(pos), _stream()),
          "qtale_index_bookkeeping")
    return dict(n_exec=n_exec, cu_exec=cu_exec, pos=pos)


# ---------------------------------------------------------------------------------
# gather / scatter
# ---------------------------------------------------------------------------------

def act_torch_dtype(act_dtype):
    return torch.float16 if act_dtype == ACT_F16 else torch.bfloat16


def compact(x, idx, n_exec, rms_gamma=None, eps=1e-5, want_xc=True, xc_out=None, hn_out=None,
            act_dtype=ACT_BF16):
    """qtale_compact.  Returns (xc, hn); either may be None.  hn is in act_dtype."""
    T, d = int(x.shape[0]), int(x.shape[1])
    xc = xc_out if xc_out is not None else (torch.zeros_like(x) if want_xc else None)
    hn = hn_out
    if hn is None and rms_gamma is not None:
        hn = torch.zeros(T, d, dtype=act_torch_dtype(act_dtype), device=x.device)
    check(lib().qtale_compact(_ptr(x), _ptr(idx), _ptr(n_exec), T, d, _ptr(rms_gamma), float(eps),
                              int(act_dtype), _ptr(xc), _ptr(hn), _stream()), "qtale_compact")
    return xc, hn


def scatter_add(x_inout, xc, f, idx, n_exec):
    T, d = int(x_inout.shape[0]), int(x_inout.shape[1])
    check(lib().qtale_scatter_add(_ptr(x_inout), _ptr(xc), _ptr(f), _ptr(idx), _ptr(n_exec), T, d,
                                  _stream()), "qtale_scatter_add")
    return x_inout


# ---------------------------------------------------------------------------------
# quantised weights
# ---------------------------------------------------------------------------------

def wq_repack(packed_codes: np.ndarray, scales: np.ndarray, zeros: np.ndarray, N, K, bits, group,
              row_mode=ROWS_PLAIN) -> np.ndarray:
    """qtale_wq_repack on host arrays; returns the native blob as a uint8 numpy array."""
    codes = np.ascontiguousarray(packed_codes, dtype=np.uint8)
    s = np.ascontiguousarray(scales).view(np.uint16)
    z = np.ascontiguousarray(zeros).view(np.uint16)
    nbytes = C.c_size_t(0)
    check(lib().qtale_wq_repack(None, None, None, N, K, bits, group, row_mode, None,
                                C.byref(nbytes)), "qtale_wq_repack(size)")
    out = np.empty(nbytes.value, dtype=np.uint8)
    check(lib().qtale_wq_repack(codes.ctypes.data, s.ctypes.data, z.ctypes.data, N, K, bits, group,
                                row_mode, out.ctypes.data, C.byref(nbytes)), "qtale_wq_repack")
    return out


class QuantWeight:
    """Device copy of a repacked quantised linear plus its C descriptor."""

    def __init__(self, wq: dict, device="cuda", row_mode=ROWS_PLAIN):
        blob = wq_repack(wq["packed"], wq["scales"], wq["zeros"], wq["N"], wq["K"], wq["bits"],
                         wq["group"], row_mode)
        self.blob = torch.from_numpy(blob).to(device)
        self.N, self.K, self.bits, self.group, self.row_mode = (wq["N"], wq["K"], wq["bits"],
                                                                 wq["group"], row_mode)
        self.c = WqWeight(self.blob.data_ptr(), self.N, self.K, self.bits, self.group, row_mode)


def wq_gemm_workspace_bytes() -> int:
    return int(lib().qtale_wq_gemm_workspace_bytes())


def wq_gemm(a, w: QuantWeight, m_dev=None, epilogue=EPI_STORE_16, y=None, idx=None, resid=None,
            dst=None, rope_cs=None, rope_features=0, ws=None):
    """qtale_wq_gemm.  a bf16 or fp16 [M_cap, K] (its dtype is the act_dtype); returns y
    (or dst for RESID_SCATTER)."""
    M_cap, lda = int(a.shape[0]), int(a.stride(0))
    act_dtype = ACT_F16 if a.dtype == torch.float16 else ACT_BF16
    epi = None
    if epilogue in (EPI_RESID_F32, EPI_RESID_SCATTER):
        epi = EpilogueArgs(idx.data_ptr(), resid.data_ptr(), int(resid.stride(0)),
                           dst.data_ptr() if dst is not None else None,
                           int(dst.stride(0)) if dst is not None else 0, None, 0)
    if epilogue == EPI_ROPE:
        epi = EpilogueArgs(None, None, 0, None, 0, rope_cs.data_ptr(), int(rope_features))
    if y is None and epilogue != EPI_RESID_SCATTER:
        n_out = w.N // 2 if epilogue == EPI_SWIGLU else w.N
        dt = a.dtype if epilogue in (EPI_STORE_16, EPI_SWIGLU, EPI_ROPE) else torch.float32
        y = torch.zeros(M_cap, n_out, dtype=dt, device=a.device)
    check(lib().qtale_wq_gemm(_ptr(a), lda, _ptr(m_dev), M_cap, C.byref(w.c), act_dtype, int(epilogue),
                              C.byref(epi) if epi is not None else None, _ptr(y),
                              int(y.stride(0)) if y is not None else 0, _ptr(ws),
                              ws.numel() * ws.element_size() if ws is not None else 0, _stream()),
          "qtale_wq_gemm")
    return dst if epilogue == EPI_RESID_SCATTER else y


# ---------------------------------------------------------------------------------
# attention
# ---------------------------------------------------------------------------------

def attention_prefill(qkv, n_heads, n_kv_heads, head_dim, cu_exec, act_dtype=ACT_F16, out=None):
    """qtale_attention_prefill on a compacted [T_cap, (H + 2 Hkv) hd] tensor of rotated q | k | v."""
    import torch
    T_cap = int(qkv.shape[0])
    if out is None:
        out = torch.zeros(T_cap, n_heads * head_dim, dtype=qkv.dtype, device=qkv.device)
    check(lib().qtale_attention_prefill(_ptr(qkv), int(qkv.stride(0)), n_heads, n_kv_heads, head_dim,
                                        int(act_dtype), _ptr(cu_exec), int(cu_exec.numel()) - 1, T_cap,
                                        _ptr(out), int(out.stride(0)), _stream()),
          "qtale_attention_prefill")
    return out


# ---------------------------------------------------------------------------------
# layer / model
# ---------------------------------------------------------------------------------

def layer_config(sh, select_mode=SELECT_THRESHOLD, theta=0.5, ratio=1.0,
                 act_dtype=ACT_F16, bits=None) -> LayerConfig:
    """bits=0: every weight carries its own width (layers of mixed 2/3/4-bit precision)."""
    return LayerConfig(sh.d, sh.n_heads, sh.n_kv_heads, sh.head_dim, sh.ffn,
                       sh.bits if bits is None else int(bits), sh.group,
                       sh.rms_eps, sh.rope_theta, int(select_mode), float(theta), float(ratio),
                       int(act_dtype))


class LayerWeights:
    """Device-resident weights of one layer (from inputs.layer_weights)."""

    def __init__(self, w: dict, device="cuda", fuse_swiglu=True, fuse_rope=True, head_dim=None):
        # head_dim is needed for the rotary row layout of the QKV matrix
        rope_mode = ROWS_PLAIN
        if fuse_rope:
            head_dim = head_dim or w.get("head_dim")
            if head_dim not in (64, 128):
                raise QtaleError("LayerWeights(fuse_rope=True) needs head_dim (64 or 128)")
            rope_mode = ROWS_ROPE64 if head_dim == 64 else ROWS_ROPE128
        self.qkv = QuantWeight(w["qkv"], device, rope_mode)
        self.o = QuantWeight(w["o"], device)
        self.gate_up = QuantWeight(w["gate_up"], device, ROWS_SWIGLU if fuse_swiglu else ROWS_PLAIN)
        self.down = QuantWeight(w["down"], device)
        self.gamma1 = torch.from_numpy(np.ascontiguousarray(w["gamma1"], np.float32)).to(device)
        self.gamma2 = torch.from_numpy(np.ascontiguousarray(w["gamma2"], np.float32)).to(device)
        self.router_w = torch.from_numpy(np.ascontiguousarray(w["router_w"], np.float32)).to(device)
        self.router_b = float(w["router_b"])
        self.c = LayerWeightsC(self.qkv.c, self.o.c, self.gate_up.c, self.down.c,
                               self.gamma1.data_ptr(), self.gamma2.data_ptr(),
                               self.router_w.data_ptr(), self.router_b)
        mlp = w.get("router_mlp")  # dict(w1 [h, d], b1 [h], w2 [2, h], b2 [2]) -> MLP router
        if mlp is not None:
            self.router_w1 = to_device_bf16(mlp["w1"], device)
            self.router_b1 = torch.from_numpy(np.ascontiguousarray(mlp["b1"], np.float32)).to(device)
            self.router_w2 = torch.from_numpy(np.ascontiguousarray(mlp["w2"], np.float32)).to(device)
            self.c.router_h = int(mlp["w1"].shape[0])
            self.c.router_w1 = self.router_w1.data_ptr()
            self.c.router_b1 = self.router_b1.data_ptr()
            self.c.router_w2 = self.router_w2.data_ptr()
            self.c.router_b2 = (C.c_float * 2)(float(mlp["b2"][0]), float(mlp["b2"][1]))

    def set_router_bias(self, b: float):
        self.router_b = float(b)
        self.c.router_b = float(b)


class KvCache:
    """Per-layer cache of the executed tokens' keys / values, [B, n_kv_heads, cap, head_dim]."""

    def __init__(self, B, cap, kv_dim, device="cuda", act_dtype=ACT_F16, head_dim=128):
        dt = act_torch_dtype(act_dtype)
        self.B, self.cap, self.head_dim, self.n_kv_heads = B, cap, head_dim, kv_dim // head_dim
        self.k = torch.zeros(B, self.n_kv_heads, cap, head_dim, dtype=dt, device=device)
        self.v = torch.zeros(B, self.n_kv_heads, cap, head_dim, dtype=dt, device=device)
        self.kv_len = torch.zeros(B, dtype=torch.int32, device=device)
        self.c = KvCacheC(self.k.data_ptr(), self.v.data_ptr(), self.kv_len.data_ptr(), cap)

    def k_view(self):
        """Keys as a [B, cap, n_kv_heads, head_dim] view (entry-major, for filling / inspecting)."""
        return self.k.permute(0, 2, 1, 3)

    def v_view(self):
        return self.v.permute(0, 2, 1, 3)

    def k_rows(self):
        """Keys as a [B, cap, n_kv_heads * head_dim] copy: one row per cached token."""
        return self.k_view().reshape(self.B, self.cap, -1)

    def v_rows(self):
        return self.v_view().reshape(self.B, self.cap, -1)


def layer_workspace_bytes(cfg: LayerConfig, T_cap: int, B_cap: int) -> int:
    return int(lib().qtale_layer_workspace_bytes(C.byref(cfg), int(T_cap), int(B_cap)))


def layer_forward(cfg: LayerConfig, w: LayerWeights, x_inout, cu_seqlens, ws, n_exec_out=None,
                  scores_out=None, pos0=None, valid=None, scores_override=None, forced_idx=None,
                  forced_n=0, kv: KvCache | None = None, phase=PHASE_PREFILL):
    """qtale_layer_forward, in place on x_inout (bf16 [T, d])."""
    T = int(x_inout.shape[0])
    B = int(cu_seqlens.shape[0]) - 1
    check(lib().qtale_layer_forward(
        C.byref(cfg), C.byref(w.c), _ptr(x_inout), T, _ptr(cu_seqlens), B, _ptr(pos0), _ptr(valid),
        _ptr(scores_override), _ptr(forced_idx), int(forced_n),
        C.byref(kv.c) if kv is not None else None, int(phase), _ptr(n_exec_out), _ptr(scores_out),
        _ptr(ws), ws.numel() * ws.element_size(), _stream()), "qtale_layer_forward")
    return x_inout


def model_workspace_bytes(cfg: ModelConfig, T_cap, B_cap, n_logit_rows) -> int:
    return int(lib().qtale_model_workspace_bytes(C.byref(cfg), int(T_cap), int(B_cap),
                                                 int(n_logit_rows)))


def model_prefill(cfg: ModelConfig, layers, embed, ids, cu_seqlens, ws, hidden_out,
                  per_layer_ratio=None, final_gamma=None, lm_head=None, logit_rows=None,
                  logits_out=None, per_layer_n_exec=None, valid=None, layer_scores_out=None,
                  caches=None):
    """qtale_model_prefill.  layers: list of LayerWeights."""
    T = int(ids.shape[0])
    B = int(cu_seqlens.shape[0]) - 1
    arr = (LayerWeightsC * len(layers))(*[l.c for l in layers])
    mw = ModelWeightsC(embed.data_ptr(), arr,
                       final_gamma.data_ptr() if final_gamma is not None else None,
                       lm_head.data_ptr() if lm_head is not None else None)
    ratios = None
    if per_layer_ratio is not None:
        ratios = (C.c_float * len(layers))(*[float(r) for r in per_layer_ratio])
    n_rows = int(logit_rows.shape[0]) if logit_rows is not None else 0
    check(lib().qtale_model_prefill(
        C.byref(cfg), C.byref(mw), _ptr(ids), T, _ptr(cu_seqlens), B, _ptr(valid),
        C.cast(_cache_array(caches), C.c_void_p) if caches is not None else None,
        C.cast(ratios, C.c_void_p) if ratios is not None else None, _ptr(hidden_out),
        _ptr(logits_out), _ptr(logit_rows), n_rows, _ptr(per_layer_n_exec), _ptr(layer_scores_out), _ptr(ws),
        ws.numel() * ws.element_size(), _stream()), "qtale_model_prefill")
    return hidden_out


def _cache_array(caches):
    return (KvCacheC * len(caches))(*[c.c for c in caches])


def model_decode_workspace_bytes(cfg: ModelConfig, B_cap) -> int:
    return int(lib().qtale_model_decode_workspace_bytes(C.byref(cfg), int(B_cap)))


def model_decode_step(cfg: ModelConfig, layers, embed, ids, pos, caches, ws, hidden_out, valid=None,
                      final_gamma=None, lm_head=None, logits_out=None, next_ids_out=None,
                      per_layer_n_exec=None, layer_scores_out=None):
    """qtale_model_decode_step.  layers: list of LayerWeights; caches: list of KvCache (one per
    layer); pos is advanced in place."""
    B = int(ids.shape[0])
    arr = (LayerWeightsC * len(layers))(*[l.c for l in layers])
    carr = _cache_array(caches)
    mw = ModelWeightsC(embed.data_ptr(), arr,
                       final_gamma.data_ptr() if final_gamma is not None else None,
                       lm_head.data_ptr() if lm_head is not None else None)
    check(lib().qtale_model_decode_step(
        C.byref(cfg), C.byref(mw), _ptr(ids), B, _ptr(pos), _ptr(valid), C.cast(carr, C.c_void_p),
        _ptr(hidden_out), _ptr(logits_out), _ptr(next_ids_out), _ptr(per_layer_n_exec),
        _ptr(layer_scores_out), _ptr(ws), ws.numel() * ws.element_size(), _stream()),
        "qtale_model_decode_step")
    return hidden_out


# ---------------------------------------------------------------------------------
# host <-> device helpers for bf16 held as float32 numpy arrays
# ---------------------------------------------------------------------------------

def to_device_bf16(a: np.ndarray, device="cuda") -> torch.Tensor:
    """float32 numpy array of bf16-representable values -> bf16 device tensor (exact)."""
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device).to(torch.bfloat16)


def to_device_act(a: np.ndarray, act_dtype, device="cuda") -> torch.Tensor:
    """float32 numpy array -> device tensor in the given 16-bit activation format (rounds)."""
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device).to(
        act_torch_dtype(act_dtype))


def to_host_f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy()
