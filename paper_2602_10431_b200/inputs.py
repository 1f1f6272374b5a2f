"""Seeded synthetic inputs for the QTALE layer path.

Everything here is input preparation only: a counter-based random stream,
value distributions, bf16 rounding of generated activations, and the recipe
that turns Gaussian fp32 weights into b-bit group-quantised codes with fp16
scale / zero-point.  None of the layer's arithmetic (router, selection,
dequantisation, attention, MLP, scatter) lives in this module; both the CPU
oracle's tests and the CUDA path's tests are fed from it.

Random stream: splitmix64 applied to a counter.  Element i of the tensor with
stream id `sid` under seed `seed` uses the 64-bit counter
(seed * 0x9E3779B97F4A7C15 + sid * 0xD1B54A32D192ED03 + i) pushed through the
splitmix64 finaliser, so any element can be regenerated without the others.
"""
from __future__ import annotations

import numpy as np

_GOLD = np.uint64(0x9E3779B97F4A7C15)
_SID = np.uint64(0xD1B54A32D192ED03)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def splitmix64(counter: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser of uint64 counters (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        z = counter.astype(np.uint64) + _GOLD
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


def _base(seed: int, sid: int) -> np.uint64:
    with np.errstate(over="ignore"):
        return np.uint64(seed) * _GOLD + np.uint64(sid) * _SID


def raw_u64(seed: int, sid: int, start: int, count: int) -> np.ndarray:
    with np.errstate(over="ignore"):
        ctr = _base(seed, sid) + np.arange(start, start + count, dtype=np.uint64)
    return splitmix64(ctr)


def uniform(seed: int, sid: int, count: int, start: int = 0) -> np.ndarray:
    """float64 uniforms in the open interval (0, 1)."""
    u = raw_u64(seed, sid, start, count)
    return ((u >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, sid: int, count: int, start: int = 0) -> np.ndarray:
    """float64 standard normals by Box-Muller; element i uses counters 2i, 2i+1."""
    u = uniform(seed, sid, 2 * count, 2 * start)
    u1, u2 = u[0::2], u[1::2]
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def beta22(seed: int, sid: int, count: int, start: int = 0) -> np.ndarray:
    """Beta(2,2) variates as the median of three independent uniforms."""
    u = uniform(seed, sid, 3 * count, 3 * start).reshape(count, 3)
    return np.median(u, axis=1)


def integers(seed: int, sid: int, count: int, high: int, start: int = 0) -> np.ndarray:
    """int32 values uniform over [0, high)."""
    u = uniform(seed, sid, count, start)
    return np.minimum((u * high).astype(np.int64), high - 1).astype(np.int32)


# ---------------------------------------------------------------------------
# bf16 helpers (storage format of the activations handed to both sides)
# ---------------------------------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even); returns uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (b >> np.uint32(16)) & np.uint32(1)
    r = b + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_bf16(x: np.ndarray) -> np.ndarray:
    """float32 values rounded to the nearest bf16, returned as float32."""
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


def activations(seed: int, sid: int, rows: int, cols: int, std: float = 1.0) -> np.ndarray:
    """[rows, cols] float32 holding bf16-representable N(0, std^2) values."""
    out = np.empty((rows, cols), dtype=np.float32)
    step = max(1, (1 << 22) // max(cols, 1))
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        z = normal(seed, sid, (r1 - r0) * cols, r0 * cols) * std
        out[r0:r1] = round_bf16(z.astype(np.float32)).reshape(r1 - r0, cols)
    return out


def gaussian_f32(seed: int, sid: int, rows: int, cols: int, std: float) -> np.ndarray:
    """[rows, cols] float32 N(0, std^2) (not rounded to bf16)."""
    out = np.empty((rows, cols), dtype=np.float32)
    step = max(1, (1 << 22) // max(cols, 1))
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        z = normal(seed, sid, (r1 - r0) * cols, r0 * cols) * std
        out[r0:r1] = z.astype(np.float32).reshape(r1 - r0, cols)
    return out


# ---------------------------------------------------------------------------
# Weight recipe: asymmetric b-bit min/max group quantisation along K
# ---------------------------------------------------------------------------

def quantize_groups(w: np.ndarray, bits: int, group: int):
    """Recipe that produces synthetic quantised weights from fp32 weights.

    Per row n and per group g of `group` consecutive input features:
      lo = min(min w, 0), hi = max(max w, 0)
      s  = fp16((hi - lo) / (2^b - 1)), replaced by 1 when it rounds to 0
      z  = clamp(rint(-lo / s), 0, 2^b - 1)          (stored as fp16, integer valued)
      q  = clamp(rint(w / s) + z, 0, 2^b - 1)        (rint = round half to even)
    The last group may be short.  Returns (codes uint8 [N,K], scales fp16 [N,ng],
    zeros fp16 [N,ng]).
    """
    assert bits in (2, 3, 4)
    w = np.ascontiguousarray(w, dtype=np.float32)
    N, K = w.shape
    ng = (K + group - 1) // group
    qmax = float((1 << bits) - 1)
    codes = np.empty((N, K), dtype=np.uint8)
    scales = np.empty((N, ng), dtype=np.float16)
    zeros = np.empty((N, ng), dtype=np.float16)
    for g in range(ng):
        blk = w[:, g * group:min(K, (g + 1) * group)]
        lo = np.minimum(blk.min(axis=1), np.float32(0))
        hi = np.maximum(blk.max(axis=1), np.float32(0))
        s16 = ((hi - lo) / np.float32(qmax)).astype(np.float32).astype(np.float16)
        s16 = np.where(s16 == 0, np.float16(1), s16)
        s = s16.astype(np.float32)
        z = np.clip(np.rint(-lo / s), 0, qmax).astype(np.float32)
        q = np.clip(np.rint(blk / s[:, None]) + z[:, None], 0, qmax)
        codes[:, g * group:min(K, (g + 1) * group)] = q.astype(np.uint8)
        scales[:, g] = s16
        zeros[:, g] = z.astype(np.float16)
    return codes, scales, zeros


def pack_codes(codes: np.ndarray, bits: int) -> np.ndarray:
    """Interface layout of the codes: row-major [N, row_bytes] uint8.

    4-bit: two codes per byte, even k in the low nibble.  3-bit: little-endian
    bit stream along K (code k occupies bits 3k .. 3k+2 of the row), 8 codes
    per 3 bytes.  2-bit: four codes per byte, code k in bits 2 (k % 4) .. + 1 of
    byte k / 4.  Rows start on a byte boundary.
    """
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    N, K = codes.shape
    if bits == 4:
        Kp = (K + 1) // 2 * 2
        c = np.zeros((N, Kp), dtype=np.uint8)
        c[:, :K] = codes
        return (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)
    if bits == 3:
        Kp = (K + 7) // 8 * 8
        c = np.zeros((N, Kp), dtype=np.uint32)
        c[:, :K] = codes
        c = c.reshape(N, Kp // 8, 8)
        word = np.zeros((N, Kp // 8), dtype=np.uint32)
        for j in range(8):
            word |= c[:, :, j] << np.uint32(3 * j)
        out = np.empty((N, Kp // 8, 3), dtype=np.uint8)
        out[:, :, 0] = word & 0xFF
        out[:, :, 1] = (word >> 8) & 0xFF
        out[:, :, 2] = (word >> 16) & 0xFF
        row_bytes = (3 * K + 7) // 8
        return np.ascontiguousarray(out.reshape(N, -1)[:, :row_bytes])
    if bits == 2:
        Kp = (K + 3) // 4 * 4
        c = np.zeros((N, Kp), dtype=np.uint8)
        c[:, :K] = codes
        return (c[:, 0::4] | (c[:, 1::4] << 2) | (c[:, 2::4] << 4) | (c[:, 3::4] << 6)).astype(np.uint8)
    raise ValueError("bits must be 2, 3 or 4")


def quantized_weight(seed: int, sid: int, N: int, K: int, bits: int, group: int, std: float = 0.02):
    """Synthetic quantised linear weight W[N, K] ~ N(0, std^2), quantised by the recipe.

    Returns dict(packed uint8 [N,row_bytes], scales fp16 [N,ng], zeros fp16 [N,ng],
    N, K, bits, group).  The fp32 weights are generated in row blocks so peak
    host memory stays bounded.
    """
    ng = (K + group - 1) // group
    row_bytes = {4: (K + 1) // 2, 3: (3 * K + 7) // 8, 2: (K + 3) // 4}[bits]
    packed = np.empty((N, row_bytes), dtype=np.uint8)
    scales = np.empty((N, ng), dtype=np.float16)
    zeros = np.empty((N, ng), dtype=np.float16)
    step = max(1, (1 << 22) // K)
    for r0 in range(0, N, step):
        r1 = min(N, r0 + step)
        w = (normal(seed, sid, (r1 - r0) * K, r0 * K) * std).astype(np.float32).reshape(r1 - r0, K)
        c, s, z = quantize_groups(w, bits, group)
        packed[r0:r1] = pack_codes(c, bits)
        scales[r0:r1] = s
        zeros[r0:r1] = z
    return dict(packed=packed, scales=scales, zeros=zeros, N=N, K=K, bits=bits, group=group)


# ---------------------------------------------------------------------------
# Layer / model level recipes
# ---------------------------------------------------------------------------

class LayerShape:
    """Shapes of one Llama-style decoder layer."""

    def __init__(self, d, n_heads, n_kv_heads, head_dim, ffn, bits=4, group=128,
                 rms_eps=1e-5, rope_theta=10000.0):
        self.d, self.n_heads, self.n_kv_heads = d, n_heads, n_kv_heads
        self.head_dim, self.ffn = head_dim, ffn
        self.bits, self.group = bits, group
        self.rms_eps, self.rope_theta = rms_eps, rope_theta

    @property
    def q_dim(self):
        return self.n_heads * self.head_dim

    @property
    def kv_dim(self):
        return self.n_kv_heads * self.head_dim

    def linear_params(self):
        d, F = self.d, self.ffn
        return d * self.q_dim + 2 * d * self.kv_dim + self.q_dim * d + 3 * d * F


CONFIG_SHAPES = {
    # single small layer: hidden 256, 4 heads of 64, FFN 688, int4 group 64
    "c1": dict(shape=LayerShape(256, 4, 4, 64, 688, 4, 64), B=2, S=128),
    # 7B-shaped layer, int4 group 128, batch 4 x 2048 prefill
    "c2": dict(shape=LayerShape(4096, 32, 32, 128, 11008, 4, 128), B=4, S=2048),
    # 7B-shaped layer for decode, int3 group 128 / int4 group 64
    "c3_int3": dict(shape=LayerShape(4096, 32, 32, 128, 11008, 3, 128), B=64, S=1),
    "c3_int4g64": dict(shape=LayerShape(4096, 32, 32, 128, 11008, 4, 64), B=64, S=1),
    # 8B-shaped (GQA) model layer
    "c4": dict(shape=LayerShape(4096, 32, 8, 128, 14336, 4, 128, 1e-5, 500000.0), B=8, S=1024),
    # 13B-shaped layer
    "c5": dict(shape=LayerShape(5120, 40, 40, 128, 13824, 4, 128), B=16, S=4096),
}


def layer_weights(seed: int, layer: int, sh: LayerShape, bits: int | None = None):
    """All tensors of one layer: four quantised linears, two norm gains, router.

    `bits` overrides the shape's bit-width for this layer (layer-interleaved
    mixed precision of the mixed 2&4-bit appendix: even layers 4-bit, odd 2-bit).

    Stream ids: layer*16 + {0:qkv, 1:o, 2:gate_up, 3:down, 4:router}.  The QKV
    matrix stacks Wq, Wk, Wv along the output dimension; gate_up stacks the
    SwiGLU gate rows then the up rows.  Norm gains are 1.  The router is a
    linear map hidden -> 1 (the difference of the two class logits) with
    N(0, 0.02^2) weights rounded to bf16 and a bias the caller sets.
    """
    b = layer * 16
    d, F = sh.d, sh.ffn
    bits = sh.bits if bits is None else bits
    w = {
        "qkv": quantized_weight(seed, b + 0, sh.q_dim + 2 * sh.kv_dim, d, bits, sh.group),
        "o": quantized_weight(seed, b + 1, d, sh.q_dim, bits, sh.group),
        "gate_up": quantized_weight(seed, b + 2, 2 * F, d, bits, sh.group),
        "down": quantized_weight(seed, b + 3, d, F, bits, sh.group),
        "gamma1": np.ones(d, dtype=np.float32),
        "gamma2": np.ones(d, dtype=np.float32),
        "router_w": round_bf16((normal(seed, b + 4, d) * 0.02).astype(np.float32)),
        "router_b": 0.0,
        "head_dim": sh.head_dim,
    }
    return w


def hidden_states(seed: int, T: int, d: int, sid: int = 1000) -> np.ndarray:
    return activations(seed, sid, T, d, 1.0)


def cu_seqlens_uniform(B: int, S: int) -> np.ndarray:
    return (np.arange(B + 1, dtype=np.int64) * S).astype(np.int32)


def ragged_seqlens(seed: int, B: int, S_max: int, sid: int = 1001) -> np.ndarray:
    """cu_seqlens for B sequences with lengths uniform in [S_max/4, S_max]."""
    lens = S_max // 4 + integers(seed, sid, B, S_max - S_max // 4 + 1)
    return np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
