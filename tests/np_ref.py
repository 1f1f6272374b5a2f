"""Independent numpy fp64 restatement of a dense Llama-style decoder layer.

Used only to pin the C oracle: different language, vectorised einsum instead
of loop nests, no index indirection.  Operates on ONE sequence of tokens with
explicit positions.
"""
import numpy as np


def rmsnorm(x, gamma, eps):
    x = x.astype(np.float64)
    return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps) * gamma.astype(np.float64)


def rope(v, pos, base):
    # v: [S, H, hd]
    S, H, hd = v.shape
    half = hd // 2
    inv = base ** (-2.0 * np.arange(half) / hd)
    ang = pos.astype(np.float64)[:, None] * inv[None, :]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = v[..., :half], v[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def dense_layer_one_sequence(x, pos, W, sh, k_prev=None, v_prev=None):
    """x: [S, d]; returns x + f(x) in fp64 (and this call's k, v).

    k_prev / v_prev: [P, Hkv, hd] keys / values already cached (all earlier)."""
    d, H, Hkv, hd, F = sh.d, sh.n_heads, sh.n_kv_heads, sh.head_dim, sh.ffn
    S = x.shape[0]
    x = x.astype(np.float64)
    h = rmsnorm(x, W["gamma1"], sh.rms_eps)
    qkv = h @ W["qkv"].astype(np.float64).T
    q = qkv[:, :H * hd].reshape(S, H, hd)
    k = qkv[:, H * hd:H * hd + Hkv * hd].reshape(S, Hkv, hd)
    v = qkv[:, H * hd + Hkv * hd:].reshape(S, Hkv, hd)
    q, k = rope(q, pos, sh.rope_theta), rope(k, pos, sh.rope_theta)
    kk, vv = k, v
    P = 0
    if k_prev is not None and k_prev.shape[0] > 0:
        P = k_prev.shape[0]
        kk = np.concatenate([k_prev.astype(np.float64), k], axis=0)
        vv = np.concatenate([v_prev.astype(np.float64), v], axis=0)
    rep = H // Hkv
    kk_r = np.repeat(kk, rep, axis=1)
    vv_r = np.repeat(vv, rep, axis=1)
    s = np.einsum("ihe,jhe->hij", q, kk_r) / np.sqrt(hd)
    causal = np.concatenate([np.ones((S, P), bool), np.tril(np.ones((S, S), bool))], axis=1)
    s = np.where(causal[None], s, -np.inf)
    s = s - s.max(axis=-1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=-1, keepdims=True)
    ao = np.einsum("hij,jhe->ihe", p, vv_r).reshape(S, H * hd)
    a = ao @ W["o"].astype(np.float64).T
    u = x + a
    h2 = rmsnorm(u, W["gamma2"], sh.rms_eps)
    gu = h2 @ W["gate_up"].astype(np.float64).T
    g, up = gu[:, :F], gu[:, F:]
    act = g / (1.0 + np.exp(-g)) * up
    m = act @ W["down"].astype(np.float64).T
    return x + a + m, k, v
