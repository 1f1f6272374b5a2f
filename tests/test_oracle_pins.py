"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA path.  Each checks the oracle against a
closed form, a value the paper prints, an invariant the paper states, a
library routine on a special case, or brute force on tiny inputs.
"""
import os

import numpy as np
import pytest

import oracle
from paper_2602_10431_b200 import accounting, inputs
from tests import np_ref

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    for line in open(os.path.join(GOLD, name)):
        line = line.split("#")[0].strip()
        if line:
            out.append(line.split())
    return out


# ---------------------------------------------------------------- router (Eq. 2, Eq. 9)

def test_two_class_softmax_closed_form_golden():
    rows = _rows("router_two_class.txt")
    g0 = np.array([float(r[0]) for r in rows])
    g1 = np.array([float(r[1]) for r in rows])
    want = np.array([float(r[2]) for r in rows])
    got = oracle.softmax2_p0(g0, g1)
    assert np.allclose(got, want, atol=1e-7)
    # linear router: w.x + b is the logit difference
    d = 8
    for a, b, p in zip(g0, g1, want):
        x = np.zeros((1, d), np.float32)
        x[0, 3] = 1.0
        w = np.zeros(d, np.float32)
        w[3] = np.float32(a - b)
        got = oracle.router_scores(x, w, 0.0)
        assert abs(got[0] - p) < 1e-6


def test_router_matches_numpy_dot_and_logistic():
    x = inputs.hidden_states(0, 37, 256)
    w = inputs.round_bf16((inputs.normal(0, 5, 256) * 0.02).astype(np.float32))
    p, z = oracle.router_scores(x, w, 0.125, return_logits=True)
    z_np = x.astype(np.float64) @ w.astype(np.float64) + 0.125
    assert np.allclose(z, z_np, rtol=0, atol=1e-12)
    assert np.array_equal(p, (1.0 / (1.0 + np.exp(-z_np))).astype(np.float32))
    # planted mistake check: a dropped bias or flipped sign would move p
    assert not np.allclose(p, 1.0 / (1.0 + np.exp(z_np)))


def test_theta_half_is_argmax_rule():
    """theta = 0.5 reproduces the argmax decision of Eq. 2 (ties execute)."""
    g0 = inputs.normal(1, 1, 500)
    g1 = inputs.normal(1, 2, 500)
    g1[:10] = g0[:10]  # exact ties
    p = oracle.softmax2_p0(g0, g1)
    m = oracle.select_threshold(p, 0.5)
    assert np.array_equal(m.astype(bool), g0 >= g1)


def test_threshold_monotone_and_extremes_and_padding():
    p = inputs.uniform(2, 1, 1000).astype(np.float32)
    valid = (inputs.uniform(2, 2, 1000) > 0.2).astype(np.uint8)
    prev = None
    for theta in [0.9, 0.5, 0.3, 0.1, 0.03]:
        m = oracle.select_threshold(p, theta, valid).astype(bool)
        assert np.array_equal(m, (p >= np.float32(theta)) & valid.astype(bool))
        if prev is not None:
            assert np.all(m[prev])  # lowering theta only adds tokens
            assert m.sum() >= prev.sum()
        prev = m
        assert not m[valid == 0].any()  # padding never executes
    assert oracle.select_threshold(p, 0.0).all()
    assert not oracle.select_threshold(p, 1.5).any()
    # tie at the threshold executes (>=)
    assert oracle.select_threshold(np.array([0.25], np.float32), 0.25)[0] == 1


def test_topk_brute_force_and_ties():
    for seed, T, k in [(0, 1, 1), (1, 17, 5), (2, 64, 64), (3, 100, 0), (4, 257, 101)]:
        p = inputs.uniform(seed, 3, T).astype(np.float32)
        if T > 8:
            p[T // 2:T // 2 + 6] = p[T // 3]  # planted equal scores
        valid = np.ones(T, np.uint8)
        if T > 20:
            valid[::7] = 0
        k = min(k, int(valid.sum()))
        m = oracle.select_topk(p, k, valid)
        order = sorted([t for t in range(T) if valid[t]], key=lambda t: (-float(p[t]), t))
        want = np.zeros(T, np.uint8)
        want[order[:k]] = 1
        assert np.array_equal(m, want)
        assert m.sum() == k


def test_topk_equals_threshold_at_kth_score_without_ties():
    p = inputs.uniform(5, 3, 300).astype(np.float32)
    assert len(np.unique(p)) == 300
    k = 123
    kth = np.sort(p)[::-1][k - 1]
    assert np.array_equal(oracle.select_topk(p, k), oracle.select_threshold(p, float(kth)))


def test_topk_count_matches_ratio():
    assert oracle.topk_count(0.5, 256) == 128
    assert oracle.topk_count(0.9, 8192) == 7373
    assert oracle.topk_count(0.75, 8192) == 6144
    assert oracle.topk_count(1.0, 77) == 77
    assert oracle.topk_count(0.0, 77) == 0
    assert oracle.topk_count(0.5, 3) == 2  # floor(1.5 + 0.5)


def test_compaction_brute_force():
    T = 103
    mask = (inputs.uniform(6, 1, T) > 0.4).astype(np.uint8)
    cu = np.array([0, 10, 10, 57, 103], np.int32)  # includes an empty sequence
    idx, n, cu_exec, pos = oracle.compact_indices(mask, cu)
    want = np.nonzero(mask)[0]
    assert n == len(want) == mask.sum()
    assert np.array_equal(idx, want)
    assert np.all(np.diff(idx) > 0)
    for b in range(4):
        assert cu_exec[b + 1] - cu_exec[b] == mask[cu[b]:cu[b + 1]].sum()
    seq = np.searchsorted(cu, idx, side="right") - 1
    assert np.array_equal(pos, idx - cu[seq])
    # empty and full
    idx, n, cu_exec, _ = oracle.compact_indices(np.zeros(T, np.uint8), cu)
    assert n == 0 and not cu_exec.any()
    idx, n, cu_exec, _ = oracle.compact_indices(np.ones(T, np.uint8), cu)
    assert n == T and np.array_equal(cu_exec, cu)


# ---------------------------------------------------------------- quantised weights (Sec. 4.1)

def test_half_conversion_all_bit_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float32)
    L = oracle.lib()
    for b in range(0, 65536, 7):
        v = L.orc_half_to_float(int(b))
        if np.isnan(ref[b]):
            assert np.isnan(v)
        else:
            assert v == ref[b]
    vals = np.concatenate([(inputs.normal(7, 1, 4000) * 0.01).astype(np.float32),
                           np.array([0, 1, -1, 65504, 65519.9, 65520, 1e-8, 5.96e-8, 3e-8,
                                     6.1e-5, 6.0e-5, 0.333333, 1e-3], np.float32)])
    for v in vals:
        with np.errstate(over="ignore"):
            assert L.orc_float_to_half(float(v)) == int(np.float32(v).astype(np.float16).view(np.uint16))


@pytest.mark.parametrize("bits,group,K", [(4, 128, 512), (4, 64, 688), (3, 128, 384), (3, 64, 200),
                                          (2, 128, 384), (2, 64, 203)])
def test_quantize_roundtrip_and_error_bound(bits, group, K):
    N = 24
    w = (inputs.normal(8, bits * 1000 + K, N * K) * 0.02).astype(np.float32).reshape(N, K)
    codes, s, z = oracle.quantize(w, bits, group)
    assert codes.max() <= (1 << bits) - 1
    packed = oracle.pack_codes(codes, bits)
    assert packed.shape[1] == (K * bits + 7) // 8
    assert np.array_equal(oracle.unpack_codes(packed, K, bits), codes)
    w_hat = oracle.dequantize(packed, s, z, K, bits, group)
    # definition written out with numpy
    sg = np.repeat(s.astype(np.float32), group, axis=1)[:, :K]
    zg = np.repeat(z.astype(np.float32), group, axis=1)[:, :K]
    assert np.array_equal(w_hat, (codes.astype(np.float32) - zg) * sg)
    # round trip of the integer codes with fixed (scale, zero)
    assert np.array_equal(oracle.requantize_fixed(w_hat, s, z, bits, group), codes)
    # error bound: in-range weights are within half a step (+ fp16 rounding of the step)
    assert np.all(np.abs(w - w_hat) <= sg * 0.5 + np.abs(w) * 2e-3 + 1e-7)
    # zero is exactly representable: zero-point is an integer code
    assert np.array_equal(z.astype(np.float32), np.rint(z.astype(np.float32)))
    zero_w = np.zeros((2, K), np.float32)
    c0, s0, z0 = oracle.quantize(zero_w, bits, group)
    assert np.all(oracle.dequantize(oracle.pack_codes(c0, bits), s0, z0, K, bits, group) == 0.0)


@pytest.mark.parametrize("bits,group,K", [(4, 128, 256), (4, 64, 688), (3, 128, 256), (3, 64, 88),
                                          (2, 128, 256), (2, 64, 90)])
def test_input_recipe_matches_oracle_quantiser(bits, group, K):
    N = 16
    w = (inputs.normal(9, K + bits, N * K) * 0.02).astype(np.float32).reshape(N, K)
    c1, s1, z1 = inputs.quantize_groups(w, bits, group)
    c2, s2, z2 = oracle.quantize(w, bits, group)
    assert np.array_equal(c1, c2)
    assert np.array_equal(s1.view(np.uint16), s2.view(np.uint16))
    assert np.array_equal(z1.view(np.uint16), z2.view(np.uint16))
    assert np.array_equal(inputs.pack_codes(c1, bits), oracle.pack_codes(c2, bits))


def test_packed_layout_hand_example():
    codes = np.array([[1, 2, 3, 4, 5, 6, 7, 0, 15 & 7]], np.uint8)
    p4 = oracle.pack_codes(codes, 4)
    assert list(p4[0]) == [0x21, 0x43, 0x65, 0x07, 0x07]
    p3 = oracle.pack_codes(codes, 3)
    word = sum(int(c) << (3 * i) for i, c in enumerate(codes[0]))
    assert list(p3[0]) == [(word >> (8 * i)) & 0xFF for i in range(4)]
    # 2-bit (mixed 2&4-bit appendix): four codes per byte, first code in the low bits
    c2 = np.array([[0, 1, 2, 3, 3, 0, 1, 0, 2]], np.uint8)
    p2 = oracle.pack_codes(c2, 2)
    assert list(p2[0]) == [0b11100100, 0b00010011, 0b00000010]
    assert np.array_equal(oracle.unpack_codes(p2, 9, 2), c2)


def test_model_size_and_bytes_per_weight():
    """Packed bytes per weight = b/8 + 4/G; model sizes of the efficiency table
    (12.6 / 3.6 / 2.8 GB for LLaMA2-7B at 16 / 4 / 3 bit) to first order."""
    P = accounting.linear_params(4096, 32, 32, 128, 11008) * 32
    other = 2 * 32000 * 4096 * 2  # embedding + LM head in 16 bit
    gib = 1024.0 ** 3
    assert abs((P * 2 + other) / gib - 12.6) < 0.15
    assert abs((P * accounting.packed_bytes_per_weight(4, 128) + other) / gib - 3.6) < 0.15
    assert abs((P * accounting.packed_bytes_per_weight(3, 128) + other) / gib - 2.8) < 0.2
    # oracle layout agrees with the byte model
    assert oracle.row_bytes(4096, 4) == 2048 and oracle.row_bytes(4096, 3) == 1536


def test_flops_model_matches_paper_table():
    full = accounting.linear_flops_per_token(4096, 32, 32, 128, 11008, n_layers=32)
    assert abs(full / 1e9 - 13.0) < 0.06
    for bits, method, ds, ratio, gflops in _rows("flops_vs_ratio_llama2_7b.txt"):
        got = accounting.linear_flops_per_token(4096, 32, 32, 128, 11008, 32, float(ratio)) / 1e9
        assert abs(got - float(gflops)) < 0.012, (bits, method, ds)
    full8 = accounting.linear_flops_per_token(4096, 32, 8, 128, 14336, n_layers=32)
    # LLaMA3.1-8B: 15.6 GFLOPs printed (includes the untied 128k-vocabulary head)
    assert abs((full8 + 2 * 4096 * 128256) / 1e9 - 15.6) < 0.6


# ---------------------------------------------------------------- dense blocks

def test_rmsnorm_linear_swiglu_against_numpy():
    x = inputs.hidden_states(10, 19, 96)
    g = (1.0 + 0.1 * inputs.normal(10, 2, 96)).astype(np.float32)
    assert np.allclose(oracle.rmsnorm(x, g, 1e-5), np_ref.rmsnorm(x, g, 1e-5), atol=1e-6)
    w = (inputs.normal(10, 3, 40 * 96) * 0.05).astype(np.float32).reshape(40, 96)
    assert np.allclose(oracle.linear(x, w), x.astype(np.float64) @ w.astype(np.float64).T, atol=1e-5)
    # a transposed operand would fail here: non-square shapes
    a, b = x[:, :40], x[:, 40:80]
    ref = a.astype(np.float64) / (1 + np.exp(-a.astype(np.float64))) * b
    assert np.allclose(oracle.swiglu(a, b), ref, atol=1e-6)
    assert oracle.swiglu(np.array([[0.0]]), np.array([[3.0]]))[0, 0] == 0.0


def test_rope_closed_forms():
    hd, H = 8, 2
    v = inputs.hidden_states(11, 6, H * hd)
    pos = np.array([0, 1, 2, 5, 9, 100], np.int32)
    r = oracle.rope(v, H, hd, pos, 10000.0)
    assert np.array_equal(r[0], v[0])  # position 0 is the identity
    assert np.allclose((r ** 2).sum(-1), (v.astype(np.float64) ** 2).sum(-1), rtol=1e-6)
    assert np.allclose(r.reshape(6, H, hd), np_ref.rope(v.reshape(6, H, hd), pos, 10000.0), atol=1e-6)
    # hd = 2: a plane rotation by the position (base irrelevant: exponent 0)
    v2 = np.array([[1.0, 0.0]], np.float32)
    r2 = oracle.rope(v2, 1, 2, np.array([1], np.int32), 10000.0)
    assert np.allclose(r2, [[np.cos(1.0), np.sin(1.0)]], atol=1e-7)
    # relative-position property: <R_m q, R_n k> depends on m - n only
    q = inputs.hidden_states(11, 1, hd, sid=7)
    k = inputs.hidden_states(11, 1, hd, sid=8)
    def dot(m, n):
        return float(oracle.rope(q, 1, hd, np.array([m], np.int32), 10000.0)[0].astype(np.float64)
                     @ oracle.rope(k, 1, hd, np.array([n], np.int32), 10000.0)[0].astype(np.float64))
    assert abs(dot(7, 3) - dot(14, 10)) < 1e-5


def test_attention_invariants():
    H, Hkv, hd, Te = 4, 2, 8, 11
    q = inputs.hidden_states(12, Te, H * hd, sid=1)
    k = inputs.hidden_states(12, Te, Hkv * hd, sid=2)
    v = inputs.hidden_states(12, Te, Hkv * hd, sid=3)
    seq_of = np.array([0] * 5 + [1] * 6, np.int32)
    pos = np.array([0, 2, 3, 7, 9, 1, 2, 3, 4, 8, 9], np.int32)
    out = oracle.attention(q, k, v, H, Hkv, hd, seq_of, pos)
    # first executed token of each sequence sees only itself
    rep = H // Hkv
    for first in (0, 5):
        want = np.repeat(v[first].reshape(Hkv, hd), rep, axis=0).reshape(-1)
        assert np.allclose(out[first], want, atol=1e-7)
    # softmax weights sum to one: constant values come back unchanged
    ones = np.ones_like(v)
    assert np.allclose(oracle.attention(q, k, ones, H, Hkv, hd, seq_of, pos), 1.0, atol=1e-6)
    # brute force, one query
    i, h = 8, 3
    js = [j for j in range(Te) if seq_of[j] == seq_of[i] and pos[j] <= pos[i]]
    s = np.array([q[i, h * hd:(h + 1) * hd].astype(np.float64)
                  @ k[j, (h // rep) * hd:(h // rep + 1) * hd].astype(np.float64) for j in js]) / np.sqrt(hd)
    pr = np.exp(s - s.max())
    pr /= pr.sum()
    want = sum(pj * v[j, (h // rep) * hd:(h // rep + 1) * hd].astype(np.float64) for pj, j in zip(pr, js))
    assert np.allclose(out[i, h * hd:(h + 1) * hd], want, atol=1e-6)


# ---------------------------------------------------------------- the layer (Eq. 1, Eq. 3)

def _small_layer(seed=0, bits=4, group=64, gqa=False):
    sh = inputs.LayerShape(64, 4, 2 if gqa else 4, 16, 176, bits, group)
    w = inputs.layer_weights(seed, 0, sh)
    w["gamma1"] = (1.0 + 0.1 * inputs.normal(seed, 90, sh.d)).astype(np.float32)
    w["gamma2"] = (1.0 + 0.1 * inputs.normal(seed, 91, sh.d)).astype(np.float32)
    for name in ("qkv", "o", "gate_up", "down"):  # larger weights so that f_l matters
        w[name] = inputs.quantized_weight(seed, 50 + len(name), w[name]["N"], w[name]["K"], bits, group, std=0.08)
    return sh, w, oracle.DenseLayer(sh, w)


def _np_weights(layer):
    return dict(qkv=layer.w_qkv, o=layer.w_o, gate_up=layer.w_gate_up, down=layer.w_down,
                gamma1=layer.gamma1, gamma2=layer.gamma2)


@pytest.mark.parametrize("gqa", [False, True])
def test_ratio_one_equals_dense_layer(gqa):
    sh, w, layer = _small_layer(gqa=gqa)
    cu = np.array([0, 13, 40], np.int32)
    x = inputs.hidden_states(0, 40, sh.d)
    out, n = oracle.layer_forward(layer, x, cu, np.ones(40, np.uint8))
    assert n == 40
    W = _np_weights(layer)
    for b in range(2):
        xs = x[cu[b]:cu[b + 1]]
        ref, _, _ = np_ref.dense_layer_one_sequence(xs, np.arange(len(xs)), W, sh)
        assert np.allclose(out[cu[b]:cu[b + 1]], ref, atol=2e-5, rtol=1e-5)
    assert np.abs(out - x).max() > 0.05  # f_l is not negligible in this fixture


def test_ratio_zero_is_identity_and_skipped_rows_untouched():
    sh, w, layer = _small_layer()
    cu = np.array([0, 20, 33], np.int32)
    x = inputs.hidden_states(1, 33, sh.d)
    out, n = oracle.layer_forward(layer, x, cu, np.zeros(33, np.uint8))
    assert n == 0 and np.array_equal(out, x)
    mask = (inputs.uniform(1, 4, 33) > 0.5).astype(np.uint8)
    out, n = oracle.layer_forward(layer, x, cu, mask)
    assert n == mask.sum()
    assert np.array_equal(out[mask == 0], x[mask == 0])
    assert np.all(np.abs(out[mask == 1] - x[mask == 1]).max(axis=1) > 0)


def test_masked_layer_equals_dense_layer_on_executed_subsequence():
    """Executed tokens attend to executed tokens of their own sequence, with RoPE
    at their original positions: same as the dense layer on the subsequence."""
    sh, w, layer = _small_layer(seed=3, gqa=True)
    cu = np.array([0, 17, 17, 48], np.int32)
    x = inputs.hidden_states(3, 48, sh.d)
    mask = (inputs.uniform(3, 4, 48) > 0.45).astype(np.uint8)
    out, _ = oracle.layer_forward(layer, x, cu, mask)
    W = _np_weights(layer)
    for b in range(3):
        t = np.arange(cu[b], cu[b + 1])
        sel = t[mask[t] == 1]
        if len(sel) == 0:
            continue
        ref, _, _ = np_ref.dense_layer_one_sequence(x[sel], sel - cu[b], W, sh)
        assert np.allclose(out[sel], ref, atol=2e-5, rtol=1e-5)


def test_sequences_are_independent():
    sh, w, layer = _small_layer(seed=4)
    x = inputs.hidden_states(4, 30, sh.d)
    mask = (inputs.uniform(4, 4, 30) > 0.3).astype(np.uint8)
    cu = np.array([0, 12, 30], np.int32)
    both, _ = oracle.layer_forward(layer, x, cu, mask)
    second, _ = oracle.layer_forward(layer, x[12:], np.array([0, 18], np.int32), mask[12:])
    assert np.array_equal(both[12:], second)


def test_decode_with_cache_equals_longer_prefill():
    """Prefill S tokens into the cache, decode one more token: the new token's
    output equals the last row of an (S+1)-token prefill with the same masks;
    bypassed tokens leave no cache entry."""
    sh, w, layer = _small_layer(seed=5, gqa=True)
    S, cap = 21, 32
    x = inputs.hidden_states(5, 2 * (S + 1), sh.d)
    mask = (inputs.uniform(5, 4, 2 * (S + 1)) > 0.4).astype(np.uint8)
    mask[S] = 1            # sequence 0's new token executes
    mask[2 * S + 1] = 0    # sequence 1's new token is bypassed
    cu_full = np.array([0, S + 1, 2 * S + 2], np.int32)
    full, _ = oracle.layer_forward(layer, x, cu_full, mask)
    kvd = sh.n_kv_heads * sh.head_dim
    ck = np.zeros((2, cap, kvd), np.float32)
    cv = np.zeros((2, cap, kvd), np.float32)
    kl = np.zeros(2, np.int32)
    pre_rows = np.concatenate([np.arange(0, S), np.arange(S + 1, 2 * S + 1)])
    _, _ = oracle.layer_forward(layer, x[pre_rows], np.array([0, S, 2 * S], np.int32), mask[pre_rows],
                                cache_k=ck, cache_v=cv, kv_len=kl)
    assert kl[0] == mask[0:S].sum() and kl[1] == mask[S + 1:2 * S + 1].sum()
    new_rows = np.array([S, 2 * S + 1])
    dec, n = oracle.layer_forward(layer, x[new_rows], np.array([0, 1, 2], np.int32), mask[new_rows],
                                  pos0=np.array([S, S], np.int32), cache_k=ck, cache_v=cv, kv_len=kl)
    assert n == 1
    assert np.allclose(dec[0], full[S], atol=1e-5)
    assert np.array_equal(dec[1], x[2 * S + 1])
    assert kl[0] == mask[0:S + 1].sum() and kl[1] == mask[S + 1:2 * S + 2].sum()


def test_gather_scatter_standalone():
    x = inputs.hidden_states(6, 20, 32)
    idx = np.array([1, 4, 5, 19], np.int32)
    xc = oracle.gather_rows(x, idx)
    assert np.array_equal(xc, x[idx])
    f = inputs.hidden_states(6, 4, 32, sid=2)
    out = oracle.scatter_add(x, xc, f, idx)
    want = x.copy()
    want[idx] = (x[idx].astype(np.float64) + f).astype(np.float32)
    assert np.array_equal(out, want)


def test_model_shares_one_theta_and_reports_counts():
    sh, w, _ = _small_layer(seed=7)
    layers = []
    for li in range(3):
        wl = inputs.layer_weights(7, li, sh)
        wl["router_w"] = inputs.round_bf16((inputs.normal(7, 300 + li, sh.d) * 0.2).astype(np.float32))
        layers.append(oracle.DenseLayer(sh, wl))
    V = 50
    embed = inputs.activations(7, 400, V, sh.d)
    ids = inputs.integers(7, 401, 24, V)
    cu = np.array([0, 10, 24], np.int32)
    x_lo, _, c_lo = oracle.model_prefill(layers, embed, ids, cu, theta=0.3)
    x_hi, _, c_hi = oracle.model_prefill(layers, embed, ids, cu, theta=0.6)
    assert c_lo[0] >= c_hi[0]          # same inputs at layer 0: lower theta executes a superset
    x_all, _, c_all = oracle.model_prefill(layers, embed, ids, cu, theta=0.0)
    assert c_all == [24, 24, 24]
    x_none, _, c_none = oracle.model_prefill(layers, embed, ids, cu, theta=1.1)
    assert c_none == [0, 0, 0] and np.array_equal(x_none, embed[ids])
    _, _, c_k = oracle.model_prefill(layers, embed, ids, cu, ratios=[0.75, 0.5, 0.25])
    assert c_k == [18, 12, 6]


def test_theta_for_ratio_is_the_exact_quantile():
    """Sec. 3.4: one theta sets the ratio.  For distinct scores the theta of ratio r is the
    k-th largest with k = round(r n): exactly k scores pass p >= theta (Eq. 9), one more as soon as
    theta drops to the next score; closed form on an arithmetic grid; padding is left out; r = 0
    gives a theta nothing passes; ties at theta can only add to the count."""
    n = 1000
    p = (np.arange(1, n + 1, dtype=np.float32) / np.float32(n + 1))        # i / (n + 1), ascending
    perm = np.argsort(inputs.uniform(11, 1, n))
    for r in [0.0, 0.001, 0.25, 0.5, 0.731, 1.0]:
        th, c = oracle.theta_for_ratio(p[perm], r)
        k = oracle.topk_count(r, n)
        if k == 0:
            assert th > 1.0 and c == 0 and oracle.select_threshold(p, th).sum() == 0
            continue
        assert th == p[n - k] and c == k                                   # closed form on the grid
        assert oracle.select_threshold(p[perm], th).sum() == k            # Eq. 9 with that theta
        assert oracle.select_threshold(p[perm], np.nextafter(np.float32(th), np.float32(2))).sum() == k - 1
        assert np.array_equal(oracle.select_threshold(p[perm], th), oracle.select_topk(p[perm], k))
    # brute force against numpy's sort on random scores with padding and planted ties
    q = inputs.beta22(12, 1, 5000).astype(np.float32)
    q[100:160] = q[7]
    valid = (inputs.uniform(12, 2, 5000) > 0.2).astype(np.uint8)
    for r in [0.1, 0.5, 0.9]:
        th, c = oracle.theta_for_ratio(q, r, valid)
        srt = np.sort(q[valid == 1])[::-1]
        k = oracle.topk_count(r, len(srt))
        assert th == srt[k - 1] and c == int((q[valid == 1] >= th).sum()) >= k
    # monotone: a higher ratio never raises theta (lowering theta raises the ratio, Sec. 3.4)
    ths = [oracle.theta_for_ratio(q, r, valid)[0] for r in np.linspace(0.05, 1.0, 20)]
    assert all(a >= b for a, b in zip(ths, ths[1:]))


def test_theta_search_loop_converges_and_falls_back_to_bisection():
    """Host logic of the ratio-targeted search on made-up response curves (no GPU)."""
    from paper_2602_10431_b200 import calibrate
    # a consistent world: the suggested theta is the right one -> two runs
    resp = lambda th: min(1.0, max(0.0, 1.2 - 1.5 * th))                  # ratio falls with theta
    inv = lambda r: (1.2 - r) / 1.5
    th, r, hist = calibrate.search_theta(lambda t: (resp(t), inv(0.75)), 0.75)
    assert abs(r - 0.75) <= 0.005 and len(hist) == 2
    # a misleading suggestion (always far too low): the bracket takes over and bisects
    th, r, hist = calibrate.search_theta(lambda t: (resp(t), 0.01), 0.6, max_iters=30)
    assert abs(r - 0.6) <= 0.005 and abs(th - inv(0.6)) < 0.01
    # unreachable target: returns the closest run seen
    th, r, hist = calibrate.search_theta(lambda t: (0.3, 0.4), 0.9, max_iters=5)
    assert r == 0.3 and len(hist) == 5


def test_router_mlp_reduces_to_the_linear_router_and_matches_numpy():
    """Eq. 2 / Eq. 9 with an MLP router.  (a) Hidden units (w, -w) with output weights (+1, -1)
    on the execute logit rebuild the linear router exactly: max(u, 0) - max(-u, 0) = u, so the
    scores must be bit-identical to orc_router_scores.  (b) Only the logit difference matters:
    adding a constant to both logits, or moving weight between the two output rows, leaves p0
    unchanged.  (c) A numpy fp64 restatement (matrix form) agrees to rounding.  (d) A hidden unit
    that is never active (large negative bias) contributes nothing."""
    T, d, h = 50, 96, 5
    x = inputs.hidden_states(71, T, d)
    w = inputs.round_bf16((inputs.normal(71, 2, d) * 0.1).astype(np.float32))
    p_lin, z_lin = oracle.router_scores(x, w, 0.25, return_logits=True)
    w1 = np.stack([w, -w])
    p, z = oracle.router_mlp_scores(x, w1, np.zeros(2, np.float32), np.array([[1, -1], [0, 0]], np.float32),
                                    np.array([0.25, 0.0], np.float32), return_logits=True)
    assert np.array_equal(p, p_lin) and np.array_equal(z, z_lin)
    w1 = inputs.round_bf16((inputs.normal(71, 3, h * d) * 0.1).astype(np.float32)).reshape(h, d)
    b1 = (inputs.normal(71, 4, h) * 0.3).astype(np.float32)
    w2 = inputs.normal(71, 5, 2 * h).astype(np.float32).reshape(2, h)
    b2 = np.array([0.1, -0.2], np.float32)
    p, z = oracle.router_mlp_scores(x, w1, b1, w2, b2, return_logits=True)
    a = np.maximum(x.astype(np.float64) @ w1.astype(np.float64).T + b1, 0)
    g = a @ w2.astype(np.float64).T + b2
    assert np.allclose(z, g[:, 0] - g[:, 1], rtol=1e-12, atol=1e-12)
    assert np.allclose(p, np.exp(g[:, 0]) / np.exp(g).sum(axis=1), atol=1e-7)
    p_shift = oracle.router_mlp_scores(x, w1, b1, w2, b2 + np.float32(3.0))
    assert np.abs(p_shift - p).max() <= 1e-7
    w2d = np.stack([w2[0] - w2[1], np.zeros(h, np.float32)]).astype(np.float32)
    p_diff = oracle.router_mlp_scores(x, w1, b1, w2d, np.array([b2[0] - b2[1], 0], np.float32))
    assert np.abs(p_diff - p).max() <= 1e-6
    b1_dead = b1.copy()
    b1_dead[2] = -1e6
    w2_zero = w2.copy()
    w2_zero[:, 2] = 0
    assert np.array_equal(oracle.router_mlp_scores(x, w1, b1_dead, w2, b2),
                          oracle.router_mlp_scores(x, w1, b1, w2_zero, b2))
