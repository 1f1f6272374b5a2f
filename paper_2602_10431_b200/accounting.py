"""Work model of the token-adaptive quantised layer (host-side bookkeeping).

Skipping a layer for a token removes that layer's linear-layer work for that
token (Eq. 3), so the per-token linear FLOPs of a model are
`execution_ratio * 2 * P_lin * n_layers`; the FLOPs table of the paper
(13.0 GFLOPs per token for LLaMA2-7B at full execution) follows this model.
"""
from __future__ import annotations


def linear_params(d, n_heads, n_kv_heads, head_dim, ffn):
    """Weights in the four quantised linears of one layer (QKV, O, gate+up, down)."""
    q, kv = n_heads * head_dim, n_kv_heads * head_dim
    return d * q + 2 * d * kv + q * d + 3 * d * ffn


def linear_flops_per_token(d, n_heads, n_kv_heads, head_dim, ffn, n_layers=1, ratio=1.0):
    return ratio * 2.0 * linear_params(d, n_heads, n_kv_heads, head_dim, ffn) * n_layers


def attention_flops(exec_lens, n_heads, head_dim):
    """Causal attention FLOPs: QK^T and PV over the lower triangle, per sequence
    2 * 2 * (S_e (S_e + 1) / 2) * H * hd."""
    return sum(2.0 * s * (s + 1) * n_heads * head_dim for s in exec_lens)


def packed_bytes_per_weight(bits, group):
    """Codes plus fp16 scale and fp16 zero-point per group."""
    return bits / 8.0 + 4.0 / group


def layer_weight_bytes(d, n_heads, n_kv_heads, head_dim, ffn, bits, group):
    return linear_params(d, n_heads, n_kv_heads, head_dim, ffn) * packed_bytes_per_weight(bits, group)


def router_bytes(T, d):
    """Router pass: every token's hidden state is read once (bf16), one score written."""
    return T * (2 * d + 4)


def gather_bytes(n_exec, d, with_norm=False):
    return n_exec * (2 * d + 2 * d * (2 if with_norm else 1))


def scatter_bytes(n_exec, d):
    return n_exec * (4 * d + 2 * d)


def layer_flops(sh, seq_lens, ratio):
    """FLOPs of one layer call on sequences of `seq_lens` tokens of which a share `ratio`
    executes (evenly per sequence): linears on the executed tokens plus causal attention
    among them."""
    ex = [ratio * s for s in seq_lens]
    lin = 2.0 * linear_params(sh.d, sh.n_heads, sh.n_kv_heads, sh.head_dim, sh.ffn) * sum(ex)
    return lin + attention_flops(ex, sh.n_heads, sh.head_dim)


def packed_weight_bytes(sh):
    """Bytes of the four packed linears of one layer (codes + per-group scale and zero-point)."""
    return int(layer_weight_bytes(sh.d, sh.n_heads, sh.n_kv_heads, sh.head_dim, sh.ffn, sh.bits, sh.group))
