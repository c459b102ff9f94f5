"""CPU oracle of one target decoder layer around the verify step's attention (the "target forward" of Sec. 3.1 whose
layers run between the early exit and the final verification; the targets of Sec. 4.1 are pre-norm decoder stacks).

TEST INFRASTRUCTURE ONLY: imported by tests/ (and nothing in the CUDA package).  Plain numpy in fp64.

The paper fixes no layer structure.  What is written out here is the common pre-norm decoder layer of the public
model families it evaluates on: RMSNorm -> Q/K/V projection -> rotary embedding (rotate-half convention) -> grouped
query attention over the cached prefix and the token tree -> output projection + residual -> RMSNorm -> gated MLP
(SiLU(gate) * up) -> down projection + residual.  Activations are STORED in bf16 between the steps (that is the
path's storage type, like the attention output that feeds the LM head), so the oracle rounds to bf16 exactly where a
tensor is stored and computes in fp64 in between.

Pins (tests/test_oracle_layer.py): rmsnorm of a constant row and its scale invariance; rotary embedding keeps pair
norms, is the identity at position 0, turns (1, 0) into (0, 1) at angle pi/2, and makes q.k depend on the position
difference only; silu(x) - silu(-x) = x; the linear map against a brute-force triple loop and the identity weight; a
layer whose output and down projections are zero returns its input; the wiring of target_layer() itself by sparse
weights with closed-form effects: one gate row, one up row and one down column (gate before up, MLP input =
RMSNorm of the post-attention stream with the MLP's own norm weight, second residual onto that stream), a layer
without MLP (x + W_o attention), and w_qkv with only its query or only its key block (block boundaries, both rotated,
values not).
"""
from __future__ import annotations

import numpy as np

from . import oracle as O


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> fp64 values."""
    return (np.ascontiguousarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def bf16_round_bits(x: np.ndarray) -> np.ndarray:
    """fp64 values -> bf16 bit patterns (round to nearest even from the fp32 value, as a device store does)."""
    b = np.ascontiguousarray(x, np.float64).astype(np.float32).view(np.uint32)
    r = ((b >> 16) & 1) + np.uint32(0x7FFF)
    return ((b + r) >> 16).astype(np.uint16)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """fp64 values rounded to the nearest bf16 value, returned as fp64."""
    return bf16_to_f64(bf16_round_bits(x))


def linear(x: np.ndarray, W: np.ndarray) -> np.ndarray:
    """y[m, n] = sum_k x[m, k] W[n, k]  (x: [M, K], W: [N, K], fp64)."""
    return x @ W.T


def rmsnorm(x: np.ndarray, gamma: np.ndarray, eps: float) -> np.ndarray:
    """y = x / sqrt(mean(x^2) + eps) * gamma, row by row."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gamma


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, rotate-half convention: x [M, heads, d], pos [M]; element i < d/2 pairs with i + d/2 and
    the pair is rotated by the angle pos * theta^(-2i/d)."""
    M, Hh, d = x.shape
    half = d // 2
    inv_freq = theta ** (-2.0 * np.arange(half, dtype=np.float64) / d)
    ang = pos.astype(np.float64)[:, None] * inv_freq[None, :]            # [M, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def swiglu(gate: np.ndarray, up: np.ndarray) -> np.ndarray:
    return silu(gate) * up


def positions(prefix_len: np.ndarray, depth: np.ndarray) -> np.ndarray:
    """Row (b, i) of the step sits at position prefix_len[b] + depth[i] (the root is the token after the prefix)."""
    return (prefix_len.astype(np.int64)[:, None] + depth.astype(np.int64)[None, :]).reshape(-1)


def target_layer(x_bits, w, k_pool_bits, v_pool_bits, page_table, prefix_len, parent, n_q_heads, n_kv_heads, head_dim,
                 rope_theta: float, eps: float, next_norm_bits=None):
    """One layer on the step's rows.

    x_bits [M, H] bf16 bits (residual stream, M = B * n rows ordered (request, node));
    w: dict of bf16 bit arrays  w_qkv [(Hq + 2 Hkv) d, H] (query rows, key rows, value rows), w_o [H, Hq d],
       w_gate_up [2 I, H] (gate rows, up rows), w_down [H, I], norm_attn [H], norm_mlp [H];
    k_pool_bits / v_pool_bits [num_pages, Hkv, 16, d]: this layer's cache (keys already rotated).
    Returns dict: x (new residual, bf16 bits), q, k_new, v_new (bf16 bits, [B, n, heads, d]), attn (bf16 bits [M, Hq d]),
    and, if next_norm_bits is given, normed = rmsnorm(x_new, next_norm) as bf16 bits (what the next layer, or the LM
    head after the final norm, reads).
    """
    B = int(np.asarray(prefix_len).shape[0])
    M, H = x_bits.shape
    n = M // B
    Hq, Hkv, d = n_q_heads, n_kv_heads, head_dim
    anc, depth = O.tree(parent)
    pos = positions(np.asarray(prefix_len), depth)
    f = {k: bf16_to_f64(v) for k, v in w.items()}
    x = bf16_to_f64(x_bits)

    h1 = bf16_round(rmsnorm(x, f["norm_attn"], eps))
    qkv = linear(h1, f["w_qkv"])
    q = rope(qkv[:, :Hq * d].reshape(M, Hq, d), pos, rope_theta)
    k = rope(qkv[:, Hq * d:(Hq + Hkv) * d].reshape(M, Hkv, d), pos, rope_theta)
    v = qkv[:, (Hq + Hkv) * d:].reshape(M, Hkv, d)
    q_b = bf16_round_bits(q).reshape(B, n, Hq, d)
    k_b = bf16_round_bits(k).reshape(B, n, Hkv, d)
    v_b = bf16_round_bits(v).reshape(B, n, Hkv, d)

    out, _, _ = O.attention_layer(q_b, k_pool_bits, v_pool_bits, np.asarray(page_table), np.asarray(prefix_len), k_b, v_b, anc,
                                  1.0 / np.sqrt(d))
    attn_b = bf16_round_bits(out.reshape(M, Hq * d))
    x1 = bf16_round(x + linear(bf16_to_f64(attn_b), f["w_o"]))

    h2 = bf16_round(rmsnorm(x1, f["norm_mlp"], eps))
    gu = linear(h2, f["w_gate_up"])
    inter = gu.shape[1] // 2
    act = bf16_round(swiglu(gu[:, :inter], gu[:, inter:]))
    x2_b = bf16_round_bits(x1 + linear(act, f["w_down"]))
    res = dict(x=x2_b, q=q_b, k_new=k_b, v_new=v_b, attn=attn_b)
    if next_norm_bits is not None:
        res["normed"] = bf16_round_bits(rmsnorm(bf16_to_f64(x2_b), bf16_to_f64(next_norm_bits), eps))
    return res
