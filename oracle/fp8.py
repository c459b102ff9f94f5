"""CPU oracle of the low-precision modes: the e4m3 rounding model of the LM head's operands and of the KV cache.

TEST INFRASTRUCTURE ONLY: imported by tests/ (and nothing in the CUDA package).  Plain numpy.

The paper states no precision for the LM head (Eq. 1, Eq. 5); the low-precision mode is this build's own option, and
its definition is written out here: every row x of a matrix (a weight row of W, a hidden row) is replaced by
scale * e4m3(x / scale) with scale = max|x| / 448 (1 for an all-zero row), where e4m3 is the 8-bit floating-point
format with 4 exponent bits (bias 7), 3 mantissa bits, subnormals, no infinities and the largest finite value 448,
rounding to nearest with ties to the even mantissa, values beyond 448 saturating.  The scale and the quotient are
computed in fp32 (that decides the 8-bit code, so both sides take that decision in the same precision); everything
after the rounding is fp64: logits = (scale_w * scale_h) * sum_k code_w[k] * code_h[k].

The 8-bit KV cache (also this build's own option: Section 3 and Eq. 1 state no storage precision) keeps one scale per
(layer, KV head): scale = max|x| / 448 over that layer's and head's K (or V) elements, codes as above.  Attention over
such a cache is the plain branch-tree attention of the decoded values, K = scale_k * code, V = scale_v * code, with the
queries rounded the same way under one scale for the call (q8 = q_scale * e4m3(q / q_scale)) and fp64 arithmetic after
the rounding: attention_layer_fp8 feeds the decoded codes (exact in bf16) to the C oracle head by head, folding
scale_k * q_scale into the score scale and multiplying the output by scale_v.

Pins (tests/test_oracle_fp8.py): all 256 code points decode to the values of the format's definition and encode back to
themselves; hand-picked ties; saturation; subnormals; monotonicity; values exactly representable are recovered, so the
quantised LM head equals the plain one on such inputs.
"""
from __future__ import annotations

import numpy as np

E4M3_MAX = 448.0


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    """uint8 e4m3 codes -> fp64 values (code 0x7f / 0xff, the NaN of the format, decodes to nan)."""
    c = np.asarray(codes, np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = (c & 7).astype(np.float64)
    val = np.where(e == 0, m * 2.0 ** -9, (1.0 + m / 8.0) * np.exp2(e.astype(np.float64) - 7.0))
    val = np.where((e == 15) & ((c & 7) == 7), np.nan, val)
    return sign * val


def e4m3_encode(x: np.ndarray) -> np.ndarray:
    """fp64 values -> uint8 e4m3 codes: round to nearest, ties to even, saturating at +-448."""
    x = np.asarray(x, np.float64)
    a = np.minimum(np.abs(x), E4M3_MAX)
    # spacing of the format at |x|: 2^-9 below 2^-6 (subnormals and the first binade), else 2^(floor(log2|x|) - 3)
    ex = np.floor(np.log2(np.maximum(a, 2.0 ** -6)))
    step = np.exp2(ex - 3.0)
    q = np.rint(a / step) * step                      # np.rint rounds half to even: a / step is exact in fp64
    q = np.minimum(q, E4M3_MAX)
    # back to (exponent, mantissa)
    ex2 = np.floor(np.log2(np.maximum(q, 2.0 ** -6)))
    sub = q < 2.0 ** -6
    e = np.where(sub, 0, ex2 + 7).astype(np.int64)
    m = np.where(sub, np.rint(q / 2.0 ** -9), np.rint((q / np.exp2(ex2) - 1.0) * 8.0)).astype(np.int64)
    code = (e << 3) | m
    code = np.where(np.signbit(x), code | 0x80, code)
    return code.astype(np.uint8)


def quantize_rows(x: np.ndarray):
    """x [rows, cols] (values that are exact in fp32, e.g. bf16) -> (codes uint8 [rows, cols], scales fp32 [rows])."""
    x32 = np.asarray(x, np.float32)
    amax = np.max(np.abs(x32), axis=1)
    scale = np.where(amax > 0, amax / np.float32(448.0), np.float32(1.0)).astype(np.float32)       # fp32 division
    ratio = (x32 / scale[:, None]).astype(np.float32)                                                # fp32 division
    return e4m3_encode(ratio.astype(np.float64)), scale


def lmhead_logits_fp8(h_codes, h_scale, w_codes, w_scale) -> np.ndarray:
    """logits[r, v] = w_scale[v] * h_scale[r] * sum_k w[v, k] h[r, k] over the decoded codes, in fp64."""
    h = e4m3_decode(h_codes)
    w = e4m3_decode(w_codes)
    acc = h @ w.T
    return acc * (np.asarray(h_scale, np.float64)[:, None] * np.asarray(w_scale, np.float64)[None, :])


def kv_scales(x: np.ndarray, head_axis: int) -> np.ndarray:
    """x [L, ..., Hkv, ...] (values exact in fp32) -> fp32 scales [L, Hkv]: max|x| / 448 per layer and head (1 if zero)."""
    x32 = np.abs(np.asarray(x, np.float32))
    axes = tuple(a for a in range(x32.ndim) if a not in (0, head_axis))
    amax = x32.max(axis=axes)
    return np.where(amax > 0, amax / np.float32(448.0), np.float32(1.0)).astype(np.float32)


def kv_quantize(x: np.ndarray, scale: np.ndarray, head_axis: int) -> np.ndarray:
    """e4m3 codes of x under scale [L, Hkv] (fp32 division, round to nearest even, saturating)."""
    x32 = np.asarray(x, np.float32)
    shape = [1] * x32.ndim
    shape[0], shape[head_axis] = scale.shape
    ratio = (x32 / np.asarray(scale, np.float32).reshape(shape)).astype(np.float32)
    return e4m3_encode(ratio.astype(np.float64))


def _codes_as_bf16_bits(codes: np.ndarray) -> np.ndarray:
    """e4m3 values have 4 significant bits: exact in bf16."""
    v = e4m3_decode(codes).astype(np.float32)
    return (v.view(np.uint32) >> 16).astype(np.uint16)


def quantize_tensor(x: np.ndarray, scale: float) -> np.ndarray:
    """e4m3 codes of x under one scale (fp32 division, round to nearest even, saturating)."""
    ratio = (np.asarray(x, np.float32) / np.float32(scale)).astype(np.float32)
    return e4m3_encode(ratio.astype(np.float64))


def attention_layer_fp8(q_codes, q_scale: float, k_codes, v_codes, k_scale, v_scale, page_table, prefix_len, k_new_codes,
                        v_new_codes, anc, scale: float):
    """Branch-tree attention of one layer over an e4m3 cache.  q_codes uint8 [B,n,Hq,d]; k_codes / v_codes uint8
    [pages,Hkv,P,d]; k_new_codes / v_new_codes uint8 [B,n,Hkv,d]; k_scale / v_scale fp32 [Hkv].
    Returns (out [B,n,Hq,d], lse [B,Hq,n]) in fp64."""
    from oracle import oracle as O
    q_bits = _codes_as_bf16_bits(q_codes)
    B, n, Hq, d = q_bits.shape
    Hkv = k_codes.shape[1]
    G = Hq // Hkv
    out = np.zeros((B, n, Hq, d), np.float64)
    lse = np.zeros((B, Hq, n), np.float64)
    for g in range(Hkv):
        o_g, lse_g, _ = O.attention_layer(
            np.ascontiguousarray(q_bits[:, :, g * G:(g + 1) * G]),
            _codes_as_bf16_bits(k_codes[:, g:g + 1]), _codes_as_bf16_bits(v_codes[:, g:g + 1]), page_table, prefix_len,
            _codes_as_bf16_bits(k_new_codes[:, :, g:g + 1]), _codes_as_bf16_bits(v_new_codes[:, :, g:g + 1]), anc,
            scale * float(k_scale[g]) * float(np.float32(q_scale)))
        out[:, :, g * G:(g + 1) * G] = o_g * float(v_scale[g])
        lse[:, g * G:(g + 1) * G] = lse_g
    return out, lse
