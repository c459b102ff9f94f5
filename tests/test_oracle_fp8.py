"""Pins for the e4m3 rounding model of the low-precision LM head (oracle/fp8.py)."""
import numpy as np

from oracle import fp8 as F


def literal_e4m3_values():
    """The format written out from its definition: sign, 4 exponent bits (bias 7), 3 mantissa bits, subnormals at
    exponent 0, no infinities, S.1111.111 is NaN."""
    vals = {}
    for code in range(256):
        s, e, m = code >> 7, (code >> 3) & 15, code & 7
        if e == 15 and m == 7:
            continue
        v = (m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7)
        vals[code] = -v if s else v
    return vals


def test_all_code_points_decode_and_encode_back():
    vals = literal_e4m3_values()
    codes = np.array(sorted(vals), np.uint8)
    dec = F.e4m3_decode(codes)
    np.testing.assert_array_equal(dec, np.array([vals[c] for c in codes]))
    enc = F.e4m3_encode(dec)
    np.testing.assert_array_equal(enc, codes)                     # (the two zeros keep their signs)
    assert max(vals.values()) == 448.0 and min(v for v in vals.values() if v > 0) == 2.0 ** -9


def test_hand_picked_ties_go_to_the_even_mantissa():
    # between 1.0 (mantissa 000) and 1.125 (001): 1.0625 -> 1.0; between 1.125 (001) and 1.25 (010): 1.1875 -> 1.25
    # between 416 (101) and 448 (110): 432 -> 448; smallest subnormal 2^-9: half of it ties to 0, 1.5 * 2^-9 ties to 2 * 2^-9
    x = np.array([1.0625, 1.1875, 432.0, 2.0 ** -10, 1.5 * 2.0 ** -9, -1.0625, 24.0 + 1.0, 26.0 + 1.0])
    want = np.array([1.0, 1.25, 448.0, 0.0, 2.0 ** -8, -1.0, 24.0, 28.0])       # 25 between 24 (100) and 26 (101): even = 24; 27 between 26 and 28 (110): 28
    np.testing.assert_array_equal(F.e4m3_decode(F.e4m3_encode(x)), want)
    # just off the tie goes to the nearer neighbour
    np.testing.assert_array_equal(F.e4m3_decode(F.e4m3_encode(np.array([1.0626, 1.0624, 431.9]))), [1.125, 1.0, 416.0])


def test_saturation_and_monotonicity():
    np.testing.assert_array_equal(F.e4m3_decode(F.e4m3_encode(np.array([500.0, 1e9, -1e9, 448.0, 464.0]))), [448.0, 448.0, -448.0, 448.0, 448.0])
    x = np.linspace(-460, 460, 20001)
    d = F.e4m3_decode(F.e4m3_encode(x))
    assert (np.diff(d) >= 0).all()
    # the rounded value is the nearest code point: never further than half the local spacing
    vals = np.array(sorted(literal_e4m3_values().values()))
    xin = x[np.abs(x) <= 448]
    nearest = np.abs(xin[:, None] - vals[None, :]).min(axis=1)
    np.testing.assert_allclose(np.abs(F.e4m3_decode(F.e4m3_encode(xin)) - xin), nearest, atol=1e-12)


def test_row_scale_maps_the_row_maximum_to_448_and_exact_inputs_are_recovered():
    rng = np.random.default_rng(0)
    # rows whose entries are code points times a power-of-two scale with the row maximum at 448 * scale: exact round trip
    vals = np.array(sorted(v for v in literal_e4m3_values().values()))
    rows = []
    for r, sc in enumerate((2.0 ** -6, 2.0 ** -3, 1.0)):
        row = rng.choice(vals, size=64) * sc
        row[r] = 448.0 * sc
        rows.append(row)
    x = np.array(rows)
    codes, scale = F.quantize_rows(x)
    np.testing.assert_array_equal(scale, np.array([2.0 ** -6, 2.0 ** -3, 1.0], np.float32))
    np.testing.assert_array_equal(F.e4m3_decode(codes) * scale[:, None].astype(np.float64), x)
    # an all-zero row keeps scale 1 and codes 0
    c0, s0 = F.quantize_rows(np.zeros((1, 8)))
    assert s0[0] == 1.0 and not c0.any()


def test_quantised_lmhead_equals_the_plain_one_on_exactly_representable_operands():
    rng = np.random.default_rng(1)
    vals = np.array(sorted(v for v in literal_e4m3_values().values() if abs(v) <= 4))
    W = rng.choice(vals, size=(40, 32)); W[:, 0] = 448.0 / 64           # every row's maximum is 7 = 448 / 64: scale 2^-6
    h = rng.choice(vals, size=(5, 32)); h[:, 0] = 448.0 / 64
    wc, ws = F.quantize_rows(W)
    hc, hs = F.quantize_rows(h)
    np.testing.assert_allclose(F.lmhead_logits_fp8(hc, hs, wc, ws), h @ W.T, rtol=1e-13)
    # and a generic case stays within the format's error bound: every operand within 2^-4 relative of itself or
    # half the smallest subnormal step, so each logit within a computable bound
    W = rng.normal(0, 0.02, size=(30, 64)); h = rng.normal(0, 1.0, size=(4, 64))
    wc, ws = F.quantize_rows(W.astype(np.float32)); hc, hs = F.quantize_rows(h.astype(np.float32))
    Wq = F.e4m3_decode(wc) * ws[:, None]; hq = F.e4m3_decode(hc) * hs[:, None]
    assert (np.abs(Wq - W) <= np.maximum(np.abs(W) * 2.0 ** -4, ws[:, None] * 2.0 ** -10) * 1.0001).all()
    assert (np.abs(hq - h) <= np.maximum(np.abs(h) * 2.0 ** -4, hs[:, None] * 2.0 ** -10) * 1.0001).all()


# ---- the 8-bit KV cache -------------------------------------------------------------------------

def _bf16_bits(v: np.ndarray) -> np.ndarray:
    return (np.asarray(v, np.float32).view(np.uint32) >> 16).astype(np.uint16)


def test_kv_scales_and_codes_per_layer_and_head():
    rng = np.random.default_rng(5)
    L, pages, Hkv, P, d = 2, 3, 2, 16, 8
    x = rng.standard_normal((L, pages, Hkv, P, d)).astype(np.float32)
    x[1, 2, 1, 7, 3] = -9.5                                       # the known extreme of (layer 1, head 1)
    x[0, :, 1] = 0.0                                              # an all-zero head keeps scale 1
    sc = F.kv_scales(x, head_axis=2)
    assert sc.shape == (L, Hkv) and sc.dtype == np.float32
    assert sc[1, 1] == np.float32(9.5) / np.float32(448.0) and sc[0, 1] == 1.0
    for l in range(L):
        for h in range(Hkv):
            if (l, h) != (0, 1):
                assert sc[l, h] == np.abs(x[l, :, h]).max() / np.float32(448.0)
    codes = F.kv_quantize(x, sc, head_axis=2)
    assert codes[1, 2, 1, 7, 3] == 0xFE                           # -448: sign bit, exponent 1111, mantissa 110
    dec = F.e4m3_decode(codes) * sc.astype(np.float64)[:, None, :, None, None]
    # every element within half a step of the format at its magnitude (step <= 2^-3 relative above the subnormals)
    err = np.abs(dec - x)
    bound = np.maximum(np.abs(x) * 2.0 ** -4, sc.astype(np.float64)[:, None, :, None, None] * 2.0 ** -10) * (1 + 1e-6)
    assert (err <= bound).all()
    # the tree's rows [L, B, n, Hkv, d] use axis 3
    y = rng.standard_normal((L, 2, 5, Hkv, d)).astype(np.float32)
    sy = F.kv_scales(y, head_axis=3)
    assert sy[1, 0] == np.abs(y[1, :, :, 0]).max() / np.float32(448.0)


def test_fp8_attention_equals_plain_attention_of_the_decoded_cache():
    """Power-of-two scales keep scale * code exact in bf16, so the same cache can be handed to the plain oracle; the
    scales differ per head, so a swapped head, a scale applied to the wrong operand or a missing one shows."""
    from oracle import oracle as O
    rng = np.random.default_rng(11)
    B, n, Hq, Hkv, d, P = 2, 5, 4, 2, 16, 16
    pages = 6
    parent = [-1, 0, 1, 0, 3]
    anc, _ = O.tree(parent)
    page_table = np.array([[4, 1, 0], [2, 5, 3]], np.int32)
    prefix_len = np.array([37, 16], np.int32)
    q_codes = rng.integers(0, 256, (B, n, Hq, d)).astype(np.uint8)
    k_codes = rng.integers(0, 256, (pages, Hkv, P, d)).astype(np.uint8)
    v_codes = rng.integers(0, 256, (pages, Hkv, P, d)).astype(np.uint8)
    kn_codes = rng.integers(0, 256, (B, n, Hkv, d)).astype(np.uint8)
    vn_codes = rng.integers(0, 256, (B, n, Hkv, d)).astype(np.uint8)
    for c in (q_codes, k_codes, v_codes, kn_codes, vn_codes):
        c[(c & 0x7F) == 0x7F] = 0x30                              # no NaN codes
        c[(c & 0x78) > 0x48] &= 0xC7                              # keep magnitudes small: scores stay moderate
    k_scale = np.array([0.25, 2.0], np.float32)
    v_scale = np.array([4.0, 0.5], np.float32)
    q = F.e4m3_decode(q_codes) * 0.125                            # q_scale = 2^-3: exact in bf16 as well
    out8, lse8 = F.attention_layer_fp8(q_codes, 0.125, k_codes, v_codes, k_scale, v_scale, page_table, prefix_len, kn_codes,
                                       vn_codes, anc, 0.3)
    def dec(c, s, axis):
        shape = [1] * c.ndim
        shape[axis] = Hkv
        return _bf16_bits(F.e4m3_decode(c) * s.astype(np.float64).reshape(shape))
    out, lse, _ = O.attention_layer(_bf16_bits(q), dec(k_codes, k_scale, 1), dec(v_codes, v_scale, 1), page_table, prefix_len,
                                    dec(kn_codes, k_scale, 2), dec(vn_codes, v_scale, 2), anc, 0.3)
    np.testing.assert_allclose(out8, out, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(lse8, lse, rtol=1e-12, atol=1e-12)
    assert np.abs(out).max() > 0.1
