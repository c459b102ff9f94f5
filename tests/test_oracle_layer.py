"""Pins of the decoder-layer oracle (oracle/target_layer.py) against closed forms, invariants and brute force."""
import numpy as np

from oracle import target_layer as T


def test_bf16_rounding_is_nearest_even():
    # 1 + 2^-8 lies halfway between 1 and 1 + 2^-7: ties go to the even mantissa (1.0); 1 + 3*2^-8 goes up to 1 + 2^-6
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -20, 1.0 + 3 * 2.0 ** -8, -2.5, 0.0])
    got = T.bf16_round(x)
    np.testing.assert_array_equal(got, [1.0, 1.0, 1.0 + 2.0 ** -7, 1.0 + 2.0 ** -6, -2.5, 0.0])
    bits = T.bf16_round_bits(np.array([1.0, -2.0]))
    assert bits.tolist() == [0x3F80, 0xC000]
    np.testing.assert_array_equal(T.bf16_to_f64(bits), [1.0, -2.0])


def test_linear_matches_a_triple_loop_and_identity_weight():
    rng = np.random.default_rng(0)
    x, W = rng.normal(size=(3, 5)), rng.normal(size=(4, 5))
    ref = np.zeros((3, 4))
    for m in range(3):
        for n in range(4):
            for k in range(5):
                ref[m, n] += x[m, k] * W[n, k]
    np.testing.assert_allclose(T.linear(x, W), ref, rtol=1e-13)
    np.testing.assert_array_equal(T.linear(x, np.eye(5)), x)
    # the weight is [N, K]: a weight with one non-zero row n picks out output column n only
    W1 = np.zeros((4, 5)); W1[2] = 1.0
    y = T.linear(x, W1)
    np.testing.assert_allclose(y[:, 2], x.sum(1)); assert np.all(y[:, [0, 1, 3]] == 0)


def test_rmsnorm_closed_forms():
    g = np.array([0.5, 2.0, -1.0, 3.0])
    # a constant row has rms |c|: the output is sign(c) * gamma
    np.testing.assert_allclose(T.rmsnorm(np.full((1, 4), -7.0), g, 0.0), -g[None, :], rtol=1e-14)
    rng = np.random.default_rng(1)
    x = rng.normal(size=(5, 4))
    np.testing.assert_allclose(T.rmsnorm(3.7 * x, g, 0.0), T.rmsnorm(x, g, 0.0), rtol=1e-13)          # scale invariance
    y = T.rmsnorm(x, np.ones(4), 0.0)
    np.testing.assert_allclose(np.mean(y * y, -1), 1.0, rtol=1e-13)                                    # unit mean square
    # eps enters under the root: x = (3, 4, 0, 0) has mean square 6.25; with eps = 2.75 the divisor is 3
    np.testing.assert_allclose(T.rmsnorm(np.array([[3.0, 4.0, 0.0, 0.0]]), np.ones(4), 2.75), [[1.0, 4.0 / 3.0, 0.0, 0.0]])


def test_rope_closed_forms_and_relative_position():
    # d = 2: one pair with frequency 1, so position p rotates (a, b) by p radians
    x = np.array([[[1.0, 0.0]]])
    np.testing.assert_allclose(T.rope(x, np.array([np.pi / 2]), 10000.0), [[[0.0, 1.0]]], atol=1e-15)
    rng = np.random.default_rng(2)
    q, k = rng.normal(size=(1, 1, 8)), rng.normal(size=(1, 1, 8))
    np.testing.assert_array_equal(T.rope(q, np.array([0]), 10000.0), q)                               # identity at position 0
    r = T.rope(q, np.array([37]), 10000.0)
    for i in range(4):                                                                                 # pair norms kept
        np.testing.assert_allclose(r[0, 0, i] ** 2 + r[0, 0, i + 4] ** 2, q[0, 0, i] ** 2 + q[0, 0, i + 4] ** 2, rtol=1e-12)
    # pair i turns by pos * theta^(-2i/d): with theta = 16, d = 8 the angles at position 1 are 1, 1/2, 1/4, 1/8
    e = np.zeros((1, 1, 8)); e[0, 0, :4] = 1.0
    np.testing.assert_allclose(T.rope(e, np.array([1]), 16.0)[0, 0], np.concatenate([np.cos([1, .5, .25, .125]), np.sin([1, .5, .25, .125])]),
                               rtol=1e-13)
    # q . k after rotation depends on the position difference only
    dot = lambda m, n: float(np.sum(T.rope(q, np.array([m]), 10000.0) * T.rope(k, np.array([n]), 10000.0)))
    np.testing.assert_allclose(dot(5, 2), dot(103, 100), rtol=1e-10)
    np.testing.assert_allclose(dot(7, 7), float(np.sum(q * k)), rtol=1e-12)
    assert abs(dot(5, 2) - dot(2, 5)) > 1e-3                                                          # and on its sign


def test_swiglu_closed_forms():
    x = np.linspace(-6, 6, 25)
    np.testing.assert_allclose(T.silu(x) - T.silu(-x), x, atol=1e-14)          # x s(x) + x s(-x) = x
    assert T.silu(np.array([0.0]))[0] == 0.0
    np.testing.assert_allclose(T.silu(np.array([40.0])), [40.0], rtol=1e-15)
    np.testing.assert_allclose(T.silu(np.array([1.0])), [1.0 / (1.0 + np.exp(-1.0))])
    np.testing.assert_allclose(T.swiglu(np.array([1.0, 2.0]), np.array([3.0, -1.0])), [3.0 * T.silu(np.array([1.0]))[0], -T.silu(np.array([2.0]))[0]])


def _tiny_layer(rng, H, Hq, Hkv, d, inter, std=0.05):
    f = lambda *s: T.bf16_round_bits(rng.normal(0, std, size=s))
    return dict(w_qkv=f((Hq + 2 * Hkv) * d, H), w_o=f(H, Hq * d), w_gate_up=f(2 * inter, H), w_down=f(H, inter),
                norm_attn=T.bf16_round_bits(1.0 + rng.normal(0, 0.1, size=H)), norm_mlp=T.bf16_round_bits(1.0 + rng.normal(0, 0.1, size=H)))


def test_layer_with_zero_output_projections_returns_its_input_and_positions_follow_depth():
    rng = np.random.default_rng(3)
    H, Hq, Hkv, d, inter, B = 64, 4, 2, 16, 96, 2
    parent = [-1, 0, 1, 0, 3]
    n = len(parent)
    w = _tiny_layer(rng, H, Hq, Hkv, d, inter)
    prefix_len = np.array([20, 33], np.int32)
    pages = 3
    page_table = np.arange(B * pages, dtype=np.int32).reshape(B, pages)
    k_pool = T.bf16_round_bits(rng.normal(size=(B * pages, Hkv, 16, d)))
    v_pool = T.bf16_round_bits(rng.normal(size=(B * pages, Hkv, 16, d)))
    x = T.bf16_round_bits(rng.normal(size=(B * n, H)))
    wz = dict(w, w_o=np.zeros_like(w["w_o"]), w_down=np.zeros_like(w["w_down"]))
    res = T.target_layer(x, wz, k_pool, v_pool, page_table, prefix_len, parent, Hq, Hkv, d, 10000.0, 1e-6)
    np.testing.assert_array_equal(res["x"], x)
    # positions: root at prefix_len, a node at depth r at prefix_len + r
    from oracle import oracle as O
    _, depth = O.tree(parent)
    assert depth.tolist() == [0, 1, 2, 1, 2]
    assert T.positions(prefix_len, depth).tolist() == [20, 21, 22, 21, 22, 33, 34, 35, 34, 35]
    # the full layer moves the residual, and the value rows are the plain projection (no rotation)
    full = T.target_layer(x, w, k_pool, v_pool, page_table, prefix_len, parent, Hq, Hkv, d, 10000.0, 1e-6, next_norm_bits=w["norm_attn"])
    assert not np.array_equal(full["x"], x)
    h1 = T.bf16_round(T.rmsnorm(T.bf16_to_f64(x), T.bf16_to_f64(w["norm_attn"]), 1e-6))
    v_ref = T.bf16_round_bits(h1 @ T.bf16_to_f64(w["w_qkv"])[(Hq + Hkv) * d:].T).reshape(B, n, Hkv, d)
    np.testing.assert_array_equal(full["v_new"], v_ref)
    # the residual after attention is x + attn W_o^T: recompute it from the returned attention rows
    x1 = T.bf16_round(T.bf16_to_f64(x) + T.bf16_to_f64(full["attn"]) @ T.bf16_to_f64(w["w_o"]).T)
    assert np.abs(T.bf16_to_f64(full["x"]) - x1).max() > 0          # the MLP added something on top
    assert full["normed"].shape == x.shape


# ---------------------------------------------------------------------------------------------
# Composition of the layer (the pre-norm decoder layer the oracle's header states): every wiring choice inside
# target_layer() is pinned by a sparse weight whose effect has a closed form in terms of the pinned pieces.
# ---------------------------------------------------------------------------------------------
def _layer_case(seed=7):
    rng = np.random.default_rng(seed)
    H, Hq, Hkv, d, inter, B = 64, 4, 2, 16, 96, 2
    parent = [-1, 0, 1, 0, 3]
    w = _tiny_layer(rng, H, Hq, Hkv, d, inter)
    prefix_len = np.array([20, 33], np.int32)
    pages = 3
    page_table = np.arange(B * pages, dtype=np.int32).reshape(B, pages)
    k_pool = T.bf16_round_bits(rng.normal(size=(B * pages, Hkv, 16, d)))
    v_pool = T.bf16_round_bits(rng.normal(size=(B * pages, Hkv, 16, d)))
    x = T.bf16_round_bits(rng.normal(size=(B * len(parent), H)))
    dims = dict(H=H, Hq=Hq, Hkv=Hkv, d=d, inter=inter, B=B, n=len(parent))
    run = lambda ww: T.target_layer(x, ww, k_pool, v_pool, page_table, prefix_len, parent, Hq, Hkv, d, 10000.0, 1e-6)
    return dims, w, x, prefix_len, parent, run


def _unit_rows(shape, entries):
    m = np.zeros(shape)
    for (r, c), v in entries.items():
        m[r, c] = v
    return T.bf16_round_bits(m)


def test_layer_mlp_half_gate_first_then_up_on_the_normed_post_attention_stream():
    """One gate row reads column 0 of the MLP's input, one up row column 1, one down column writes column 2:
    the layer must add silu(h_0) * h_1 to column 2 of the post-attention stream x1 and nothing anywhere else, with
    h = RMSNorm(x1; norm_mlp).  Fails if gate and up rows are swapped, if the MLP reads norm(x) instead of norm(x1),
    if the second residual is taken from x instead of x1, or if the wrong norm weight is used."""
    dims, w, x, _, _, run = _layer_case()
    H, inter = dims["H"], dims["inter"]
    ww = dict(w, w_gate_up=_unit_rows((2 * inter, H), {(0, 0): 1.0, (inter, 1): 1.0}),      # gate row 0 <- col 0, up row 0 <- col 1
              w_down=_unit_rows((H, inter), {(2, 0): 1.0}))
    res = run(ww)
    x1 = T.bf16_round(T.bf16_to_f64(x) + T.bf16_to_f64(res["attn"]) @ T.bf16_to_f64(w["w_o"]).T)
    assert np.abs(x1 - T.bf16_to_f64(x)).max() > 1e-2                     # attention really moved the stream
    h = T.bf16_round(T.rmsnorm(x1, T.bf16_to_f64(w["norm_mlp"]), 1e-6))
    a, b = h[:, 0], h[:, 1]
    act = T.bf16_round(a / (1.0 + np.exp(-a)) * b)                         # silu(gate) * up, stored in bf16
    want = x1.copy()
    want[:, 2] = x1[:, 2] + act
    np.testing.assert_array_equal(res["x"], T.bf16_round_bits(want))
    swapped = x1[:, 2] + T.bf16_round(b / (1.0 + np.exp(-b)) * a)
    assert np.abs(T.bf16_round(swapped) - T.bf16_to_f64(res["x"])[:, 2]).max() > 1e-3   # the case tells the two orders apart


def test_layer_without_mlp_is_x_plus_output_projection_of_attention():
    dims, w, x, _, _, run = _layer_case()
    res = run(dict(w, w_down=np.zeros_like(w["w_down"])))
    x1 = T.bf16_round_bits(T.bf16_to_f64(x) + T.bf16_to_f64(res["attn"]) @ T.bf16_to_f64(w["w_o"]).T)
    np.testing.assert_array_equal(res["x"], x1)


def test_layer_qkv_split_and_rotation_of_queries_and_keys():
    """w_qkv rows are (query rows, key rows, value rows).  With only the key block non-zero the queries and values
    come out zero and the keys are the ROTATED projection; with only the query block non-zero the queries are the
    rotated projection and keys / values are zero.  Fails on a wrong Q/K/V boundary and on a missing rotation."""
    dims, w, x, prefix_len, parent, run = _layer_case()
    H, Hq, Hkv, d, B, n = (dims[k] for k in ("H", "Hq", "Hkv", "d", "B", "n"))
    from oracle import oracle as O
    _, depth = O.tree(parent)
    pos = T.positions(prefix_len, depth)
    h1 = T.bf16_round(T.rmsnorm(T.bf16_to_f64(x), T.bf16_to_f64(w["norm_attn"]), 1e-6))
    Wf = T.bf16_to_f64(w["w_qkv"])
    blocks = {"q": (0, Hq * d, Hq), "k": (Hq * d, (Hq + Hkv) * d, Hkv)}
    for name, (lo, hi, heads) in blocks.items():
        only = np.zeros_like(w["w_qkv"])
        only[lo:hi] = w["w_qkv"][lo:hi]
        res = run(dict(w, w_qkv=only))
        proj = (h1 @ Wf[lo:hi].T).reshape(B * n, heads, d)
        rotated = T.bf16_round_bits(T.rope(proj, pos, 10000.0)).reshape(B, n, heads, d)
        got = res["q"] if name == "q" else res["k_new"]
        np.testing.assert_array_equal(got, rotated)
        assert not np.array_equal(got, T.bf16_round_bits(proj).reshape(B, n, heads, d))     # positions > 0: rotation matters
        for other in ("q", "k_new", "v_new"):
            if other != ("q" if name == "q" else "k_new"):
                assert (T.bf16_to_f64(res[other]) == 0).all(), (name, other)        # (+0 or -0)
