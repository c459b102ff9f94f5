"""GPU parity: branch-tree attention over an e4m3 KV cache (mirror_attn_verify_fp8) and the cache quantiser against the
oracle's rounding model (oracle/fp8.py)."""
import numpy as np
import pytest
import torch

from oracle import fp8 as F
from oracle import oracle as O
from paper_2510_13161_b200 import inputs as I
from paper_2510_13161_b200.binding import MirrorError
from tests.helpers import make_mirror

pytestmark = pytest.mark.gpu

# Tolerance against the oracle (8-bit Q, K and V, fp64 after the rounding).  The kernel also rounds the unnormalised softmax
# weights to e4m3: each weight is off by at most 2^-4 of itself, so an output element is off by at most
# 2^-4 * sum_j w_j |v_j| (checked element by element below: the derived bound).  The errors are independent from key to key
# and mostly cancel: 1% .. 3% of the largest output on these shapes, depending on how the CTAs cut the units; FP8_REL is a
# coarse gate on top of the derived bound.  The row sums are taken before that rounding: the log-sum-exp keeps the bf16
# path's bound.
FP8_REL = 5e-2
LSE_ATOL = 2e-3


def small(**kw):
    base = dict(hidden=1024, n_q_heads=8, n_kv_heads=2, head_dim=128, layers=2, batch=2, prefix_lo=1, prefix_hi=300,
                kappa=2, gamma=4, vocab=64, mode="greedy", kv_std=1.0)
    base.update(kw)
    return I.VerifyConfig("t", **base)


def f32(t):
    return t.float().cpu().numpy()


def quantise(m, x):
    """The library's own quantiser; the codes are checked against the oracle's in test_quantiser_is_bit_exact."""
    P, d = x.k_pool.shape[3], x.k_pool.shape[4]
    ks, vs = m.mirror_kv_scales_fp8(x.k_pool, P * d), m.mirror_kv_scales_fp8(x.v_pool, P * d)
    k8, v8 = m.mirror_kv_quantize_fp8(x.k_pool, P * d, ks), m.mirror_kv_quantize_fp8(x.v_pool, P * d, vs)
    kn8, vn8 = m.mirror_kv_quantize_fp8(x.k_new, d, ks), m.mirror_kv_quantize_fp8(x.v_new, d, vs)
    return ks, vs, k8, v8, kn8, vn8


def run_and_compare(cfg, seed, parent=None, q_std=1.0, layers=None, tweak=None):
    x = I.gen_verify_inputs(cfg, seed, "cuda", parent=parent, with_lm_head=False, q_std=q_std)
    if tweak is not None:
        tweak(x)
    m = make_mirror(cfg)
    ks, vs, k8, v8, kn8, vn8 = quantise(m, x)
    kv = m.kv_fp8(k8, v8, x.page_table, x.prefix_len)
    tree = m.tree(x.tokens, cfg.kappa, cfg.gamma, parent=x.parent)
    L, B, n, Hq, d = x.q.shape
    lse = torch.empty((L, B, Hq, n), dtype=torch.float32, device="cuda")
    q_scale = float(np.float32(max(float(x.q.float().abs().max()), 1e-30)) / np.float32(448.0))
    out = m.mirror_attn_verify_fp8(kv, tree, x.q, kn8, vn8, ks, vs, q_scale, lse_out=lse)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    anc, _ = O.tree(x.parent)
    pt, pl = x.page_table.cpu().numpy(), x.prefix_len.cpu().numpy()
    ks_h, vs_h = ks.cpu().numpy(), vs.cpu().numpy()
    worst = 0.0
    for l in (range(L) if layers is None else layers):
        ref, lse_ref = F.attention_layer_fp8(F.quantize_tensor(f32(x.q[l]), q_scale), q_scale, k8[l].cpu().numpy(), v8[l].cpu().numpy(), ks_h[l], vs_h[l], pt, pl,
                                             kn8[l].cpu().numpy(), vn8[l].cpu().numpy(), anc, 1.0 / np.sqrt(d))
        got = f32(out[l]).astype(np.float64)
        err, scale = np.abs(got - ref).max(), np.abs(ref).max()
        assert err <= FP8_REL * scale, (l, err, scale)
        # the worst case, element by element: every weight off by 2^-4 of itself in the direction of its |v|
        # (sum_j w_j |v_j|: the oracle again with the sign bits of the V codes cleared), plus the output's bf16 rounding
        # and the weights that fall below the 8-bit format's range
        a_ref, _ = F.attention_layer_fp8(F.quantize_tensor(f32(x.q[l]), q_scale), q_scale, k8[l].cpu().numpy(), v8[l].cpu().numpy() & 0x7F,
                                         ks_h[l], vs_h[l], pt, pl, kn8[l].cpu().numpy(), vn8[l].cpu().numpy() & 0x7F, anc, 1.0 / np.sqrt(d))
        assert (np.abs(got - ref) <= 2.0 ** -4 * a_ref + 2.0 ** -8 * np.abs(ref) + 2.0 ** -7 * scale).all(), l
        np.testing.assert_allclose(lse[l].cpu().numpy(), lse_ref, atol=LSE_ATOL)
        worst = max(worst, err / scale)
    return worst


def test_quantiser_is_bit_exact():
    cfg = small(batch=3, layers=3)
    x = I.gen_verify_inputs(cfg, 4, "cuda", with_lm_head=False)
    x.k_pool[1, :, 1] = 0                                           # an all-zero (layer, head): scale 1, codes 0
    m = make_mirror(cfg)
    ks, vs, k8, v8, kn8, vn8 = quantise(m, x)
    torch.cuda.synchronize()
    for pool, new, s, c, cn in ((x.k_pool, x.k_new, ks, k8, kn8), (x.v_pool, x.v_new, vs, v8, vn8)):
        s_ref = F.kv_scales(f32(pool), head_axis=2)
        np.testing.assert_array_equal(s.cpu().numpy(), s_ref)
        np.testing.assert_array_equal(c.cpu().numpy(), F.kv_quantize(f32(pool), s_ref, head_axis=2))
        np.testing.assert_array_equal(cn.cpu().numpy(), F.kv_quantize(f32(new), s_ref, head_axis=3))     # (saturating where beyond)


@pytest.mark.parametrize("kw", [
    dict(),                                                          # 17 rows, ragged prefixes, 2 layers
    dict(n_q_heads=10, hidden=1280, kappa=4, gamma=4, batch=3, layers=3),            # G = 5 (85 rows)
    dict(prefix_lo=0, prefix_hi=0),                                  # tree tokens only
    dict(prefix_lo=15, prefix_hi=17, batch=4),                       # around a page boundary
    dict(prefix_lo=33, prefix_hi=33, batch=1),                       # three slots and the tree's: odd last slots
    dict(n_q_heads=16, hidden=2048, kappa=4, gamma=4, batch=2, prefix_hi=700),        # 136 rows: two row blocks
    dict(n_q_heads=16, hidden=2048, kappa=8, gamma=8, batch=2, prefix_hi=500),        # 520 rows, n = 65
    dict(kappa=8, gamma=15, batch=1, prefix_hi=100),                 # n = 121 tree tokens
    dict(prefix_lo=3000, prefix_hi=5000, batch=2, layers=1),         # units cut across many CTAs
])
def test_shapes_and_ragged_cases(kw):
    run_and_compare(small(**kw), 1)


def test_general_tree_mask():
    cfg = small(kappa=1, gamma=6, batch=2)
    run_and_compare(cfg, 2, parent=I.random_tree_parent(24, 5, max_depth=6))


def test_uniform_scores_make_the_weights_exact():
    """Zero queries: every visible key has the same weight (exactly representable), so the output is the plain mean of
    the decoded V rows and only the bf16 rounding of the output is left: the P V path on its own."""
    cfg = small(prefix_lo=200, prefix_hi=900, batch=2, layers=1)

    def zero_q(x):
        x.q.zero_()
    x = I.gen_verify_inputs(cfg, 6, "cuda", with_lm_head=False)
    zero_q(x)
    m = make_mirror(cfg)
    ks, vs, k8, v8, kn8, vn8 = quantise(m, x)
    out = m.mirror_attn_verify_fp8(m.kv_fp8(k8, v8, x.page_table, x.prefix_len), m.tree(x.tokens, cfg.kappa, cfg.gamma, parent=x.parent),
                                   x.q, kn8, vn8, ks, vs, 1.0)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    anc, _ = O.tree(x.parent)
    ref, _ = F.attention_layer_fp8(F.quantize_tensor(f32(x.q[0]), 1.0), 1.0, k8[0].cpu().numpy(), v8[0].cpu().numpy(), ks[0].cpu().numpy(), vs[0].cpu().numpy(),
                                   x.page_table.cpu().numpy(), x.prefix_len.cpu().numpy(), kn8[0].cpu().numpy(), vn8[0].cpu().numpy(),
                                   anc, 1.0 / np.sqrt(cfg.head_dim))
    got = f32(out[0]).astype(np.float64)
    assert np.abs(got - ref).max() <= 2.0 ** -8 * np.abs(ref).max() + 1e-6


def test_peaked_scores_move_the_offset():
    cfg = small(prefix_lo=4096, prefix_hi=4096, batch=1, layers=1)

    def plant(x):
        qv = x.q[0, 0, 0, 0].float()
        for t, gain in ((5, 0.5), (1023, 0.8), (1024, 1.0), (2047, 1.2), (3000, 1.5), (4095, 2.0)):
            page = int(x.page_table[0, t // 16])
            x.k_pool[0, page, 0, t % 16] = (qv * gain / qv.norm() * 4.0).to(torch.bfloat16)
    run_and_compare(cfg, 3, q_std=3.0, tweak=plant)


def test_head_dim_64_is_refused():
    cfg = small(head_dim=64, n_q_heads=4, hidden=256)
    x = I.gen_verify_inputs(cfg, 1, "cuda", with_lm_head=False)
    m = make_mirror(cfg)
    z8 = torch.zeros(x.k_pool.shape, dtype=torch.uint8, device="cuda")
    n8 = torch.zeros(x.k_new.shape, dtype=torch.uint8, device="cuda")
    s = torch.ones((cfg.layers, cfg.n_kv_heads), dtype=torch.float32, device="cuda")
    with pytest.raises(MirrorError) as e:
        m.mirror_attn_verify_fp8(m.kv_fp8(z8, z8, x.page_table, x.prefix_len), m.tree(x.tokens, cfg.kappa, cfg.gamma, parent=x.parent),
                                 x.q, n8, n8, s, s, 1.0)
    assert e.value.code == 3


def test_commit_of_codes_then_attention_on_the_committed_cache():
    """The accepted path's codes are appended to the 8-bit cache byte for byte (oracle: kv_commit on the code arrays), and
    the next step's attention over that cache matches the oracle over the oracle's committed cache."""
    from paper_2510_13161_b200 import binding
    cfg = small(batch=3, prefix_lo=20, prefix_hi=120, kappa=2, gamma=3)
    x = I.gen_verify_inputs(cfg, 9, "cuda", with_lm_head=False, headroom=cfg.gamma + 1)
    m = make_mirror(cfg)
    ks, vs, k8, v8, kn8, vn8 = quantise(m, x)
    paths = [[1, 2], [], [4, 5, 6]]
    res = binding.AcceptResult(cfg.batch, cfg.gamma, "cuda")
    acc = np.full((cfg.batch, cfg.gamma), -1, np.int32)
    n_acc = np.array([len(p) for p in paths], np.int32)
    for b, p in enumerate(paths):
        acc[b, :len(p)] = p
    res.accepted_nodes.copy_(torch.from_numpy(acc))
    res.n_accepted.copy_(torch.from_numpy(n_acc))
    k_ref, v_ref, pl_ref = O.kv_commit(k8.cpu().numpy(), v8.cpu().numpy(), x.page_table.cpu().numpy(), x.prefix_len.cpu().numpy(),
                                       kn8.cpu().numpy(), vn8.cpu().numpy(), acc, n_acc)
    pl = x.prefix_len.clone()
    kv = m.kv_fp8(k8, v8, x.page_table, pl)
    tree = m.tree(x.tokens, cfg.kappa, cfg.gamma, parent=x.parent)
    m.mirror_kv_commit_fp8(kv, tree, kn8, vn8, res, pl)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    assert np.array_equal(k8.cpu().numpy(), k_ref) and np.array_equal(v8.cpu().numpy(), v_ref)
    assert np.array_equal(pl.cpu().numpy(), pl_ref)
    # next step: same tree rows on the longer prefixes
    L, B, n, Hq, d = x.q.shape
    q_scale = float(np.float32(float(x.q.float().abs().max())) / np.float32(448.0))
    out = m.mirror_attn_verify_fp8(kv, tree, x.q, kn8, vn8, ks, vs, q_scale)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    anc, _ = O.tree(x.parent)
    for l in range(L):
        ref, _ = F.attention_layer_fp8(F.quantize_tensor(f32(x.q[l]), q_scale), q_scale, k_ref[l], v_ref[l], ks[l].cpu().numpy(),
                                       vs[l].cpu().numpy(), x.page_table.cpu().numpy(), pl_ref, kn8[l].cpu().numpy(), vn8[l].cpu().numpy(),
                                       anc, 1.0 / np.sqrt(d))
        got = f32(out[l]).astype(np.float64)
        assert np.abs(got - ref).max() <= FP8_REL * np.abs(ref).max(), l


def test_fused_step_over_the_8_bit_cache_equals_its_parts():
    """mirror_verify_step_fp8 = mirror_attn_verify_fp8 -> LM head -> acceptance: the same attention bits and the same
    decision as the three calls made one after the other (each part has its own parity test against the oracle)."""
    from paper_2510_13161_b200 import binding
    cfg = small(batch=3, layers=2, prefix_lo=40, prefix_hi=400, kappa=3, gamma=3, vocab=1500)
    x = I.gen_verify_inputs(cfg, 12, "cuda")
    m = make_mirror(cfg)
    ks, vs, k8, v8, kn8, vn8 = quantise(m, x)
    kv = m.kv_fp8(k8, v8, x.page_table, x.prefix_len)
    tree = m.tree(x.tokens, cfg.kappa, cfg.gamma, parent=x.parent)
    q_scale = float(np.float32(float(x.q.float().abs().max())) / np.float32(448.0))
    acc = m.accept_in(binding.ACCEPT_GREEDY, True)
    attn_fused = torch.empty_like(x.q)
    argmax_fused = torch.empty(cfg.batch * cfg.n_nodes, dtype=torch.int32, device="cuda")
    res = m.mirror_verify_step_fp8(kv, tree, x.q, kn8, vn8, ks, vs, q_scale, None, x.W, acc, attn_fused, argmax_out=argmax_fused)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    attn = m.mirror_attn_verify_fp8(kv, tree, x.q, kn8, vn8, ks, vs, q_scale)
    rows = attn[-1].reshape(cfg.batch * cfg.n_nodes, cfg.hidden)
    lm = m.mirror_lmhead_reduce(rows, x.W)
    acc2 = m.accept_in(binding.ACCEPT_GREEDY, True, target_argmax=lm["argmax"])
    res2 = m.mirror_accept_select(tree, acc2)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    assert torch.equal(attn_fused, attn)
    assert torch.equal(argmax_fused, lm["argmax"])
    a, b = res.cpu(), res2.cpu()
    for f in ("n_accepted", "best_branch", "n_emitted", "emitted", "accepted_nodes", "decide_row"):
        assert np.array_equal(a[f], b[f]), f
