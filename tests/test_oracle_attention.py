"""Pins for the oracle's branch-tree attention (O1): it must equal what decoding each
branch alone with ordinary causal attention gives, agree with a library attention
routine under an explicit mask, and satisfy the softmax invariants."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2510_13161_b200 import inputs as I


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def small_cfg(**kw):
    base = dict(hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=16, layers=1, batch=2, prefix_lo=5,
                prefix_hi=45, kappa=3, gamma=3, vocab=32, mode="greedy", kv_std=1.0)
    base.update(kw)
    return I.VerifyConfig("t", **base)


def run_oracle(x, layer=0, parent=None, want_weights=False):
    anc, _ = O.tree(x.parent if parent is None else parent)
    scale = 1.0 / np.sqrt(x.cfg.head_dim)
    return O.attention_layer(I.bf16_bits(x.q[layer]), I.bf16_bits(x.k_pool[layer]), I.bf16_bits(x.v_pool[layer]),
                             x.page_table.numpy(), x.prefix_len.numpy(), I.bf16_bits(x.k_new[layer]),
                             I.bf16_bits(x.v_new[layer]), anc, scale, want_weights)


def gather_prefix(x, layer, b, g):
    """Prefix K and V of request b, kv head g, in logical token order, as fp64 [L,d]."""
    L = int(x.prefix_len[b])
    kp = bf16_to_f64(I.bf16_bits(x.k_pool[layer]))
    vp = bf16_to_f64(I.bf16_bits(x.v_pool[layer]))
    ks, vs = [], []
    for t in range(L):
        page = int(x.page_table[b, t // I.PAGE_SIZE])
        ks.append(kp[page, g, t % I.PAGE_SIZE])
        vs.append(vp[page, g, t % I.PAGE_SIZE])
    d = x.cfg.head_dim
    return np.array(ks).reshape(L, d), np.array(vs).reshape(L, d)


def causal_attention(qs, ks, vs, n_ctx, scale):
    """Textbook causal decode: query j (j-th of the trailing len(qs) positions) sees keys 0..n_ctx+j."""
    outs = []
    for j, qv in enumerate(qs):
        kk, vv = ks[: n_ctx + j + 1], vs[: n_ctx + j + 1]
        s = scale * kk @ qv
        w = np.exp(s - s.max())
        w /= w.sum()
        outs.append(w @ vv)
    return np.array(outs)


@pytest.mark.parametrize("seed", [0, 1])
@pytest.mark.parametrize("tree_kind", ["comb", "random"])
def test_tree_attention_equals_per_branch_causal_decoding(seed, tree_kind):
    cfg = small_cfg()
    parent = None if tree_kind == "comb" else I.random_tree_parent(cfg.n_nodes, seed, max_depth=4)
    x = I.gen_verify_inputs(cfg, seed, parent=parent, with_lm_head=False)
    out, _, _ = run_oracle(x)
    par = x.parent
    n = len(par)
    qf = bf16_to_f64(I.bf16_bits(x.q[0])); knf = bf16_to_f64(I.bf16_bits(x.k_new[0])); vnf = bf16_to_f64(I.bf16_bits(x.v_new[0]))
    G = cfg.n_q_heads // cfg.n_kv_heads
    scale = 1.0 / np.sqrt(cfg.head_dim)
    seen = np.zeros((cfg.batch, n), bool)
    for b in range(cfg.batch):
        L = int(x.prefix_len[b])
        for leaf in range(n):
            path = []
            j = leaf
            while j != -1:
                path.append(j)
                j = par[j]
            path = path[::-1]          # root .. leaf: this branch decoded on its own
            for h in range(cfg.n_q_heads):
                g = h // G
                kp, vp = gather_prefix(x, 0, b, g)
                ks = np.concatenate([kp, knf[b, path, g]], 0)
                vs = np.concatenate([vp, vnf[b, path, g]], 0)
                ref = causal_attention(qf[b, path, h], ks, vs, L, scale)
                for pos, node in enumerate(path):
                    np.testing.assert_allclose(out[b, node, h], ref[pos], rtol=0, atol=1e-12)
                    seen[b, node] = True
    assert seen.all()


def test_matches_library_attention_with_explicit_mask():
    cfg = small_cfg(batch=1, prefix_lo=37, prefix_hi=37)
    x = I.gen_verify_inputs(cfg, 3, with_lm_head=False)
    out, lse, _ = run_oracle(x)
    anc, _ = O.tree(x.parent)
    n, L, G = cfg.n_nodes, 37, cfg.n_q_heads // cfg.n_kv_heads
    qf = torch.from_numpy(bf16_to_f64(I.bf16_bits(x.q[0])))[0]          # [n,Hq,d]
    knf = torch.from_numpy(bf16_to_f64(I.bf16_bits(x.k_new[0])))[0]     # [n,Hkv,d]
    vnf = torch.from_numpy(bf16_to_f64(I.bf16_bits(x.v_new[0])))[0]
    mask = torch.cat([torch.ones(n, L, dtype=torch.bool), torch.from_numpy(anc.astype(bool))], 1)
    for h in range(cfg.n_q_heads):
        kp, vp = gather_prefix(x, 0, 0, h // G)
        K = torch.cat([torch.from_numpy(kp), knf[:, h // G]], 0)
        V = torch.cat([torch.from_numpy(vp), vnf[:, h // G]], 0)
        ref = torch.nn.functional.scaled_dot_product_attention(qf[:, h][None], K[None], V[None], attn_mask=mask[None])
        np.testing.assert_allclose(out[0, :, h], ref[0].numpy(), rtol=0, atol=1e-12)
        s = (qf[:, h] @ K.T) / np.sqrt(cfg.head_dim)
        ref_lse = torch.logsumexp(s.masked_fill(~mask, -float("inf")), -1)
        np.testing.assert_allclose(lse[0, h], ref_lse.numpy(), rtol=0, atol=1e-12)


def test_weights_sum_to_one_and_masked_weights_are_zero():
    cfg = small_cfg()
    x = I.gen_verify_inputs(cfg, 5, with_lm_head=False)
    _, _, w = run_oracle(x, want_weights=True)
    anc, _ = O.tree(x.parent)
    Lmax = x.page_table.shape[1] * I.PAGE_SIZE
    np.testing.assert_allclose(w.sum(-1), 1.0, atol=1e-13)
    for b in range(cfg.batch):
        L = int(x.prefix_len[b])
        assert (w[b, :, :, L:Lmax] == 0).all()                 # beyond the prefix: nothing
        assert (w[b, :, :, :L] > 0).all()                      # the whole verified prefix is visible
        for i in range(cfg.n_nodes):
            for j in range(cfg.n_nodes):
                col = w[b, i, :, Lmax + j]
                assert (col > 0).all() if anc[i, j] else (col == 0).all()


def test_root_sees_only_prefix_and_itself_and_ignores_other_branches():
    cfg = small_cfg(batch=1)
    x = I.gen_verify_inputs(cfg, 7, with_lm_head=False)
    out0, _, _ = run_oracle(x)
    x.k_new[0][:, 1:] = 0
    x.v_new[0][:, 1:] += 3.0
    out1, _, _ = run_oracle(x)
    np.testing.assert_array_equal(out0[:, 0], out1[:, 0])
    # a node's output does not move when a sibling branch's K/V change
    y = I.gen_verify_inputs(cfg, 7, with_lm_head=False)
    g = cfg.gamma
    y.k_new[0][:, 1 + g:] = 1.5      # branches 1.. altered, branch 0 (nodes 1..g) untouched
    out2, _, _ = run_oracle(y)
    np.testing.assert_array_equal(out0[:, 1:1 + g], out2[:, 1:1 + g])


def test_constant_values_give_constant_output_and_equal_keys_give_the_mean():
    cfg = small_cfg(batch=1, prefix_lo=20, prefix_hi=20)
    x = I.gen_verify_inputs(cfg, 9, with_lm_head=False)
    x.v_pool.fill_(0.75); x.v_new.fill_(0.75)
    out, _, _ = run_oracle(x)
    np.testing.assert_allclose(out, 0.75, atol=1e-14)
    y = I.gen_verify_inputs(cfg, 9, with_lm_head=False)
    y.k_pool.fill_(0.5); y.k_new.fill_(0.5)
    out, _, _ = run_oracle(y)
    anc, depth = O.tree(y.parent)
    vnf = bf16_to_f64(I.bf16_bits(y.v_new[0]))[0]
    G = cfg.n_q_heads // cfg.n_kv_heads
    for i in range(cfg.n_nodes):
        for h in range(cfg.n_q_heads):
            _, vp = gather_prefix(y, 0, 0, h // G)
            vis = np.concatenate([vp, vnf[anc[i].astype(bool), h // G]], 0)
            assert vis.shape[0] == 20 + depth[i] + 1
            np.testing.assert_allclose(out[0, i, h], vis.mean(0), atol=1e-13)


def test_score_shift_and_physical_page_permutation_change_nothing():
    cfg = small_cfg(batch=2)
    x = I.gen_verify_inputs(cfg, 11, with_lm_head=False)
    out0, lse0, _ = run_oracle(x)
    # same logical cache laid out contiguously instead of through a shuffled page table
    y = I.gen_verify_inputs(cfg, 11, with_lm_head=False, shuffle_pages=False)
    for b in range(cfg.batch):
        for p in range((int(x.prefix_len[b]) + 15) // 16):
            y.k_pool[0][int(y.page_table[b, p])] = x.k_pool[0][int(x.page_table[b, p])]
            y.v_pool[0][int(y.page_table[b, p])] = x.v_pool[0][int(x.page_table[b, p])]
    out1, lse1, _ = run_oracle(y)
    np.testing.assert_array_equal(out0, out1)
    np.testing.assert_array_equal(lse0, lse1)
    # reversing the logical order of the prefix tokens (a permutation) leaves o unchanged
    z = I.gen_verify_inputs(cfg, 11, with_lm_head=False)
    G = cfg.n_q_heads // cfg.n_kv_heads
    for b in range(cfg.batch):
        L = int(z.prefix_len[b])
        for pool_x, pool_z in ((x.k_pool, z.k_pool), (x.v_pool, z.v_pool)):
            for t in range(L):
                s = L - 1 - t
                pool_z[0][int(z.page_table[b, t // 16]), :, t % 16] = pool_x[0][int(x.page_table[b, s // 16]), :, s % 16]
    out2, _, _ = run_oracle(z)
    np.testing.assert_allclose(out0, out2, atol=1e-13)


def test_empty_prefix_root_returns_its_own_value():
    cfg = small_cfg(batch=1, prefix_lo=0, prefix_hi=0)
    x = I.gen_verify_inputs(cfg, 13, with_lm_head=False)
    out, lse, _ = run_oracle(x)
    vnf = bf16_to_f64(I.bf16_bits(x.v_new[0]))[0]
    G = cfg.n_q_heads // cfg.n_kv_heads
    for h in range(cfg.n_q_heads):
        np.testing.assert_allclose(out[0, 0, h], vnf[0, h // G], atol=1e-15)


def test_single_branch_reduces_to_plain_causal_decode():
    cfg = small_cfg(kappa=1, gamma=5, batch=1, prefix_lo=33, prefix_hi=33)
    x = I.gen_verify_inputs(cfg, 15, with_lm_head=False)
    out, _, _ = run_oracle(x)
    qf = bf16_to_f64(I.bf16_bits(x.q[0]))[0]; knf = bf16_to_f64(I.bf16_bits(x.k_new[0]))[0]; vnf = bf16_to_f64(I.bf16_bits(x.v_new[0]))[0]
    G = cfg.n_q_heads // cfg.n_kv_heads
    for h in range(cfg.n_q_heads):
        kp, vp = gather_prefix(x, 0, 0, h // G)
        ref = causal_attention(qf[:, h], np.concatenate([kp, knf[:, h // G]]), np.concatenate([vp, vnf[:, h // G]]), 33,
                               1 / np.sqrt(cfg.head_dim))
        np.testing.assert_allclose(out[0, :, h], ref, atol=1e-12)


def test_multi_stream_attention_mask_is_the_chain_tree():
    """The draft-side multi-stream mask (Speculative Streaming, Sec. 3.1: the main stream attends to the prefix only,
    stream j to the prefix and the streams up to j) is the tree mask of a single chain: node 0 = main stream."""
    n = 9
    want = np.zeros((n, n), np.uint8)
    for j in range(n):
        want[j, :j + 1] = 1                      # streams <= j (itself included), written from the sentence
    anc, depth = O.tree(I.comb_parent(1, n - 1))
    np.testing.assert_array_equal(anc, want)
    assert depth.tolist() == list(range(n))


def test_kv_commit_then_root_only_attention_equals_attention_over_the_accepted_path():
    """Roll-forward pin: after committing the root and an accepted path into the paged cache, a fresh query that sees
    only the (longer) prefix must get exactly what it would get from the old prefix plus those tree tokens as visible
    tree nodes -- the commit puts the right rows at the right positions of the right pages, for every layer and head."""
    from paper_2510_13161_b200 import inputs as I
    cfg = I.VerifyConfig("c", 256, 4, 2, 64, 2, 3, 20, 70, 2, 3, 512, "greedy")
    x = I.gen_verify_inputs(cfg, 3, "cpu", with_lm_head=False, headroom=cfg.gamma + 1)
    n = cfg.n_nodes
    kp, vp = I.bf16_bits(x.k_pool), I.bf16_bits(x.v_pool)
    kn, vn = I.bf16_bits(x.k_new), I.bf16_bits(x.v_new)
    pt, pl = x.page_table.numpy(), x.prefix_len.numpy()
    accepted = np.array([[1, 2, 3], [4, 5, -1], [-1, -1, -1]], np.int32)      # paths of length 3, 2, 0
    n_acc = np.array([3, 2, 0], np.int32)
    kp2, vp2, pl2 = O.kv_commit(kp, vp, pt, pl, kn, vn, accepted, n_acc)
    assert (pl2 == pl + n_acc + 1).all() and (kp == I.bf16_bits(x.k_pool)).all()       # inputs untouched
    parent = x.parent
    anc, _ = O.tree(parent)
    scale = 1.0 / np.sqrt(cfg.head_dim)
    q = I.bf16_bits(x.q)
    for layer in range(cfg.layers):
        # (a) new cache, every node a root-like query that sees no tree token but itself; node 0's row is the probe
        eye = np.eye(n, dtype=np.uint8)
        out_new, _, _ = O.attention_layer(q[layer], kp2[layer], vp2[layer], pt, pl2, kn[layer], vn[layer], eye, scale)
        for b in range(cfg.batch):
            path = [0] + [int(c) for c in accepted[b, :n_acc[b]]]
            # (b) old cache, the probe row sees exactly the committed tree tokens plus itself
            vis = np.eye(n, dtype=np.uint8)
            probe = n - 1                                  # a node outside every committed path
            assert probe not in path
            vis[probe, path] = 1
            out_old, _, _ = O.attention_layer(q[layer], kp[layer], vp[layer], pt, pl, kn[layer], vn[layer], vis, scale)
            # the same query vector must be used on both sides: compare row `probe` of (b) with row `probe` of (a)
            np.testing.assert_allclose(out_new[b, probe], out_old[b, probe], rtol=1e-9, atol=1e-12)
