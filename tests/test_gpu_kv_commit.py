"""Roll-forward of the paged cache (mirror_kv_commit) against the oracle: byte-exact pools and lengths, a second
verify step on the committed cache, and the bounds report."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2510_13161_b200 import binding, inputs as I
from tests.helpers import make_mirror, oracle_attention

pytestmark = pytest.mark.gpu


def accepted_result(B, gamma, paths, device="cuda"):
    res = binding.AcceptResult(B, gamma, device)
    acc = np.full((B, max(gamma, 1)), -1, np.int32)
    n_acc = np.zeros(B, np.int32)
    for b, p in enumerate(paths):
        acc[b, :len(p)] = p
        n_acc[b] = len(p)
    res.accepted_nodes.copy_(torch.from_numpy(acc))
    res.n_accepted.copy_(torch.from_numpy(n_acc))
    return res, acc, n_acc


@pytest.mark.parametrize("d,Hkv,layers,B,kappa,gamma", [(64, 2, 2, 3, 2, 3), (128, 8, 3, 4, 4, 4), (128, 2, 1, 1, 1, 7)])
def test_commit_matches_oracle_bytes(d, Hkv, layers, B, kappa, gamma):
    cfg = I.VerifyConfig("c", 256, Hkv * 2, Hkv, d, layers, B, 5, 90, kappa, gamma, 512, "greedy")
    x = I.gen_verify_inputs(cfg, 7, "cuda", with_lm_head=False, headroom=gamma + 1)
    rng = np.random.default_rng(0)
    paths = []
    for b in range(B):                                   # a random prefix of a random branch (length 0 .. gamma)
        br = int(rng.integers(0, kappa)); ln = int(rng.integers(0, gamma + 1))
        paths.append([1 + br * gamma + j for j in range(ln)])
    res, acc, n_acc = accepted_result(B, gamma, paths)
    m = make_mirror(cfg)
    k_pool, v_pool, pl = x.k_pool.clone(), x.v_pool.clone(), x.prefix_len.clone()
    kv = m.kv(k_pool, v_pool, x.page_table, pl)
    tree = m.tree(x.tokens, kappa, gamma)
    m.mirror_kv_commit(kv, tree, x.k_new, x.v_new, res, pl)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    kp, vp, pl_ref = O.kv_commit(I.bf16_bits(x.k_pool), I.bf16_bits(x.v_pool), x.page_table.cpu().numpy(),
                                 x.prefix_len.cpu().numpy(), I.bf16_bits(x.k_new), I.bf16_bits(x.v_new), acc, n_acc)
    assert np.array_equal(I.bf16_bits(k_pool), kp) and np.array_equal(I.bf16_bits(v_pool), vp)
    assert np.array_equal(pl.cpu().numpy(), pl_ref)


def test_second_step_on_the_committed_cache():
    """verify step -> commit -> attention of the next step: the GPU's second attention over the cache it committed
    must match the oracle's attention over the oracle's committed cache."""
    cfg = I.VerifyConfig("c2", 512, 8, 2, 64, 2, 3, 30, 120, 2, 3, 1500, "greedy")
    x = I.gen_verify_inputs(cfg, 2, "cuda", headroom=cfg.gamma + 1)
    m = make_mirror(cfg)
    k_pool, v_pool, pl = x.k_pool.clone(), x.v_pool.clone(), x.prefix_len.clone()
    kv = m.kv(k_pool, v_pool, x.page_table, pl)
    tree = m.tree(x.tokens, cfg.kappa, cfg.gamma)
    attn_out = torch.empty_like(x.q)
    acc = m.accept_in(binding.ACCEPT_GREEDY, True)
    res = m.mirror_verify_step(kv, tree, x.q, x.k_new, x.v_new, x.hidden, x.W, acc, attn_out)
    m.mirror_kv_commit(kv, tree, x.k_new, x.v_new, res, pl)
    # next step: fresh tree inputs on the longer prefix
    y = I.gen_verify_inputs(cfg, 3, "cuda", with_lm_head=False, headroom=cfg.gamma + 1)
    out2 = m.mirror_attn_verify(kv, tree, y.q, y.k_new, y.v_new)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    got = res.cpu()
    kp, vp, pl_ref = O.kv_commit(I.bf16_bits(x.k_pool), I.bf16_bits(x.v_pool), x.page_table.cpu().numpy(),
                                 x.prefix_len.cpu().numpy(), I.bf16_bits(x.k_new), I.bf16_bits(x.v_new),
                                 got["accepted_nodes"], got["n_accepted"])
    assert np.array_equal(pl.cpu().numpy(), pl_ref)
    anc, _ = O.tree(x.parent)
    scale = 1.0 / np.sqrt(cfg.head_dim)
    for layer in range(cfg.layers):
        ref, _, _ = O.attention_layer(I.bf16_bits(y.q[layer]), kp[layer], vp[layer], x.page_table.cpu().numpy(), pl_ref,
                                      I.bf16_bits(y.k_new[layer]), I.bf16_bits(y.v_new[layer]), anc, scale)
        err = np.abs(out2[layer].float().cpu().numpy() - ref).max() / max(np.abs(ref).max(), 1e-9)
        assert err < 1e-2, (layer, err)


def test_commit_beyond_the_page_table_is_reported_not_written():
    cfg = I.VerifyConfig("c3", 256, 4, 2, 64, 1, 2, 32, 32, 1, 4, 512, "greedy")      # prefix 32 = exactly two pages, no headroom
    x = I.gen_verify_inputs(cfg, 1, "cuda", with_lm_head=False)
    res, _, _ = accepted_result(2, 4, [[1, 2], []])
    m = make_mirror(cfg)
    k_pool, v_pool, pl = x.k_pool.clone(), x.v_pool.clone(), x.prefix_len.clone()
    kv = m.kv(k_pool, v_pool, x.page_table, pl)
    tree = m.tree(x.tokens, 1, 4)
    m.mirror_kv_commit(kv, tree, x.k_new, x.v_new, res, pl)
    torch.cuda.synchronize()
    assert m.device_status() == (6, 801)
    assert torch.equal(k_pool, x.k_pool) and torch.equal(v_pool, x.v_pool)
