"""GPU parity on randomly drawn shapes: head dimension, GQA factor, tree shape, batch, layers and prefix lengths around the
page and tile boundaries, bf16 cache and (head dimension 128) e4m3 cache, each against its oracle at the bounds of
tests/test_gpu_attn.py and tests/test_gpu_attn_fp8.py."""
import numpy as np
import pytest
import torch

from oracle import fp8 as F
from oracle import oracle as O
from paper_2510_13161_b200 import inputs as I
from tests.helpers import make_mirror, oracle_attention

pytestmark = pytest.mark.gpu


def draw(rng):
    d = int(rng.choice([64, 128]))
    Hkv, G = int(rng.choice([1, 2, 4])), int(rng.choice([1, 2, 4, 5, 8]))
    kappa, gamma = int(rng.integers(1, 9)), int(rng.integers(1, 9))
    B, L = int(rng.integers(1, 5)), int(rng.integers(1, 4))
    lo = int(rng.choice([0, 1, 15, 16, 17, 63, 64, 65, 127, 129, 500]))
    hi = lo + int(rng.choice([0, 1, 30, 200, 1500]))
    parent = None
    if rng.random() < 0.3:                                   # a general tree instead of the comb
        n = int(rng.integers(2, 33))
        parent = I.random_tree_parent(n, int(rng.integers(0, 1000)), max_depth=int(rng.integers(1, 8)))
        kappa, gamma = 1, n - 1
    cfg = I.VerifyConfig("r", Hkv * G * d, Hkv * G, Hkv, d, L, B, lo, hi, kappa, gamma, 64, "greedy", kv_std=1.0)
    return cfg, parent, bool(d == 128 and rng.random() < 0.5)


@pytest.mark.parametrize("seed", [7, 8])
def test_random_shapes(seed):
    rng = np.random.default_rng(seed)
    for case in range(25):
        cfg, parent, fp8 = draw(rng)
        x = I.gen_verify_inputs(cfg, 100 * seed + case, "cuda", parent=parent, with_lm_head=False)
        m = make_mirror(cfg)
        tree = m.tree(x.tokens, cfg.kappa, cfg.gamma, parent=x.parent)
        L, B, n, Hq, d = x.q.shape
        lse = torch.empty((L, B, Hq, n), dtype=torch.float32, device="cuda")
        what = (seed, case, cfg, "fp8" if fp8 else "bf16")
        if not fp8:
            out = m.mirror_attn_verify(m.kv(x.k_pool, x.v_pool, x.page_table, x.prefix_len), tree, x.q, x.k_new, x.v_new, lse_out=lse)
            torch.cuda.synchronize()
            assert m.device_status() == (0, 0), what
            ref = oracle_attention(x)
            for l in range(L):
                o_ref, lse_ref = ref[l]
                err, sc = np.abs(out[l].float().cpu().numpy() - o_ref).max(), np.abs(o_ref).max()
                assert err <= 1e-2 * sc + 1e-5, (what, l, err, sc)
                np.testing.assert_allclose(lse[l].cpu().numpy(), lse_ref, atol=2e-3)
            continue
        P = x.k_pool.shape[3]
        ks, vs = m.mirror_kv_scales_fp8(x.k_pool, P * d), m.mirror_kv_scales_fp8(x.v_pool, P * d)
        k8, v8 = m.mirror_kv_quantize_fp8(x.k_pool, P * d, ks), m.mirror_kv_quantize_fp8(x.v_pool, P * d, vs)
        kn8, vn8 = m.mirror_kv_quantize_fp8(x.k_new, d, ks), m.mirror_kv_quantize_fp8(x.v_new, d, vs)
        q_scale = float(np.float32(max(float(x.q.float().abs().max()), 1e-30)) / np.float32(448.0))
        out = m.mirror_attn_verify_fp8(m.kv_fp8(k8, v8, x.page_table, x.prefix_len), tree, x.q, kn8, vn8, ks, vs, q_scale, lse_out=lse)
        torch.cuda.synchronize()
        assert m.device_status() == (0, 0), what
        anc, _ = O.tree(x.parent)
        pt, pl = x.page_table.cpu().numpy(), x.prefix_len.cpu().numpy()
        for l in range(L):
            qc = F.quantize_tensor(x.q[l].float().cpu().numpy(), q_scale)
            common = (ks[l].cpu().numpy(), vs[l].cpu().numpy(), pt, pl)
            k_l, v_l, kn_l, vn_l = k8[l].cpu().numpy(), v8[l].cpu().numpy(), kn8[l].cpu().numpy(), vn8[l].cpu().numpy()
            o_ref, lse_ref = F.attention_layer_fp8(qc, q_scale, k_l, v_l, *common, kn_l, vn_l, anc, 1.0 / np.sqrt(d))
            a_ref, _ = F.attention_layer_fp8(qc, q_scale, k_l, v_l & 0x7F, *common, kn_l, vn_l & 0x7F, anc, 1.0 / np.sqrt(d))
            got = out[l].float().cpu().numpy().astype(np.float64)
            sc = np.abs(o_ref).max()
            assert (np.abs(got - o_ref) <= 2.0 ** -4 * a_ref + 2.0 ** -8 * np.abs(o_ref) + 2.0 ** -7 * sc).all(), (what, l)
            np.testing.assert_allclose(lse[l].cpu().numpy(), lse_ref, atol=2e-3)
