"""Top-kappa (Eq. 6) selected inside the LM-head GEMM's epilogue: the sorted (logit, id) list per CTA or unit and row,
merged afterwards, against the oracle's definition (logit descending, id ascending) -- weight streams (few rows, running
lists), several row chunks (lists per unit), kappa from 1 to 32, a vocabulary with a ragged last tile, planted ties at
the kappa-th place across CTAs, and the workspace that holds no [M, V] buffer."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2510_13161_b200 import binding, inputs as I
from tests.helpers import make_mirror

pytestmark = pytest.mark.gpu
TOL = 2e-3


def rand_bf16(shape, std, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.empty(shape, dtype=torch.bfloat16).normal_(0, std, generator=g)


def lm_cfg(V, H, T=1.0):
    return I.VerifyConfig("t", H, 4, 2, 64, 1, 1, 16, 16, 2, 4, V, "greedy", temperature=T)


def check_topk(res, logits, T, k):
    ref = O.row_reduce(logits, T, k)
    tid = res["topk_id"].cpu().numpy(); tlp = res["topk_logprob"].cpu().numpy()
    for r in range(logits.shape[0]):
        assert len(set(tid[r].tolist())) == k, r                           # k different ids
        if not np.array_equal(tid[r], ref["topk_id"][r]):
            # the order (or the k-th member) may differ only between logits closer than the GEMM's error bound
            assert np.abs(np.sort(logits[r, tid[r]]) - np.sort(logits[r, ref["topk_id"][r]])).max() < TOL, r
        np.testing.assert_allclose(tlp[r], logits[r, tid[r]] / T - ref["lse"][r], atol=2 * TOL)
        assert (np.diff(logits[r, tid[r]]) <= TOL).all()                   # descending


@pytest.mark.parametrize("M,V,H,k,T", [(17, 40000, 512, 8, 1.0), (57, 152064, 256, 8, 0.9), (128, 9000, 512, 32, 1.0),
                                        (300, 5000, 256, 5, 1.0), (520, 20011, 256, 32, 0.7), (9, 3000, 128, 1, 1.0)])
def test_fused_topk_matches_the_oracle(M, V, H, k, T):
    W = rand_bf16((V, H), 0.05, 3); hid = rand_bf16((M, H), 1.0, 4)
    m = make_mirror(lm_cfg(V, H, T), temperature=T)
    res = m.mirror_lmhead_reduce(hid.cuda(), W.cuda(), topk=k)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    logits = O.lmhead_logits(I.bf16_bits(hid), I.bf16_bits(W))
    check_topk(res, logits, T, k)
    # the workspace this took holds no [M, V] fp32 buffer (when the vocabulary is large against the lists)
    t = binding.Tree(1, 1, 0, 0, None, None); t.batch, t.n_nodes = (M + 127) // 128, min(M, 128)
    if V >= 100000:
        assert m.workspace_bytes(t, None, binding.WS_LMHEAD_TOPK) < m.workspace_bytes(t, None, binding.WS_LMHEAD_LOGITS)


def test_ties_at_the_kth_place_across_ctas_go_to_the_lower_id():
    """Identical weight rows give identical logits.  Copies of one strong row are planted far apart in the vocabulary
    (different tiles, different CTAs), more of them than kappa: the Top-kappa must hold the LOWEST ids, in order."""
    V, H, M, k = 30000, 256, 12, 4
    W = rand_bf16((V, H), 0.05, 5); hid = rand_bf16((M, H), 1.0, 6)
    big = (hid[0].float() * 0.2).to(torch.bfloat16)
    planted = [29990, 17, 15000, 7777, 22222, 301]                  # six copies, kappa = 4
    for v in planted:
        W[v] = big
    m = make_mirror(lm_cfg(V, H))
    res = m.mirror_lmhead_reduce(hid.cuda(), W.cuda(), topk=k)
    torch.cuda.synchronize()
    assert res["topk_id"][0].cpu().tolist() == sorted(planted)[:k]
    logits = O.lmhead_logits(I.bf16_bits(hid), I.bf16_bits(W))
    check_topk(res, logits, 1.0, k)


def test_early_exit_tap_needs_no_logits_buffer():
    V, H, M, k = 152064, 256, 57, 8
    W = rand_bf16((V, H), 0.05, 7).cuda(); hid = rand_bf16((M, H), 1.0, 8).cuda()
    m = make_mirror(lm_cfg(V, H))
    ids, lp = m.mirror_early_exit_tap(hid, W, k)
    torch.cuda.synchronize()
    assert m._ws.numel() < M * V * 4                                       # below the 34.7 MB that the fp32 logits alone would take
    logits = O.lmhead_logits(I.bf16_bits(hid.cpu()), I.bf16_bits(W.cpu()))
    ref = O.row_reduce(logits, 1.0, k)
    got = ids.cpu().numpy()
    for r in range(M):
        if not np.array_equal(got[r], ref["topk_id"][r]):
            assert np.abs(np.sort(logits[r, got[r]]) - np.sort(logits[r, ref["topk_id"][r]])).max() < TOL
    np.testing.assert_allclose(lp.float().cpu().numpy(), ref["topk_logprob"], atol=0.05)      # bf16 payload
