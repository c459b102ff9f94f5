"""GPU parity: mirror_lmhead_reduce (tcgen05 GEMM + fused row reductions) against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2510_13161_b200 import inputs as I
from tests.helpers import make_mirror

pytestmark = pytest.mark.gpu

LOGIT_TOL = 5e-2          # the stated bound for bf16 logits against the fp64 oracle
LOGIT_TOL_TIGHT = 2e-3    # what fp32 accumulation of exact bf16 products should meet on these inputs


def lm_cfg(V, H):
    return I.VerifyConfig("t", H, 4, 2, 64, 1, 1, 16, 16, 2, 4, V, "greedy")


def rand_bf16(shape, std, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.empty(shape, dtype=torch.bfloat16).normal_(0, std, generator=g)


def check_reductions(res, logits, T=1.0, topk=0):
    ref = O.row_reduce(logits, T, topk)
    M, V = logits.shape
    srt = np.sort(logits, -1)
    gap = srt[:, -1] - srt[:, -2]
    am = res["argmax"].cpu().numpy()
    flips = int((am != ref["argmax"]).sum())
    for r in np.nonzero(am != ref["argmax"])[0]:
        # a different argmax is legitimate only inside the logit error bound
        assert logits[r, ref["argmax"][r]] - logits[r, am[r]] < LOGIT_TOL_TIGHT, (r, gap[r])
    np.testing.assert_allclose(res["maxlogit"].cpu().numpy(), ref["maxlogit"], atol=LOGIT_TOL_TIGHT)
    if res["lse"] is not None:
        np.testing.assert_allclose(res["lse"].cpu().numpy(), ref["lse"], atol=LOGIT_TOL_TIGHT)
    return ref, flips


@pytest.mark.parametrize("M,V,H", [(9, 1024, 256), (17, 5000, 512), (1, 1024, 64), (33, 5003, 320), (16, 152, 128),
                                   (64, 2048, 1024), (130, 3000, 256)])
def test_logits_and_reductions_match_oracle(M, V, H):
    W = rand_bf16((V, H), 0.05, 1); hid = rand_bf16((M, H), 1.0, 2)
    m = make_mirror(lm_cfg(V, H))
    res = m.mirror_lmhead_reduce(hid.cuda(), W.cuda(), want_logits=True)
    assert m.device_status() == (0, 0)
    logits = O.lmhead_logits(I.bf16_bits(hid), I.bf16_bits(W))
    got = res["logits"].cpu().numpy().astype(np.float64)
    err = np.abs(got - logits).max()
    assert err < LOGIT_TOL and err < LOGIT_TOL_TIGHT, err
    check_reductions(res, logits)
    # the reductions are the same with and without the logits spill
    res2 = m.mirror_lmhead_reduce(hid.cuda(), W.cuda(), want_logits=False)
    assert torch.equal(res["argmax"], res2["argmax"])
    assert torch.equal(res["maxlogit"], res2["maxlogit"]) and torch.equal(res["lse"], res2["lse"])


@pytest.mark.parametrize("M,V,H", [(300, 4096, 256), (392, 4096, 256), (520, 5003, 320), (1040, 2600, 192)])
def test_row_chunking(M, V, H):
    """More than 256 rows: several row chunks per vocabulary tile, one partial per unit (ragged last tile included)."""
    W = rand_bf16((V, H), 0.05, 3); hid = rand_bf16((M, H), 1.0, 4)
    m = make_mirror(lm_cfg(V, H))
    res = m.mirror_lmhead_reduce(hid.cuda(), W.cuda(), want_logits=True)
    assert m.device_status() == (0, 0)
    logits = O.lmhead_logits(I.bf16_bits(hid), I.bf16_bits(W))
    assert np.abs(res["logits"].cpu().numpy() - logits).max() < LOGIT_TOL_TIGHT
    check_reductions(res, logits)


@pytest.mark.parametrize("M,V,H", [(17, 5000, 512), (130, 3000, 256), (300, 4096, 256)])
def test_single_cta_fallback_kernel_matches_oracle_and_pair_kernel(M, V, H, monkeypatch):
    """The one-CTA-per-SM kernel that serves when the scratch cannot hold the pair kernel's partials: forced here."""
    W = rand_bf16((V, H), 0.05, 11); hid = rand_bf16((M, H), 1.0, 12)
    m = make_mirror(lm_cfg(V, H))
    res_pair = m.mirror_lmhead_reduce(hid.cuda(), W.cuda(), want_logits=True)
    monkeypatch.setenv("MIRROR_LM_PAIR_MIN_ROWS", "1000000")      # (tuning values are read when a context is created)
    m1 = make_mirror(lm_cfg(V, H))
    monkeypatch.delenv("MIRROR_LM_PAIR_MIN_ROWS")
    res = m1.mirror_lmhead_reduce(hid.cuda(), W.cuda(), want_logits=True)
    assert m.device_status() == (0, 0) and m1.device_status() == (0, 0)
    logits = O.lmhead_logits(I.bf16_bits(hid), I.bf16_bits(W))
    assert np.abs(res["logits"].cpu().numpy() - logits).max() < LOGIT_TOL_TIGHT
    check_reductions(res, logits)
    # same accumulation order per logit in both kernels (K ascending): the logits agree bit for bit
    assert torch.equal(res["logits"], res_pair["logits"])
    assert torch.equal(res["argmax"], res_pair["argmax"]) and torch.equal(res["maxlogit"], res_pair["maxlogit"])


def test_ties_go_to_lowest_id_and_topk_gather_temperature():
    V, H, M, T = 3000, 256, 12, 0.8
    W = rand_bf16((V, H), 0.05, 5); hid = rand_bf16((M, H), 1.0, 6)
    big = (hid[0].float() * 0.2).to(torch.bfloat16)          # a row strongly aligned with hidden row 0
    for v in (2900, 17, 1500):                               # identical weight rows: identical logits; spread over tiles / CTAs
        W[v] = big
    m = make_mirror(lm_cfg(V, H), temperature=T)
    rows = torch.tensor([0, 3, 11, 5], dtype=torch.int32); toks = torch.tensor([17, 2999, 0, 1500], dtype=torch.int32)
    res = m.mirror_lmhead_reduce(hid.cuda(), W.cuda(), topk=8, gather_row=rows.cuda(), gather_tok=toks.cuda())
    assert m.device_status() == (0, 0)
    logits = O.lmhead_logits(I.bf16_bits(hid), I.bf16_bits(W))
    assert logits[0, 17] == logits[0, 2900] == logits[0, 1500] == logits[0].max()
    assert int(res["argmax"][0]) == 17
    ref, _ = check_reductions(res, logits, T, topk=8)
    tid = res["topk_id"].cpu().numpy(); tlp = res["topk_logprob"].cpu().numpy()
    assert tid[0, :3].tolist() == [17, 1500, 2900]
    for r in range(M):
        if not np.array_equal(tid[r], ref["topk_id"][r]):   # order may differ only between near-equal logits
            assert np.abs(np.sort(logits[r, tid[r]]) - np.sort(logits[r, ref["topk_id"][r]])).max() < LOGIT_TOL_TIGHT
        np.testing.assert_allclose(tlp[r], logits[r, tid[r]] / T - ref["lse"][r], atol=2 * LOGIT_TOL_TIGHT)
    np.testing.assert_allclose(res["gather_logit"].cpu().numpy(), logits[rows.numpy(), toks.numpy()], atol=LOGIT_TOL_TIGHT)


def test_full_vocab_sampled_rows():
    """The bench launch configuration (M = 17, V = 152064, H = 5120): every reduction against the oracle,
    and the logits themselves on sampled columns."""
    cfg = I.CONFIGS["qwen14b"]
    x = I.gen_verify_inputs(cfg, 0, "cuda", layers=1, force_hidden=True)
    m = make_mirror(cfg)
    res = m.mirror_lmhead_reduce(x.hidden, x.W, want_logits=True)
    assert m.device_status() == (0, 0)
    logits = O.lmhead_logits(I.bf16_bits(x.hidden), I.bf16_bits(x.W))
    err = np.abs(res["logits"].cpu().numpy() - logits).max()
    assert err < LOGIT_TOL_TIGHT, err
    _, flips = check_reductions(res, logits)
    print("argmax flips", flips, "max logit err", err)


@pytest.mark.parametrize("M,V,H", [(17, 20000, 512), (392, 6000, 512), (1040, 3000, 256)])
def test_repeated_runs_are_bitwise_equal(M, V, H):
    """Partials are merged in a fixed order whichever CTA pair ran which unit: twelve runs, bit for bit."""
    W = rand_bf16((V, H), 0.05, 21).cuda(); hid = rand_bf16((M, H), 1.0, 22).cuda()
    m = make_mirror(lm_cfg(V, H))
    first = m.mirror_lmhead_reduce(hid, W, want_logits=True)
    first = {k: v.clone() for k, v in first.items() if isinstance(v, torch.Tensor)}
    for _ in range(11):
        res = m.mirror_lmhead_reduce(hid, W, want_logits=True)
        for k, v in first.items():
            assert torch.equal(res[k], v), k
    assert m.device_status() == (0, 0)
