"""The bounded device-side waits, exercised the allowed way: nothing traps, spins without limit or touches bad memory.
A context created with a short wait limit and the test aid that makes a producer stop issuing copies after one stage
(it neither arms the stage's barrier nor issues its copies) runs a small problem: a consumer's wait runs out, the
kernel records MIRROR_ERR_TIMEOUT, every role unwinds (copies in flight are waited for, tensor memory is released
behind the block / cluster barrier) and the launch returns.  The next call on the SAME context is a normal one and
must match the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2510_13161_b200 import inputs as I
from tests.helpers import make_mirror, oracle_attention

pytestmark = pytest.mark.gpu
LIMIT = "4000000"          # SM cycles: about 2 ms


def stalled_mirror(cfg, monkeypatch):
    monkeypatch.setenv("MIRROR_WAIT_LIMIT_CYCLES", LIMIT)
    monkeypatch.setenv("MIRROR_TEST_STALL_AFTER_STAGES", "1")
    m = make_mirror(cfg)                       # tuning values are read when the context is created
    monkeypatch.delenv("MIRROR_WAIT_LIMIT_CYCLES")
    monkeypatch.delenv("MIRROR_TEST_STALL_AFTER_STAGES")
    return m


def test_attention_wait_runs_out_and_the_context_stays_usable(monkeypatch):
    cfg = I.shrink(I.CONFIGS["tiny"], layers=2, batch=2, prefix_lo=500, prefix_hi=700, kappa=3, gamma=4)
    x = I.gen_verify_inputs(cfg, 3, "cuda", with_lm_head=False)
    m = stalled_mirror(cfg, monkeypatch)
    kv = m.kv(x.k_pool, x.v_pool, x.page_table, x.prefix_len)
    tree = m.tree(x.tokens, cfg.kappa, cfg.gamma)
    out = torch.zeros_like(x.q)
    m.mirror_attn_verify(kv, tree, x.q, x.k_new, x.v_new, out=out)          # the K producer stops after one stage
    code, detail = m.device_status()
    assert code == 7, (code, detail)                                        # MIRROR_ERR_TIMEOUT
    assert detail in (10, 20, 21, 23, 24, 30, 32, 33, 34, 35, 36), detail   # one of the attention kernel's waits
    assert m.device_status() == (0, 0)                                      # read once, then cleared
    # the same context, next call: normal, and right
    m.mirror_attn_verify(kv, tree, x.q, x.k_new, x.v_new, out=out)
    assert m.device_status() == (0, 0)
    ref = oracle_attention(x)
    for l in range(cfg.layers):
        r = ref[l][0]
        err = np.abs(out[l].float().cpu().numpy() - r).max()
        assert err <= 1e-2 * np.abs(r).max() + 1e-5, (l, err)


@pytest.mark.parametrize("M", [17, 300])          # a weight stream (two CTAs per SM) and several row chunks
def test_lmhead_pair_wait_runs_out_and_the_context_stays_usable(M, monkeypatch):
    V, H = 6000, 512
    cfg = I.VerifyConfig("t", H, 4, 2, 64, 1, 1, 16, 16, 2, 4, V, "greedy")
    g = torch.Generator().manual_seed(5)
    W = torch.empty((V, H), dtype=torch.bfloat16).normal_(0, 0.05, generator=g).cuda()
    hid = torch.empty((M, H), dtype=torch.bfloat16).normal_(0, 1.0, generator=g).cuda()
    m = stalled_mirror(cfg, monkeypatch)
    m.mirror_lmhead_reduce(hid, W)                                           # both CTAs of every pair stop after one stage
    code, detail = m.device_status()
    assert code == 7, (code, detail)
    assert detail in (11, 12, 13, 16), detail                                # one of the pair kernel's waits
    res = m.mirror_lmhead_reduce(hid, W)
    assert m.device_status() == (0, 0)
    logits = O.lmhead_logits(I.bf16_bits(hid), I.bf16_bits(W))
    red = O.row_reduce(logits)
    got = res["argmax"].cpu().numpy()
    for r in np.nonzero(got != red["argmax"])[0]:
        assert logits[r, red["argmax"][r]] - logits[r, got[r]] < 2e-3
    assert np.abs(res["lse"].cpu().numpy() - red["lse"]).max() <= 2e-3
