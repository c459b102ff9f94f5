"""Early-exit tap (Eq. 5, Eq. 6), overlap mass (Eq. 7) and the reuse decision end to end against the oracle."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2510_13161_b200 import binding, inputs as I
from tests.helpers import make_mirror

pytestmark = pytest.mark.gpu


def cfg_for(V, H, kappa, gamma, B):
    return I.VerifyConfig("ee", H, 4, 2, 64, 1, B, 16, 16, kappa, gamma, V, "greedy")


@pytest.mark.parametrize("M,V,H,kappa,T", [(9, 3000, 256, 4, 1.0), (17, 152064, 512, 8, 1.0), (40, 5003, 256, 8, 0.7)])
def test_tap_message_and_overlap_mass_match_oracle(M, V, H, kappa, T):
    g = torch.Generator().manual_seed(M)
    hid_e = (torch.randn((M, H), generator=g) * 1.0).to(torch.bfloat16)        # early-exit hidden rows
    hid_f = (hid_e.float() + 0.5 * torch.randn((M, H), generator=g)).to(torch.bfloat16)   # final rows: correlated with them
    W = (torch.randn((V, H), generator=g) * 0.05).to(torch.bfloat16)
    m = make_mirror(cfg_for(V, H, 1, M - 1, 1), temperature=T)
    ids, lp = m.mirror_early_exit_tap(hid_e.cuda(), W.cuda(), kappa)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    # oracle: fp64 logits of the early-exit rows, Top-kappa by (logit descending, id ascending), log-probs at temperature T
    logits_e = O.lmhead_logits(I.bf16_bits(hid_e), I.bf16_bits(W))
    ref = O.row_reduce(logits_e, T, kappa)
    ids_h = ids.cpu().numpy(); lp_h = lp.float().cpu().numpy()
    for r in range(M):
        if not np.array_equal(ids_h[r], ref["topk_id"][r]):       # order may differ only between near-equal logits
            assert np.abs(np.sort(logits_e[r, ids_h[r]]) - np.sort(logits_e[r, ref["topk_id"][r]])).max() < 2e-3
        want = logits_e[r, ids_h[r]] / T - ref["lse"][r]
        np.testing.assert_allclose(lp_h[r], want, rtol=2 ** -8, atol=3e-3)     # bf16 payload
    # overlap mass of the message under the final distribution
    fin = m.mirror_lmhead_reduce(hid_f.cuda(), W.cuda(), want_logits=True)
    omega = m.mirror_overlap_mass(fin["logits"], fin["lse"], ids).cpu().numpy()
    assert m.device_status() == (0, 0)
    logits_f = O.lmhead_logits(I.bf16_bits(hid_f), I.bf16_bits(W))
    q = np.exp(logits_f / T - np.log(np.exp(logits_f / T - (logits_f / T).max(1, keepdims=True)).sum(1, keepdims=True)) - (logits_f / T).max(1, keepdims=True))
    want_omega = np.array([O.overlap_mass(q[r], ids_h[r]) for r in range(M)])
    np.testing.assert_allclose(omega, want_omega, rtol=2e-3, atol=1e-6)
    assert (omega > 0).all() and (omega <= 1 + 1e-5).all()
    # Omega grows with kappa (Proposition 1): the message of kappa ids contains the message of fewer ids
    ids2, _ = m.mirror_early_exit_tap(hid_e.cuda(), W.cuda(), max(1, kappa // 2))
    omega2 = m.mirror_overlap_mass(fin["logits"], fin["lse"], ids2).cpu().numpy()
    assert (omega2 <= omega + 1e-6).all()


def test_reuse_decision_follows_the_message_end_to_end():
    """Tap on early-exit rows -> message ids as cand_ids of the acceptance -> reuse_slot is the position of the
    correction / bonus token in the deciding row's message, or -1 (fallback) when the message misses it."""
    V, H, kappa, gamma, B = 4001, 256, 4, 3, 6
    cfg = cfg_for(V, H, 2, gamma, B)
    n = cfg.n_nodes
    g = torch.Generator().manual_seed(11)
    hid_f = torch.randn((B * n, H), generator=g).to(torch.bfloat16)
    hid_e = (hid_f.float() + 0.8 * torch.randn((B * n, H), generator=g)).to(torch.bfloat16)
    W = (torch.randn((V, H), generator=g) * 0.05).to(torch.bfloat16)
    m = make_mirror(cfg)
    ids, _ = m.mirror_early_exit_tap(hid_e.cuda(), W.cuda(), kappa)
    fin = m.mirror_lmhead_reduce(hid_f.cuda(), W.cuda())
    am = fin["argmax"].cpu().numpy().reshape(B, n)
    tok = torch.randint(0, V, (B, n), generator=g, dtype=torch.int32)
    par = I.comb_parent(2, gamma)
    for b in range(B):                                   # plant agreement of different depths on branch b % 2
        r = 0
        for j in range(b % (gamma + 1)):
            c = 1 + (b % 2) * gamma + j
            tok[b, c] = int(am[b, r]); r = c
    tree = m.tree(tok.cuda(), 2, gamma)
    acc = m.accept_in(binding.ACCEPT_GREEDY, True, target_argmax=fin["argmax"], cand_ids=ids)
    got = m.mirror_accept_select(tree, acc).cpu()
    ref = O.accept_greedy(tok.numpy(), am, par, gamma, cand_ids=ids.cpu().numpy())
    for f in ("n_accepted", "best_branch", "decide_row", "n_emitted", "emitted", "accepted_nodes", "reuse_slot"):
        np.testing.assert_array_equal(got[f], ref[f], err_msg=f)
    ids_h = ids.cpu().numpy().reshape(B, n, kappa)
    reused = 0
    for b in range(B):
        R, extra = int(got["decide_row"][b]), int(got["emitted"][b, got["n_emitted"][b] - 1])
        where = np.nonzero(ids_h[b, R] == extra)[0]
        assert got["reuse_slot"][b] == (where[0] if len(where) else -1)
        reused += int(got["reuse_slot"][b] >= 0)
    assert reused > 0
