"""GPU parity: mirror_accept_select against the oracle's acceptance rules (bit-exact outputs)."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2510_13161_b200 import binding, inputs as I
from tests.helpers import make_mirror

pytestmark = pytest.mark.gpu
FIELDS = ["n_accepted", "best_branch", "decide_row", "n_emitted", "emitted", "accepted_nodes", "reuse_slot"]


def cfg_for(V, kappa, gamma, B):
    return I.VerifyConfig("t", 256, 4, 2, 64, 1, B, 16, 16, kappa, gamma, V, "greedy")


def planted_greedy_case(B, kappa, gamma, V, seed, parent=None):
    """Random tokens / target argmax with agreement planted to random depths on random branches."""
    rng = np.random.default_rng(seed)
    par = I.comb_parent(kappa, gamma) if parent is None else parent
    n = len(par)
    tok = rng.integers(0, V, size=(B, n)).astype(np.int32)
    am = rng.integers(0, V, size=(B, n)).astype(np.int32)
    paths, plen = O.branches(par, gamma)
    for b in range(B):
        for i in range(len(paths)):
            depth = rng.integers(0, plen[i] + 1)
            for j in range(depth):
                c = paths[i, j]
                am[b, par[c]] = tok[b, c]
    return par, tok, am


@pytest.mark.parametrize("kappa,gamma,B", [(2, 4, 1), (4, 4, 3), (8, 6, 8), (8, 8, 16), (1, 7, 2), (8, 7, 1), (1, 1, 1)])
@pytest.mark.parametrize("emit_bonus", [True, False])
def test_greedy_matches_oracle_bit_exact(kappa, gamma, B, emit_bonus):
    V = 97
    m = make_mirror(cfg_for(V, kappa, gamma, B))
    for seed in range(3):
        par, tok, am = planted_greedy_case(B, kappa, gamma, V, seed)
        cand = np.random.default_rng(seed).integers(0, V, size=(B, len(par), 5)).astype(np.int32)
        # make some reuse hits likely
        cand[:, :, 2] = am
        if seed == 1:
            cand[:, :, 2] = -7
        ref = O.accept_greedy(tok, am, par, gamma, emit_bonus, cand)
        tok_d = torch.from_numpy(tok).cuda(); am_d = torch.from_numpy(am).cuda(); cand_d = torch.from_numpy(cand).cuda()
        tree = m.tree(tok_d, kappa, gamma)
        acc = m.accept_in(0, emit_bonus, target_argmax=am_d, cand_ids=cand_d)
        got = m.mirror_accept_select(tree, acc).cpu()
        for f in FIELDS:
            np.testing.assert_array_equal(got[f], ref[f], err_msg=f)
        assert m.device_status() == (0, 0)


def test_greedy_general_tree_and_all_accept():
    V, gamma = 50, 5
    par = [-1, 0, 1, 1, 0, 4, 5, 5, 2, 8, 3]
    m = make_mirror(cfg_for(V, 1, gamma, 4))
    for seed in range(4):
        par_, tok, am = planted_greedy_case(4, 0, gamma, V, seed, parent=par)
        if seed == 3:                       # everything agrees: every branch fully accepted, lowest index wins
            for b in range(4):
                for c in range(1, len(par)):
                    am[b, par[c]] = tok[b, c] = 7
        ref = O.accept_greedy(tok, am, par, gamma)
        tok_d = torch.from_numpy(tok).cuda(); am_d = torch.from_numpy(am).cuda()
        tree = m.tree(tok_d, 0, gamma, parent=par)
        got = m.mirror_accept_select(tree, m.accept_in(0, True, target_argmax=am_d)).cpu()
        for f in FIELDS:
            np.testing.assert_array_equal(got[f], ref[f], err_msg=f)


def spec_case(B, kappa, gamma, V, seed, peaked=False):
    g = torch.Generator().manual_seed(seed)
    n = 1 + kappa * gamma
    logits = torch.randn((B * n, V), generator=g) * (3.0 if peaked else 1.0)
    qp = torch.softmax(torch.randn((B, n - 1, V), generator=g) * (3.0 if peaked else 1.0), -1)
    tok = torch.randint(0, V, (B, n), generator=g, dtype=torch.int32)
    # draw the drafted tokens from q so that acceptance actually happens
    for b in range(B):
        for c in range(1, n):
            tok[b, c] = int(torch.multinomial(qp[b, c - 1], 1, generator=g))
    ua = torch.rand((B, n), generator=g); ur = torch.rand((B, n), generator=g)
    return logits.float(), qp.float(), tok, ua.float(), ur.float()


@pytest.mark.parametrize("kappa,gamma,B,V,T", [(1, 4, 4, 1000, 1.0), (2, 4, 3, 1024, 1.0), (8, 6, 8, 5003, 0.7),
                                               (4, 4, 2, 152064, 1.0), (8, 8, 2, 128256, 1.3)])
def test_spec_sampling_matches_oracle(kappa, gamma, B, V, T):
    m = make_mirror(cfg_for(V, kappa, gamma, B), temperature=T)
    par = I.comb_parent(kappa, gamma)
    accepted_total = 0
    for seed in range(3):
        logits, qp, tok, ua, ur = spec_case(B, kappa, gamma, V, seed, peaked=(seed == 2))
        if seed == 1:
            qp[:, 0] = torch.softmax(logits.view(B, -1, V)[:, 0] / T, -1)     # p == q at the first node: residual has no mass
        lse = torch.logsumexp(logits.double() / T, -1).float()
        cand = torch.topk(logits, 4, dim=-1).indices.to(torch.int32)
        ref = O.accept_spec(tok.numpy(), logits.numpy(), lse.numpy(), qp.numpy(), ua.numpy(), ur.numpy(), par, gamma,
                            True, T, cand.numpy())
        tree = m.tree(tok.cuda(), kappa, gamma)
        acc = m.accept_in(1, True, logits=logits.cuda(), lse=lse.cuda(), q_probs=qp.cuda(), u_accept=ua.cuda(),
                          u_resample=ur.cuda(), cand_ids=cand.cuda())
        got = m.mirror_accept_select(tree, acc).cpu()
        assert m.device_status() == (0, 0)
        for b in range(B):
            same = all(np.array_equal(got[f][b], ref[f][b]) for f in FIELDS)
            # a disagreement is tolerated only on a knife edge of the fp64 decision (exp implementations differ in the last ulp)
            assert same or ref["margin"][b] < 1e-9, (b, ref["margin"][b], {f: (got[f][b], ref[f][b]) for f in FIELDS})
        accepted_total += int(ref["n_accepted"].sum())
    assert accepted_total > 0


def tree_case(B, parent, V, seed, peaked=False, iid_siblings=True):
    """Drafts on an arbitrary tree: the children of a node are independent draws from one q (the lossless setting)
    or each from its own q."""
    g = torch.Generator().manual_seed(seed)
    n = len(parent)
    scale = 3.0 if peaked else 1.0
    logits = torch.randn((B * n, V), generator=g) * scale
    qp = torch.softmax(torch.randn((B, n - 1, V), generator=g) * scale, -1)
    if iid_siblings:
        first_child = {}
        for c in range(1, n):
            first_child.setdefault(parent[c], c)
            qp[:, c - 1] = qp[:, first_child[parent[c]] - 1]
    tok = torch.zeros((B, n), dtype=torch.int32)
    for b in range(B):
        for c in range(1, n):
            tok[b, c] = int(torch.multinomial(qp[b, c - 1], 1, generator=g))
    ua = torch.rand((B, n), generator=g); ur = torch.rand((B, n), generator=g)
    return logits.float(), qp.float(), tok, ua.float(), ur.float()


@pytest.mark.parametrize("shape,B,V,T", [(("comb", 1, 4), 4, 1000, 1.0), (("comb", 4, 4), 6, 1024, 1.0),
                                         (("comb", 8, 6), 8, 5003, 0.7), (("random", 24, 5), 6, 3001, 1.0),
                                         (("wide", 12, 1), 6, 2000, 1.0), (("comb", 8, 8), 2, 128256, 1.3)])
def test_lossless_tree_acceptance_matches_oracle(shape, B, V, T):
    kind, a, b_ = shape
    if kind == "comb":
        par, gamma, kappa = I.comb_parent(a, b_), b_, a
    elif kind == "random":
        par, gamma, kappa = I.random_tree_parent(a, 3, max_depth=b_), b_, 0
    else:                                   # one level of many siblings
        par, gamma, kappa = [-1] + [0] * a, 1, 0
    n = len(par)
    m = make_mirror(cfg_for(V, 1, n - 1, B), temperature=T)
    accepted_total = rejected_siblings = 0
    for seed in range(4):
        logits, qp, tok, ua, ur = tree_case(B, par, V, seed, peaked=(seed == 2), iid_siblings=(seed != 3))
        if seed == 1:
            qp[:, 0] = torch.softmax(logits.view(B, -1, V)[:, 0] / T, -1)     # p == q at the first node: residual has no mass
        lse = torch.logsumexp(logits.double() / T, -1).float()
        cand = torch.topk(logits, 4, dim=-1).indices.to(torch.int32)
        ref = O.accept_tree(tok.numpy(), logits.numpy(), lse.numpy(), qp.numpy(), ua.numpy(), ur.numpy(), par, gamma,
                            True, T, cand.numpy())
        tree = m.tree(tok.cuda(), kappa, gamma, parent=par)
        acc = m.accept_in(binding.ACCEPT_SPEC_TREE, True, logits=logits.cuda(), lse=lse.cuda(), q_probs=qp.cuda(),
                          u_accept=ua.cuda(), u_resample=ur.cuda(), cand_ids=cand.cuda())
        got = m.mirror_accept_select(tree, acc, tree_scratch=(seed % 2 == 0)).cpu()      # with and without the fp64 scratch
        assert m.device_status() == (0, 0)
        for b in range(B):
            same = all(np.array_equal(got[f][b], ref[f][b]) for f in FIELDS)
            # a disagreement is tolerated only on a knife edge of the fp64 decision (the normalisers are summed in a
            # different order, exp implementations differ in the last ulp)
            assert same or ref["margin"][b] < 1e-9, (b, ref["margin"][b], {f: (got[f][b], ref[f][b]) for f in FIELDS})
        accepted_total += int(ref["n_accepted"].sum())
        rejected_siblings += int((ref["n_accepted"] == 0).sum())
    assert accepted_total > 0 and rejected_siblings > 0


def test_spec_root_only_tree_draws_from_the_root_row():
    V, B = 777, 5
    m = make_mirror(cfg_for(V, 0, 0, B))
    g = torch.Generator().manual_seed(0)
    logits = torch.randn((B, V), generator=g)
    lse = torch.logsumexp(logits.double(), -1).float()
    tok = torch.zeros((B, 1), dtype=torch.int32)
    ua = torch.rand((B, 1), generator=g); ur = torch.rand((B, 1), generator=g)
    ref = O.accept_spec(tok.numpy(), logits.numpy(), lse.numpy(), np.zeros((B, 0, V), np.float32), ua.numpy(), ur.numpy(), [-1], 0)
    tree = m.tree(tok.cuda(), 0, 0)
    acc = m.accept_in(1, True, logits=logits.cuda(), lse=lse.cuda(), u_accept=ua.cuda(), u_resample=ur.cuda())
    got = m.mirror_accept_select(tree, acc).cpu()
    for f in ("n_accepted", "n_emitted", "decide_row", "reuse_slot"):
        np.testing.assert_array_equal(got[f], ref[f])
    np.testing.assert_array_equal(got["emitted"][:, 0], ref["emitted"][:, 0])


def test_bad_arguments_are_rejected_on_the_host():
    from paper_2510_13161_b200.binding import MirrorError
    m = make_mirror(cfg_for(100, 2, 2, 1))
    tok = torch.zeros((1, 5), dtype=torch.int32).cuda()
    with pytest.raises(MirrorError) as e:
        m.mirror_accept_select(m.tree(tok, 2, 2), m.accept_in(0, True))        # no target_argmax
    assert e.value.code == 1
    with pytest.raises(MirrorError) as e:
        m.mirror_accept_select(m.tree(tok, 3, 2), m.accept_in(0, True, target_argmax=tok))   # n != 1 + kappa*gamma
    assert e.value.code == 2
    with pytest.raises(MirrorError) as e:
        m.mirror_accept_select(m.tree(tok, 0, 2, parent=[-1, 0, 2, 1, 0]), m.accept_in(0, True, target_argmax=tok))
    assert e.value.code == 2


def test_deduplicated_tree_commits_the_same_tokens_as_the_comb_tree():
    """kappa branches that share prefixes: verifying the tree of distinct prefixes (mirror_trie_build) commits exactly
    what verifying the kappa separate chains commits, with fewer rows to score."""
    V, kappa, gamma, B = 11, 6, 5, 1
    m = make_mirror(cfg_for(V, kappa, gamma, B))
    rng = np.random.default_rng(5)
    fewer = 0
    for trial in range(20):
        bt = rng.integers(0, 3, size=(kappa, gamma)).astype(np.int32)           # tiny alphabet: many shared prefixes
        root = int(rng.integers(0, V))
        parent, tokens, node_of = binding.mirror_trie_build(bt, root)
        n_t = len(parent)
        fewer += (1 + kappa * gamma) - n_t
        # the target's greedy token per tree node; a row of the comb tree that repeats a prefix sees the same one
        am_t = rng.integers(0, 3, size=(B, n_t)).astype(np.int32)
        am_c = np.zeros((B, 1 + kappa * gamma), np.int32)
        am_c[:, 0] = am_t[:, 0]
        for i in range(kappa):
            for j in range(gamma):
                am_c[:, 1 + i * gamma + j] = am_t[:, node_of[i][j]]
        tok_c = np.concatenate([[root], bt.reshape(-1)]).astype(np.int32)[None, :]
        tok_t = np.asarray(tokens, np.int32)[None, :]
        tree_c = m.tree(torch.from_numpy(tok_c).cuda(), kappa, gamma)
        tree_t = m.tree(torch.from_numpy(tok_t).cuda(), 0, gamma, parent=parent)
        got_c = m.mirror_accept_select(tree_c, m.accept_in(0, True, target_argmax=torch.from_numpy(am_c).cuda())).cpu()
        got_t = m.mirror_accept_select(tree_t, m.accept_in(0, True, target_argmax=torch.from_numpy(am_t).cuda())).cpu()
        ref_t = O.accept_greedy(tok_t, am_t, parent, gamma)
        for f in FIELDS:
            np.testing.assert_array_equal(got_t[f], ref_t[f], err_msg=f)
        np.testing.assert_array_equal(got_t["n_accepted"], got_c["n_accepted"])
        np.testing.assert_array_equal(got_t["n_emitted"], got_c["n_emitted"])
        np.testing.assert_array_equal(got_t["emitted"], got_c["emitted"])
        # the accepted path is the same sequence of tokens, node ids differ
        a = int(got_t["n_accepted"][0])
        path_t = [int(tok_t[0, v]) for v in got_t["accepted_nodes"][0][:a]]
        path_c = [int(tok_c[0, v]) for v in got_c["accepted_nodes"][0][:a]]
        assert path_t == path_c
    assert fewer > 0
    assert m.device_status() == (0, 0)
