"""Pins for the oracle's acceptance rules (O3, O3'): the greedy operator against a literal
set-comprehension over every input of a tiny case, fixed cases, the Fig. 1 example, exact
integration of the speculative-sampling rule (losslessness for one branch), the reuse
probability of Proposition 1, and the lossless rule over sibling sets of a tree (exact integration
for two and three independent siblings, the chain special case, fixed walk-order cases)."""
import itertools
import os

import numpy as np
import pytest

from oracle import oracle as O
from paper_2510_13161_b200.inputs import comb_parent

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def literal_accept_len(draft, target):
    """Eq. 3 as printed: the largest r in {0..gamma} with draft_j == target_j for all j <= r."""
    gamma = len(draft)
    return max(r for r in range(gamma + 1) if all(draft[j] == target[j] for j in range(r)))


def test_greedy_rule_exhaustively_on_a_tiny_case():
    V, kappa, gamma = 3, 2, 2
    parent = comb_parent(kappa, gamma)           # nodes: 0 | 1,2 | 3,4
    n = len(parent)
    toks, ams = [], []
    for tok in itertools.product(range(V), repeat=n - 1):
        for am in itertools.product(range(V), repeat=n):
            toks.append((0,) + tok); ams.append(am)
    toks = np.array(toks, np.int32); ams = np.array(ams, np.int32)
    o = O.accept_greedy(toks, ams, parent, gamma)
    for k in range(len(toks)):
        tok, am = toks[k], ams[k]
        lens = []
        for i in range(kappa):
            nodes = [1 + i * gamma + j for j in range(gamma)]
            draft = [tok[c] for c in nodes]
            target = [am[parent[c]] for c in nodes]      # row of the parent checks the child
            lens.append(literal_accept_len(draft, target))
        A = max(lens)
        best = min(i for i in range(kappa) if lens[i] == A)
        R = 0 if A == 0 else 1 + best * gamma + A - 1
        assert o["n_accepted"][k] == A
        assert o["best_branch"][k] == best
        assert o["decide_row"][k] == R
        assert o["n_emitted"][k] == A + 1
        exp = [tok[1 + best * gamma + j] for j in range(A)] + [am[R]]
        assert o["emitted"][k, :A + 1].tolist() == exp
        assert (o["emitted"][k, A + 1:] == -1).all()
        assert o["accepted_nodes"][k, :A].tolist() == [1 + best * gamma + j for j in range(A)]


def test_greedy_fixed_cases():
    kappa, gamma = 2, 3
    parent = comb_parent(kappa, gamma)
    n = len(parent)
    am = np.array([[5, 6, 7, 8, 1, 1, 1]], np.int32)
    # all-accept on branch 0: bonus token from the last node's row
    tok = np.array([[0, 5, 6, 7, 9, 9, 9]], np.int32)
    o = O.accept_greedy(tok, am, parent, gamma)
    assert (o["n_accepted"][0], o["best_branch"][0], o["decide_row"][0], o["n_emitted"][0]) == (3, 0, 3, 4)
    assert o["emitted"][0].tolist() == [5, 6, 7, 8]
    o = O.accept_greedy(tok, am, parent, gamma, emit_bonus=False)
    assert o["n_emitted"][0] == 3 and o["emitted"][0].tolist() == [5, 6, 7, -1]
    # first-token reject everywhere: A = 0, branch 0, correction = argmax of the root row
    tok = np.array([[0, 4, 6, 7, 4, 1, 1]], np.int32)
    o = O.accept_greedy(tok, am, parent, gamma)
    assert (o["n_accepted"][0], o["best_branch"][0], o["decide_row"][0]) == (0, 0, 0)
    assert o["emitted"][0].tolist() == [5, -1, -1, -1]
    # two identical branches: the lower index wins
    am2 = np.array([[5, 6, 0, 0, 6, 0, 0]], np.int32)
    tok = np.array([[0, 5, 6, 2, 5, 6, 2]], np.int32)
    o = O.accept_greedy(tok, am2, parent, gamma)
    assert (o["n_accepted"][0], o["best_branch"][0], o["decide_row"][0]) == (2, 0, 2)
    # the longer agreement wins even on the higher branch index
    tok = np.array([[0, 5, 9, 2, 5, 6, 2]], np.int32)
    o = O.accept_greedy(tok, am2, parent, gamma)
    assert (o["n_accepted"][0], o["best_branch"][0], o["decide_row"][0]) == (2, 1, 5)
    assert o["accepted_nodes"][0].tolist() == [4, 5, -1]
    # a mismatch hides later matches (prefix semantics, not a count of matches)
    tok = np.array([[0, 4, 6, 7, 4, 1, 1]], np.int32)
    assert O.accept_greedy(tok, am, parent, gamma)["n_accepted"][0] == 0


def read_golden(name):
    d = {}
    for line in open(os.path.join(GOLDEN, name)):
        if line.startswith("#") or ":" not in line:
            continue
        k, v = line.split(":", 1)
        d[k.strip()] = [int(t) for t in v.split()]
    return d


def test_fig1_worked_example():
    g = read_golden("fig1_example.txt")
    gamma, kappa = g["gamma"][0], g["kappa"][0]
    parent = comb_parent(kappa, gamma)
    tok = np.array([[0] + g["draft_window"]], np.int32)
    # row r holds the target's token for the position after node r (root row checks the first draft token)
    am = np.array([g["target_tokens"]], np.int32)
    for cands, want in ((g["candidates_with_reuse"], g["expected_reuse_slot_with"][0]),
                        (g["candidates_without_reuse"], g["expected_reuse_slot_without"][0])):
        cand = np.tile(np.array(cands, np.int32), (1, len(parent), 1))
        o = O.accept_greedy(tok, am, parent, gamma, cand_ids=cand)
        assert o["n_accepted"][0] == g["expected_accepted"][0]
        A = o["n_accepted"][0]
        assert o["emitted"][0, :A + 1].tolist() == g["expected_emitted"]
        assert o["emitted"][0, A] == g["expected_correction"][0]
        assert o["decide_row"][0] == 2          # the correction sits at 0-based depth tau = 2
        assert o["reuse_slot"][0] == want


# ---------------------------------------------------------------------------------------------
# speculative sampling
# ---------------------------------------------------------------------------------------------
def spec_inputs_chain(p_rows, q_rows, xs, u_acc, u_res):
    """One request: a chain root -> node1 -> ... ; p_rows[r] is row r's target distribution,
    q_rows[c-1] node c's draft distribution, xs the drafted tokens."""
    n = len(xs) + 1
    logits = np.log(np.maximum(np.array(p_rows, np.float64), 1e-300)).astype(np.float32)
    lse = np.zeros(n, np.float32)
    return (np.array([0] + list(xs), np.int32), logits, lse, np.array(q_rows, np.float32),
            np.array(u_acc, np.float32), np.array(u_res, np.float32))


def batch_spec(items, parent, gamma, **kw):
    tok = np.stack([i[0] for i in items]); logits = np.stack([i[1] for i in items]).reshape(-1, items[0][1].shape[-1])
    lse = np.concatenate([i[2] for i in items]); q = np.stack([i[3] for i in items])
    ua = np.stack([i[4] for i in items]); ur = np.stack([i[5] for i in items])
    return O.accept_spec(tok, logits, lse, q, ua, ur, parent, gamma, **kw)


def test_spec_rule_is_lossless_for_one_branch_exact_integration():
    # gamma = 1, kappa = 1, |V| = 4.  p, q are sixteenths; every boundary of the rule (accept
    # thresholds p/q in {1/4, 1/3}, residual CDF steps in sevenths) lies on a grid edge, so the
    # midpoint rule integrates the emitted-token law exactly: it must equal p (the speculative
    # sampling theorem of the works the paper cites for its lossless claim, Sec. 4.1).
    p = np.array([1, 5, 2, 8]) / 16.0
    q = np.array([4, 4, 6, 2]) / 16.0
    Na, Nr = 12, 7
    parent = comb_parent(1, 1)
    items, weights = [], []
    for x in range(4):
        for a in range(Na):
            for r in range(Nr):
                ua, ur = (a + 0.5) / Na, (r + 0.5) / Nr
                items.append(spec_inputs_chain([p, p], [q], [x], [0.0, ua], [ur, ur]))
                weights.append(q[x] / (Na * Nr))
    o = batch_spec(items, parent, 1)
    w = np.array(weights)
    law = np.zeros(4)
    for k in range(len(items)):
        law[o["emitted"][k, 0]] += w[k]
    np.testing.assert_allclose(law, p, atol=1e-12)
    # P[accept] = sum_v min(p_v, q_v)
    np.testing.assert_allclose((w * (o["n_accepted"] == 1)).sum(), np.minimum(p, q).sum(), atol=1e-12)
    assert (o["n_emitted"] == o["n_accepted"] + 1).all()


def test_spec_rule_two_step_chain_law():
    # gamma = 2: the first emitted token follows p0; given that the draft's first token v was
    # accepted, the second emitted token follows the row of that node, p1.
    V = 4
    p0 = np.array([1, 5, 2, 8]) / 16.0; q1 = np.array([4, 4, 6, 2]) / 16.0
    p1 = np.array([6, 2, 7, 1]) / 16.0; q2 = np.array([2, 8, 3, 3]) / 16.0
    p2 = np.array([3, 3, 5, 5]) / 16.0
    parent = comb_parent(1, 2)
    items, weights = [], []
    # accept thresholds: p0/q1 in {1/4, 1/3}, p1/q2 in {1/4, 1/3}: a 12-cell grid holds them all.
    # CDF steps: residual of row 0 in 7ths, of row 1 in 8ths, bonus row p2 in 16ths: 112 = lcm(7, 8, 16).
    sub = [(a + 0.5) / 12 for a in range(12)]
    res_grid = [(r + 0.5) / 112 for r in range(112)]
    for x1 in range(V):
        for x2 in range(V):
            for ua1 in sub:
                for ua2 in sub:
                    for ur in res_grid:
                        items.append(spec_inputs_chain([p0, p1, p2], [q1, q2], [x1, x2], [0.0, ua1, ua2], [ur, ur, ur]))
                        weights.append(q1[x1] * q2[x2] / (12 * 12 * 112))
    o = batch_spec(items, parent, 2)
    w = np.array(weights)
    law1 = np.zeros(V); joint = np.zeros((V, V)); law3 = np.zeros(V)
    for k in range(len(items)):
        e = o["emitted"][k]
        law1[e[0]] += w[k]
        if o["n_accepted"][k] >= 1:
            joint[e[0], e[1]] += w[k]
        if o["n_accepted"][k] == 2:
            law3[e[2]] += w[k]
    np.testing.assert_allclose(law1, p0, atol=1e-12)
    acc1 = np.minimum(p0, q1)
    np.testing.assert_allclose(joint, acc1[:, None] * p1[None, :], atol=1e-12)
    # all accepted: the bonus token follows the last node's row
    np.testing.assert_allclose(law3, acc1.sum() * np.minimum(p1, q2).sum() * p2, atol=1e-12)


def test_spec_rule_special_cases():
    parent = comb_parent(1, 1)
    p = np.array([0.1, 0.2, 0.3, 0.4])
    # p == q: always accept, whatever u
    for u in (0.0, 0.5, 0.999999):
        for x in range(4):
            o = batch_spec([spec_inputs_chain([p, p], [p], [x], [0, u], [0.3, 0.3])], parent, 1)
            assert o["n_accepted"][0] == 1 and o["emitted"][0, 0] == x
    # q one-hot on a token the target gives zero mass: always reject, correction ~ p (residual == p)
    pz = np.array([0.0, 0.5, 0.25, 0.25]); q = np.array([1.0, 0, 0, 0])
    cdf = np.cumsum(pz)
    for ur in (0.01, 0.49, 0.51, 0.74, 0.76, 0.99):
        o = batch_spec([spec_inputs_chain([pz, pz], [q], [0], [0, 0.5], [ur, ur])], parent, 1)
        assert o["n_accepted"][0] == 0
        assert o["emitted"][0, 0] == int(np.searchsorted(cdf, ur, side="right"))
    # u = 0 accepts anything the target gives positive mass
    o = batch_spec([spec_inputs_chain([p, p], [np.array([0.97, 0.01, 0.01, 0.01])], [0], [0, 0.0], [0.3, 0.3])], parent, 1)
    assert o["n_accepted"][0] == 1


def spec_inputs_tree(p_rows, q_rows, xs, u_acc, u_res):
    """One request over an arbitrary tree: p_rows[r] is the target distribution of node r's row, q_rows[c] node c's
    draft distribution (c >= 1), xs[c] its token, u_acc[c] the uniform of its accept test, u_res[r] the uniform of an
    extra token drawn at row r."""
    n = len(xs)
    logits = np.log(np.maximum(np.array(p_rows, np.float64), 1e-300)).astype(np.float32)
    return (np.array(xs, np.int32), logits, np.zeros(n, np.float32), np.array(q_rows[1:], np.float32),
            np.array(u_acc, np.float32), np.array(u_res, np.float32))


def test_spec_rule_over_several_branches_hand_worked_cases():
    """The independent per-branch rule for kappa > 1 (each branch tested as a chain with its own uniforms, the longest
    wins, ties and A = 0 go to the lowest branch, the extra token is drawn at the chosen branch's deciding row from the
    residual against the draft distribution of THAT branch's first rejected node).  Expected values are worked by hand
    with deterministic devices: u_accept = 0 always passes; a token the target gives no mass always fails.
    Tree: kappa = 3, gamma = 2; nodes 0 | 1,2 | 3,4 | 5,6."""
    parent = comb_parent(3, 2)
    V = 4
    P0 = [0.0, 0.5, 0.25, 0.25]            # a row that gives token 0 no mass
    PA = [0.1, 0.2, 0.3, 0.4]
    QA = [0.5, 0.5, 0.0, 0.0]              # residual of P0 against QA: [0, 0, .25, .25]
    QB = [0.5, 0.0, 0.5, 0.0]              # residual of P0 against QB: [0, .5, 0, .25]
    flat = [0.25] * 4

    def run(p_rows, q_rows, xs, u_acc, u_res, **kw):
        return batch_spec([spec_inputs_tree(p_rows, q_rows, xs, u_acc, u_res)], parent, 2, **kw)

    def check(o, A, best, R, emitted, nodes):
        assert o["n_accepted"][0] == A and o["best_branch"][0] == best and o["decide_row"][0] == R
        assert o["n_emitted"][0] == len(emitted)
        assert o["emitted"][0].tolist() == emitted + [-1] * (3 - len(emitted))
        assert o["accepted_nodes"][0].tolist() == nodes + [-1] * (2 - len(nodes))

    # 1. every branch accepts its first node and fails its second: tie at A = 1 -> branch 0.  Deciding row = node 1;
    #    rejected node 2 proposed token 0 from QA; residual [0, 0, .25, .25], Z = .5, u_res[1] = .6 -> threshold .3 -> id 3.
    #    (QB, the other branches' distribution, would give id 1; u_res of another row (.1) id 2.)
    p_rows = [PA, P0, PA, P0, PA, P0, PA]
    q_rows = [None, flat, QA, flat, QB, flat, QB]
    xs = [0, 1, 0, 2, 0, 3, 0]
    u_acc = [0, 0.0, 0.5, 0.0, 0.5, 0.0, 0.5]
    u_res = [0.1, 0.6, 0.1, 0.1, 0.1, 0.1, 0.1]
    check(run(p_rows, q_rows, xs, u_acc, u_res), 1, 0, 1, [1, 3], [1])

    # 2. the longer branch sits at the highest index: branch 0 accepts one node, branch 1 none, branch 2 both.
    #    Whole branch accepted -> bonus from the last node's own row PA with u_res[6] = .35: cdf .1 .3 .6 -> id 2.
    p_rows = [PA, P0, PA, PA, PA, PA, PA]
    q_rows = [None, flat, QA, [0, 0, 0, 1.0], flat, flat, flat]
    xs = [0, 1, 0, 3, 1, 2, 3]
    u_acc = [0, 0.0, 0.5, 0.99, 0.0, 0.0, 0.0]          # node 3: .99 * 1 > PA[3] = .4 fails
    u_res = [0.9, 0.9, 0.9, 0.9, 0.9, 0.9, 0.35]
    check(run(p_rows, q_rows, xs, u_acc, u_res), 2, 2, 6, [2, 3, 2], [5, 6])
    #    the same with emit_bonus off: nothing beyond the accepted tokens
    check(run(p_rows, q_rows, xs, u_acc, u_res, emit_bonus=False), 2, 2, 6, [2, 3], [5, 6])

    # 3. every branch fails at depth 0: A = 0, branch 0, deciding row = root; the residual uses branch 0's first node's
    #    distribution (QA -> [0, 0, .25, .25]) and u_res[root] = .6 -> id 3; QB of branches 1, 2 would give id 1.
    p_rows = [P0, PA, PA, PA, PA, PA, PA]
    q_rows = [None, QA, flat, QB, flat, QB, flat]
    xs = [0, 0, 1, 0, 1, 0, 1]
    u_acc = [0, 0.5, 0.0, 0.5, 0.0, 0.5, 0.0]
    u_res = [0.6, 0.1, 0.1, 0.1, 0.1, 0.1, 0.1]
    check(run(p_rows, q_rows, xs, u_acc, u_res), 0, 0, 0, [3], [])

    # 4. the winner is branch 1, rejected at depth 1: deciding row = node 3, residual of its row P0 against node 4's QA
    #    with u_res[3] = .6 -> id 3 (node 2's or node 6's QB would give id 1; u_res of rows 0, 1, 5 (.1) id 2).
    p_rows = [P0, PA, PA, P0, PA, PA, PA]
    q_rows = [None, QB, QB, flat, QA, QB, QB]
    xs = [0, 0, 1, 2, 0, 0, 1]
    u_acc = [0, 0.5, 0.0, 0.0, 0.5, 0.5, 0.0]           # nodes 1 and 5 propose token 0 (no mass at the root): fail
    u_res = [0.1, 0.1, 0.1, 0.6, 0.1, 0.1, 0.1]
    check(run(p_rows, q_rows, xs, u_acc, u_res), 1, 1, 3, [2, 3], [3])

    # 5. the accept test of a node reads ITS OWN uniform and its PARENT's row: node 4 (branch 1, depth 1) proposes
    #    token 3 from a one-hot q; the parent row PA gives it .4: u = .39 passes, u = .41 fails.
    p_rows = [PA, PA, PA, PA, P0, PA, PA]               # node 4's own row gives token 3 mass .25: not the one tested
    q_rows = [None, flat, flat, flat, [0, 0, 0, 1.0], flat, flat]
    xs = [0, 0, 0, 1, 3, 0, 0]
    for u4, A in ((0.39, 2), (0.41, 1)):
        u_acc = [0, 0.99, 0.99, 0.0, u4, 0.99, 0.99]    # nodes 1, 5: .99 * .25 > PA[0] = .1 fail
        o = run(p_rows, q_rows, xs, u_acc, [0.5] * 7)
        assert o["n_accepted"][0] == A and o["best_branch"][0] == 1


def test_spec_rule_generic_grid_is_close_to_p():
    # the same law on values that are not grid-aligned: midpoint integration, tolerance ~ 1/N
    rng = np.random.default_rng(3)
    p = rng.dirichlet(np.ones(5)); q = rng.dirichlet(np.ones(5))
    parent = comb_parent(1, 1)
    N = 200
    items, weights = [], []
    for x in range(5):
        for a in range(N):
            for r in range(N):
                items.append(spec_inputs_chain([p, p], [q], [x], [0, (a + 0.5) / N], [(r + 0.5) / N] * 2))
                weights.append(q[x] / N / N)
    o = batch_spec(items, parent, 1)
    law = np.bincount(o["emitted"][:, 0], weights=np.array(weights), minlength=5)
    np.testing.assert_allclose(law, p, atol=2.0 / N)


def test_spec_temperature_uses_scaled_logits():
    # with lse given for logits/T, the accept test compares against Softmax(logits/T)
    parent = comb_parent(1, 1)
    logits = np.array([[1.0, 2.0, 0.5, -1.0]] * 2, np.float32)
    T = 2.0
    pT = np.exp(logits[0] / T); pT /= pT.sum()
    lse = np.full(2, np.log(np.exp(logits[0].astype(np.float64) / T).sum()), np.float32)
    q = np.array([[[0.25, 0.25, 0.25, 0.25]]], np.float32)
    x = 3                                         # p/q = pT[3]/0.25 < 1
    thr = pT[x] / 0.25
    for u, want in ((thr * 0.99, 1), (thr * 1.01, 0)):
        o = O.accept_spec(np.array([[0, x]], np.int32), logits, lse, q, np.array([[0, u]], np.float32),
                          np.array([[0.5, 0.5]], np.float32), parent, 1, temperature=T)
        assert o["n_accepted"][0] == want


def test_reuse_probability_equals_overlap_mass():
    # Proposition 1: with A = 0 reuse succeeds iff the target's token is in the early-exit Top-kappa
    # set, so P[reuse] = Omega_kappa.  A root-only tree draws the token from the root row.
    rng = np.random.default_rng(5)
    V = 8
    final = np.array([3, 1, 4, 1, 5, 9, 2, 7]) / 32.0
    early_logits = np.log(final)[None] + rng.normal(size=(1, V))
    N = 32                                       # CDF steps of `final` are 32nds
    prev = -1.0
    for kappa in (1, 2, 4, 8):
        ids = O.row_reduce(early_logits, topk=kappa)["topk_id"][0]
        omega = O.overlap_mass(final, ids)
        B = N
        tok = np.zeros((B, 1), np.int32)
        logits = np.tile(np.log(final).astype(np.float32), (B, 1))
        o = O.accept_spec(tok, logits, np.zeros(B, np.float32), np.zeros((B, 0, V), np.float32),
                          np.zeros((B, 1), np.float32), ((np.arange(B) + 0.5) / N).astype(np.float32)[:, None],
                          [-1], 1, cand_ids=np.tile(ids, (B, 1, 1)))
        p_reuse = (o["reuse_slot"] >= 0).mean()
        assert abs(p_reuse - omega) < 1e-12
        assert p_reuse >= prev                    # monotone in kappa; reaches 1 at kappa = |V|
        prev = p_reuse
    assert prev == 1.0


def test_branches_of_general_tree():
    parent = [-1, 0, 1, 1, 0, 4]
    paths, plen = O.branches(parent, 3)
    assert paths.tolist() == [[1, 2, -1], [1, 3, -1], [4, 5, -1]]
    assert plen.tolist() == [2, 2, 2]
    with pytest.raises(ValueError):
        O.tree([-1, 1])


# ---------------------------------------------------------------------------------------------
# O3'': lossless acceptance over a tree (sequential multi-round rejection over siblings)
# ---------------------------------------------------------------------------------------------
def tree_inputs(p_rows, q_rows, xs, u_acc, u_res):
    """One request on an arbitrary tree: p_rows[r] row r's target distribution, q_rows[c-1] node c's draft
    distribution, xs[c-1] node c's token."""
    n = len(xs) + 1
    logits = np.log(np.maximum(np.array(p_rows, np.float64), 1e-300)).astype(np.float32)
    return (np.array([0] + list(xs), np.int32), logits, np.zeros(n, np.float32), np.array(q_rows, np.float32),
            np.array(u_acc, np.float32), np.array(u_res, np.float32))


def batch_tree(items, parent, max_len, **kw):
    tok = np.stack([i[0] for i in items]); logits = np.stack([i[1] for i in items]).reshape(-1, items[0][1].shape[-1])
    lse = np.concatenate([i[2] for i in items]); q = np.stack([i[3] for i in items])
    ua = np.stack([i[4] for i in items]); ur = np.stack([i[5] for i in items])
    return O.accept_tree(tok, logits, lse, q, ua, ur, parent, max_len, **kw)


@pytest.mark.parametrize("p16,q16,m,grids", [
    # thresholds of sibling 1: p/q in {1/4, 1/3} (12 cells); of sibling 2: residual/q = 4/7 (7 cells); the last
    # residual is a point mass
    ([1, 5, 2, 8], [4, 4, 6, 2], 2, (12, 7, 3)),
    ([1, 5, 2, 8], [4, 4, 6, 2], 3, (12, 7, 3)),
    # thresholds 1/3 and 3/5 (15 cells); after two rejections the residual is (7, 26)/33 on ids 2, 3 (33 cells)
    ([2, 3, 5, 6], [6, 5, 3, 2], 2, (15, 2, 33)),
])
def test_tree_rule_is_lossless_for_iid_siblings_exact_integration(p16, q16, m, grids):
    """m sibling drafts drawn independently from q under the root: whatever m is, the first emitted token must
    follow the target distribution p exactly (the property that makes multi-branch verification lossless).  Every
    decision boundary lies on a grid edge, so the midpoint rule integrates the law exactly."""
    V = 4
    p = np.array(p16) / 16.0
    q = np.array(q16) / 16.0
    parent = np.array([-1] + [0] * m, np.int32)
    Na1, Na2, Nr = grids
    items, weights = [], []
    for xs in itertools.product(range(V), repeat=m):
        for a1 in range(Na1):
            for a2 in range(Na2):
                for r in range(Nr):
                    ua = [0.0, (a1 + 0.5) / Na1] + [(a2 + 0.5) / Na2] * (m - 1)
                    ur = [(r + 0.5) / Nr] * (m + 1)
                    items.append(tree_inputs([p] * (m + 1), [q] * m, xs, ua, ur))
                    weights.append(np.prod([q[x] for x in xs]) / (Na1 * Na2 * Nr))
    # (with three siblings the third one's threshold is 0 or above 1 for these numbers, so sharing sibling 2's
    # uniform integrates it exactly too)
    o = batch_tree(items, parent, 1)
    w = np.array(weights)
    law = np.zeros(V)
    for k in range(len(items)):
        law[o["emitted"][k, 0]] += w[k]
    np.testing.assert_allclose(law, p, atol=1e-12)
    # more siblings can only help: the acceptance probability is at least that of one draft
    assert (w * (o["n_accepted"] == 1)).sum() >= np.minimum(p, q).sum() - 1e-12


def test_tree_rule_on_a_chain_is_the_single_branch_rule():
    rng = np.random.default_rng(5)
    V, gamma, B = 23, 4, 200
    parent = comb_parent(1, gamma)
    n = gamma + 1
    logits = rng.normal(0, 2, (B * n, V)).astype(np.float32)
    lse = np.log(np.exp(logits.astype(np.float64)).sum(1)).astype(np.float32)
    q = rng.dirichlet(np.ones(V), (B, n - 1)).astype(np.float32)
    tok = rng.integers(0, V, (B, n)).astype(np.int32)
    ua = rng.random((B, n)).astype(np.float32); ur = rng.random((B, n)).astype(np.float32)
    a = O.accept_spec(tok, logits, lse, q, ua, ur, parent, gamma)
    b = O.accept_tree(tok, logits, lse, q, ua, ur, parent, gamma)
    for key in ("n_accepted", "best_branch", "decide_row", "n_emitted", "emitted", "accepted_nodes", "reuse_slot"):
        assert (a[key] == b[key]).all(), key
    assert (a["n_accepted"] > 0).any() and (a["n_accepted"] < gamma).any()


def test_tree_rule_walk_order_on_a_two_level_tree():
    # nodes: 1, 2 under the root; 3, 4 under node 1; 5 under node 2.  Branches (leaves in order): [1,3], [1,4], [2,5].
    parent = np.array([-1, 0, 0, 1, 1, 2], np.int32)
    V = 3
    flat = np.full(V, 1.0 / V)
    peaked = np.array([0.98, 0.01, 0.01])
    # node 1 proposes token 1 from a draft that is sure of it, the target gives it 1%: rejected for u = 0.9;
    # node 2 (u = 0) and node 5 (u = 0) pass whatever their numbers are; node 5 is a leaf: bonus from its row
    p_rows = [peaked, flat, flat, flat, flat, np.array([0.0, 0.0, 1.0])]
    q_rows = [np.array([0.01, 0.98, 0.01]), flat, flat, flat, flat]
    item = tree_inputs(p_rows, q_rows, [1, 0, 2, 2, 1], [0.0, 0.9, 0.0, 0.5, 0.5, 0.0], [0.5] * 6)
    o = batch_tree([item], parent, 2)
    assert o["n_accepted"][0] == 2 and o["accepted_nodes"][0].tolist() == [2, 5]
    assert o["best_branch"][0] == 2 and o["decide_row"][0] == 5
    assert o["emitted"][0].tolist() == [0, 1, 2] and o["n_emitted"][0] == 3
    # both children of the root rejected (u close to 1 against drafts that overrate their tokens): the extra token
    # comes from the twice-reduced distribution at the root, which has lost ids 1 and 2 entirely -> id 0
    q_over = [np.array([0.0, 1.0, 0.0]), np.array([0.0, 0.0, 1.0]), flat, flat, flat]
    item = tree_inputs([np.array([0.5, 0.25, 0.25])] + [flat] * 5, q_over, [1, 2, 0, 0, 0], [0.0, 0.99, 0.99, 0.5, 0.5, 0.5], [0.7] * 6)
    o = batch_tree([item], parent, 2)
    assert o["n_accepted"][0] == 0 and o["decide_row"][0] == 0 and o["n_emitted"][0] == 1
    assert o["emitted"][0].tolist() == [0, -1, -1]
    # without a bonus a fully accepted path emits only its own tokens
    item = tree_inputs(p_rows, q_rows, [1, 0, 2, 2, 1], [0.0, 0.9, 0.0, 0.5, 0.5, 0.0], [0.5] * 6)
    o = batch_tree([item], parent, 2, emit_bonus=False)
    assert o["n_emitted"][0] == 2 and o["emitted"][0].tolist() == [0, 1, -1]


def test_trie_build_shares_exactly_the_common_prefixes():
    """Pins of the de-duplicated tree: a hand-worked case, and on random branches the brute-force properties that
    define it (one node per distinct prefix, every branch recovered by walking up from its leaf)."""
    bt = [[5, 7, 9], [5, 7, 2], [5, 1, 9], [4, 7, 9]]
    parent, tokens, node_of = O.trie_build(bt, 99)
    # prefixes in order of appearance: (5) (5,7) (5,7,9) | (5,7,2) | (5,1) (5,1,9) | (4) (4,7) (4,7,9)
    assert parent.tolist() == [-1, 0, 1, 2, 2, 1, 5, 0, 7, 8]
    assert tokens.tolist() == [99, 5, 7, 9, 2, 1, 9, 4, 7, 9]
    assert node_of.tolist() == [[1, 2, 3], [1, 2, 4], [1, 5, 6], [7, 8, 9]]
    rng = np.random.default_rng(0)
    for _ in range(50):
        kappa, gamma = int(rng.integers(1, 7)), int(rng.integers(1, 6))
        bt = rng.integers(0, 3, size=(kappa, gamma))                      # tiny alphabet: many shared prefixes
        parent, tokens, node_of = O.trie_build(bt, 7)
        prefixes = {tuple(bt[i, :j + 1]) for i in range(kappa) for j in range(gamma)}
        assert len(parent) == 1 + len(prefixes)
        assert all(parent[i] < i for i in range(1, len(parent))) and parent[0] == -1
        for i in range(kappa):
            node, seq = int(node_of[i, gamma - 1]), []
            while node != 0:
                seq.append(int(tokens[node])); node = int(parent[node])
            assert seq[::-1] == bt[i].tolist()
        # identical branches end in the same leaf; branches that differ somewhere do not
        for a in range(kappa):
            for b in range(kappa):
                assert (node_of[a, gamma - 1] == node_of[b, gamma - 1]) == bool(np.array_equal(bt[a], bt[b]))
    # no sharing at all reproduces the comb tree
    parent, tokens, node_of = O.trie_build([[1, 2], [3, 4]], 0)
    assert parent.tolist() == [-1, 0, 1, 0, 3] and node_of.tolist() == [[1, 2], [3, 4]]
