"""End to end on the GPU: greedy speculative decoding through the library (embedding rows -> target layers -> LM head ->
acceptance -> roll-forward of the paged cache, step after step) emits exactly what plain one-token-at-a-time decoding
through the same library emits.  This is the rule-level equivalence of Sec. "Correctness": the acceptance operator
(Eq. 3 / Eq. 10) keeps the longest prefix the target agrees with and adds the target's own token, so whatever the
draft proposes the committed sequence is the target's greedy sequence."""
import numpy as np
import pytest
import torch

from paper_2510_13161_b200 import binding, inputs as I
from tests.helpers import make_mirror

pytestmark = pytest.mark.gpu

H, HQ, HKV, D, INTER, LAYERS, V = 256, 4, 2, 64, 512, 2, 1000
THETA, EPS = 1.0e4, 1e-6
PROMPT, GEN = 8, 40
MIN_GAP = 0.2            # a greedy token whose logit leads by less than this could flip between the two evaluations
                         # (logits here have a standard deviation of about 16; the two runs differ by bf16 roundings)


class Model:
    def __init__(self, seed):
        cfg = I.VerifyConfig("loop", H, HQ, HKV, D, LAYERS, 1, 0, 0, 1, 1, V, "greedy", 0.05)
        self.cfg = cfg
        self.m = make_mirror(cfg)
        layers, norm_final, _ = I.gen_layer_weights(cfg, INTER, LAYERS, seed, "cuda")
        self.target = self.m.target(layers, norm_final, INTER, THETA, EPS)
        g = torch.Generator(device="cuda").manual_seed(seed + 1)
        self.embed = torch.empty((V, H), dtype=torch.bfloat16, device="cuda").normal_(0, 1.0, generator=g)
        self.W = torch.empty((V, H), dtype=torch.bfloat16, device="cuda").normal_(0, 1.0, generator=g)      # peaked logits
        self.pages = 8
        self.reset()

    def reset(self):
        shape = (LAYERS, self.pages, HKV, I.PAGE_SIZE, D)
        self.k_pool = torch.zeros(shape, dtype=torch.bfloat16, device="cuda")
        self.v_pool = torch.zeros(shape, dtype=torch.bfloat16, device="cuda")
        self.page_table = torch.arange(self.pages, dtype=torch.int32, device="cuda").flip(0).reshape(1, -1).contiguous()
        self.prefix_len = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.kv = self.m.kv(self.k_pool, self.v_pool, self.page_table, self.prefix_len)

    def forward(self, tokens, kappa, gamma, parent=None):
        """One target pass over a token tree: (tree, forward outputs, greedy token and top-2 logit gap per row)."""
        m = self.m
        tok = torch.tensor([tokens], dtype=torch.int32, device="cuda")
        tree = m.tree(tok, kappa, gamma, parent=parent)
        x = m.mirror_embed_rows(self.embed, tok)
        out = m.mirror_target_forward(self.target, self.kv, tree, x)
        red = m.mirror_lmhead_reduce(out["hidden"], self.W, topk=2)
        gap = (red["topk_logprob"][:, 0] - red["topk_logprob"][:, 1]).cpu().numpy()
        return tree, out, red["argmax"], gap

    def commit(self, tree, out, gamma, accepted_nodes):
        res = binding.AcceptResult(1, gamma, "cuda")
        res.accepted_nodes.zero_()
        if accepted_nodes:
            res.accepted_nodes[0, :len(accepted_nodes)] = torch.tensor(accepted_nodes, dtype=torch.int32, device="cuda")
        res.n_accepted[0] = len(accepted_nodes)
        self.m.mirror_kv_commit(self.kv, tree, out["k_new"], out["v_new"], res, self.prefix_len)

    def prefill(self, prompt):
        """The prompt as one chain: every token's K/V goes into the cache; returns the first generated token."""
        n = len(prompt)
        tree, out, am, gap = self.forward(prompt, 1, n - 1)
        self.commit(tree, out, n - 1, list(range(1, n)))
        return int(am[n - 1]), float(gap[n - 1])


def decode_plain(model, prompt, n_tokens):
    model.reset()
    tok, gap = model.prefill(prompt)
    seq, gaps = [tok], [gap]
    while len(seq) < n_tokens:
        tree, out, am, g = model.forward([seq[-1]], 1, 1, parent=[-1])
        model.commit(tree, out, 1, [])
        seq.append(int(am[0])); gaps.append(float(g[0]))
    assert model.m.device_status() == (0, 0)
    return seq, gaps


def decode_speculative(model, prompt, n_tokens, drafts, kappa, gamma):
    """drafts(generated so far) -> kappa x gamma proposed continuations of the last generated token."""
    m = model.m
    model.reset()
    tok, _ = model.prefill(prompt)
    seq, accepted_hist = [tok], []
    while len(seq) < n_tokens:
        branches = drafts(seq)
        tokens = [seq[-1]] + [t for br in branches for t in br]
        tree, out, am, _ = model.forward(tokens, kappa, gamma)
        res = m.mirror_accept_select(tree, m.accept_in(binding.ACCEPT_GREEDY, True, target_argmax=am))
        r = res.cpu()
        a, n_e = int(r["n_accepted"][0]), int(r["n_emitted"][0])
        assert n_e == a + 1
        m.mirror_kv_commit(model.kv, tree, out["k_new"], out["v_new"], res, model.prefix_len)
        seq.extend(int(t) for t in r["emitted"][0][:n_e])
        accepted_hist.append(a)
    assert m.device_status() == (0, 0)
    assert int(model.prefix_len[0]) == len(prompt) + len(seq) - 1          # everything but the newest token is cached
    return seq[:n_tokens], accepted_hist


@pytest.mark.parametrize("seed,min_stable", [(3, 40), (2, 16), (0, 12)])
def test_greedy_speculative_decoding_emits_the_plain_greedy_sequence(seed, min_stable):
    model = Model(seed)
    rng = np.random.default_rng(seed)
    prompt = [int(t) for t in rng.integers(0, V, size=PROMPT)]
    ref, gaps = decode_plain(model, prompt, GEN)
    # compare up to the first token whose lead is too small to be stable across the two evaluations
    stable = next((i for i, g in enumerate(gaps) if g < MIN_GAP), GEN)
    assert stable >= min_stable, (stable, gaps[:stable + 1])
    kappa, gamma = 3, 4

    def drafts_mixed(seq):
        """Branch 0: the true continuation, broken at a random depth; branch 1: noise; branch 2: the true continuation."""
        pos = len(seq)
        truth = [ref[pos + j] if pos + j < len(ref) else int(rng.integers(0, V)) for j in range(gamma)]
        b0 = list(truth); cut = int(rng.integers(0, gamma + 1))
        for j in range(cut, gamma):
            b0[j] = int(rng.integers(0, V))
        b1 = [int(t) for t in rng.integers(0, V, size=gamma)]
        b2 = list(truth) if rng.random() < 0.5 else [int(t) for t in rng.integers(0, V, size=gamma)]
        return [b0, b1, b2]

    def drafts_noise(seq):
        return [[int(t) for t in rng.integers(0, V, size=gamma)] for _ in range(kappa)]

    got, acc = decode_speculative(model, prompt, GEN, drafts_mixed, kappa, gamma)
    assert got[:stable] == ref[:stable]
    assert max(acc) == gamma and min(acc) < gamma          # whole branches were accepted, and some were cut short
    got2, acc2 = decode_speculative(model, prompt, GEN, drafts_noise, kappa, gamma)
    assert got2[:stable] == ref[:stable]
    assert sum(acc2) <= 2                                   # noise is (almost) never accepted: one token per step
