"""The decoding loop of tests/test_gpu_decode_loop.py over an e4m3 KV cache: embedding rows -> target layers (new K/V rows
quantised under the cache's scales, 8-bit attention) -> LM head -> acceptance -> roll-forward of the code cache.  Plain
one-token-at-a-time decoding and greedy speculative decoding go through the same 8-bit path, so they commit the same
sequence (the rule-level equivalence of Sec. "Correctness" does not depend on the cache's precision)."""
import numpy as np
import pytest
import torch

from paper_2510_13161_b200 import binding, inputs as I
from tests.helpers import make_mirror

pytestmark = pytest.mark.gpu

H, HQ, HKV, D, INTER, LAYERS, V = 512, 4, 2, 128, 1024, 2, 1000
THETA, EPS = 1.0e4, 1e-6
PROMPT, GEN = 8, 32
MIN_GAP = 0.3            # a greedy token whose logit leads by less than this could flip between the two evaluations


class Model8:
    def __init__(self, seed):
        cfg = I.VerifyConfig("loop8", H, HQ, HKV, D, LAYERS, 1, 0, 0, 1, 1, V, "greedy", 0.05)
        self.m = make_mirror(cfg)
        layers, norm_final, _ = I.gen_layer_weights(cfg, INTER, LAYERS, seed, "cuda")
        self.target = self.m.target(layers, norm_final, INTER, THETA, EPS)
        g = torch.Generator(device="cuda").manual_seed(seed + 1)
        self.embed = torch.empty((V, H), dtype=torch.bfloat16, device="cuda").normal_(0, 1.0, generator=g)
        self.W = torch.empty((V, H), dtype=torch.bfloat16, device="cuda").normal_(0, 1.0, generator=g)
        self.pages = 8
        self.page_table = torch.arange(self.pages, dtype=torch.int32, device="cuda").flip(0).reshape(1, -1).contiguous()
        self.calibrate()
        self.reset()

    def calibrate(self):
        """Scales from one bf16 pass over random tokens: magnitudes of K, V and Q per layer (and KV head), with head room."""
        m = self.m
        tok = torch.randint(0, V, (1, 33), dtype=torch.int32, device="cuda", generator=torch.Generator(device="cuda").manual_seed(99))
        shape = (LAYERS, self.pages, HKV, I.PAGE_SIZE, D)
        z = torch.zeros(shape, dtype=torch.bfloat16, device="cuda")
        pl = torch.zeros(1, dtype=torch.int32, device="cuda")
        tree = m.tree(tok, 1, 32)
        out = m.mirror_target_forward(self.target, m.kv(z, z.clone(), self.page_table, pl), tree, m.mirror_embed_rows(self.embed, tok))
        self.k_scale = (out["k_new"].float().abs().amax(dim=(1, 2, 4)) * 1.5 / 448.0).contiguous()
        self.v_scale = (out["v_new"].float().abs().amax(dim=(1, 2, 4)) * 1.5 / 448.0).contiguous()
        self.q_scales = [float(out["q"][l].float().abs().max()) * 1.5 / 448.0 for l in range(LAYERS)]

    def reset(self):
        shape = (LAYERS, self.pages, HKV, I.PAGE_SIZE, D)
        self.k8 = torch.zeros(shape, dtype=torch.uint8, device="cuda")
        self.v8 = torch.zeros(shape, dtype=torch.uint8, device="cuda")
        self.prefix_len = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.kv = self.m.kv_fp8(self.k8, self.v8, self.page_table, self.prefix_len)

    def forward(self, tokens, kappa, gamma, parent=None):
        m = self.m
        tok = torch.tensor([tokens], dtype=torch.int32, device="cuda")
        tree = m.tree(tok, kappa, gamma, parent=parent)
        out = m.mirror_target_forward_fp8(self.target, self.kv, tree, m.mirror_embed_rows(self.embed, tok), self.k_scale, self.v_scale,
                                          self.q_scales)
        red = m.mirror_lmhead_reduce(out["hidden"], self.W, topk=2)
        gap = (red["topk_logprob"][:, 0] - red["topk_logprob"][:, 1]).cpu().numpy()
        return tree, out, red["argmax"], gap

    def commit(self, tree, out, res):
        self.m.mirror_kv_commit_fp8(self.kv, tree, out["k_new8"], out["v_new8"], res, self.prefix_len)

    def commit_nodes(self, tree, out, gamma, nodes):
        res = binding.AcceptResult(1, gamma, "cuda")
        res.accepted_nodes.zero_()
        if nodes:
            res.accepted_nodes[0, :len(nodes)] = torch.tensor(nodes, dtype=torch.int32, device="cuda")
        res.n_accepted[0] = len(nodes)
        self.commit(tree, out, res)

    def prefill(self, prompt):
        n = len(prompt)
        tree, out, am, gap = self.forward(prompt, 1, n - 1)
        self.commit_nodes(tree, out, n - 1, list(range(1, n)))
        return int(am[n - 1]), float(gap[n - 1])


def decode_plain(model, prompt, n_tokens):
    model.reset()
    tok, gap = model.prefill(prompt)
    seq, gaps = [tok], [gap]
    while len(seq) < n_tokens:
        tree, out, am, g = model.forward([seq[-1]], 1, 1, parent=[-1])
        model.commit_nodes(tree, out, 1, [])
        seq.append(int(am[0])); gaps.append(float(g[0]))
    assert model.m.device_status() == (0, 0)
    return seq, gaps


def decode_speculative(model, prompt, n_tokens, drafts, kappa, gamma):
    m = model.m
    model.reset()
    tok, _ = model.prefill(prompt)
    seq, accepted = [tok], []
    while len(seq) < n_tokens:
        tokens = [seq[-1]] + [t for br in drafts(seq) for t in br]
        tree, out, am, _ = model.forward(tokens, kappa, gamma)
        res = m.mirror_accept_select(tree, m.accept_in(binding.ACCEPT_GREEDY, True, target_argmax=am))
        r = res.cpu()
        a, n_e = int(r["n_accepted"][0]), int(r["n_emitted"][0])
        model.commit(tree, out, res)
        seq.extend(int(t) for t in r["emitted"][0][:n_e])
        accepted.append(a)
    assert m.device_status() == (0, 0)
    assert int(model.prefix_len[0]) == len(prompt) + len(seq) - 1
    return seq[:n_tokens], accepted


@pytest.mark.parametrize("seed,min_stable", [(5, 32), (2, 20), (4, 16)])
def test_speculative_decoding_over_the_8_bit_cache_emits_the_plain_sequence(seed, min_stable):
    model = Model8(seed)
    rng = np.random.default_rng(seed)
    prompt = [int(t) for t in rng.integers(0, V, size=PROMPT)]
    ref, gaps = decode_plain(model, prompt, GEN)
    stable = next((i for i, g in enumerate(gaps) if g < MIN_GAP), GEN)
    assert stable >= min_stable, (stable, gaps[:stable + 1])
    kappa, gamma = 3, 4

    def drafts(seq):
        pos = len(seq)
        truth = [ref[pos + j] if pos + j < len(ref) else int(rng.integers(0, V)) for j in range(gamma)]
        b0 = list(truth); cut = int(rng.integers(0, gamma + 1))
        for j in range(cut, gamma):
            b0[j] = int(rng.integers(0, V))
        return [b0, [int(t) for t in rng.integers(0, V, size=gamma)], list(truth)]

    got, acc = decode_speculative(model, prompt, GEN, drafts, kappa, gamma)
    assert got[:stable] == ref[:stable]
    assert max(acc) == gamma


def test_layers_over_the_8_bit_cache_are_their_parts():
    """mirror_target_forward_fp8, first layer: the new rows' codes are the oracle's quantisation of the bf16 rows it
    returns, and its attention output is what mirror_attn_verify_fp8 gives on those codes (bit for bit)."""
    from oracle import fp8 as F
    model = Model8(5)
    m = model.m
    rng = np.random.default_rng(5)
    # some history in the cache first
    model.prefill([int(t) for t in rng.integers(0, V, size=20)])
    tokens = [int(t) for t in rng.integers(0, V, size=1 + 3 * 4)]
    tree, out, _, _ = model.forward(tokens, 3, 4)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    ks, vs = model.k_scale.cpu().numpy(), model.v_scale.cpu().numpy()
    for name, name8, sc in (("k_new", "k_new8", ks), ("v_new", "v_new8", vs)):
        ref = F.kv_quantize(out[name].float().cpu().numpy(), sc, head_axis=3)
        assert np.array_equal(out[name8].cpu().numpy(), ref), name
    kv0 = m.kv_fp8(model.k8[:1], model.v8[:1], model.page_table, model.prefix_len)
    a0 = m.mirror_attn_verify_fp8(kv0, tree, out["q"][:1], out["k_new8"][:1], out["v_new8"][:1], model.k_scale[:1].contiguous(),
                                  model.v_scale[:1].contiguous(), model.q_scales[0])
    torch.cuda.synchronize()
    assert torch.equal(a0[0], out["attn_out"][0])
