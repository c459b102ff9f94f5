"""GPU parity of the fused verify step (attention -> LM head -> acceptance) against the oracle chain."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2510_13161_b200 import binding, inputs as I
from tests.helpers import make_mirror, oracle_attention, to_device

pytestmark = pytest.mark.gpu
FIELDS = ["n_accepted", "best_branch", "decide_row", "n_emitted", "emitted", "accepted_nodes", "reuse_slot"]


def oracle_step_greedy(x, logits=None):
    """Oracle chain: last-layer attention (fp64, unrounded) -> LM head -> argmax -> greedy acceptance."""
    cfg = x.cfg
    L = x.q.shape[0]
    if logits is None:
        if x.hidden is not None:
            logits = O.lmhead_logits(I.bf16_bits(x.hidden), I.bf16_bits(x.W))
        else:
            out, _ = oracle_attention(x, [L - 1])[L - 1]
            logits = O.lmhead_logits(out.reshape(-1, cfg.hidden), I.bf16_bits(x.W))
    red = O.row_reduce(logits)
    return logits, red


def gpu_step(m, x, mode=0, **acc_kw):
    kv = m.kv(x.k_pool, x.v_pool, x.page_table, x.prefix_len)
    tree = m.tree(x.tokens, x.cfg.kappa, x.cfg.gamma, parent=x.parent)
    attn_out = torch.empty_like(x.q)
    argmax = torch.empty(x.tokens.numel(), dtype=torch.int32, device="cuda")
    acc = m.accept_in(mode, True, **acc_kw)
    res = m.mirror_verify_step(kv, tree, x.q, x.k_new, x.v_new, x.hidden, x.W, acc, attn_out, argmax_out=argmax)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    return res.cpu(), argmax.cpu().numpy(), attn_out


def count_flips(argmax_gpu, logits, tol=2e-3):
    red = O.row_reduce(logits)
    flips = np.nonzero(argmax_gpu != red["argmax"])[0]
    for r in flips:      # a flip is legitimate only when the oracle's gap is inside the logit error bound
        assert logits[r, red["argmax"][r]] - logits[r, argmax_gpu[r]] < tol, r
    return len(flips)


def test_tiny_config_uniform_and_planted():
    cfg = I.CONFIGS["tiny"]
    x = I.gen_verify_inputs(cfg, 0, "cuda")
    m = make_mirror(cfg)
    logits, red = oracle_step_greedy(x)
    got, am, _ = gpu_step(m, x)
    flips = count_flips(am, logits)
    tok = x.tokens.cpu().numpy()
    ref = O.accept_greedy(tok, am.reshape(tok.shape), x.parent, cfg.gamma)      # identical argmax in: outputs bit-exact
    for f in FIELDS:
        np.testing.assert_array_equal(got[f], ref[f], err_msg=f)
    # planted variant: branch 1 copies the oracle's target argmax for its first 3 positions
    g = cfg.gamma
    tok2 = tok.copy()
    rows = [0, 1 + g, 2 + g]
    for j, r in enumerate(rows):
        tok2[0, 1 + g + j] = red["argmax"][r]
    x.tokens = torch.from_numpy(tok2).cuda()
    got, am, _ = gpu_step(m, x)
    ref = O.accept_greedy(tok2, red["argmax"].reshape(tok.shape), x.parent, cfg.gamma)
    if flips == 0 and count_flips(am, logits) == 0:
        for f in FIELDS:
            np.testing.assert_array_equal(got[f], ref[f], err_msg=f)
        assert got["n_accepted"][0] >= 3 and got["best_branch"][0] == 1


@pytest.mark.parametrize("mode", [1, 2])            # independent per-branch rule; lossless rule over the tree
def test_spec_sampling_step_small(mode):
    cfg = I.VerifyConfig("s", 512, 8, 2, 64, 2, 3, 40, 200, 3, 3, 2000, "spec_sampling")
    x = I.gen_verify_inputs(cfg, 1, "cuda")
    # draft tokens drawn from q so that some are accepted
    g = torch.Generator().manual_seed(0)
    tok = x.tokens.cpu()
    for b in range(cfg.batch):
        for c in range(1, cfg.n_nodes):
            tok[b, c] = int(torch.multinomial(x.q_probs[b, c - 1].cpu(), 1, generator=g))
    x.tokens = tok.cuda()
    m = make_mirror(cfg)
    got, am, attn_out = gpu_step(m, x, mode, q_probs=x.q_probs, u_accept=x.u_accept, u_resample=x.u_resample)
    # feed the oracle the identical logits the GPU used: recompute them with the same kernel and the spill on
    rows = attn_out[-1].reshape(cfg.rows, cfg.hidden)
    lm = m.mirror_lmhead_reduce(rows, x.W, want_logits=True)
    rule = O.accept_spec if mode == 1 else O.accept_tree
    ref = rule(tok.numpy(), lm["logits"].cpu().numpy(), lm["lse"].cpu().numpy(), x.q_probs.cpu().numpy(),
               x.u_accept.cpu().numpy(), x.u_resample.cpu().numpy(), x.parent, cfg.gamma)
    for b in range(cfg.batch):
        same = all(np.array_equal(got[f][b], ref[f][b]) for f in FIELDS)
        assert same or ref["margin"][b] < 1e-9, (b, ref["margin"][b])


def test_full_size_14b_step_flip_count():
    cfg = I.CONFIGS["qwen14b"]
    x = I.gen_verify_inputs(cfg, 0, "cuda")
    m = make_mirror(cfg)
    got, am, attn_out = gpu_step(m, x)
    logits, red = oracle_step_greedy(x)
    flips = count_flips(am, logits)
    print("end-to-end argmax flips:", flips, "of", len(am))
    tok = x.tokens.cpu().numpy()
    ref = O.accept_greedy(tok, am.reshape(tok.shape), x.parent, cfg.gamma)
    for f in FIELDS:
        np.testing.assert_array_equal(got[f], ref[f], err_msg=f)


@pytest.mark.parametrize("layers", [1, 2, 6])
def test_host_buffer_step_equals_the_device_buffer_step(layers):
    """mirror_verify_step_host (inputs in pinned host memory, copied in pieces on its own stream) decides exactly what
    mirror_verify_step decides on the same inputs, call after call with changing inputs."""
    cfg = I.shrink(I.CONFIGS["tiny"], layers=layers, batch=3, prefix_lo=40, prefix_hi=300, kappa=3, gamma=4, vocab=3000)
    m = make_mirror(cfg)
    x0 = to_device(I.gen_verify_inputs(cfg, 0, "cpu"))
    kv = m.kv(x0.k_pool, x0.v_pool, x0.page_table, x0.prefix_len)
    d_in = {k: torch.empty_like(getattr(x0, k)) for k in ("q", "k_new", "v_new", "tokens")}
    tree_h = m.tree(d_in["tokens"], cfg.kappa, cfg.gamma)
    acc = m.accept_in(binding.ACCEPT_GREEDY, True)
    attn_h, attn_d = torch.empty_like(x0.q), torch.empty_like(x0.q)
    res_h, res_d = binding.AcceptResult(cfg.batch, cfg.gamma, "cuda"), binding.AcceptResult(cfg.batch, cfg.gamma, "cuda")
    h_out = {"n_accepted": torch.empty(cfg.batch, dtype=torch.int32).pin_memory(), "emitted": torch.empty((cfg.batch, cfg.gamma + 1), dtype=torch.int32).pin_memory(),
             "n_emitted": torch.empty(cfg.batch, dtype=torch.int32).pin_memory(), "best_branch": torch.empty(cfg.batch, dtype=torch.int32).pin_memory()}
    for seed in range(4):
        xs = I.gen_verify_inputs(cfg, seed, "cpu")            # same cache (same config and page draw), new step inputs
        h_in = {k: getattr(xs, k).contiguous().pin_memory() for k in ("q", "k_new", "v_new", "tokens")}
        m.mirror_verify_step_host(kv, tree_h, h_in, d_in, x0.hidden, x0.W, acc, attn_h, res_h, h_out=h_out)
        torch.cuda.synchronize()
        xd = {k: v.cuda() for k, v in h_in.items()}
        tree_d = m.tree(xd["tokens"], cfg.kappa, cfg.gamma)
        m.mirror_verify_step(kv, tree_d, xd["q"], xd["k_new"], xd["v_new"], x0.hidden, x0.W, acc, attn_d, out=res_d)
        torch.cuda.synchronize()
        assert torch.equal(attn_h, attn_d)
        for f in ("n_accepted", "best_branch", "n_emitted", "emitted", "accepted_nodes"):
            assert torch.equal(getattr(res_h, f), getattr(res_d, f)), f
        for f, t in h_out.items():
            assert torch.equal(t, getattr(res_d, f).cpu()), f
        for k in d_in:
            assert torch.equal(d_in[k], xd[k]), k
    assert m.device_status() == (0, 0)


def test_verify_step_replays_from_a_cuda_graph():
    """The step only enqueues kernels (no allocation, no synchronisation once the workspace is attached), so it can be
    captured in a CUDA graph; replays with new inputs in the same buffers decide like direct calls."""
    cfg = I.shrink(I.CONFIGS["tiny"], layers=3, batch=2, prefix_lo=40, prefix_hi=200, kappa=3, gamma=4, vocab=3000)
    m = make_mirror(cfg)
    x = to_device(I.gen_verify_inputs(cfg, 0, "cpu"))
    kv = m.kv(x.k_pool, x.v_pool, x.page_table, x.prefix_len)
    tree = m.tree(x.tokens, cfg.kappa, cfg.gamma)
    acc = m.accept_in(binding.ACCEPT_GREEDY, True)
    attn_g, attn_d = torch.empty_like(x.q), torch.empty_like(x.q)
    res_g, res_d = binding.AcceptResult(cfg.batch, cfg.gamma, "cuda"), binding.AcceptResult(cfg.batch, cfg.gamma, "cuda")
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        m.mirror_verify_step(kv, tree, x.q, x.k_new, x.v_new, x.hidden, x.W, acc, attn_g, out=res_g, stream=s)    # attaches the workspace
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            m.mirror_verify_step(kv, tree, x.q, x.k_new, x.v_new, x.hidden, x.W, acc, attn_g, out=res_g, stream=s)
    for seed in (1, 2, 3):
        xs = I.gen_verify_inputs(cfg, seed, "cpu")
        for k in ("q", "k_new", "v_new", "tokens"):
            getattr(x, k).copy_(getattr(xs, k))                 # new step inputs in the captured buffers
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        m.mirror_verify_step(kv, tree, x.q, x.k_new, x.v_new, x.hidden, x.W, acc, attn_d, out=res_d)
        torch.cuda.synchronize()
        assert torch.equal(attn_g, attn_d)
        for f in FIELDS:
            assert torch.equal(getattr(res_g, f), getattr(res_d, f)), f
    assert m.device_status() == (0, 0)


def test_step_when_no_unit_is_cut_by_the_partition():
    """Equal prefixes in a batch whose unit count the CTA groups divide: every group holds whole units, the merge kernel has
    nothing to merge, and the LM head behind it must still see the finished attention rows (the merge kernel's blocks wait
    for the attention kernel before they leave).  Many repetitions: a missing wait shows up now and then only."""
    cfg = I.VerifyConfig("nocut", 1024, 8, 8, 128, 16, 2, 600, 600, 2, 3, 4096, "greedy")     # 16 x 2 x 8 = 256 units
    x = I.gen_verify_inputs(cfg, 5, "cuda")
    m = make_mirror(cfg)
    logits, red = oracle_step_greedy(x)
    ref_attn = oracle_attention(x, [cfg.layers - 1])[cfg.layers - 1][0]
    tok = x.tokens.cpu().numpy()
    for rep in range(20):
        got, am, attn_out = gpu_step(m, x)
        err = np.abs(attn_out[-1].float().cpu().numpy() - ref_attn).max()
        assert err <= 1e-2 * np.abs(ref_attn).max() + 1e-5, (rep, err)
        count_flips(am, logits)
        ref = O.accept_greedy(tok, am.reshape(tok.shape), x.parent, cfg.gamma)
        for f in FIELDS:
            np.testing.assert_array_equal(got[f], ref[f], err_msg=f)
