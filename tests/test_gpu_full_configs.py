"""GPU parity at the full sizes of the larger configurations (batched / long-context / 66B-class), on
sampled outputs the oracle can afford: sampled layers and requests for attention, sampled rows for the LM
head, and the acceptance decision re-derived by the oracle from the very logits the GPU produced."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2510_13161_b200 import binding, inputs as I
from tests.helpers import make_mirror

pytestmark = pytest.mark.gpu
FIELDS = ["n_accepted", "best_branch", "decide_row", "n_emitted", "emitted", "accepted_nodes", "reuse_slot"]


def check_attention_samples(x, out, lse, layers, requests):
    """Oracle attention for a few (layer, request) pairs; the request is cut out of the batch on the host."""
    cfg = x.cfg
    anc, _ = O.tree(x.parent)
    scale = 1.0 / np.sqrt(cfg.head_dim)
    worst = 0.0
    for l in layers:
        kp, vp = I.bf16_bits(x.k_pool[l]), I.bf16_bits(x.v_pool[l])
        for b in requests:
            o_ref, lse_ref, _ = O.attention_layer(I.bf16_bits(x.q[l, b:b + 1]), kp, vp, x.page_table[b:b + 1].cpu().numpy(),
                                                  x.prefix_len[b:b + 1].cpu().numpy(), I.bf16_bits(x.k_new[l, b:b + 1]),
                                                  I.bf16_bits(x.v_new[l, b:b + 1]), anc, scale)
            got = out[l, b].float().cpu().numpy()
            err = np.abs(got - o_ref[0]).max()
            ref_scale = np.abs(o_ref).max()
            assert err < 2e-2 and err <= 1e-2 * ref_scale + 1e-5, (l, b, err, ref_scale)
            np.testing.assert_allclose(lse[l, b].cpu().numpy(), lse_ref[0], atol=2e-3)
            worst = max(worst, err / ref_scale)
    return worst


def check_lmhead_rows(hidden_rows, W, res, rows):
    logits = O.lmhead_logits(I.bf16_bits(hidden_rows[rows]), I.bf16_bits(W))
    red = O.row_reduce(logits)
    am = res["argmax"].cpu().numpy()[rows]
    for k in np.nonzero(am != red["argmax"])[0]:
        assert logits[k, red["argmax"][k]] - logits[k, am[k]] < 2e-3
    np.testing.assert_allclose(res["maxlogit"].cpu().numpy()[rows], red["maxlogit"], atol=2e-3)
    np.testing.assert_allclose(res["lse"].cpu().numpy()[rows], red["lse"], atol=2e-3)
    if res.get("logits") is not None:
        assert np.abs(res["logits"][torch.as_tensor(rows)].cpu().numpy() - logits).max() < 2e-3


def run_config(name, layers, requests, lm_rows, n_layers=None):
    cfg = I.CONFIGS[name]
    x = I.gen_verify_inputs(cfg, 0, "cuda", layers=n_layers)
    L = x.q.shape[0]
    m = make_mirror(cfg, temperature=cfg.temperature)
    kv = m.kv(x.k_pool, x.v_pool, x.page_table, x.prefix_len)
    tree = m.tree(x.tokens, cfg.kappa, cfg.gamma)
    spec = cfg.mode == "spec_sampling"
    # --- attention alone (with lse)
    lse = torch.empty((L, cfg.batch, cfg.n_q_heads, cfg.n_nodes), dtype=torch.float32, device="cuda")
    out = m.mirror_attn_verify(kv, tree, x.q, x.k_new, x.v_new, lse_out=lse)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    worst = check_attention_samples(x, out, lse, [l for l in layers if l < L], requests)
    # --- fused step
    attn_out = torch.empty_like(x.q)
    argmax = torch.empty(cfg.rows, dtype=torch.int32, device="cuda")
    acc = m.accept_in(binding.ACCEPT_SPEC_SAMPLING if spec else binding.ACCEPT_GREEDY, True, q_probs=x.q_probs,
                      u_accept=x.u_accept, u_resample=x.u_resample)
    res = m.mirror_verify_step(kv, tree, x.q, x.k_new, x.v_new, x.hidden, x.W, acc, attn_out, argmax_out=argmax).cpu()
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    assert torch.equal(attn_out, out)                           # same kernel, same inputs: bitwise equal
    # --- LM head on the step's rows, sampled rows against the oracle
    rows_t = x.hidden if x.hidden is not None else attn_out[-1].reshape(cfg.rows, cfg.hidden)
    lm = m.mirror_lmhead_reduce(rows_t, x.W, want_logits=spec)
    assert torch.equal(lm["argmax"], argmax)
    check_lmhead_rows(rows_t, x.W, lm, lm_rows)
    # --- acceptance from the GPU's own logits / argmax: outputs must be bit-exact (spec: up to knife edges)
    tok = x.tokens.cpu().numpy()
    if spec:
        ref = O.accept_spec(tok, lm["logits"].cpu().numpy(), lm["lse"].cpu().numpy(), x.q_probs.cpu().numpy(),
                            x.u_accept.cpu().numpy(), x.u_resample.cpu().numpy(), x.parent, cfg.gamma, True, cfg.temperature)
        for b in range(cfg.batch):
            same = all(np.array_equal(res[f][b], ref[f][b]) for f in FIELDS)
            assert same or ref["margin"][b] < 1e-9, (b, ref["margin"][b])
    else:
        ref = O.accept_greedy(tok, argmax.cpu().numpy().reshape(tok.shape), x.parent, cfg.gamma)
        for f in FIELDS:
            np.testing.assert_array_equal(res[f], ref[f], err_msg=f)
    print(name, "worst relative attention error", worst)


def test_qwen14b_batch8_spec_sampling_full_size():
    run_config("qwen14b_b8", layers=[0, 47], requests=[0, 5], lm_rows=[0, 49, 200, 391])


def test_qwen32b_long_context_full_size():
    run_config("qwen32b_long", layers=[63], requests=[0], lm_rows=list(range(0, 33, 4)))


def test_opt66b_batch16_spec_sampling_full_size():
    run_config("opt66b_b16", layers=[79], requests=[3], lm_rows=[0, 65, 1039])


def test_paper_native_operating_point():
    run_config("paper_native", layers=[0, 47], requests=[0], lm_rows=list(range(0, 57, 8)))
