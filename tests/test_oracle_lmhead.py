"""Pins for the oracle's LM head and row reductions (O2): closed forms, library fp64
routines, normalisation, tie-breaking."""
import numpy as np
import torch

from oracle import oracle as O
from paper_2510_13161_b200 import inputs as I


def bf16_to_f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def rand_bf16(shape, std, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.empty(shape, dtype=torch.bfloat16).normal_(0, std, generator=g)


def test_unit_vector_hidden_reads_out_a_weight_column():
    V, H = 50, 24
    W = rand_bf16((V, H), 0.02, 1)
    hid = torch.zeros((3, H), dtype=torch.bfloat16)
    hid[0, 5] = 2.0; hid[1, 0] = -0.5; hid[2, 23] = 1.0
    logits = O.lmhead_logits(I.bf16_bits(hid), I.bf16_bits(W))
    Wf = bf16_to_f64(I.bf16_bits(W))
    np.testing.assert_array_equal(logits[0], 2.0 * Wf[:, 5])
    np.testing.assert_array_equal(logits[1], -0.5 * Wf[:, 0])
    np.testing.assert_array_equal(logits[2], Wf[:, 23])


def test_matches_fp64_library_matmul_and_logsumexp():
    V, H, M = 300, 96, 7
    W = rand_bf16((V, H), 0.05, 2); hid = rand_bf16((M, H), 1.0, 3)
    logits = O.lmhead_logits(I.bf16_bits(hid), I.bf16_bits(W))
    ref = hid.double() @ W.double().T
    np.testing.assert_allclose(logits, ref.numpy(), rtol=0, atol=1e-13)
    # W is [V,H] and hidden is [M,H]: a transposed operand would not even have this shape
    assert logits.shape == (M, V)
    for T in (1.0, 0.7):
        red = O.row_reduce(logits, temperature=T, topk=5)
        np.testing.assert_allclose(red["lse"], torch.logsumexp(ref / T, -1).numpy(), atol=1e-12)
        np.testing.assert_array_equal(red["argmax"], ref.argmax(-1).numpy())
        np.testing.assert_array_equal(red["maxlogit"], ref.max(-1).values.numpy())
        tv, ti = torch.topk(ref, 5, dim=-1)
        np.testing.assert_array_equal(red["topk_id"], ti.numpy())
        np.testing.assert_allclose(red["topk_logprob"], (tv / T - torch.logsumexp(ref / T, -1, keepdim=True)).numpy(), atol=1e-12)
    # the f64-hidden entry point computes the same contraction
    logits2 = O.lmhead_logits(hid.double().numpy(), I.bf16_bits(W))
    np.testing.assert_array_equal(logits, logits2)


def test_logprobs_normalise_and_top1_is_argmax():
    V = 40
    logits = np.random.default_rng(0).normal(size=(4, V)) * 3
    red = O.row_reduce(logits, temperature=1.3, topk=V)
    np.testing.assert_allclose(np.exp(red["topk_logprob"]).sum(-1), 1.0, atol=1e-13)
    np.testing.assert_array_equal(red["topk_id"][:, 0], red["argmax"])
    assert (np.diff(red["topk_logprob"], axis=-1) <= 0).all()
    for r in range(4):
        assert sorted(red["topk_id"][r].tolist()) == list(range(V))


def test_ties_go_to_the_lowest_token_id():
    V, H = 20, 16
    W = rand_bf16((V, H), 0.1, 4)
    W[11] = W[3]; W[17] = W[3]            # duplicate rows give exactly equal logits
    hid = rand_bf16((2, H), 1.0, 5)
    logits = O.lmhead_logits(I.bf16_bits(hid), I.bf16_bits(W))
    assert (logits[:, 3] == logits[:, 11]).all() and (logits[:, 3] == logits[:, 17]).all()
    logits[:, [3, 11, 17]] = logits.max() + 1.0
    red = O.row_reduce(logits, topk=4)
    np.testing.assert_array_equal(red["argmax"], [3, 3])
    np.testing.assert_array_equal(red["topk_id"][:, :3], [[3, 11, 17], [3, 11, 17]])


def test_overlap_mass_is_monotone_and_reaches_one():
    # Eq. 7: Omega_kappa is nondecreasing in kappa and tends to 1 as kappa -> |V|
    rng = np.random.default_rng(1)
    V = 30
    early = rng.normal(size=(1, V)) * 2
    final = early + rng.normal(size=(1, V))
    qf = np.exp(final[0] - final.max()); qf /= qf.sum()
    prev = 0.0
    for kappa in range(1, V + 1):
        ids = O.row_reduce(early, topk=kappa)["topk_id"][0]
        om = O.overlap_mass(qf, ids)
        assert om >= prev - 1e-15
        assert abs(om - qf[ids].sum()) < 1e-15
        prev = om
    assert abs(prev - 1.0) < 1e-12
