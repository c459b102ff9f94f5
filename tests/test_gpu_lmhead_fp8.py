"""GPU parity of the low-precision LM head (e4m3 operands with one scale per row) against the oracle's rounding model:
the 8-bit codes and scales bit for bit, the logits of the quantised operands within the fp32-accumulation tolerance of
the bf16 head, argmax flips only inside that tolerance."""
import numpy as np
import pytest
import torch

from oracle import fp8 as F
from oracle import oracle as O
from paper_2510_13161_b200 import inputs as I
from tests.helpers import make_mirror

pytestmark = pytest.mark.gpu
LOGIT_TOL = 2e-3


def rand_bf16(shape, std, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.empty(shape, dtype=torch.bfloat16).normal_(0, std, generator=g)


def lm_cfg(V, H, T=1.0):
    return I.VerifyConfig("t", H, 4, 2, 64, 1, 1, 16, 16, 2, 4, V, "greedy", temperature=T)


@pytest.mark.parametrize("rows,cols", [(7, 128), (130, 512), (33, 5120)])
def test_row_quantisation_is_bit_exact(rows, cols):
    x = rand_bf16((rows, cols), 0.7, 3)
    x[2] = 0                                        # an all-zero row
    x[1, 5] = 448.0                                  # and one whose maximum is a power-of-two multiple of the format's
    m = make_mirror(lm_cfg(1024, 128))
    codes, scale = m.mirror_quantize_rows_fp8(x.cuda())
    rc, rs = F.quantize_rows(x.float().numpy())
    np.testing.assert_array_equal(scale.cpu().numpy(), rs)
    np.testing.assert_array_equal(codes.cpu().numpy(), rc)


@pytest.mark.parametrize("M,V,H,T", [(17, 6000, 512, 1.0), (300, 4100, 256, 0.8), (128, 20000, 1024, 1.0)])
def test_fp8_lmhead_matches_the_oracle_of_the_quantised_operands(M, V, H, T):
    W = rand_bf16((V, H), 0.05, 11); hid = rand_bf16((M, H), 1.0, 12)
    m = make_mirror(lm_cfg(V, H, T), temperature=T)
    W8, ws = m.mirror_quantize_rows_fp8(W.cuda())
    h8, hs = m.mirror_quantize_rows_fp8(hid.cuda())
    res = m.mirror_lmhead_reduce_fp8(h8, hs, W8, ws, want_logits=True)
    torch.cuda.synchronize()
    assert m.device_status() == (0, 0)
    logits = F.lmhead_logits_fp8(h8.cpu().numpy(), hs.cpu().numpy(), W8.cpu().numpy(), ws.cpu().numpy())
    assert np.abs(res["logits"].cpu().numpy() - logits).max() < LOGIT_TOL
    red = O.row_reduce(logits, temperature=T)
    got = res["argmax"].cpu().numpy()
    for r in np.nonzero(got != red["argmax"])[0]:
        assert logits[r, red["argmax"][r]] - logits[r, got[r]] < LOGIT_TOL, r
    assert np.abs(res["maxlogit"].cpu().numpy() - red["maxlogit"]).max() < LOGIT_TOL
    assert np.abs(res["lse"].cpu().numpy() - red["lse"]).max() < LOGIT_TOL
    # the quantised head is a coarse copy of the bf16 head: close, not equal (sanity of the scales' orientation)
    plain = O.lmhead_logits(I.bf16_bits(hid), I.bf16_bits(W))
    assert np.abs(plain - logits).max() < 0.5 and np.corrcoef(plain.ravel(), logits.ravel())[0, 1] > 0.99
