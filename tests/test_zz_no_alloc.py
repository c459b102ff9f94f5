"""mirror_lmhead_reduce_noalloc: the LM-head reductions for hosts that may not allocate device memory
(all memory owned by the host's own pool, allocator-guarded plugin regions).  Its scratch is a fixed
array inside the library, so it needs neither a context nor a workspace.  The test calls it through the
C ABI twice in a row and checks each result against the regular entry point, which uses a caller
workspace, and against the CPU oracle.  Collected last on purpose: a failure here cannot hide any other test."""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2510_13161_b200 import binding, inputs as I
from tests.helpers import make_mirror

pytestmark = pytest.mark.gpu


def rand_bf16(shape, std, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.empty(shape, dtype=torch.bfloat16).normal_(0, std, generator=g).cuda()


def call_noalloc(lib, hid, W, T, argmax, maxlogit, lse):
    M, H = hid.shape
    code = lib.mirror_lmhead_reduce_noalloc(0, C.c_void_p(hid.data_ptr()), M, C.c_void_p(W.data_ptr()), W.shape[0], H,
                                            C.c_float(T), C.c_void_p(argmax.data_ptr()), C.c_void_p(maxlogit.data_ptr()),
                                            C.c_void_p(lse.data_ptr()), C.c_void_p(torch.cuda.current_stream().cuda_stream))
    return code


def test_noalloc_matches_workspace_entry_point_on_two_calls_in_a_row():
    lib = binding.load_library()
    V, H, T = 20000, 512, 0.9
    cfg = I.VerifyConfig("t", H, 4, 2, 64, 1, 1, 16, 16, 2, 4, V, "greedy")
    m = make_mirror(cfg, temperature=T)
    W = rand_bf16((V, H), 0.05, 11)
    # outputs are allocated up front: the entry point itself must not need the allocator
    outs = [(torch.empty(M, dtype=torch.int32, device="cuda"), torch.empty(M, dtype=torch.float32, device="cuda"),
             torch.empty(M, dtype=torch.float32, device="cuda")) for M in (17, 100)]
    hids = [rand_bf16((17, H), 1.0, 12), rand_bf16((100, H), 1.0, 13)]
    refs = [m.mirror_lmhead_reduce(h, W) for h in hids]
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    for h, (am, mx, ls) in zip(hids, outs):            # second call reuses the scratch the first one left behind
        assert call_noalloc(lib, h, W, T, am, mx, ls) == 0
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    for ref, (am, mx, ls) in zip(refs, outs):
        assert torch.equal(am, ref["argmax"])
        torch.testing.assert_close(mx, ref["maxlogit"], atol=2e-3, rtol=0)
        torch.testing.assert_close(ls, ref["lse"], atol=2e-3, rtol=0)


def test_noalloc_rejects_sizes_beyond_its_scratch():
    lib = binding.load_library()
    H, V = 128, 1024
    W = rand_bf16((V, H), 0.05, 1); hid = rand_bf16((129, H), 1.0, 2)
    am = torch.empty(129, dtype=torch.int32, device="cuda")
    f = torch.empty(129, dtype=torch.float32, device="cuda")
    assert call_noalloc(lib, hid, W, 1.0, am, f, f.clone()) == 2          # MIRROR_ERR_SHAPE: more than 128 rows
    assert lib.mirror_lmhead_reduce_noalloc(0, None, 1, None, V, H, C.c_float(1.0), None, None, None, None) == 1
    res = binding.mirror_lmhead_reduce_noalloc(hid[:128], W)              # the limit itself is accepted
    ref = make_mirror(I.VerifyConfig("t", H, 4, 2, 64, 1, 1, 16, 16, 2, 4, V, "greedy")).mirror_lmhead_reduce(hid[:128], W)
    assert torch.equal(res["argmax"], ref["argmax"])


@pytest.mark.parametrize("rows", [(111, 128), (128, 17)])
def test_noalloc_against_the_oracle_at_row_counts_where_every_sm_holds_two_ctas(rows):
    """Up to 128 rows two CTAs share an SM, so a launch leaves twice as many partials as the GPU has SMs: the fixed
    array holds them (111 rows was the first count that did not fit an array sized by the SM count).  Two calls in a
    row, the second on fewer or more rows than the first, each compared with the fp64 oracle."""
    lib = binding.load_library()
    V, H, T = 40960, 512, 1.0
    W = rand_bf16((V, H), 0.05, 21)
    Wb = I.bf16_bits(W)
    for seed, M in enumerate(rows):
        hid = rand_bf16((M, H), 1.0, 30 + seed)
        am = torch.empty(M, dtype=torch.int32, device="cuda")
        mx = torch.empty(M, dtype=torch.float32, device="cuda")
        ls = torch.empty(M, dtype=torch.float32, device="cuda")
        assert call_noalloc(lib, hid, W, T, am, mx, ls) == 0
        assert binding.mirror_lmhead_noalloc_status(0) == (0, 0)
        logits = O.lmhead_logits(I.bf16_bits(hid), Wb)
        red = O.row_reduce(logits)
        got = am.cpu().numpy()
        for r in np.nonzero(got != red["argmax"])[0]:          # a flip only inside the logit error bound
            assert logits[r, red["argmax"][r]] - logits[r, got[r]] < 2e-3, r
        assert np.abs(mx.cpu().numpy() - red["maxlogit"]).max() <= 2e-3
        assert np.abs(ls.cpu().numpy() - red["lse"]).max() <= 2e-3
