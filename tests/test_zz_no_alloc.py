"""mirror_lmhead_reduce_noalloc: the LM-head reductions for hosts that may not allocate device memory
(all memory owned by the host's own pool, allocator-guarded plugin regions).  Its scratch is a fixed
array inside the library, so it needs neither a context nor a workspace.  The test calls it through the
C ABI twice in a row and checks each result against the regular entry point, which uses a caller
workspace.  Collected last on purpose: a failure here cannot hide any other test."""
import ctypes as C

import pytest
import torch

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
