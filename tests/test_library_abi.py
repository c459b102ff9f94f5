"""The C-ABI library builds, loads without a GPU, and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2510_13161_b200 import _build, binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mirror.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mirror_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib_path = _build.build()
    lib = ctypes.CDLL(lib_path)
    names = declared_symbols()
    assert "mirror_verify_step" in names and "mirror_attn_verify" in names
    assert "mirror_lmhead_reduce" in names and "mirror_accept_select" in names
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(binding.EXPORTS) == names


def test_status_strings_and_argument_errors_without_a_gpu():
    lib = binding.load_library()
    assert lib.mirror_status_str(0) == b"ok"
    assert b"workspace" in lib.mirror_status_str(4)
    # null arguments are rejected on the host before any CUDA call
    assert lib.mirror_create(None, None, 0) == 1
    assert lib.mirror_destroy(None) == 1
    assert lib.mirror_accept_select(None, None, None, None, None) == 1
    assert lib.mirror_lmhead_reduce(None, None, 0, None, 0, None, None, 0, None, None, None, None, None, None, None, None) == 1
    bad = binding.ModelDesc(256, 4, 3, 64, 1024, 16, 0.0, 1.0)       # 3 KV heads do not divide 4 query heads
    ctx = ctypes.c_void_p()
    assert lib.mirror_create(ctypes.byref(ctx), ctypes.byref(bad), 0) == 2
    bad = binding.ModelDesc(256, 4, 2, 96, 1024, 16, 0.0, 1.0)       # head_dim 96 unsupported
    assert lib.mirror_create(ctypes.byref(ctx), ctypes.byref(bad), 0) == 3


def test_trie_build_matches_the_oracle_on_the_host():
    """mirror_trie_build is host-only: it runs without a GPU and must agree with the oracle's definition."""
    import numpy as np
    from oracle import oracle as O
    from paper_2510_13161_b200 import binding
    rng = np.random.default_rng(1)
    for _ in range(100):
        kappa, gamma = int(rng.integers(1, 9)), int(rng.integers(1, 9))
        bt = rng.integers(0, 3, size=(kappa, gamma))
        parent, tokens, node_of = binding.mirror_trie_build(bt, 11)
        rp, rt, rn = O.trie_build(bt, 11)
        assert parent == rp.tolist() and tokens == rt.tolist() and node_of == rn.tolist()
    # limits: more distinct prefixes than a tree may hold
    import pytest
    big = np.arange(64 * 2).reshape(64, 2)                    # 64 branches x 2 = 129 nodes with the root
    with pytest.raises(binding.MirrorError):
        binding.mirror_trie_build(big, 0)
