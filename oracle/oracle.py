"""numpy/ctypes front end of the CPU oracle (oracle/mirror_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, the smoke check and the benchmark's
cpu_baseline / reference legs.  It imports nothing from the CUDA package.

All functions take host numpy arrays.  bf16 tensors are passed as uint16 bit
patterns (shape unchanged); results are fp64 / int32 numpy arrays.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional, Sequence

import numpy as np

from . import build as _build

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.oracle_overlap_mass.restype = C.c_double
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def tree(parent: Sequence[int]):
    """Ancestor matrix anc[i,j] (j == i or j above i) and node depths of the hypothesis tree (Sec. 3.1)."""
    par = _c(parent, np.int32)
    n = par.shape[0]
    anc = np.zeros((n, n), np.uint8)
    depth = np.zeros(n, np.int32)
    rc = lib().oracle_tree(_p(par), n, _p(anc), _p(depth))
    if rc != 0:
        raise ValueError("malformed parent array")
    return anc, depth


def branches(parent: Sequence[int], max_len: int):
    par = _c(parent, np.int32)
    n = par.shape[0]
    paths = np.full((max(n, 1), max_len), -1, np.int32)
    plen = np.zeros(max(n, 1), np.int32)
    nb = lib().oracle_branches(_p(par), n, max_len, _p(paths), _p(plen))
    if nb < 0:
        raise ValueError("a branch is longer than max_len")
    return paths[:nb].copy(), plen[:nb].copy()


def attention_layer(q, k_pool, v_pool, page_table, prefix_len, k_new, v_new, anc, scale: float,
                    want_weights: bool = False):
    """O1: branch-tree attention of one layer.  q [B,n,Hq,d], pools [pages,Hkv,P,d],
    k_new/v_new [B,n,Hkv,d] as uint16 bf16 bits.  Returns (out [B,n,Hq,d], lse [B,Hq,n], weights|None)."""
    q = _c(q, np.uint16); k_pool = _c(k_pool, np.uint16); v_pool = _c(v_pool, np.uint16)
    k_new = _c(k_new, np.uint16); v_new = _c(v_new, np.uint16)
    page_table = _c(page_table, np.int32); prefix_len = _c(prefix_len, np.int32)
    anc = _c(anc, np.uint8)
    B, n, Hq, d = q.shape
    _, Hkv, P, _ = k_pool.shape
    max_pages = page_table.shape[1]
    out = np.zeros((B, n, Hq, d), np.float64)
    lse = np.zeros((B, Hq, n), np.float64)
    w = np.zeros((B, n, Hq, max_pages * P + n), np.float64) if want_weights else None
    lib().oracle_attention_layer(_p(q), _p(k_pool), _p(v_pool), _p(page_table), C.c_int(max_pages),
                                 _p(prefix_len), _p(k_new), _p(v_new), _p(anc),
                                 B, n, Hq, Hkv, d, P, C.c_double(scale), _p(out), _p(lse), _p(w))
    return out, lse, w


def lmhead_logits(hidden, W):
    """O2: logits = hidden @ W^T in fp64.  hidden: uint16 bf16 bits [M,H] or float64 [M,H]; W uint16 [V,H]."""
    W = _c(W, np.uint16)
    V, H = W.shape
    if hidden.dtype == np.float64:
        hidden = _c(hidden, np.float64)
        M = hidden.shape[0]
        out = np.zeros((M, V), np.float64)
        lib().oracle_lmhead_logits_f64(_p(hidden), _p(W), M, V, H, _p(out))
    else:
        hidden = _c(hidden, np.uint16)
        M = hidden.shape[0]
        out = np.zeros((M, V), np.float64)
        lib().oracle_lmhead_logits(_p(hidden), _p(W), M, V, H, _p(out))
    return out


def row_reduce(logits, temperature: float = 1.0, topk: int = 0):
    """Per-row argmax (lowest id on ties), max logit, log-sum-exp of logits/T, and the sorted Top-k
    (ids, log-probs) message of Eq. 6."""
    logits = _c(logits, np.float64)
    M, V = logits.shape
    argmax = np.zeros(M, np.int32); mx = np.zeros(M, np.float64); lse = np.zeros(M, np.float64)
    tid = np.zeros((M, max(topk, 1)), np.int32); tlp = np.zeros((M, max(topk, 1)), np.float64)
    lib().oracle_row_reduce(_p(logits), M, V, C.c_double(temperature), topk, _p(argmax), _p(mx), _p(lse),
                            _p(tid), _p(tlp))
    return dict(argmax=argmax, maxlogit=mx, lse=lse, topk_id=tid[:, :topk], topk_logprob=tlp[:, :topk])


def _accept_out(B, max_len):
    return dict(n_accepted=np.zeros(B, np.int32), best_branch=np.zeros(B, np.int32),
                decide_row=np.zeros(B, np.int32), n_emitted=np.zeros(B, np.int32),
                emitted=np.full((B, max_len + 1), -1, np.int32),
                accepted_nodes=np.full((B, max_len), -1, np.int32), reuse_slot=np.zeros(B, np.int32))


def accept_greedy(tokens, target_argmax, parent, max_len: int, emit_bonus: bool = True, cand_ids=None):
    """O3: greedy acceptance (Eq. 3 / Eq. 10), branch selection, correction/bonus token, reuse lookup."""
    tokens = _c(tokens, np.int32); target_argmax = _c(target_argmax, np.int32); par = _c(parent, np.int32)
    B, n = tokens.shape
    cand = None if cand_ids is None else _c(cand_ids, np.int32)
    n_cand = 0 if cand is None else cand.shape[-1]
    o = _accept_out(B, max_len)
    rc = lib().oracle_accept_greedy(_p(tokens), _p(target_argmax), _p(par), B, n, max_len, int(emit_bonus),
                                    _p(cand), n_cand, _p(o["n_accepted"]), _p(o["best_branch"]),
                                    _p(o["decide_row"]), _p(o["n_emitted"]), _p(o["emitted"]),
                                    _p(o["accepted_nodes"]), _p(o["reuse_slot"]))
    if rc != 0:
        raise ValueError("bad tree")
    return o


def accept_spec(tokens, logits, lse, q_probs, u_accept, u_resample, parent, max_len: int,
                emit_bonus: bool = True, temperature: float = 1.0, cand_ids=None):
    """O3': speculative-sampling acceptance with residual resampling; also returns per-request margins."""
    tokens = _c(tokens, np.int32); par = _c(parent, np.int32)
    logits = _c(logits, np.float32); lse = _c(lse, np.float32); q_probs = _c(q_probs, np.float32)
    u_accept = _c(u_accept, np.float32); u_resample = _c(u_resample, np.float32)
    B, n = tokens.shape
    V = logits.shape[-1]
    cand = None if cand_ids is None else _c(cand_ids, np.int32)
    n_cand = 0 if cand is None else cand.shape[-1]
    o = _accept_out(B, max_len)
    o["margin"] = np.zeros(B, np.float64)
    rc = lib().oracle_accept_spec(_p(tokens), _p(logits), _p(lse), _p(q_probs), _p(u_accept), _p(u_resample),
                                  _p(par), B, n, V, max_len, int(emit_bonus), C.c_double(temperature),
                                  _p(cand), n_cand, _p(o["n_accepted"]), _p(o["best_branch"]),
                                  _p(o["decide_row"]), _p(o["n_emitted"]), _p(o["emitted"]),
                                  _p(o["accepted_nodes"]), _p(o["reuse_slot"]), _p(o["margin"]))
    if rc != 0:
        raise ValueError("bad tree")
    return o


def accept_tree(tokens, logits, lse, q_probs, u_accept, u_resample, parent, max_len: int,
                emit_bonus: bool = True, temperature: float = 1.0, cand_ids=None):
    """O3'': lossless acceptance over a token tree (sequential multi-round rejection over siblings)."""
    tokens = _c(tokens, np.int32); par = _c(parent, np.int32)
    logits = _c(logits, np.float32); lse = _c(lse, np.float32); q_probs = _c(q_probs, np.float32)
    u_accept = _c(u_accept, np.float32); u_resample = _c(u_resample, np.float32)
    B, n = tokens.shape
    V = logits.shape[-1]
    cand = None if cand_ids is None else _c(cand_ids, np.int32)
    n_cand = 0 if cand is None else cand.shape[-1]
    o = _accept_out(B, max_len)
    o["margin"] = np.zeros(B, np.float64)
    rc = lib().oracle_accept_tree(_p(tokens), _p(logits), _p(lse), _p(q_probs), _p(u_accept), _p(u_resample),
                                  _p(par), B, n, V, max_len, int(emit_bonus), C.c_double(temperature),
                                  _p(cand), n_cand, _p(o["n_accepted"]), _p(o["best_branch"]),
                                  _p(o["decide_row"]), _p(o["n_emitted"]), _p(o["emitted"]),
                                  _p(o["accepted_nodes"]), _p(o["reuse_slot"]), _p(o["margin"]))
    if rc != 0:
        raise ValueError("bad tree")
    return o


def kv_commit(k_pool, v_pool, page_table, prefix_len, k_new, v_new, accepted_nodes, n_accepted, page_size: int = 16):
    """Roll-forward of the paged cache after a verify step (Sec. 3.1): for every request the K/V rows of the root and
    of its accepted nodes, in path order, become tokens prefix_len .. prefix_len + A of every layer and head; the
    prefix grows by A + 1.  Pools are [L, num_pages, Hkv, page, d] arrays of bf16 bit patterns (uint16), k_new / v_new
    [L, B, n, Hkv, d].  Returns new (k_pool, v_pool, prefix_len); the inputs are not modified."""
    k_pool = np.array(k_pool, copy=True); v_pool = np.array(v_pool, copy=True)
    page_table = np.asarray(page_table); prefix_len = np.array(prefix_len, copy=True)
    accepted_nodes = np.asarray(accepted_nodes); n_accepted = np.asarray(n_accepted)
    B = prefix_len.shape[0]
    for b in range(B):
        nodes = [0] + [int(c) for c in accepted_nodes[b, :int(n_accepted[b])]]
        for j, node in enumerate(nodes):
            pos = int(prefix_len[b]) + j
            page, slot = int(page_table[b, pos // page_size]), pos % page_size
            k_pool[:, page, :, slot, :] = k_new[:, b, node]
            v_pool[:, page, :, slot, :] = v_new[:, b, node]
        prefix_len[b] += len(nodes)
    return k_pool, v_pool, prefix_len


def overlap_mass(q_final, ids) -> float:
    """Eq. 7: Omega_kappa, the final distribution's mass on the early-exit Top-kappa ids."""
    q_final = _c(q_final, np.float64); ids = _c(ids, np.int32)
    return float(lib().oracle_overlap_mass(_p(q_final), _p(ids), ids.shape[0]))


def trie_build(branch_tokens, root_token: int):
    """Token tree without duplicated prefixes out of kappa branches of gamma tokens (the branch-complete proposal of
    Sec. 3.1 as a tree, "tree drafts"): branches that agree on their first r tokens share their first r nodes.  Written
    as the definition: a node per distinct non-empty prefix, numbered in order of first appearance (branch by branch,
    left to right), parent = the node of the prefix one token shorter (the root for length 1).
    Returns (parent [n], tokens [n], node_of [kappa, gamma])."""
    bt = np.asarray(branch_tokens, np.int64)
    kappa, gamma = bt.shape
    ids = {(): 0}
    parent, tokens = [-1], [int(root_token)]
    node_of = np.zeros((kappa, gamma), np.int32)
    for i in range(kappa):
        for j in range(gamma):
            pre = tuple(int(t) for t in bt[i, :j + 1])
            if pre not in ids:
                ids[pre] = len(parent)
                parent.append(ids[pre[:-1]])
                tokens.append(pre[-1])
            node_of[i, j] = ids[pre]
    return np.asarray(parent, np.int32), np.asarray(tokens, np.int32), node_of
