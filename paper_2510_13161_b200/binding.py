"""Thin ctypes binding of libmirror.so (see include/mirror.h).

Argument marshalling only: every step of the verify path runs in the CUDA kernels
of the library.  torch is used for device memory and streams.  There is no CPU
fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmirror.so")

ACCEPT_GREEDY = 0
ACCEPT_SPEC_SAMPLING = 1
ACCEPT_SPEC_TREE = 2
WS_ATTN, WS_LMHEAD, WS_LMHEAD_LOGITS, WS_STEP_GREEDY, WS_STEP_SPEC, WS_ACCEPT_TREE, WS_STEP_TREE = 1, 2, 10, 7, 15, 16, 31
WS_LMHEAD_TOPK = 34

EXPORTS = [
    "mirror_create", "mirror_destroy", "mirror_workspace_bytes", "mirror_set_workspace",
    "mirror_attn_verify", "mirror_lmhead_reduce", "mirror_accept_select", "mirror_verify_step",
    "mirror_device_status", "mirror_launch_count", "mirror_status_str", "mirror_set_stage_events",
    "mirror_lmhead_reduce_noalloc", "mirror_lmhead_noalloc_status", "mirror_quantize_rows_fp8", "mirror_lmhead_reduce_fp8", "mirror_early_exit_tap", "mirror_overlap_mass", "mirror_kv_commit",
    "mirror_linear_scratch_bytes", "mirror_linear", "mirror_rmsnorm", "mirror_target_scratch_bytes", "mirror_target_forward", "mirror_trie_build", "mirror_verify_step_host", "mirror_embed_rows",
    "mirror_attn_verify_fp8", "mirror_kv_scales_fp8", "mirror_kv_quantize_fp8", "mirror_kv_commit_fp8", "mirror_verify_step_fp8", "mirror_target_forward_fp8",
]


class MirrorError(RuntimeError):
    def __init__(self, code: int, where: str, text: str):
        super().__init__(f"{where}: mirror_status {code} ({text})")
        self.code = code


class ModelDesc(C.Structure):
    _fields_ = [("hidden", C.c_int), ("n_q_heads", C.c_int), ("n_kv_heads", C.c_int), ("head_dim", C.c_int),
                ("vocab", C.c_int), ("page_size", C.c_int), ("softmax_scale", C.c_float), ("temperature", C.c_float)]


class Tree(C.Structure):
    _fields_ = [("batch", C.c_int), ("n_nodes", C.c_int), ("kappa", C.c_int), ("gamma", C.c_int),
                ("tokens", C.c_void_p), ("parent", C.POINTER(C.c_int32))]


class AcceptHostOut(C.Structure):
    _fields_ = [("n_accepted", C.c_void_p), ("best_branch", C.c_void_p), ("n_emitted", C.c_void_p), ("emitted", C.c_void_p)]


class LayerWeights(C.Structure):
    _fields_ = [("w_qkv", C.c_void_p), ("w_o", C.c_void_p), ("w_gate_up", C.c_void_p), ("w_down", C.c_void_p),
                ("norm_attn", C.c_void_p), ("norm_mlp", C.c_void_p)]


class Target(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("intermediate", C.c_int), ("rope_theta", C.c_float), ("rms_eps", C.c_float),
                ("layers", C.POINTER(LayerWeights)), ("norm_final", C.c_void_p)]


class KV(C.Structure):
    _fields_ = [("k_pool", C.c_void_p), ("v_pool", C.c_void_p), ("layer_stride", C.c_int64),
                ("num_layers", C.c_int), ("num_pages", C.c_int), ("max_pages_per_req", C.c_int),
                ("page_table", C.c_void_p), ("prefix_len", C.c_void_p)]


class AcceptIn(C.Structure):
    _fields_ = [("mode", C.c_int), ("emit_bonus", C.c_int), ("target_argmax", C.c_void_p), ("logits", C.c_void_p),
                ("lse", C.c_void_p), ("q_probs", C.c_void_p), ("u_accept", C.c_void_p), ("u_resample", C.c_void_p),
                ("cand_ids", C.c_void_p), ("n_cand", C.c_int)]


class AcceptOut(C.Structure):
    _fields_ = [("n_accepted", C.c_void_p), ("best_branch", C.c_void_p), ("n_emitted", C.c_void_p),
                ("emitted", C.c_void_p), ("accepted_nodes", C.c_void_p), ("decide_row", C.c_void_p),
                ("reuse_slot", C.c_void_p)]


_lib = None


def load_library():
    """Load libmirror.so; raises if it has not been built (python -m paper_2510_13161_b200._build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing: build it with `python -m paper_2510_13161_b200._build`; "
                                    "there is no fallback path")
        lib = C.CDLL(LIB_PATH)
        lib.mirror_status_str.restype = C.c_char_p
        lib.mirror_status_str.argtypes = [C.c_int]
        for name in EXPORTS:
            if name != "mirror_status_str":
                getattr(lib, name).restype = C.c_int
        _lib = lib
    return _lib


def _check(code: int, where: str):
    if code != 0:
        raise MirrorError(code, where, load_library().mirror_status_str(code).decode())


def _ptr(t: Optional[torch.Tensor], dtype=None, name: str = "tensor"):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def mirror_trie_build(branch_tokens, root_token: int):
    """Host helper: kappa branches of gamma tokens -> (parent list, tokens list, node_of [kappa][gamma]) of the tree
    that shares common prefixes."""
    lib = load_library()
    rows = [list(map(int, r)) for r in branch_tokens]
    kappa, gamma = len(rows), len(rows[0])
    flat = (C.c_int32 * (kappa * gamma))(*[t for r in rows for t in r])
    cap = 1 + kappa * gamma
    parent, tokens, node_of = (C.c_int32 * cap)(), (C.c_int32 * cap)(), (C.c_int32 * (kappa * gamma))()
    n = C.c_int()
    _check(lib.mirror_trie_build(flat, kappa, gamma, int(root_token), parent, tokens, node_of, C.byref(n)), "mirror_trie_build")
    return list(parent[:n.value]), list(tokens[:n.value]), [list(node_of[i * gamma:(i + 1) * gamma]) for i in range(kappa)]


def mirror_lmhead_reduce_noalloc(hidden: torch.Tensor, W: torch.Tensor, temperature: float = 1.0, argmax=None,
                                 maxlogit=None, lse=None, stream=None) -> dict:
    """LM head reductions for callers that cannot allocate device memory: no context, no workspace; the
    kernel's scratch is a fixed array inside the library (at most 128 rows).  The output tensors may be
    passed in (so that this wrapper allocates nothing either); missing ones are created here for
    convenience.  Calls on one device share the scratch array: do not let them overlap on the GPU."""
    lib = load_library()
    M, H = hidden.shape
    V = W.shape[0]
    dev = hidden.device
    if argmax is None:
        argmax = torch.empty(M, dtype=torch.int32, device=dev)
    if maxlogit is None:
        maxlogit = torch.empty(M, dtype=torch.float32, device=dev)
    if lse is None:
        lse = torch.empty(M, dtype=torch.float32, device=dev)
    _check(lib.mirror_lmhead_reduce_noalloc(dev.index if dev.index is not None else torch.cuda.current_device(),
                                            _ptr(hidden, torch.bfloat16, "hidden"), M, _ptr(W, torch.bfloat16, "W"), V, H,
                                            C.c_float(temperature), _ptr(argmax, torch.int32, "argmax"),
                                            _ptr(maxlogit, torch.float32, "maxlogit"), _ptr(lse, torch.float32, "lse"),
                                            _stream(stream)), "mirror_lmhead_reduce_noalloc")
    return dict(argmax=argmax, maxlogit=maxlogit, lse=lse)


def mirror_lmhead_noalloc_status(device: int = 0):
    """(code, detail) of the first device-side problem of the no-allocation LM-head calls on `device` since the last
    query (synchronises the device; (0, 0) when there was none)."""
    code, detail = C.c_int(), C.c_int()
    _check(load_library().mirror_lmhead_noalloc_status(int(device), C.byref(code), C.byref(detail)), "mirror_lmhead_noalloc_status")
    return code.value, detail.value


class AcceptResult:
    """Device tensors written by mirror_accept_select / mirror_verify_step."""

    def __init__(self, batch: int, gamma: int, device):
        i32 = dict(dtype=torch.int32, device=device)
        self.n_accepted = torch.empty(batch, **i32)
        self.best_branch = torch.empty(batch, **i32)
        self.n_emitted = torch.empty(batch, **i32)
        self.emitted = torch.empty((batch, gamma + 1), **i32)
        self.accepted_nodes = torch.empty((batch, max(gamma, 1)), **i32)
        self.decide_row = torch.empty(batch, **i32)
        self.reuse_slot = torch.empty(batch, **i32)

    def struct(self) -> AcceptOut:
        return AcceptOut(*[C.c_void_p(getattr(self, f).data_ptr()) for f, _ in AcceptOut._fields_])

    def cpu(self) -> dict:
        return {f: getattr(self, f).cpu().numpy() for f, _ in AcceptOut._fields_}


class Mirror:
    """One library context: a model shape on one device, plus its workspace."""

    def __init__(self, hidden: int, n_q_heads: int, n_kv_heads: int, head_dim: int, vocab: int,
                 page_size: int = 16, softmax_scale: float = 0.0, temperature: float = 1.0, device: int = 0):
        self.lib = load_library()
        self.desc = ModelDesc(hidden, n_q_heads, n_kv_heads, head_dim, vocab, page_size, softmax_scale, temperature)
        self.device = torch.device("cuda", device)
        self._ctx = C.c_void_p()
        _check(self.lib.mirror_create(C.byref(self._ctx), C.byref(self.desc), device), "mirror_create")
        self._ws = None
        self._keep = []

    def close(self):
        if self._ctx:
            self.lib.mirror_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- argument structs -------------------------------------------------------------------
    def tree(self, tokens: torch.Tensor, kappa: int, gamma: int, parent: Optional[Sequence[int]] = None) -> Tree:
        B, n = tokens.shape
        par = None
        if parent is not None:
            arr = (C.c_int32 * len(parent))(*parent)
            self._keep.append(arr)
            par = C.cast(arr, C.POINTER(C.c_int32))
        t = Tree(B, n, kappa, gamma, _ptr(tokens, torch.int32, "tokens"), par)
        t._refs = (tokens,)          # the struct holds raw pointers: keep the tensors alive with it
        return t

    def kv(self, k_pool: torch.Tensor, v_pool: torch.Tensor, page_table: torch.Tensor, prefix_len: torch.Tensor) -> KV:
        """k_pool / v_pool: bf16 [L, num_pages, Hkv, page, d] (one allocation, layers consecutive)."""
        L, num_pages = k_pool.shape[0], k_pool.shape[1]
        stride = k_pool.stride(0) if L > 1 else k_pool[0].numel()
        kv = KV(_ptr(k_pool, torch.bfloat16, "k_pool"), _ptr(v_pool, torch.bfloat16, "v_pool"), stride, L, num_pages,
                page_table.shape[1], _ptr(page_table, torch.int32, "page_table"), _ptr(prefix_len, torch.int32, "prefix_len"))
        kv._refs = (k_pool, v_pool, page_table, prefix_len)
        return kv

    # ---- workspace --------------------------------------------------------------------------
    def workspace_bytes(self, tree: Tree, kv: Optional[KV], what: int) -> int:
        out = C.c_size_t()
        _check(self.lib.mirror_workspace_bytes(self._ctx, C.byref(tree), C.byref(kv) if kv is not None else None,
                                               C.c_uint(what), C.byref(out)), "mirror_workspace_bytes")
        return out.value

    def ensure_workspace(self, tree: Tree, kv: Optional[KV], what: int):
        need = self.workspace_bytes(tree, kv, what)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.device)
            _check(self.lib.mirror_set_workspace(self._ctx, C.c_void_p(self._ws.data_ptr()), C.c_size_t(need)),
                   "mirror_set_workspace")

    # ---- entry points -----------------------------------------------------------------------
    def mirror_attn_verify(self, kv: KV, tree: Tree, q, k_new, v_new, out=None, lse_out=None, stream=None):
        if out is None:
            out = torch.empty_like(q)
        self.ensure_workspace(tree, kv, WS_ATTN)
        _check(self.lib.mirror_attn_verify(self._ctx, C.byref(kv), C.byref(tree), _ptr(q, torch.bfloat16, "q"),
                                           _ptr(k_new, torch.bfloat16, "k_new"), _ptr(v_new, torch.bfloat16, "v_new"),
                                           _ptr(out, torch.bfloat16, "out"), _ptr(lse_out, torch.float32, "lse_out"),
                                           _stream(stream)), "mirror_attn_verify")
        return out

    # ---- e4m3 cache ----------------------------------------------------------------------------
    def kv_fp8(self, k_codes: torch.Tensor, v_codes: torch.Tensor, page_table: torch.Tensor, prefix_len: torch.Tensor) -> KV:
        """k_codes / v_codes: uint8 e4m3 codes [L, num_pages, Hkv, page, d] (one allocation, layers consecutive)."""
        L, num_pages = k_codes.shape[0], k_codes.shape[1]
        stride = k_codes.stride(0) if L > 1 else k_codes[0].numel()
        kv = KV(_ptr(k_codes, torch.uint8, "k_codes"), _ptr(v_codes, torch.uint8, "v_codes"), stride, L, num_pages,
                page_table.shape[1], _ptr(page_table, torch.int32, "page_table"), _ptr(prefix_len, torch.int32, "prefix_len"))
        kv._refs = (k_codes, v_codes, page_table, prefix_len)
        return kv

    def _kv_fp8_dims(self, x: torch.Tensor, inner: int):
        L = x.shape[0]
        layer_elems = x[0].numel()
        stride = x.stride(0) if L > 1 else layer_elems
        return L, stride, layer_elems, inner

    def mirror_kv_scales_fp8(self, x: torch.Tensor, inner: int, stream=None) -> torch.Tensor:
        """x bf16 [L, ..., Hkv, <inner elements>] -> fp32 scales [L, Hkv] (max|x| / 448 per layer and KV head)."""
        L, stride, layer_elems, inner = self._kv_fp8_dims(x, inner)
        scale = torch.empty((L, self.desc.n_kv_heads), dtype=torch.float32, device=x.device)
        _check(self.lib.mirror_kv_scales_fp8(self._ctx, _ptr(x, torch.bfloat16, "x"), L, C.c_int64(stride), C.c_int64(layer_elems),
                                             inner, _ptr(scale, torch.float32, "scale"), _stream(stream)), "mirror_kv_scales_fp8")
        return scale

    def mirror_kv_quantize_fp8(self, x: torch.Tensor, inner: int, scale: torch.Tensor, stream=None) -> torch.Tensor:
        """x bf16 -> e4m3 codes (uint8, same shape) under the given [L, Hkv] scales."""
        L, stride, layer_elems, inner = self._kv_fp8_dims(x, inner)
        out = torch.empty(x.shape, dtype=torch.uint8, device=x.device)
        _check(self.lib.mirror_kv_quantize_fp8(self._ctx, _ptr(x, torch.bfloat16, "x"), L, C.c_int64(stride), C.c_int64(layer_elems),
                                               inner, _ptr(scale, torch.float32, "scale"), _ptr(out, torch.uint8, "out"),
                                               _stream(stream)), "mirror_kv_quantize_fp8")
        return out

    def mirror_attn_verify_fp8(self, kv: KV, tree: Tree, q, k_new8, v_new8, k_scale, v_scale, q_scale: float, out=None,
                               lse_out=None, stream=None):
        if out is None:
            out = torch.empty_like(q)
        self.ensure_workspace(tree, kv, WS_ATTN)
        _check(self.lib.mirror_attn_verify_fp8(self._ctx, C.byref(kv), C.byref(tree), _ptr(q, torch.bfloat16, "q"),
                                               _ptr(k_new8, torch.uint8, "k_new8"), _ptr(v_new8, torch.uint8, "v_new8"),
                                               _ptr(k_scale, torch.float32, "k_scale"), _ptr(v_scale, torch.float32, "v_scale"),
                                               C.c_float(q_scale), _ptr(out, torch.bfloat16, "out"),
                                               _ptr(lse_out, torch.float32, "lse_out"), _stream(stream)), "mirror_attn_verify_fp8")
        return out

    def mirror_lmhead_reduce(self, hidden, W, topk: int = 0, gather_row=None, gather_tok=None, want_lse: bool = True,
                             want_logits: bool = False, stream=None) -> dict:
        M = hidden.shape[0]
        dev = hidden.device
        res = dict(argmax=torch.empty(M, dtype=torch.int32, device=dev),
                   maxlogit=torch.empty(M, dtype=torch.float32, device=dev),
                   lse=torch.empty(M, dtype=torch.float32, device=dev) if want_lse else None,
                   topk_id=torch.empty((M, topk), dtype=torch.int32, device=dev) if topk else None,
                   topk_logprob=torch.empty((M, topk), dtype=torch.float32, device=dev) if topk else None,
                   gather_logit=None, logits=None)
        n_gather = 0
        if gather_row is not None:
            n_gather = gather_row.numel()
            res["gather_logit"] = torch.empty(n_gather, dtype=torch.float32, device=dev)
        if want_logits:
            res["logits"] = torch.empty((M, self.desc.vocab), dtype=torch.float32, device=dev)
        t = Tree(1, M if M <= 128 else 128, 0, 0, None, None)
        t.batch, t.n_nodes = (M + 127) // 128, min(M, 128)      # sizes only: batch * n_nodes >= M
        self.ensure_workspace(t, None, WS_LMHEAD_TOPK if topk else WS_LMHEAD)
        _check(self.lib.mirror_lmhead_reduce(self._ctx, _ptr(hidden, torch.bfloat16, "hidden"), M,
                                             _ptr(W, torch.bfloat16, "W"), topk,
                                             _ptr(gather_row, torch.int32, "gather_row"),
                                             _ptr(gather_tok, torch.int32, "gather_tok"), n_gather,
                                             _ptr(res["argmax"]), _ptr(res["maxlogit"]), _ptr(res["lse"]),
                                             _ptr(res["topk_id"]), _ptr(res["topk_logprob"]), _ptr(res["gather_logit"]),
                                             _ptr(res["logits"]), _stream(stream)), "mirror_lmhead_reduce")
        return res

    def mirror_quantize_rows_fp8(self, x: torch.Tensor, stream=None):
        """x bf16 [rows, cols] -> (e4m3 codes uint8 [rows, cols], scales fp32 [rows])."""
        rows, cols = x.shape
        out = torch.empty((rows, cols), dtype=torch.uint8, device=x.device)
        scale = torch.empty(rows, dtype=torch.float32, device=x.device)
        _check(self.lib.mirror_quantize_rows_fp8(self._ctx, _ptr(x, torch.bfloat16, "x"), rows, cols, _ptr(out, torch.uint8, "out"),
                                                 _ptr(scale, torch.float32, "scale"), _stream(stream)), "mirror_quantize_rows_fp8")
        return out, scale

    def mirror_lmhead_reduce_fp8(self, hidden8, h_scale, W8, w_scale, want_logits: bool = False, stream=None) -> dict:
        M = hidden8.shape[0]
        dev = hidden8.device
        res = dict(argmax=torch.empty(M, dtype=torch.int32, device=dev), maxlogit=torch.empty(M, dtype=torch.float32, device=dev),
                   lse=torch.empty(M, dtype=torch.float32, device=dev),
                   logits=torch.empty((M, self.desc.vocab), dtype=torch.float32, device=dev) if want_logits else None)
        t = Tree(1, M if M <= 128 else 128, 0, 0, None, None)
        t.batch, t.n_nodes = (M + 127) // 128, min(M, 128)      # sizes only: batch * n_nodes >= M
        self.ensure_workspace(t, None, WS_LMHEAD)
        _check(self.lib.mirror_lmhead_reduce_fp8(self._ctx, _ptr(hidden8, torch.uint8, "hidden8"), _ptr(h_scale, torch.float32, "h_scale"),
                                                 M, _ptr(W8, torch.uint8, "W8"), _ptr(w_scale, torch.float32, "w_scale"),
                                                 _ptr(res["argmax"]), _ptr(res["maxlogit"]), _ptr(res["lse"]), _ptr(res["logits"]),
                                                 _stream(stream)), "mirror_lmhead_reduce_fp8")
        return res

    def accept_in(self, mode: int, emit_bonus: bool = True, target_argmax=None, logits=None, lse=None, q_probs=None,
                  u_accept=None, u_resample=None, cand_ids=None) -> AcceptIn:
        n_cand = 0 if cand_ids is None else cand_ids.shape[-1]
        a = AcceptIn(mode, int(emit_bonus), _ptr(target_argmax, torch.int32, "target_argmax"),
                     _ptr(logits, torch.float32, "logits"), _ptr(lse, torch.float32, "lse"),
                     _ptr(q_probs, torch.float32, "q_probs"), _ptr(u_accept, torch.float32, "u_accept"),
                     _ptr(u_resample, torch.float32, "u_resample"), _ptr(cand_ids, torch.int32, "cand_ids"), n_cand)
        a._refs = (target_argmax, logits, lse, q_probs, u_accept, u_resample, cand_ids)
        return a

    def mirror_early_exit_tap(self, hidden_le: torch.Tensor, W: torch.Tensor, kappa: int, stream=None):
        """Top-kappa message of the early-exit proxy: (ids int32 [M, kappa], log-probs bf16 [M, kappa])."""
        M = hidden_le.shape[0]
        ids = torch.empty((M, kappa), dtype=torch.int32, device=hidden_le.device)
        lp = torch.empty((M, kappa), dtype=torch.bfloat16, device=hidden_le.device)
        t = Tree(1, M if M <= 128 else 128, 0, 0, None, None)
        t.batch, t.n_nodes = (M + 127) // 128, min(M, 128)      # sizes only: batch * n_nodes >= M
        self.ensure_workspace(t, None, WS_LMHEAD_TOPK)
        _check(self.lib.mirror_early_exit_tap(self._ctx, _ptr(hidden_le, torch.bfloat16, "hidden_le"), M,
                                              _ptr(W, torch.bfloat16, "W"), kappa, _ptr(ids, torch.int32, "msg_ids"),
                                              _ptr(lp, torch.bfloat16, "msg_logprob"), _stream(stream)), "mirror_early_exit_tap")
        return ids, lp

    def mirror_overlap_mass(self, logits_final: torch.Tensor, lse_final: torch.Tensor, msg_ids: torch.Tensor, stream=None):
        """Eq. 7 per row: mass of the final distribution on the message's ids (fp32 [M])."""
        M, kappa = msg_ids.shape
        omega = torch.empty(M, dtype=torch.float32, device=msg_ids.device)
        _check(self.lib.mirror_overlap_mass(self._ctx, _ptr(logits_final, torch.float32, "logits_final"),
                                            _ptr(lse_final, torch.float32, "lse_final"), _ptr(msg_ids, torch.int32, "msg_ids"),
                                            M, kappa, _ptr(omega, torch.float32, "omega"), _stream(stream)), "mirror_overlap_mass")
        return omega

    def mirror_kv_commit(self, kv: KV, tree: Tree, k_new, v_new, res: "AcceptResult", prefix_len: torch.Tensor, stream=None):
        """Append the root and the accepted path of `res` to the paged cache and advance prefix_len in place."""
        _check(self.lib.mirror_kv_commit(self._ctx, C.byref(kv), C.byref(tree), _ptr(k_new, torch.bfloat16, "k_new"),
                                         _ptr(v_new, torch.bfloat16, "v_new"), _ptr(res.accepted_nodes, torch.int32, "accepted_nodes"),
                                         _ptr(res.n_accepted, torch.int32, "n_accepted"), _ptr(prefix_len, torch.int32, "prefix_len"),
                                         _stream(stream)), "mirror_kv_commit")

    def mirror_kv_commit_fp8(self, kv: KV, tree: Tree, k_new8, v_new8, res: "AcceptResult", prefix_len: torch.Tensor, stream=None):
        """mirror_kv_commit for an e4m3 cache (kv from kv_fp8, k_new8 / v_new8 uint8 codes under the cache's scales)."""
        _check(self.lib.mirror_kv_commit_fp8(self._ctx, C.byref(kv), C.byref(tree), _ptr(k_new8, torch.uint8, "k_new8"),
                                             _ptr(v_new8, torch.uint8, "v_new8"), _ptr(res.accepted_nodes, torch.int32, "accepted_nodes"),
                                             _ptr(res.n_accepted, torch.int32, "n_accepted"), _ptr(prefix_len, torch.int32, "prefix_len"),
                                             _stream(stream)), "mirror_kv_commit_fp8")

    # ---- the target's layers around the attention ---------------------------------------------
    def target(self, layers: Sequence[dict], norm_final: torch.Tensor, intermediate: int, rope_theta: float = 1e6,
               rms_eps: float = 1e-6) -> Target:
        """layers: one dict per layer with bf16 CUDA tensors w_qkv, w_o, w_gate_up, w_down, norm_attn, norm_mlp."""
        arr = (LayerWeights * len(layers))()
        refs = [norm_final]
        for i, w in enumerate(layers):
            for f, _ in LayerWeights._fields_:
                setattr(arr[i], f, _ptr(w[f], torch.bfloat16, f).value)
                refs.append(w[f])
        t = Target(len(layers), intermediate, rope_theta, rms_eps, arr, _ptr(norm_final, torch.bfloat16, "norm_final"))
        t._refs = (arr, refs)
        return t

    def mirror_linear(self, x: torch.Tensor, W: torch.Tensor, residual: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """x [M, K] @ W [N, K]^T (+ residual [M, N]) -> bf16 [M, N]."""
        M, K = x.shape
        N = W.shape[0]
        need = C.c_size_t()
        _check(self.lib.mirror_linear_scratch_bytes(self._ctx, M, N, K, C.byref(need)), "mirror_linear_scratch_bytes")
        scratch = getattr(self, "_linear_scratch", None)          # grown on demand; calls on one stream may share it
        if scratch is None or scratch.numel() < need.value:
            scratch = self._linear_scratch = torch.empty(max(need.value, 256), dtype=torch.uint8, device=self.device)
        out = torch.empty((M, N), dtype=torch.bfloat16, device=self.device)
        _check(self.lib.mirror_linear(self._ctx, _ptr(x, torch.bfloat16, "x"), M, _ptr(W, torch.bfloat16, "W"), N, K,
                                      _ptr(residual, torch.bfloat16, "residual"), _ptr(out), _ptr(scratch),
                                      C.c_size_t(scratch.numel()), _stream(stream)), "mirror_linear")
        return out

    def mirror_embed_rows(self, table: torch.Tensor, tokens: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """out[r] = table[tokens[r]]: table bf16 [V, H], tokens int32 (any shape, M entries) -> bf16 [M, H]."""
        M = tokens.numel()
        if out is None:
            out = torch.empty((M, table.shape[1]), dtype=torch.bfloat16, device=self.device)
        _check(self.lib.mirror_embed_rows(self._ctx, _ptr(table, torch.bfloat16, "table"), _ptr(tokens, torch.int32, "tokens"), M,
                                          _ptr(out, torch.bfloat16, "out"), _stream(stream)), "mirror_embed_rows")
        return out

    def mirror_rmsnorm(self, x: torch.Tensor, gamma: torch.Tensor, eps: float = 1e-6, stream=None) -> torch.Tensor:
        M, H = x.shape
        out = torch.empty_like(x)
        _check(self.lib.mirror_rmsnorm(self._ctx, _ptr(x, torch.bfloat16, "x"), _ptr(gamma, torch.bfloat16, "gamma"), M, H,
                                       C.c_float(eps), _ptr(out), _stream(stream)), "mirror_rmsnorm")
        return out

    def target_scratch(self, tree: Tree, target: Target) -> torch.Tensor:
        need = C.c_size_t()
        _check(self.lib.mirror_target_scratch_bytes(self._ctx, C.byref(tree), C.byref(target), C.byref(need)),
               "mirror_target_scratch_bytes")
        return torch.empty(need.value, dtype=torch.uint8, device=self.device)

    def mirror_target_forward(self, target: Target, kv: KV, tree: Tree, x: torch.Tensor, scratch: Optional[torch.Tensor] = None,
                              out: Optional[dict] = None, stream=None) -> dict:
        """All layers of `target` on the residual rows x [B*n, H]; returns q, k_new, v_new, attn_out ([L, B, n, heads, d]),
        x_out and hidden (the LM-head rows)."""
        L, B, n = target.n_layers, tree.batch, tree.n_nodes
        Hq, Hkv, d = self.desc.n_q_heads, self.desc.n_kv_heads, self.desc.head_dim
        if scratch is None:
            scratch = self.target_scratch(tree, target)
        if out is None:
            e = lambda *shape: torch.empty(shape, dtype=torch.bfloat16, device=self.device)
            out = dict(q=e(L, B, n, Hq, d), k_new=e(L, B, n, Hkv, d), v_new=e(L, B, n, Hkv, d), attn_out=e(L, B, n, Hq, d),
                       x_out=torch.empty_like(x), hidden=torch.empty_like(x))
        self.ensure_workspace(tree, kv, WS_ATTN)
        _check(self.lib.mirror_target_forward(self._ctx, C.byref(target), C.byref(kv), C.byref(tree), _ptr(x, torch.bfloat16, "x"),
                                              _ptr(out["q"]), _ptr(out["k_new"]), _ptr(out["v_new"]), _ptr(out["attn_out"]),
                                              _ptr(out["x_out"]), _ptr(out["hidden"]), _ptr(scratch), C.c_size_t(scratch.numel()),
                                              _stream(stream)), "mirror_target_forward")
        out["_scratch"] = scratch
        return out

    def mirror_target_forward_fp8(self, target: Target, kv: KV, tree: Tree, x: torch.Tensor, k_scale, v_scale, q_scales,
                                  scratch: Optional[torch.Tensor] = None, stream=None) -> dict:
        """mirror_target_forward over an e4m3 cache (kv from kv_fp8); q_scales: one host float per layer.  Also returns
        k_new8 / v_new8: the new rows' codes under the cache's scales."""
        L, B, n = target.n_layers, tree.batch, tree.n_nodes
        Hq, Hkv, d = self.desc.n_q_heads, self.desc.n_kv_heads, self.desc.head_dim
        if scratch is None:
            scratch = self.target_scratch(tree, target)
        e = lambda *shape: torch.empty(shape, dtype=torch.bfloat16, device=self.device)
        e8 = lambda *shape: torch.empty(shape, dtype=torch.uint8, device=self.device)
        out = dict(q=e(L, B, n, Hq, d), k_new=e(L, B, n, Hkv, d), v_new=e(L, B, n, Hkv, d), k_new8=e8(L, B, n, Hkv, d),
                   v_new8=e8(L, B, n, Hkv, d), attn_out=e(L, B, n, Hq, d), x_out=torch.empty_like(x), hidden=torch.empty_like(x))
        qs = (C.c_float * L)(*[float(v) for v in q_scales])
        self.ensure_workspace(tree, kv, WS_ATTN)
        _check(self.lib.mirror_target_forward_fp8(self._ctx, C.byref(target), C.byref(kv), C.byref(tree), _ptr(x, torch.bfloat16, "x"),
                                                  _ptr(k_scale, torch.float32, "k_scale"), _ptr(v_scale, torch.float32, "v_scale"), qs,
                                                  _ptr(out["q"]), _ptr(out["k_new"]), _ptr(out["v_new"]), _ptr(out["k_new8"]),
                                                  _ptr(out["v_new8"]), _ptr(out["attn_out"]), _ptr(out["x_out"]), _ptr(out["hidden"]),
                                                  _ptr(scratch), C.c_size_t(scratch.numel()), _stream(stream)),
               "mirror_target_forward_fp8")
        out["_scratch"] = scratch
        return out

    def mirror_accept_select(self, tree: Tree, acc: AcceptIn, out: Optional[AcceptResult] = None, stream=None,
                             tree_scratch: bool = False) -> AcceptResult:
        """tree_scratch: size the workspace so that the tree rule can keep its running distribution in memory."""
        if out is None:
            out = AcceptResult(tree.batch, tree.gamma, self.device)
        if tree_scratch:
            self.ensure_workspace(tree, None, WS_STEP_TREE)
        o = out.struct()
        _check(self.lib.mirror_accept_select(self._ctx, C.byref(tree), C.byref(acc), C.byref(o), _stream(stream)),
               "mirror_accept_select")
        return out

    def mirror_verify_step_host(self, kv: KV, tree: Tree, h_in: dict, d_in: dict, hidden, W, acc: AcceptIn, attn_out,
                                out: "AcceptResult", h_out: Optional[dict] = None, stream=None) -> "AcceptResult":
        """mirror_verify_step with this step's inputs in (pinned) host tensors h_in = {q, k_new, v_new, tokens}; d_in holds
        the device staging tensors of the same shapes (d_in["tokens"] must be the tensor `tree` was built on); h_out:
        optional pinned host tensors n_accepted, best_branch, n_emitted, emitted that receive the decision."""
        def hp(t, dtype, name):
            if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
                raise ValueError(f"{name} must be a contiguous host tensor of {dtype}")
            return C.c_void_p(t.data_ptr())
        ho = AcceptHostOut(*[(C.c_void_p(h_out[f].data_ptr()) if h_out and f in h_out else None) for f, _ in AcceptHostOut._fields_])
        self.ensure_workspace(tree, kv, {ACCEPT_GREEDY: WS_STEP_GREEDY, ACCEPT_SPEC_TREE: WS_STEP_TREE}.get(acc.mode, WS_STEP_SPEC))
        o = out.struct()
        _check(self.lib.mirror_verify_step_host(self._ctx, C.byref(kv), C.byref(tree), hp(h_in["q"], torch.bfloat16, "q"),
                                                hp(h_in["k_new"], torch.bfloat16, "k_new"), hp(h_in["v_new"], torch.bfloat16, "v_new"),
                                                hp(h_in["tokens"], torch.int32, "tokens"), _ptr(d_in["q"], torch.bfloat16, "d_q"),
                                                _ptr(d_in["k_new"], torch.bfloat16, "d_k_new"), _ptr(d_in["v_new"], torch.bfloat16, "d_v_new"),
                                                _ptr(hidden, torch.bfloat16, "hidden"), _ptr(W, torch.bfloat16, "W"), C.byref(acc),
                                                C.byref(o), C.byref(ho), _ptr(attn_out, torch.bfloat16, "attn_out"), _stream(stream)),
               "mirror_verify_step_host")
        return out

    def mirror_verify_step(self, kv: KV, tree: Tree, q, k_new, v_new, hidden, W, acc: AcceptIn, attn_out,
                           out: Optional[AcceptResult] = None, argmax_out=None, stream=None) -> AcceptResult:
        if out is None:
            out = AcceptResult(tree.batch, tree.gamma, self.device)
        self.ensure_workspace(tree, kv, {ACCEPT_GREEDY: WS_STEP_GREEDY, ACCEPT_SPEC_TREE: WS_STEP_TREE}.get(acc.mode, WS_STEP_SPEC))
        o = out.struct()
        _check(self.lib.mirror_verify_step(self._ctx, C.byref(kv), C.byref(tree), _ptr(q, torch.bfloat16, "q"),
                                           _ptr(k_new, torch.bfloat16, "k_new"), _ptr(v_new, torch.bfloat16, "v_new"),
                                           _ptr(hidden, torch.bfloat16, "hidden"), _ptr(W, torch.bfloat16, "W"),
                                           C.byref(acc), C.byref(o), _ptr(attn_out, torch.bfloat16, "attn_out"),
                                           _ptr(argmax_out, torch.int32, "argmax_out"), _stream(stream)),
               "mirror_verify_step")
        return out

    def mirror_verify_step_fp8(self, kv: KV, tree: Tree, q, k_new8, v_new8, k_scale, v_scale, q_scale: float, hidden, W,
                               acc: AcceptIn, attn_out, out: Optional[AcceptResult] = None, argmax_out=None, stream=None) -> AcceptResult:
        """mirror_verify_step over an e4m3 cache (kv from kv_fp8; k_new8 / v_new8 uint8 codes under the cache's scales)."""
        if out is None:
            out = AcceptResult(tree.batch, tree.gamma, self.device)
        self.ensure_workspace(tree, kv, {ACCEPT_GREEDY: WS_STEP_GREEDY, ACCEPT_SPEC_TREE: WS_STEP_TREE}.get(acc.mode, WS_STEP_SPEC))
        o = out.struct()
        _check(self.lib.mirror_verify_step_fp8(self._ctx, C.byref(kv), C.byref(tree), _ptr(q, torch.bfloat16, "q"),
                                               _ptr(k_new8, torch.uint8, "k_new8"), _ptr(v_new8, torch.uint8, "v_new8"),
                                               _ptr(k_scale, torch.float32, "k_scale"), _ptr(v_scale, torch.float32, "v_scale"),
                                               C.c_float(q_scale), _ptr(hidden, torch.bfloat16, "hidden"), _ptr(W, torch.bfloat16, "W"),
                                               C.byref(acc), C.byref(o), _ptr(attn_out, torch.bfloat16, "attn_out"),
                                               _ptr(argmax_out, torch.int32, "argmax_out"), _stream(stream)),
               "mirror_verify_step_fp8")
        return out

    def set_stage_events(self, events):
        """events: four torch.cuda.Event(enable_timing=True) recorded by later mirror_verify_step calls, or None."""
        if events is None:
            _check(self.lib.mirror_set_stage_events(self._ctx, None), "mirror_set_stage_events")
            return
        for e in events:
            if e.cuda_event == 0:       # torch creates the CUDA event lazily, on first record
                e.record()
        arr = (C.c_void_p * 4)(*[C.c_void_p(e.cuda_event) for e in events])
        _check(self.lib.mirror_set_stage_events(self._ctx, arr), "mirror_set_stage_events")

    def device_status(self):
        code, detail = C.c_int(), C.c_int()
        _check(self.lib.mirror_device_status(self._ctx, C.byref(code), C.byref(detail)), "mirror_device_status")
        return code.value, detail.value

    def launch_count(self) -> int:
        n = C.c_longlong()
        _check(self.lib.mirror_launch_count(self._ctx, C.byref(n)), "mirror_launch_count")
        return n.value
