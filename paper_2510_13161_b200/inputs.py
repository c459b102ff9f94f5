"""Seeded synthetic inputs for the Mirror-SD target-side verify step.

This module only *draws* inputs (shapes, value distributions, page tables, token
trees).  It holds none of the method's arithmetic and imports neither the CUDA
binding nor the CPU oracle, so both sides can consume exactly the same tensors.

The paper evaluates on SpecBench prompts with 14B-66B targets (Sec. 4.1); it
prints no tensor shapes, so the shapes below are the synthetic stand-ins for
those workloads: a shared verified prefix held in a paged KV cache, a token tree
of kappa branches x gamma lookahead tokens hanging off the last committed token
(the hypothesis tree of Sec. 3.1), target LM-head weights, and, for stochastic
verification, the draft distributions and per-node uniforms.

Every tensor is generated in its storage dtype (bf16 for activations, weights
and KV), so the rounded value is the one value both sides see.
"""
from __future__ import annotations

import zlib
from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Sequence

import torch

PAGE_SIZE = 16


@dataclass(frozen=True)
class VerifyConfig:
    name: str
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    layers: int
    batch: int
    prefix_lo: int          # prefix lengths drawn uniformly from [prefix_lo, prefix_hi]
    prefix_hi: int
    kappa: int              # branches
    gamma: int              # lookahead tokens per branch
    vocab: int
    mode: str               # "greedy" | "spec_sampling" (independent per-branch rule) | "spec_tree" (lossless rule over the tree)
    w_std: float = 0.02
    kv_std: float = 1.0
    explicit_hidden: bool = False   # LM-head rows given as an input instead of the last layer's attention output
    temperature: float = 1.0

    @property
    def n_nodes(self) -> int:
        return 1 + self.kappa * self.gamma

    @property
    def rows(self) -> int:
        return self.batch * self.n_nodes

    @property
    def draft_tokens(self) -> int:
        return self.batch * self.kappa * self.gamma


CONFIGS: Dict[str, VerifyConfig] = {
    # configs[0]: the oracle finishes it in well under a second
    "tiny": VerifyConfig("tiny", 256, 4, 2, 64, 1, 1, 128, 128, 2, 4, 1024, "greedy", 0.02, 0.02),
    # configs[1]: 14B-shaped target, batch 1 -- the bench workload
    "qwen14b": VerifyConfig("qwen14b", 5120, 40, 8, 128, 48, 1, 2048, 2048, 4, 4, 152064, "greedy"),
    # configs[2]: 14B-shaped, batch 8, ragged prefixes, stochastic acceptance
    "qwen14b_b8": VerifyConfig("qwen14b_b8", 5120, 40, 8, 128, 48, 8, 512, 4096, 8, 6, 152064, "spec_sampling"),
    # configs[3]: 32B-shaped, long context (Hq*d != hidden, so hidden rows are explicit)
    "qwen32b_long": VerifyConfig("qwen32b_long", 5120, 64, 8, 128, 64, 1, 32768, 32768, 4, 8, 152064, "greedy",
                                 explicit_hidden=True),
    # configs[4]: 66B-class, batch 16, ragged prefixes, stochastic acceptance
    "opt66b_b16": VerifyConfig("opt66b_b16", 8192, 64, 8, 128, 80, 16, 1024, 8192, 8, 8, 128256, "spec_sampling"),
    # the paper's own operating point (Sec. 4.1: gamma=7, kappa=8, batch 1) on the 14B shape
    "paper_native": VerifyConfig("paper_native", 5120, 40, 8, 128, 48, 1, 2048, 2048, 8, 7, 152064, "greedy"),
}


def shrink(cfg: VerifyConfig, **kw) -> VerifyConfig:
    """A copy of `cfg` with some fields replaced (used to cut big configs down for parity tests)."""
    return replace(cfg, **kw)


def _seed_for(seed: int, name: str) -> int:
    return (int(seed) * 1000003 + zlib.crc32(name.encode())) & 0x7FFFFFFFFFFFFFFF


def _gen(device, seed: int, name: str) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_seed_for(seed, name))
    return g


def comb_parent(kappa: int, gamma: int) -> List[int]:
    """Parent array of the canonical token tree: node 0 is the root (last committed
    token); branch i is the chain of nodes 1+i*gamma .. 1+i*gamma+gamma-1 whose first
    node hangs off the root."""
    parent = [-1]
    for i in range(kappa):
        for j in range(gamma):
            parent.append(0 if j == 0 else 1 + i * gamma + j - 1)
    return parent


def random_tree_parent(n_nodes: int, seed: int, max_depth: int = 8) -> List[int]:
    """A seeded random tree with parent[i] < i and bounded depth (general-tree test cases)."""
    g = torch.Generator().manual_seed(_seed_for(seed, "tree"))
    parent, depth = [-1], [0]
    for i in range(1, n_nodes):
        while True:
            p = int(torch.randint(0, i, (1,), generator=g))
            if depth[p] < max_depth:
                break
        parent.append(p)
        depth.append(depth[p] + 1)
    return parent


def draw_prefix_lens(cfg: VerifyConfig, seed: int) -> torch.Tensor:
    g = _gen("cpu", seed, "prefix_len")
    if cfg.prefix_lo == cfg.prefix_hi:
        return torch.full((cfg.batch,), cfg.prefix_lo, dtype=torch.int32)
    return torch.randint(cfg.prefix_lo, cfg.prefix_hi + 1, (cfg.batch,), generator=g, dtype=torch.int32)


def gen_page_table(prefix_len: torch.Tensor, seed: int, spare_pages: int = 3, shuffle: bool = True, headroom: int = 0):
    """Physical pages handed out by a seeded random permutation of the pool (a fragmented
    cache); unused table slots hold -1.  `headroom` tokens beyond each prefix get pages too (room to commit
    accepted tokens).  Returns (page_table [B,max_pages] int32, num_pages)."""
    pages = [(int(l) + headroom + PAGE_SIZE - 1) // PAGE_SIZE for l in prefix_len]
    total = sum(pages)
    num_pages = total + spare_pages
    max_pages = max(1, max(pages) if pages else 1)
    g = _gen("cpu", seed, "page_table")
    perm = torch.randperm(num_pages, generator=g) if shuffle else torch.arange(num_pages)
    table = torch.full((len(pages), max_pages), -1, dtype=torch.int32)
    at = 0
    for b, p in enumerate(pages):
        table[b, :p] = perm[at:at + p].to(torch.int32)
        at += p
    return table, num_pages


def _normal(shape, std, dtype, device, gen) -> torch.Tensor:
    t = torch.empty(shape, dtype=dtype, device=device)
    t.normal_(0.0, std, generator=gen)
    return t


@dataclass
class VerifyInputs:
    cfg: VerifyConfig
    seed: int
    parent: List[int]
    prefix_len: torch.Tensor          # [B] int32
    page_table: torch.Tensor          # [B, max_pages] int32
    num_pages: int
    q: torch.Tensor                   # [L,B,n,Hq,d] bf16
    k_pool: torch.Tensor              # [L,num_pages,Hkv,16,d] bf16
    v_pool: torch.Tensor
    k_new: torch.Tensor               # [L,B,n,Hkv,d] bf16
    v_new: torch.Tensor
    W: Optional[torch.Tensor]         # [V,H] bf16
    hidden: Optional[torch.Tensor]    # [B*n,H] bf16 or None (chain the last layer's attention output)
    tokens: torch.Tensor              # [B,n] int32 (node 0 = last committed token)
    q_probs: Optional[torch.Tensor] = None    # [B,n-1,V] fp32, draft distribution that proposed node i+1
    u_accept: Optional[torch.Tensor] = None   # [B,n] fp32 in [0,1)
    u_resample: Optional[torch.Tensor] = None  # [B,n] fp32 in [0,1)
    extras: dict = field(default_factory=dict)


def gen_verify_inputs(cfg: VerifyConfig, seed: int = 0, device: str = "cpu", *,
                      parent: Optional[Sequence[int]] = None, with_lm_head: bool = True,
                      layers: Optional[int] = None, shuffle_pages: bool = True,
                      q_std: float = 1.0, force_hidden: bool = False, headroom: int = 0) -> VerifyInputs:
    """Draw one verify-step problem.  `layers` overrides cfg.layers (parity tests on big
    configs generate a few layers only; each layer's tensors depend on (seed, layer) alone,
    so layer l is the same tensor whatever `layers` is)."""
    L = cfg.layers if layers is None else layers
    B, n, Hq, Hkv, d = cfg.batch, cfg.n_nodes, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    par = list(parent) if parent is not None else comb_parent(cfg.kappa, cfg.gamma)
    n = len(par)
    bf = torch.bfloat16
    prefix_len = draw_prefix_lens(cfg, seed)
    page_table, num_pages = gen_page_table(prefix_len, seed, shuffle=shuffle_pages, headroom=headroom)

    q = torch.empty((L, B, n, Hq, d), dtype=bf, device=device)
    k_pool = torch.empty((L, num_pages, Hkv, PAGE_SIZE, d), dtype=bf, device=device)
    v_pool = torch.empty_like(k_pool)
    k_new = torch.empty((L, B, n, Hkv, d), dtype=bf, device=device)
    v_new = torch.empty_like(k_new)
    for l in range(L):
        q[l].normal_(0.0, q_std, generator=_gen(device, seed, f"q{l}"))
        k_pool[l].normal_(0.0, cfg.kv_std, generator=_gen(device, seed, f"k_pool{l}"))
        v_pool[l].normal_(0.0, cfg.kv_std, generator=_gen(device, seed, f"v_pool{l}"))
        k_new[l].normal_(0.0, cfg.kv_std, generator=_gen(device, seed, f"k_new{l}"))
        v_new[l].normal_(0.0, cfg.kv_std, generator=_gen(device, seed, f"v_new{l}"))

    W = hidden = None
    if with_lm_head:
        W = _normal((cfg.vocab, cfg.hidden), cfg.w_std, bf, device, _gen(device, seed, "W"))
        if cfg.explicit_hidden or force_hidden or Hq * d != cfg.hidden:
            hidden = _normal((B * n, cfg.hidden), 1.0, bf, device, _gen(device, seed, "hidden"))

    tokens = torch.randint(0, cfg.vocab, (B, n), generator=_gen("cpu", seed, "tokens"), dtype=torch.int32)

    out = VerifyInputs(cfg, seed, par, prefix_len.to(device), page_table.to(device), num_pages,
                       q, k_pool, v_pool, k_new, v_new, W, hidden, tokens.to(device))
    if cfg.mode in ("spec_sampling", "spec_tree"):
        out.u_accept = torch.rand((B, n), generator=_gen("cpu", seed, "u_accept"), dtype=torch.float32).to(device)
        out.u_resample = torch.rand((B, n), generator=_gen("cpu", seed, "u_resample"), dtype=torch.float32).to(device)
        if with_lm_head:
            qp = torch.empty((B, n - 1, cfg.vocab), dtype=torch.float32, device=device)
            for b in range(B):
                z = torch.empty((n - 1, cfg.vocab), dtype=torch.float32, device=device)
                z.normal_(0.0, 1.0, generator=_gen(device, seed, f"q_logits{b}"))
                qp[b] = torch.softmax(z, dim=-1)
            out.q_probs = qp
    return out


def gen_layer_weights(cfg: VerifyConfig, intermediate: int, layers: int, seed: int = 0, device: str = "cpu",
                      w_std: Optional[float] = None):
    """Seeded weights of `layers` pre-norm decoder layers for the shape of `cfg` (bf16): per layer a dict with w_qkv
    [(Hq + 2 Hkv) d, H] (query, key, value rows), w_o [H, Hq d], w_gate_up [2 I, H] (gate, up rows), w_down [H, I] and
    the two RMSNorm weights [H] (around 1); plus the final norm weight and the residual rows x [B n, H] that enter
    layer 0 (stand-ins for the embeddings of the tree's tokens).  Returns (list of dicts, norm_final, x)."""
    H, Hq, Hkv, d = cfg.hidden, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    std = cfg.w_std if w_std is None else w_std
    bf = torch.bfloat16
    out = []
    for l in range(layers):
        g = lambda name: _gen(device, seed, f"layer{l}.{name}")
        norm = lambda name: (1.0 + 0.1 * torch.empty(H, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=g(name))).to(bf)
        out.append(dict(w_qkv=_normal(((Hq + 2 * Hkv) * d, H), std, bf, device, g("w_qkv")),
                        w_o=_normal((H, Hq * d), std, bf, device, g("w_o")),
                        w_gate_up=_normal((2 * intermediate, H), std, bf, device, g("w_gate_up")),
                        w_down=_normal((H, intermediate), std, bf, device, g("w_down")),
                        norm_attn=norm("norm_attn"), norm_mlp=norm("norm_mlp")))
    norm_final = (1.0 + 0.1 * torch.empty(H, dtype=torch.float32, device=device).normal_(0.0, 1.0, generator=_gen(device, seed, "norm_final"))).to(bf)
    x = _normal((cfg.rows, H), 1.0, bf, device, _gen(device, seed, "x_embed"))
    return out, norm_final, x


def bf16_bits(t: torch.Tensor):
    """numpy uint16 view of a bf16 tensor's bits (host copy)."""
    return t.detach().to("cpu").contiguous().view(torch.uint16).numpy()
