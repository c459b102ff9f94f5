"""Shared helpers for the parity tests: run the CPU oracle on generated inputs."""
import numpy as np
import torch

from oracle import oracle as O
from paper_2510_13161_b200 import inputs as I


def oracle_attention(x: I.VerifyInputs, layers=None):
    """fp64 oracle attention for the given layers -> dict layer -> (out [B,n,Hq,d], lse [B,Hq,n])."""
    anc, _ = O.tree(x.parent)
    scale = 1.0 / np.sqrt(x.cfg.head_dim)
    pt, pl = x.page_table.cpu().numpy(), x.prefix_len.cpu().numpy()
    res = {}
    for l in (range(x.q.shape[0]) if layers is None else layers):
        out, lse, _ = O.attention_layer(I.bf16_bits(x.q[l]), I.bf16_bits(x.k_pool[l]), I.bf16_bits(x.v_pool[l]), pt, pl,
                                        I.bf16_bits(x.k_new[l]), I.bf16_bits(x.v_new[l]), anc, scale)
        res[l] = (out, lse)
    return res


def to_device(x: I.VerifyInputs, device="cuda"):
    for f in ("prefix_len", "page_table", "q", "k_pool", "v_pool", "k_new", "v_new", "W", "hidden", "tokens",
              "q_probs", "u_accept", "u_resample"):
        v = getattr(x, f)
        if isinstance(v, torch.Tensor):
            setattr(x, f, v.to(device))
    return x


def make_mirror(cfg, temperature=1.0):
    from paper_2510_13161_b200.binding import Mirror
    return Mirror(cfg.hidden, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.vocab, temperature=temperature)
