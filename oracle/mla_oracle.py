"""fp64 CPU oracle for Multi-Latent Attention (MLA), the comparison method of the paper's Section 2.1 (Eq. 3-6).

TEST INFRASTRUCTURE ONLY, like cca_oracle.py: the slow, plain definition that the library's MLA baseline
configuration is checked against.  torch CPU float64, bf16-rounded inputs widened exactly, no intermediate rounding,
whole score rows, no fusion.  It imports nothing from the product.

Steps, in the paper's order:
  Eq. 3   C_KV = x W_DKV, C_Q = x W_DQ                              (down-projections to the two latents)
  Eq. 4   q_i = W_UQ C_Q, k_i = W_UK C_KV, v_i = W_UV C_KV          (per-head up-projections)
  Eq. 6   q^r_i = RoPE(W_UQR C_Q), k^r = RoPE(W_KR x), one k^r shared by all heads;
          q_i <- [q_i, q^r_i], k_i <- [k_i, k^r]; attention as in MHA (Eq. 1-2), then W_O.
Eq. 5 (the absorbed, MQA-mode form without RoPE) is used as a pin, not as the implementation.

Readings taken where the paper is silent: no biases; softmax scale 1/sqrt(d_nope + d_rope) (the per-head query/key
size after concatenation); RoPE as in cca_oracle (pairs (c, c + d_rope/2), base 10000, positions from 0); causal mask;
linear weights are [out, in] like torch.nn.Linear.  The comparison table's MLA row leaves the RoPE projections out of
its counts; `describe` does the same and reports them separately.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict

import torch

from oracle import cca_oracle as O

F64 = torch.float64


@dataclasses.dataclass(frozen=True)
class MlaConfig:
    d_model: int        # E
    n_heads: int        # n_h
    d_nope: int         # per-head size of the up-projected (position-free) query / key part
    d_rope: int         # size of the RoPE part (per head for queries, one shared key part)
    d_v: int            # per-head value size
    d_ckv: int          # width of the shared KV latent, E / c_kv
    d_cq: int           # width of the query latent, E / c_q
    causal: int = 1
    rope_base: float = 10000.0

    @property
    def d_qk(self):
        return self.d_nope + self.d_rope


def forward(cfg: MlaConfig, w: Dict[str, torch.Tensor], x):
    """Eq. 3, 4, 6 and the output projection.  w: w_dq [d_cq,E], w_dkv [d_ckv,E], w_uq [n_h*d_nope,d_cq],
    w_uqr [n_h*d_rope,d_cq], w_uk [n_h*d_nope,d_ckv], w_uv [n_h*d_v,d_ckv], w_kr [d_rope,E], w_o [E,n_h*d_v].
    Returns (out [B,S,E], intermediates)."""
    x = O._f64(x)
    B, S, E = x.shape
    nh, dn, dr, dv = cfg.n_heads, cfg.d_nope, cfg.d_rope, cfg.d_v
    W = {n: O._f64(t) for n, t in w.items()}
    I = {"x": x}
    c_kv = x @ W["w_dkv"].T                                   # Eq. 3
    c_q = x @ W["w_dq"].T
    I["c_kv"], I["c_q"] = c_kv, c_q
    q_n = (c_q @ W["w_uq"].T).reshape(B, S, nh, dn)           # Eq. 4
    k_n = (c_kv @ W["w_uk"].T).reshape(B, S, nh, dn)
    v = (c_kv @ W["w_uv"].T).reshape(B, S, nh, dv)
    I["q_nope"], I["k_nope"], I["v"] = q_n, k_n, v
    if dr > 0:                                                # Eq. 6
        ang = O.rope_angles(S, dr, cfg.rope_base)
        q_r = O.rope((c_q @ W["w_uqr"].T).reshape(B, S, nh, dr), ang)
        k_r = O.rope((x @ W["w_kr"].T).reshape(B, S, 1, dr), ang)
        q = torch.cat([q_n, q_r], dim=-1)
        k = torch.cat([k_n, k_r.expand(B, S, nh, dr)], dim=-1)
        I["k_rope"] = k_r
    else:
        q, k = q_n, k_n
    I["q"], I["k"] = q, k
    o, lse = attention_mha(q, k, v, bool(cfg.causal))
    I["o"], I["lse"] = o, lse
    out = o.reshape(B, S, nh * dv) @ W["w_o"].T
    I["out"] = out
    return out, I


def attention_mha(q, k, v, causal):
    """Eq. 1-2 per head with query/key size d_qk and value size d_v: softmax(q k^T / sqrt(d_qk)) v."""
    B, S, nh, dqk = q.shape
    dv = v.shape[-1]
    o = torch.zeros(B, S, nh, dv, dtype=F64)
    lse = torch.zeros(B, nh, S, dtype=F64)
    inv = 1.0 / math.sqrt(dqk)
    ar = torch.arange(S)
    for b in range(B):
        for i in range(nh):
            s = (q[b, :, i, :] @ k[b, :, i, :].T) * inv
            if causal:
                s = s.masked_fill(ar[None, :] > ar[:, None], float("-inf"))
            m = s.max(dim=-1, keepdim=True).values
            e = torch.exp(s - m)
            z = e.sum(dim=-1, keepdim=True)
            o[b, :, i, :] = (e / z) @ v[b, :, i, :]
            lse[b, i, :] = (m + torch.log(z)).squeeze(-1)
    return o, lse


def forward_absorbed_nope(cfg: MlaConfig, w: Dict[str, torch.Tensor], x):
    """Eq. 5: without RoPE the up-projections can be folded into the query and the output side, and every head
    attends to the shared latent C_KV itself (multi-query attention over the latent):
        softmax(C_Q W_UQ,i^T W_UK,i C_KV^T / sqrt(d_nope)) C_KV W_UV,i^T W_O,i^T.
    Only defined for d_rope = 0; used to pin forward()."""
    assert cfg.d_rope == 0
    x = O._f64(x)
    B, S, E = x.shape
    nh, dn, dv = cfg.n_heads, cfg.d_nope, cfg.d_v
    W = {n: O._f64(t) for n, t in w.items()}
    c_kv = x @ W["w_dkv"].T
    c_q = x @ W["w_dq"].T
    w_uq = W["w_uq"].reshape(nh, dn, cfg.d_cq)
    w_uk = W["w_uk"].reshape(nh, dn, cfg.d_ckv)
    w_uv = W["w_uv"].reshape(nh, dv, cfg.d_ckv)
    w_o = W["w_o"].reshape(E, nh, dv)
    out = torch.zeros(B, S, E, dtype=F64)
    ar = torch.arange(S)
    for i in range(nh):
        q_abs = c_q @ (w_uq[i].T @ w_uk[i])                   # [B,S,d_ckv]: the query in the latent's coordinates
        s = torch.einsum("bsc,btc->bst", q_abs, c_kv) / math.sqrt(dn)
        if cfg.causal:
            s = s.masked_fill(ar[None, None, :] > ar[None, :, None], float("-inf"))
        p = torch.softmax(s, dim=-1)
        ctx = torch.einsum("bst,btc->bsc", p, c_kv)           # attention output in the latent
        out += ctx @ (w_o[:, i, :] @ w_uv[i]).T
    return out


def describe(cfg: MlaConfig, B: int, S: int) -> Dict[str, int]:
    """Counts of the comparison table's MLA row (c_q = E / d_cq, c_kv = E / d_ckv; per-head sizes with
    n_h * d_nope = n_h * d_v = E), which leaves the RoPE projections out; those are reported separately."""
    E = cfg.d_model
    nh, dn, dr, dv = cfg.n_heads, cfg.d_nope, cfg.d_rope, cfg.d_v
    params = E * nh * dv + cfg.d_ckv * E + cfg.d_ckv * nh * dn + cfg.d_ckv * nh * dv + cfg.d_cq * E + cfg.d_cq * nh * dn
    rope_params = dr * E + nh * dr * cfg.d_cq
    T = B * S
    return {
        "params": params,
        "rope_params": rope_params,
        "kv_cache_elems": B * S * cfg.d_ckv + B * S * dr,
        "fwd_flops": 2 * T * (E * nh * dv + cfg.d_cq * E + cfg.d_cq * nh * dn + cfg.d_ckv * E + cfg.d_ckv * nh * dn
                              + cfg.d_ckv * nh * dv) + 2 * B * S * S * nh * dn + 2 * B * S * S * nh * dv,
        "rope_fwd_flops": 2 * T * rope_params + 2 * B * S * S * nh * dr,
    }
