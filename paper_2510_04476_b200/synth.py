"""Seeded synthetic inputs for the CCA / CCGQA block.

This module only draws random tensors and names the benchmark shapes.  It holds
none of the method's arithmetic, so both the CUDA path's callers and the fp64
oracle's callers can take their inputs from here without sharing any compute.

Recipe (the paper's kernel study used random activations, no dataset):
  x, d_out ~ N(0,1); projection weights ~ N(0,0.02); conv weights ~ N(0,0.1);
  temp ~ U(-0.5,0.5).  Every tensor is drawn in fp32 on the host from one
  torch.Generator in the fixed order
      x, w_qk, w_v1, w_v2, w_o, conv0_w, conv1_w, temp, d_out
  and rounded to bf16 (temp stays fp32), so that both paths see identical bits.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict

import torch

# Flag bits of the block's optional stages (ablation table of the paper).
CCA_CONV1 = 1
CCA_CONV2 = 2
CCA_QK_MEAN = 4
CCA_V_SHIFT = 8
CCA_QK_NORM = 16
CCA_ROPE = 32
CCA_ALL = 63


@dataclasses.dataclass(frozen=True)
class Shape:
    """The paper's parameters plus batch and sequence length."""
    name: str
    B: int
    S: int
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    k_seq: int = 2
    k_ch: int = 2
    causal: int = 1
    flags: int = CCA_ALL
    rope_base: float = 10000.0
    seed: int = 0

    @property
    def L_q(self) -> int:
        return self.n_q_heads * self.head_dim

    @property
    def L_k(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def L(self) -> int:
        return self.L_q + self.L_k

    @property
    def compression(self) -> int:
        return self.d_model // self.L_q

    def replace(self, **kw) -> "Shape":
        return dataclasses.replace(self, **kw)


# The benchmark configurations (index = config number, 1-based in the text).
CONFIGS: Dict[str, Shape] = {
    "cfg1_tiny": Shape("cfg1_tiny", 1, 128, 256, 4, 4, 32, seed=0),
    "cfg2_small": Shape("cfg2_small", 2, 2048, 2048, 16, 4, 64, seed=2),
    "cfg3_prefill16k": Shape("cfg3_prefill16k", 1, 16384, 4096, 8, 2, 128, seed=3),
    "cfg4_train": Shape("cfg4_train", 8, 4096, 2048, 8, 2, 64, seed=4),
}


def mha_like(shape: Shape) -> Shape:
    """Same d_model and head_dim, no compression, no latent transforms: the
    in-house multi-head-attention configuration of the same kernels."""
    h = shape.d_model // shape.head_dim
    return shape.replace(name=shape.name + "_mha", n_q_heads=h, n_kv_heads=h, flags=0)


def sweep_shape(S: int, C: int) -> Shape:
    """Context x compression sweep: d_model 2048, latent head dim 64,
    32/C query heads, a quarter as many kv heads (at least 1), 64k tokens."""
    hq = 32 // C
    hk = max(1, hq // 4)
    seed = 1000 * int(math.log2(C)) + int(math.log2(S))
    return Shape(f"sweep_S{S}_C{C}", max(1, 65536 // S), S, 2048, hq, hk, 64, seed=seed)


def make_inputs(shape: Shape, want_dout: bool = True) -> Dict[str, torch.Tensor]:
    """Draw the block's inputs and parameters on the host (bf16 except temp)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(shape.seed)
    E, L, Lq, Lk, dh = shape.d_model, shape.L, shape.L_q, shape.L_k, shape.head_dim

    def normal(size, std):
        return (torch.randn(size, generator=g, dtype=torch.float32) * std).to(torch.bfloat16)

    t = {}
    t["x"] = normal((shape.B, shape.S, E), 1.0)
    t["w_qk"] = normal((L, E), 0.02)
    t["w_v1"] = normal((Lk // 2, E), 0.02)
    t["w_v2"] = normal((Lk // 2, E), 0.02)
    t["w_o"] = normal((E, Lq), 0.02)
    t["conv0_w"] = normal((L, shape.k_seq), 0.1)
    t["conv1_w"] = normal((L, dh, shape.k_ch), 0.1)
    t["temp"] = torch.rand((shape.n_kv_heads,), generator=g, dtype=torch.float32) - 0.5
    if want_dout:
        t["d_out"] = normal((shape.B, shape.S, E), 1.0)
    return t


@dataclasses.dataclass(frozen=True)
class MlaShape:
    """Multi-Latent Attention (the paper's Section 2.1) as a baseline: E, heads, per-head part sizes, latent widths."""
    name: str
    B: int
    S: int
    d_model: int
    n_heads: int
    d_nope: int
    d_rope: int
    d_ckv: int
    d_cq: int
    causal: int = 1
    rope_base: float = 10000.0
    seed: int = 0

    @property
    def head_dim(self) -> int:
        return self.d_nope + self.d_rope


def mla_like(shape: Shape) -> MlaShape:
    """The MLA baseline of equal d_model and head size: E / d_h heads, half of each query / key head position-free
    and half RoPE (one RoPE key part shared by all heads), value heads of size d_h, KV latent E / 4, query latent
    E / 2.  The paper gives no MLA dimensions for its kernel study; these keep the attention FLOPs at MHA's, as
    its text describes."""
    dh = shape.head_dim
    return MlaShape(shape.name + "_mla", shape.B, shape.S, shape.d_model, shape.d_model // dh, dh // 2, dh // 2,
                    shape.d_model // 4, shape.d_model // 2, causal=shape.causal, seed=shape.seed)


def make_mla_inputs(m: MlaShape) -> Dict[str, torch.Tensor]:
    """x ~ N(0,1), every projection ~ N(0,0.02), drawn in the order x, w_dq, w_dkv, w_uq, w_uqr, w_uk, w_uv, w_kr,
    w_o and rounded to bf16."""
    g = torch.Generator(device="cpu")
    g.manual_seed(m.seed)
    E, nh, dh = m.d_model, m.n_heads, m.head_dim

    def normal(size, std):
        return (torch.randn(size, generator=g, dtype=torch.float32) * std).to(torch.bfloat16)

    t = {"x": normal((m.B, m.S, E), 1.0)}
    t["w_dq"] = normal((m.d_cq, E), 0.02)
    t["w_dkv"] = normal((m.d_ckv, E), 0.02)
    t["w_uq"] = normal((nh * m.d_nope, m.d_cq), 0.02)
    t["w_uqr"] = normal((nh * m.d_rope, m.d_cq), 0.02)
    t["w_uk"] = normal((nh * m.d_nope, m.d_ckv), 0.02)
    t["w_uv"] = normal((nh * dh, m.d_ckv), 0.02)
    t["w_kr"] = normal((m.d_rope, E), 0.02)
    t["w_o"] = normal((E, nh * dh), 0.02)
    return t
