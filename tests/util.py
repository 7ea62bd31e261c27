"""Helpers shared by the parity tests: oracle config mapping and the tolerance rule."""
import math

import torch

from oracle import cca_oracle as O

ATOL, RTOL = 1e-2, 1e-2     # max |err| <= 1e-2 + 1e-2 |ref|  (bf16 operands, fp32 accumulate)


def oracle_cfg(sh):
    return O.OracleConfig(d_model=sh.d_model, n_q_heads=sh.n_q_heads, n_kv_heads=sh.n_kv_heads,
                          head_dim=sh.head_dim, k_seq=sh.k_seq, k_ch=sh.k_ch, causal=sh.causal, flags=sh.flags,
                          rope_base=sh.rope_base)


def check_close(name, got, ref, scale_abs=False):
    """Element-wise |got - ref| <= ATOL*s + RTOL*|ref|.

    s = 1 for activations and the input gradient.  For parameter gradients (sums over all B*S
    tokens of products with unit-variance upstream gradients) s = max(1, rms(ref)): every bf16
    operand contributes a relative error of 2^-9 to each of the B*S terms, so the error of the sum
    scales with the typical magnitude of the sum, not with 1."""
    got = got.detach().to("cpu").to(torch.float64)
    ref = ref.detach().to("cpu").to(torch.float64)
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    assert torch.isfinite(got).all(), f"{name}: non-finite values"
    s = max(1.0, float(ref.pow(2).mean().sqrt())) if scale_abs else 1.0
    err = (got - ref).abs()
    tol = ATOL * s + RTOL * ref.abs()
    bad = err > tol
    if bad.any():
        idx = torch.nonzero(bad)[0].tolist()
        worst = float((err / tol).max())
        raise AssertionError(f"{name}: {int(bad.sum())}/{bad.numel()} outside tolerance; worst err/tol {worst:.2f}; "
                             f"first at {idx}: got {float(got[tuple(idx)])} ref {float(ref[tuple(idx)])}")
    return float((err / tol).max())


PARAM_NAMES = ["w_qk", "w_v1", "w_v2", "w_o", "conv0_w", "conv1_w", "temp"]


def to_device(t, device="cuda"):
    return {k: v.to(device).contiguous() for k, v in t.items()}
