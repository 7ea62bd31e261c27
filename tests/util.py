"""Helpers shared by the parity tests: oracle config mapping and the tolerance rule."""
import math

import torch

from oracle import cca_oracle as O

ATOL, RTOL = 1e-2, 1e-2     # max |err| <= 1e-2 + 1e-2 |ref|  (bf16 operands, fp32 accumulate)


def oracle_cfg(sh):
    return O.OracleConfig(d_model=sh.d_model, n_q_heads=sh.n_q_heads, n_kv_heads=sh.n_kv_heads,
                          head_dim=sh.head_dim, k_seq=sh.k_seq, k_ch=sh.k_ch, causal=sh.causal, flags=sh.flags,
                          rope_base=sh.rope_base)


def check_close(name, got, ref, tail=None):
    """Element-wise |got - ref| <= 1e-2 + 1e-2 |ref|: outputs, saved activations, the input gradient.

    tail = (fraction, factor), only for an input gradient of tens of millions of elements: at most `fraction` of the
    elements may exceed the bound, none by more than `factor`.  (With Gaussian rounding noise of standard deviation
    sigma the largest of 7e7 errors is about 6 sigma, so a bound that the typical element meets five times over is
    still grazed by a handful.)  Outputs never get a tail."""
    got = got.detach().to("cpu").to(torch.float64)
    ref = ref.detach().to("cpu").to(torch.float64)
    assert got.shape == ref.shape, (name, got.shape, ref.shape)
    assert torch.isfinite(got).all(), f"{name}: non-finite values"
    err = (got - ref).abs()
    tol = ATOL + RTOL * ref.abs()
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


def check_out_wide(cfg, t, I, name, got, ref, rows=None, model=None):
    """Block outputs of shapes outside the benchmark configurations whose output scale may be large (d_model 4096
    against a few dozen keys gives outputs of rms 1, where the bf16 rounding of o alone is a third of the absolute
    1e-2): 1e-2 + 1e-2 |ref| + 6 sigma with sigma = kappa 2^-9 sqrt(sum_c (o_c W_ec)^2) per element, kappa from the
    bf16-storage model as for the parameter gradients.  rows: token positions of `got` / `ref` (decode steps)."""
    from tests import noise_model as NM
    rss = NM.out_term_rss(t, I)
    model = model if model is not None else NM.storage_model_gradients(cfg, t)
    kap = NM.kappa(model["out"], I["out"], rss)
    if rows is not None:
        rss = rss[:, rows]
    got = got.detach().to("cpu").to(torch.float64).reshape(ref.shape)
    assert torch.isfinite(got).all(), f"{name}: non-finite values"
    err = (got - ref).abs()
    tol = ATOL + RTOL * ref.abs() + N_SIGMA * kap * NM.U * rss.reshape(ref.shape)
    bad = err > tol
    if bad.any():
        idx = torch.nonzero(bad)[0].tolist()
        raise AssertionError(f"{name}: {int(bad.sum())}/{bad.numel()} outside 1e-2 + 1e-2|ref| + 6 sigma; worst err/tol "
                             f"{float((err / tol).max()):.2f}; first at {idx}")
    return model


N_SIGMA = 6.0
LAST_PARAM_REPORT = {}        # name -> figures of the most recent check_param_grads call (for -s runs and reports)


def check_param_grads(cfg, t, I, G, grads, names=None, report=None, model=None, kappas=None):
    """Parameter gradients against the oracle.  Each is a sum over all B*S tokens of products whose factors went
    through bf16 on the way (q, k, v, o, P, d_o, dS, the latent gradient), so its error is a random walk over the
    terms of the sum and grows with their size, not with the size of the result: an absolute 1e-2 cannot hold on a
    sum of rms 5..80 whose terms are each known to 2^-9.  The rule is therefore, per element,

        |got - ref| <= 1e-2 + 1e-2 |ref| + 6 sigma,    sigma = kappa * 2^-9 * sqrt(sum_t term_t^2),

    with the root-sum-square of the terms taken from the oracle for that very element and kappa (the effective
    number of roundings per term, 1.4 .. 2.5) from the oracle's steps re-run with bf16 storage (tests/noise_model.py);
    neither comes from the CUDA path.  The overall noise level is held to the model as well:
    rms(err / (2^-9 rss)) <= 2 kappa.  d_temp is one heavily cancelling sum per kv head over all (query, key)
    pairs of dS * logit: same rule with those terms (noise_model.temp_term_rss); h_k samples cannot calibrate a
    kappa, so it takes that of d_w_qk, whose terms pass through the same attention adjoint.  The fraction of
    elements that meets the plain rule 1e-2 + 1e-2 |ref| is recorded in `report` / LAST_PARAM_REPORT.

    model: gradients of noise_model.storage_model_gradients if the caller has them already.  kappas: {name: kappa}
    taken from a shorter sequence of the same configuration, for the longest contexts where a second pass of the
    oracle's steps would take minutes (kappa counts roundings per term; it does not depend on the number of terms).
    The level check is 2 kappa: the model leaves out the order of the fp32 accumulations and the approximate
    exponentials, and small cases fluctuate; a systematic error raises the level by multiples
    (tests/test_tolerance_rule.py)."""
    from tests import noise_model as NM
    names = list(names or PARAM_NAMES)
    rss = NM.term_rss(cfg, t, I, G)
    # A sum of fewer than 32 terms (B * S tokens) is no random walk: its bound is the worst case instead, every one of
    # the 3 kappa^2 roundings of a term (kappa^2 = number of roundings / 3 for uniform rounding errors) in the same
    # direction: 3 kappa^2 * 2^-9 * sum |term|.
    few_terms = I["x"].shape[0] * I["x"].shape[1] < 32
    l1 = NM.term_rss(cfg, t, I, G, power=1) if few_terms else None
    if kappas is None:
        model = model if model is not None else NM.storage_model_gradients(cfg, t)
        kappas = {n: NM.kappa(model["d_" + n], G["d_" + n], rss[n]) for n in rss}
    rep = {}
    kap_qk = kappas["w_qk"]
    for n in names:
        ref = G["d_" + n].to(torch.float64)
        got = grads["d_" + n].detach().to("cpu").to(torch.float64).reshape(ref.shape)
        assert torch.isfinite(got).all(), f"d_{n}: non-finite values"
        err = (got - ref).abs()
        plain = ATOL + RTOL * ref.abs()
        if n == "temp":
            kap = kap_qk
            noise = (3 * kap * kap * NM.U * NM.temp_term_rss(cfg, I, G, power=1) if few_terms
                     else N_SIGMA * kap * NM.U * NM.temp_term_rss(cfg, I, G))
        else:
            kap = kappas[n]
            noise = 3 * kap * kap * NM.U * l1[n] if few_terms else N_SIGMA * kap * NM.U * rss[n]
            m = NM.noisy(rss[n])
            if int(m.sum()) >= NM.MIN_NOISY and not few_terms:
                level = float((err[m] / (NM.U * rss[n][m])).pow(2).mean().sqrt())
                assert level <= 2.0 * kap, f"d_{n}: noise level {level:.2f} x 2^-9 rss, the bf16-storage model gives {kap:.2f}"
        tol = plain + noise
        rep[n] = {"kappa": kap, "plain_fraction": float((err <= plain).double().mean()),
                  "worst_err_over_tol": float((err / tol).max())}
        bad = err > tol
        if bad.any():
            idx = torch.nonzero(bad)[0].tolist()
            raise AssertionError(f"d_{n}: {int(bad.sum())}/{bad.numel()} outside 1e-2 + 1e-2|ref| + 6 sigma; worst err/tol "
                                 f"{rep[n]['worst_err_over_tol']:.2f}; first at {idx}: got {float(got[tuple(idx)])} "
                                 f"ref {float(ref[tuple(idx)])} noise bound {float(noise[tuple(idx)])}")
    LAST_PARAM_REPORT.clear()
    LAST_PARAM_REPORT.update(rep)
    if report is not None:
        report.update(rep)
    print("parameter gradients: " + "; ".join(
        f"d_{n} kappa {r['kappa']:.2f}, {100 * r['plain_fraction']:.1f}% within the plain rule, worst {r['worst_err_over_tol']:.2f} of bound"
        for n, r in rep.items()))
    return rep


PARAM_NAMES = ["w_qk", "w_v1", "w_v2", "w_o", "conv0_w", "conv1_w", "temp"]


def to_device(t, device="cuda"):
    return {k: v.to(device).contiguous() for k, v in t.items()}
