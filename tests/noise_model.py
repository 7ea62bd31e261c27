"""Test infrastructure: the error scale of the parameter gradients, derived from the oracle alone.

A parameter gradient is a sum over all B*S tokens of products, e.g. d_w_qk[c,e] = sum_t d_qk0[t,c] x[t,e].  An
implementation that keeps its activations in bf16 (q, k, v, o, P, d_o, dS, the latent gradient: "bf16 in, fp32
accumulate") perturbs every term of that sum by an independent relative error of a few 2^-9, so the error of the
sum is a random walk over the terms:

    sigma[c,e] = kappa * 2^-9 * sqrt( sum_t term_t[c,e]^2 ).

`term_rss` evaluates the square root for every element of every matrix-shaped parameter gradient from the oracle's
intermediates (one contraction of the squared factors each), `temp_term_rss` for d_temp (its terms are the
(query, key) pairs' dS * logit).  kappa, the number of bf16 roundings a term has
effectively been through, is not guessed: `storage_model_gradients` runs the oracle's own steps once more with a
round-to-bf16 at each place where such an implementation stores a tensor or hands it to a tensor-core contraction
(nothing else is changed), and kappa = rms((model - exact) / (2^-9 * rss)) per gradient.  Nothing here looks at
the CUDA path's results.
"""
import math

import torch

from oracle import cca_oracle as O

F64 = torch.float64
U = 2.0 ** -9


def _r(x):
    """Round to bf16 and widen back (the model's only deviation from the oracle)."""
    return x.to(torch.bfloat16).to(F64)


def term_rss(cfg, t, I, G, power=2):
    """power = 2: sqrt(sum over tokens of term^2) for every element of every matrix-shaped parameter gradient (the
    scale of a random walk over the terms).  power = 1: sum of |term| (the scale of the worst case, every rounding
    in the same direction; used where a sum has too few terms for a random walk)."""
    B, S, E = I["x"].shape
    T = B * S
    L, Lk, dh = cfg.L, cfg.L_k, cfg.head_dim
    H = cfg.n_q_heads + cfg.n_kv_heads

    def pw(v):
        return v ** 2 if power == 2 else v.abs()

    def root(v):
        return v.sqrt() if power == 2 else v

    def noisy_factor(v):
        """|v| of the computed (hence noisy) factor of a term, floored per token by the rms over its head's channels:
        the rounding noise of a latent-gradient element is at the scale of its head's typical element, not of its
        own value, which may be a cancelling sum (over the query heads of a group, over the queries of a key)."""
        vh = v.reshape(*v.shape[:-1], -1, dh)
        floor = vh.pow(2).mean(dim=-1, keepdim=True).sqrt()
        return torch.maximum(vh.abs(), floor).reshape(v.shape)

    x2 = pw(I["x"].reshape(T, E))
    r = {}
    r["w_qk"] = root(pw(noisy_factor(G["d_qk0"].reshape(T, L))).T @ x2)
    dv = noisy_factor(G["d_v"].reshape(T, Lk))
    r["w_v1"] = root(pw(dv[:, :Lk // 2]).T @ x2)
    r["w_v2"] = root(pw(dv[:, Lk // 2:]).T @ pw(I["xs"].reshape(T, E)))
    r["w_o"] = root(pw(O._f64(t["d_out"]).reshape(T, E)).T @ pw(noisy_factor(I["o"].reshape(T, -1))))
    k = cfg.k_seq
    c0 = torch.zeros(L, k, dtype=F64)
    if cfg.flags & O.CONV1:
        dy1 = noisy_factor(G["d_y1"])
        for j in range(k):
            lag = k - 1 - j
            if lag < S:
                c0[:, j] = (pw(dy1[:, lag:]) * pw(I["qk0"][:, :S - lag])).sum(dim=(0, 1))
    r["conv0_w"] = root(c0)
    k = cfg.k_ch
    c1 = torch.zeros(H, dh, dh, k, dtype=F64)
    if cfg.flags & O.CONV2:
        dy2 = pw(noisy_factor(G["d_y2"]).reshape(B, S, H, dh))
        y1 = pw(I["y1"].reshape(B, S, H, dh))
        for j in range(k):
            lag = k - 1 - j
            if lag < S:
                c1[..., j] = torch.einsum("bsho,bshi->hoi", dy2[:, lag:], y1[:, :S - lag])
    r["conv1_w"] = root(c1.reshape(L, dh, k))
    return r


def out_term_rss(t, I):
    """sqrt(sum_c (o[t,c] W_o[e,c])^2) for every element of the block's output (Eq. 11, up-projection)."""
    B, S = I["x"].shape[:2]
    o2 = I["o"].reshape(B, S, -1) ** 2
    return (o2 @ (O._f64(t["w_o"]) ** 2).transpose(0, 1)).sqrt()


def temp_term_rss(cfg, I, G, power=2):
    """Noise scale of d_temp, one number per kv head.  d_temp[j] = sum over the (query, key) pairs of the group's
    heads of dS * logit (Eq. 11: the temperature scales every logit of its kv head), so the terms are those
    products, formed from the oracle's q, k, v, o and d_o exactly as its attention adjoint forms them: sqrt(sum of
    term^2) (power = 2) or sum of |term| (power = 1).  One more contribution enters in quadrature (power = 2) or
    is added (power = 1): a row of dS sums to zero only as far as delta = rowsum(dO * O) agrees with the
    probabilities the backward recomputes, and O was accumulated from bf16-rounded probabilities; the residual of row
    t, of scale sqrt(sum_s (P_s (dP_s - delta_t))^2) roundings, multiplies the row's mean logit sum_s P_s s_s, which
    is not small when the keys a row attends to are aligned with its query."""
    q, k, v, o, do = I["q"], I["k"], I["v"], I["o"], G["d_o"]
    B, S, hq, dh = q.shape
    g = cfg.g
    inv = 1.0 / math.sqrt(dh)
    acc = torch.zeros(cfg.n_kv_heads, dtype=F64)
    if not cfg.flags & O.QK_NORM:
        return acc
    ar = torch.arange(S)
    blk = max(1, (1 << 24) // max(S, 1))
    for b in range(B):
        for i in range(hq):
            j = i // g
            kj, vj = k[b, :, j, :], v[b, :, j, :]
            for r0 in range(0, S, blk):
                r1 = min(S, r0 + blk)
                s = (q[b, r0:r1, i, :] @ kj.transpose(0, 1)) * inv
                sm = s.masked_fill(ar[None, :] > ar[r0:r1, None], float("-inf")) if cfg.causal else s
                p = torch.softmax(sm, dim=-1)
                doi = do[b, r0:r1, i, :]
                D = (doi * o[b, r0:r1, i, :]).sum(dim=-1, keepdim=True)
                ds = p * (doi @ vj.transpose(0, 1) - D)
                s0 = torch.where(torch.isfinite(sm), s, torch.zeros_like(s))
                sbar = (p * s0).sum(dim=-1)
                if power == 2:
                    acc[j] += (ds * s0).pow(2).sum() + (sbar.pow(2) * ds.pow(2).sum(dim=-1)).sum()
                else:
                    acc[j] += (ds * s0).abs().sum() + (sbar.abs() * ds.abs().sum(dim=-1)).sum()
    return acc.sqrt() if power == 2 else acc


def _attention_bf16_storage(q, k, v, do, g, causal):
    """Eq. 11 and its adjoint with the probabilities rounded where a bf16-operand implementation rounds them:
    the forward's P before it multiplies V (row sums over the rounded values), the backward's P^T before it
    multiplies dO, dS before it multiplies K and Q.  Returns o (unrounded), dq, dk, dv."""
    B, S, hq, dh = q.shape
    inv = 1.0 / math.sqrt(dh)
    o = torch.zeros_like(q)
    dq = torch.zeros_like(q)
    dk = torch.zeros_like(k)
    dv = torch.zeros_like(v)
    blk = max(1, (1 << 24) // max(S, 1))
    ar = torch.arange(S)
    for b in range(B):
        for i in range(hq):
            j = i // g
            kj, vj = k[b, :, j, :], v[b, :, j, :]
            for r0 in range(0, S, blk):
                r1 = min(S, r0 + blk)
                qi = q[b, r0:r1, i, :]
                s = (qi @ kj.transpose(0, 1)) * inv
                if causal:
                    s = s.masked_fill(ar[None, :] > ar[r0:r1, None], float("-inf"))
                m = s.max(dim=-1, keepdim=True).values
                e = _r(torch.exp(s - m))
                z = e.sum(dim=-1, keepdim=True)
                oi = (e @ vj) / z
                o[b, r0:r1, i, :] = oi
                p = torch.exp(s - m) / z                                   # 2^(s - lse) with the forward's lse
                doi = do[b, r0:r1, i, :]
                dp = doi @ vj.transpose(0, 1)
                D = (doi * oi).sum(dim=-1, keepdim=True)
                ds = _r(p * (dp - D))
                dq[b, r0:r1, i, :] = (ds @ kj) * inv
                dk[b, :, j, :] += (ds.transpose(0, 1) @ qi) * inv
                dv[b, :, j, :] += _r(p).transpose(0, 1) @ doi
    return o, dq, dk, dv


def storage_model_gradients(cfg, t):
    """The oracle's forward and backward steps, composed as in oracle.forward / oracle.backward, with a bf16
    rounding at each storage point of a "bf16 in, fp32 accumulate" implementation: conv1's output (operand of the
    conv2 contraction), q, k, v, o, P, d_o, dS, the pre-norm latent gradient (operand of the conv2-adjoint
    contraction), and the latent gradient that enters the projection gradients.  Returns the parameter gradients."""
    x = O._f64(t["x"])
    B, S, E = x.shape
    hq, hk, dh, g = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.g
    Lq, Lk, L = cfg.L_q, cfg.L_k, cfg.L
    w = {n: O._f64(t[n]) for n in ("w_qk", "w_v1", "w_v2", "w_o", "conv0_w", "conv1_w", "temp")}
    qk0 = O.down_projection(x, w["w_qk"])
    y1 = O.conv1_seq(qk0, w["conv0_w"]) if cfg.flags & O.CONV1 else qk0
    y1r = _r(y1) if cfg.flags & O.CONV2 else y1
    y2 = O.conv2_seq_ch(y1r, w["conv1_w"], hq + hk, dh) if cfg.flags & O.CONV2 else y1
    q0 = qk0[..., :Lq].reshape(B, S, hq, dh)
    k0 = qk0[..., Lq:].reshape(B, S, hk, dh)
    yq = y2[..., :Lq].reshape(B, S, hq, dh)
    yk = y2[..., Lq:].reshape(B, S, hk, dh)
    qh, kh = O.qk_mean(q0, k0, yq, yk, g) if cfg.flags & O.QK_MEAN else (yq, yk)
    v_flat, xs = O.value_shift(x, w["w_v1"], w["w_v2"], bool(cfg.flags & O.V_SHIFT))
    v = _r(v_flat).reshape(B, S, hk, dh)
    if cfg.flags & O.QK_NORM:
        beta = torch.exp(w["temp"])
        qn = O.l2norm_scale(qh, math.sqrt(dh))
        kn = O.l2norm_scale(kh, math.sqrt(dh) * beta)
    else:
        qn, kn = qh, kh
    ang = O.rope_angles(S, dh, cfg.rope_base) if cfg.flags & O.ROPE else None
    q = _r(O.rope(qn, ang) if ang is not None else qn)
    k = _r(O.rope(kn, ang) if ang is not None else kn)
    d_out = O._f64(t["d_out"])
    do = _r(d_out @ w["w_o"]).reshape(B, S, hq, dh)
    o, dq, dk, dv = _attention_bf16_storage(q, k, v, do, g, bool(cfg.causal))
    G = {"d_w_o": torch.einsum("bse,bsc->ec", d_out, _r(o).reshape(B, S, Lq))}
    G["out"] = O.up_projection(_r(o).reshape(B, S, Lq), w["w_o"])
    dqn = O.rope_adjoint(dq, ang) if ang is not None else dq
    dkn = O.rope_adjoint(dk, ang) if ang is not None else dk
    if cfg.flags & O.QK_NORM:
        k_n = O.rope_adjoint(k, ang) if ang is not None else k          # the stored (rounded) key, rotated back
        G["d_temp"] = (dkn * k_n).sum(dim=(0, 1, 3))
        dqh = O.l2norm_scale_adjoint(dqn, qh, math.sqrt(dh))
        dkh = O.l2norm_scale_adjoint(dkn, kh, math.sqrt(dh) * beta)
    else:
        G["d_temp"] = torch.zeros(hk, dtype=F64)
        dqh, dkh = dqn, dkn
    dq0 = torch.zeros(B, S, hq, dh, dtype=F64)
    dk0 = torch.zeros(B, S, hk, dh, dtype=F64)
    if cfg.flags & O.QK_MEAN:
        dmu = dqh + dkh.unsqueeze(3).expand(B, S, hk, g, dh).reshape(B, S, hq, dh) / g
        dq0 += 0.5 * dmu
        dk0 += 0.5 * dmu.reshape(B, S, hk, g, dh).sum(dim=3)
    dy2 = torch.cat([dqh.reshape(B, S, Lq), dkh.reshape(B, S, Lk)], dim=-1)
    if cfg.flags & O.CONV2:
        dy1, G["d_conv1_w"] = O.conv2_seq_ch_adjoint(_r(dy2), y1r, w["conv1_w"], hq + hk, dh)
    else:
        dy1, G["d_conv1_w"] = dy2, torch.zeros(L, dh, cfg.k_ch, dtype=F64)
    if cfg.flags & O.CONV1:
        dqk0, G["d_conv0_w"] = O.conv1_seq_adjoint(dy1, qk0, w["conv0_w"])
    else:
        dqk0, G["d_conv0_w"] = dy1, torch.zeros(L, cfg.k_seq, dtype=F64)
    dqk0 = _r(dqk0 + torch.cat([dq0.reshape(B, S, Lq), dk0.reshape(B, S, Lk)], dim=-1))
    dvf = _r(dv.reshape(B, S, Lk))
    G["d_w_qk"] = torch.einsum("bsl,bse->le", dqk0, x)
    G["d_w_v1"] = torch.einsum("bsl,bse->le", dvf[..., : Lk // 2], x)
    G["d_w_v2"] = torch.einsum("bsl,bse->le", dvf[..., Lk // 2:], xs)
    return G


NOISE_FLOOR = 1e-4       # sums whose noise scale 2^-9 rss is below this (1 % of the absolute tolerance) count as exact


def noisy(rss):
    """Elements whose sum has terms large enough for rounding noise to matter next to the absolute 1e-2 (a gradient
    that is zero in exact arithmetic, e.g. through a one-key softmax, has terms of 1e-16 and is left to the plain rule)."""
    return U * rss > NOISE_FLOOR


MIN_NOISY = 64            # fewer noisy elements than this measure nothing


def kappa(model, exact, rss):
    """Effective number of bf16 roundings per term: rms of the model's error in units of 2^-9 * rss, over the
    `noisy` elements (over every element with terms at all if fewer than MIN_NOISY are noisy: the gradient is then
    tiny against the absolute 1e-2 and the figure hardly matters).  Never below 1 (one rounding is the least such a
    path can have)."""
    m = noisy(rss)
    if int(m.sum()) < MIN_NOISY:
        m = rss > 0
    if not bool(m.any()):
        return 1.0
    z = (model - exact)[m] / (U * rss[m])
    return max(1.0, float(z.pow(2).mean().sqrt()))
