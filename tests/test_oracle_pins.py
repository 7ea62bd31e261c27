"""Pins for the fp64 oracle: each test checks it against something other than itself --
brute force in pure Python, a textbook or library routine, a closed form, an invariant
the paper states, finite differences or autograd.  CPU only."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import cca_oracle as O
from paper_2510_04476_b200 import synth

F64 = torch.float64


def small_shape(**kw):
    base = dict(name="t", B=2, S=12, d_model=32, n_q_heads=4, n_kv_heads=2, head_dim=4, seed=11)
    base.update(kw)
    return synth.Shape(**base)


def cfg_of(sh, **kw):
    d = dict(d_model=sh.d_model, n_q_heads=sh.n_q_heads, n_kv_heads=sh.n_kv_heads, head_dim=sh.head_dim,
             k_seq=sh.k_seq, k_ch=sh.k_ch, causal=sh.causal, flags=sh.flags, rope_base=sh.rope_base)
    d.update(kw)
    return O.OracleConfig(**d)


def inputs64(sh, scale_w=10.0):
    """fp64 inputs; projection weights are scaled up so tiny shapes have O(1) latents."""
    t = synth.make_inputs(sh)
    t = {k: v.to(F64) for k, v in t.items()}
    for n in ("w_qk", "w_v1", "w_v2", "w_o"):
        t[n] = t[n] * scale_w
    return t


# ------------------------------------------------------------------ attention core

def brute_attention(q, k, v, g, causal):
    """Pure-Python softmax attention, one scalar at a time (Eq. 1-2 / Eq. 11)."""
    B, S, hq, dh = q.shape
    o = np.zeros((B, S, hq, dh))
    q, k, v = q.numpy(), k.numpy(), v.numpy()
    for b in range(B):
        for i in range(hq):
            j = i // g
            for t in range(S):
                last = t if causal else S - 1
                sc = [sum(q[b, t, i, c] * k[b, u, j, c] for c in range(dh)) / math.sqrt(dh) for u in range(last + 1)]
                m = max(sc)
                e = [math.exp(s - m) for s in sc]
                z = sum(e)
                for c in range(dh):
                    o[b, t, i, c] = sum(e[u] / z * v[b, u, j, c] for u in range(last + 1))
    return torch.from_numpy(o)


@pytest.mark.parametrize("causal", [1, 0])
@pytest.mark.parametrize("hq,hk", [(4, 4), (4, 2), (4, 1)])
def test_attention_matches_brute_force(causal, hq, hk):
    torch.manual_seed(0)
    B, S, dh = 2, 9, 6
    q = torch.randn(B, S, hq, dh, dtype=F64)
    k = torch.randn(B, S, hk, dh, dtype=F64)
    v = torch.randn(B, S, hk, dh, dtype=F64)
    o, lse, p = O.attention(q, k, v, hq // hk, bool(causal), want_p=True)
    ref = brute_attention(q, k, v, hq // hk, causal)
    assert torch.allclose(o, ref, atol=1e-13, rtol=1e-12)
    assert torch.allclose(p.sum(-1), torch.ones_like(p.sum(-1)), atol=1e-14)
    if causal:
        assert float(p.triu(1).abs().max()) == 0.0
    # lse is the log of the softmax denominator of the scaled scores
    s00 = (q[0, S - 1, 0] @ k[0, :, 0].T) / math.sqrt(dh)
    assert abs(float(torch.logsumexp(s00, 0)) - float(lse[0, 0, S - 1])) < 1e-12


def test_attention_rows_subset_equals_full():
    torch.manual_seed(1)
    q = torch.randn(1, 20, 4, 8, dtype=F64)
    k = torch.randn(1, 20, 2, 8, dtype=F64)
    v = torch.randn(1, 20, 2, 8, dtype=F64)
    o, lse, _ = O.attention(q, k, v, 2, True)
    rows = [0, 7, 19]
    o2, lse2, _ = O.attention(q, k, v, 2, True, rows=rows)
    assert torch.allclose(o[:, rows], o2, atol=1e-14) and torch.allclose(lse[:, :, rows], lse2, atol=1e-14)


# ------------------------------------------------------------------ causality / halo / v-shift

def test_causality_bit_identical():
    sh = small_shape(S=16)
    t = inputs64(sh)
    cfg = cfg_of(sh)
    out, _ = O.forward(cfg, t, t["x"])
    t0 = 9
    x2 = t["x"].clone()
    x2[:, t0:] += torch.randn_like(x2[:, t0:])
    out2, _ = O.forward(cfg, t, x2)
    assert torch.equal(out[:, :t0], out2[:, :t0])
    assert not torch.equal(out[:, t0:], out2[:, t0:])


@pytest.mark.parametrize("k_seq,k_ch", [(2, 2), (3, 1), (1, 4), (4, 3)])
def test_conv_halo_is_constant_size(k_seq, k_ch):
    """q[t], k[t] depend on x[t-pad .. t] only, pad = k_seq + k_ch - 2."""
    sh = small_shape(S=16, k_seq=k_seq, k_ch=k_ch)
    t = inputs64(sh)
    cfg = cfg_of(sh)
    I = O.pre_attention(cfg, t, t["x"])
    pad = k_seq + k_ch - 2
    tt = 12
    x2 = t["x"].clone()
    x2[:, : tt - pad] += 1.0
    I2 = O.pre_attention(cfg, t, x2)
    assert torch.equal(I["q"][:, tt], I2["q"][:, tt]) and torch.equal(I["k"][:, tt], I2["k"][:, tt])
    if pad > 0:
        x3 = t["x"].clone()
        x3[:, tt - pad] += 1.0
        I3 = O.pre_attention(cfg, t, x3)
        assert not torch.equal(I["q"][:, tt], I3["q"][:, tt])


def test_value_shift_half_cannot_see_present():
    sh = small_shape(S=8)
    t = inputs64(sh)
    cfg = cfg_of(sh)
    I = O.pre_attention(cfg, t, t["x"])
    tt = 5
    x2 = t["x"].clone()
    x2[:, tt] += 1.0
    I2 = O.pre_attention(cfg, t, x2)
    v = I["v"].reshape(sh.B, sh.S, -1)
    v2 = I2["v"].reshape(sh.B, sh.S, -1)
    half = sh.L_k // 2
    assert torch.equal(v[:, tt, half:], v2[:, tt, half:])          # built from x[t-1]
    assert not torch.equal(v[:, tt, :half], v2[:, tt, :half])      # built from x[t]
    assert not torch.equal(v[:, tt + 1, half:], v2[:, tt + 1, half:])
    assert float(v[:, 0, half:].abs().max()) == 0.0                # x[-1] = 0
    # h_k even: the last h_k/2 heads are exactly the shifted ones
    assert torch.equal(I["v"][:, tt, sh.n_kv_heads // 2:], I2["v"][:, tt, sh.n_kv_heads // 2:])


# ------------------------------------------------------------------ reductions

def test_reduces_to_plain_mha():
    """C = 1, every latent transform off, h_k = h_q: Eq. 1-2 with W_V = [W_v1; W_v2]."""
    sh = small_shape(S=7, d_model=16, n_q_heads=4, n_kv_heads=4, head_dim=4, flags=0)
    t = inputs64(sh)
    cfg = cfg_of(sh)
    out, _ = O.forward(cfg, t, t["x"])
    x = t["x"]
    wq, wk = t["w_qk"][: sh.L_q], t["w_qk"][sh.L_q:]
    wv = torch.cat([t["w_v1"], t["w_v2"]], 0)
    B, S = sh.B, sh.S
    q = (x @ wq.T).reshape(B, S, 4, 4)
    k = (x @ wk.T).reshape(B, S, 4, 4)
    v = (x @ wv.T).reshape(B, S, 4, 4)
    o = brute_attention(q, k, v, 1, 1)
    ref = o.reshape(B, S, -1) @ t["w_o"].T
    assert torch.allclose(out, ref, atol=1e-12, rtol=1e-12)


def test_identity_convs_equal_convs_off():
    sh = small_shape(k_seq=3, k_ch=2)
    t = inputs64(sh)
    t["conv0_w"] = torch.zeros_like(t["conv0_w"])
    t["conv0_w"][:, -1] = 1.0
    w1 = torch.zeros_like(t["conv1_w"])
    for c in range(sh.L):
        w1[c, c % sh.head_dim, -1] = 1.0
    t["conv1_w"] = w1
    out_on, _ = O.forward(cfg_of(sh), t, t["x"])
    out_off, _ = O.forward(cfg_of(sh, flags=sh.flags & ~(O.CONV1 | O.CONV2)), t, t["x"])
    assert torch.allclose(out_on, out_off, atol=1e-13)


def _repeat_kv_heads(t, sh, g):
    """CCA weights whose k / v heads are the g-fold repeated heads of a CCGQA set."""
    dh, hk, Lq, E = sh.head_dim, sh.n_kv_heads, sh.L_q, sh.d_model
    rep = lambda a: a.reshape(hk, dh, *a.shape[1:]).repeat_interleave(g, dim=0).reshape(hk * g * dh, *a.shape[1:])
    u = dict(t)
    u["w_qk"] = torch.cat([t["w_qk"][:Lq], rep(t["w_qk"][Lq:])], 0)
    u["conv0_w"] = torch.cat([t["conv0_w"][:Lq], rep(t["conv0_w"][Lq:])], 0)
    u["conv1_w"] = torch.cat([t["conv1_w"][:Lq], rep(t["conv1_w"][Lq:])], 0)
    wv = rep(torch.cat([t["w_v1"], t["w_v2"]], 0))
    u["w_v1"], u["w_v2"] = wv[: wv.shape[0] // 2], wv[wv.shape[0] // 2:]
    u["temp"] = t["temp"].repeat_interleave(g)
    return u


def test_ccgqa_equals_cca_with_repeated_heads():
    fl = O.ALL_FLAGS & ~(O.QK_MEAN | O.V_SHIFT)
    sh = small_shape(flags=fl)
    t = inputs64(sh)
    g = sh.n_q_heads // sh.n_kv_heads
    out_g, _ = O.forward(cfg_of(sh), t, t["x"])
    u = _repeat_kv_heads(t, sh, g)
    out_c, _ = O.forward(cfg_of(sh, n_kv_heads=sh.n_q_heads), u, t["x"])
    assert torch.allclose(out_g, out_c, atol=1e-12)
    # with q-k-mean on, E_group's mean over the group breaks the equivalence
    out_g2, _ = O.forward(cfg_of(sh, flags=fl | O.QK_MEAN), t, t["x"])
    out_c2, _ = O.forward(cfg_of(sh, n_kv_heads=sh.n_q_heads, flags=fl | O.QK_MEAN), u, t["x"])
    assert not torch.allclose(out_g2, out_c2, atol=1e-6)


def test_group_of_one_makes_group_ops_identity():
    sh = small_shape(n_kv_heads=4)
    t = inputs64(sh)
    I = O.pre_attention(cfg_of(sh), t, t["x"])
    B, S = sh.B, sh.S
    q0 = I["qk0"][..., : sh.L_q].reshape(B, S, 4, 4)
    k0 = I["qk0"][..., sh.L_q:].reshape(B, S, 4, 4)
    mu = 0.5 * (q0 + k0)
    assert torch.allclose(I["q_hat"], I["y2"][..., : sh.L_q].reshape(B, S, 4, 4) + mu, atol=1e-14)
    assert torch.allclose(I["k_hat"], I["y2"][..., sh.L_q:].reshape(B, S, 4, 4) + mu, atol=1e-14)


def test_qk_mean_group_mean_by_loops():
    sh = small_shape()
    t = inputs64(sh)
    I = O.pre_attention(cfg_of(sh), t, t["x"])
    g, dh = 2, sh.head_dim
    b, s = 1, 5
    qk0, y2 = I["qk0"][b, s], I["y2"][b, s]
    for j in range(sh.n_kv_heads):
        acc = torch.zeros(dh, dtype=F64)
        for i in range(j * g, (j + 1) * g):
            mu = 0.5 * (qk0[i * dh:(i + 1) * dh] + qk0[sh.L_q + j * dh: sh.L_q + (j + 1) * dh])
            assert torch.allclose(I["q_hat"][b, s, i], y2[i * dh:(i + 1) * dh] + mu, atol=1e-14)
            acc += mu
        assert torch.allclose(I["k_hat"][b, s, j], y2[sh.L_q + j * dh: sh.L_q + (j + 1) * dh] + acc / g, atol=1e-14)


# ------------------------------------------------------------------ norm / temperature / softmax closed forms

def test_norms_and_logit_bound_and_scale_invariance():
    sh = small_shape()
    t = inputs64(sh)
    cfg = cfg_of(sh)
    out, I = O.forward(cfg, t, t["x"], want_p=True)
    dh = sh.head_dim
    assert torch.allclose(I["q"].norm(dim=-1), torch.full_like(I["q"].norm(dim=-1), math.sqrt(dh)), atol=1e-12)
    beta = torch.exp(t["temp"])
    assert torch.allclose(I["k"].norm(dim=-1), (math.sqrt(dh) * beta).expand_as(I["k"].norm(dim=-1)), atol=1e-12)
    s = torch.einsum("bthd,bujd->bhtuj", I["q"], I["k"]) / math.sqrt(dh)
    assert float(s.abs().max()) <= math.sqrt(dh) * float(beta.max()) + 1e-12
    t2 = dict(t)
    t2["w_qk"] = t["w_qk"] * 3.7
    out2, _ = O.forward(cfg, t2, t["x"])
    assert torch.allclose(out, out2, atol=1e-12)


def test_cold_keys_give_running_mean_of_values():
    sh = small_shape()
    t = inputs64(sh)
    t["temp"] = torch.full_like(t["temp"], -50.0)
    _, I = O.forward(cfg_of(sh), t, t["x"])
    v, g = I["v"], 2
    run = torch.cumsum(v, dim=1) / torch.arange(1, sh.S + 1, dtype=F64)[None, :, None, None]
    ref = run.repeat_interleave(g, dim=2)
    assert torch.allclose(I["o"], ref, atol=1e-12)


def test_single_token_closed_form():
    sh = small_shape(S=1)
    t = inputs64(sh)
    out, I = O.forward(cfg_of(sh), t, t["x"])
    x0 = t["x"][:, 0]
    v = torch.cat([x0 @ t["w_v1"].T, torch.zeros(sh.B, sh.L_k // 2, dtype=F64)], -1)
    o = v.reshape(sh.B, sh.n_kv_heads, sh.head_dim).repeat_interleave(2, dim=1).reshape(sh.B, -1)
    assert torch.allclose(out[:, 0], o @ t["w_o"].T, atol=1e-13)


# ------------------------------------------------------------------ RoPE

def test_rope_position_zero_identity_and_textbook_2d():
    u = torch.randn(1, 5, 3, 2, dtype=F64)
    ang = O.rope_angles(5, 2, 10000.0)
    r = O.rope(u, ang)
    assert torch.equal(r[:, 0], u[:, 0])
    for tpos in range(5):                                   # theta_0 = 1: rotation by t radians
        c, s = math.cos(tpos), math.sin(tpos)
        R = torch.tensor([[c, -s], [s, c]], dtype=F64)
        assert torch.allclose(r[0, tpos], u[0, tpos] @ R.T, atol=1e-14)
    ang8 = O.rope_angles(4, 8, 10000.0)
    assert torch.allclose(ang8[1], torch.tensor([1.0, 10000 ** -0.25, 10000 ** -0.5, 10000 ** -0.75], dtype=F64))


def test_rope_relative_shift_invariance():
    sh = small_shape()
    t = inputs64(sh)
    cfg = cfg_of(sh)
    Ia = O.pre_attention(cfg, t, t["x"], pos0=0)
    Ib = O.pre_attention(cfg, t, t["x"], pos0=37)
    _, _, pa = O.attention(Ia["q"], Ia["k"], Ia["v"], cfg.g, True, want_p=True)
    _, _, pb = O.attention(Ib["q"], Ib["k"], Ib["v"], cfg.g, True, want_p=True)
    assert not torch.allclose(Ia["q"], Ib["q"])
    assert torch.allclose(pa, pb, atol=1e-12)
    # rotation keeps the norm
    assert torch.allclose(Ia["q"].norm(dim=-1), Ia["q_n"].norm(dim=-1), atol=1e-12)


# ------------------------------------------------------------------ convs against library routines

@pytest.mark.parametrize("k", [1, 2, 3, 4])
def test_conv1_impulse_and_numpy_convolve(k):
    L, S = 5, 10
    w0 = torch.randn(L, k, dtype=F64)
    u = torch.zeros(1, S, L, dtype=F64)
    u[0, 3] = 1.0
    y = O.conv1_seq(u, w0)
    for j in range(k):                                       # tap j acts at lag k-1-j
        tpos = 3 + (k - 1 - j)
        assert torch.equal(y[0, tpos], w0[:, j])
    u = torch.randn(2, S, L, dtype=F64)
    y = O.conv1_seq(u, w0)
    for c in range(L):
        ref = np.convolve(u[1, :, c].numpy(), w0[c].numpy()[::-1])[:S]
        assert np.allclose(y[1, :, c].numpy(), ref, atol=1e-13)


@pytest.mark.parametrize("k_seq,k_ch", [(2, 2), (3, 4), (1, 1)])
def test_both_convs_match_torch_conv1d(k_seq, k_ch):
    """Library restatement: left-pad once by k_seq+k_ch-2, depth-wise conv1d, grouped conv1d."""
    H, dh, S, B = 3, 4, 9, 2
    L = H * dh
    u = torch.randn(B, S, L, dtype=F64)
    w0 = torch.randn(L, k_seq, dtype=F64)
    w1 = torch.randn(L, dh, k_ch, dtype=F64)
    y = O.conv2_seq_ch(O.conv1_seq(u, w0), w1, H, dh)
    z = F.pad(u.permute(0, 2, 1), (k_seq + k_ch - 2, 0))
    z = F.conv1d(z, w0[:, None, :], groups=L)
    z = F.conv1d(z, w1, groups=H).permute(0, 2, 1)
    assert torch.allclose(y, z, atol=1e-12)


# ------------------------------------------------------------------ the paper's closed-form counts

@pytest.mark.parametrize("E,hq,hk,dh", [(2048, 16, 4, 64), (4096, 8, 2, 128), (2048, 8, 8, 64)])
def test_formulas_match_comparison_table(E, hq, hk, dh):
    B, S, ks, kc = 3, 4096, 2, 2
    cfg = O.OracleConfig(E, hq, hk, dh, ks, kc)
    d = O.describe(cfg, B, S)
    C1, C2 = E // (hq * dh), E // (hk * dh)
    conv = d["conv_params"]
    assert d["params"] - conv == 2 * E * E // C1 + 2 * E * E // C2
    assert d["kv_cache_elems"] == 2 * B * S * E // C2
    assert d["fwd_flops"] - 2 * B * S * conv == 4 * B * S * E * E // C1 + 4 * B * S * E * E // C2 + 4 * B * E * S * S // C1
    assert d["decode_flops"] - 2 * B * conv == 4 * B * E * E // C1 + 4 * B * E * E // C2 + 4 * B * E * S // C1
    # conv footnote with the CCGQA substitution (e_bar, h_q + h_k): the grouped term is
    # e_bar^2/(h_q+h_k)*k_ch; the depth-wise term is one tap set per latent channel, which lies
    # between zero and the footnote's doubled 2*e_bar*k_seq
    e_bar = E // C1 + E // C2
    grouped = e_bar * e_bar // (hq + hk) * kc
    assert grouped == (hq + hk) * dh * dh * kc
    assert conv == e_bar * ks + grouped
    assert grouped < conv <= 2 * e_bar * ks + grouped
    if hq == hk:                                            # CCA row recovered at C1 = C2
        C = C1
        assert d["params"] - conv == 4 * E * E // C
        assert d["kv_cache_elems"] == 2 * B * S * E // C


# ------------------------------------------------------------------ backward

def _loss_fn(cfg, t, names):
    def f(*args):
        u = dict(t)
        for n, a in zip(names, args):
            u[n] = a
        out, _ = O.forward(cfg, u, u["x"])
        return (out * t["d_out"]).sum()
    return f


@pytest.mark.parametrize("flags", [O.ALL_FLAGS, 0, O.ALL_FLAGS & ~O.QK_MEAN, O.ALL_FLAGS & ~O.V_SHIFT,
                                   O.CONV1 | O.QK_NORM, O.CONV2 | O.ROPE | O.QK_MEAN])
@pytest.mark.parametrize("hk,causal", [(2, 1), (4, 1), (1, 0)])
def test_backward_matches_finite_differences(flags, hk, causal):
    sh = small_shape(B=2, S=6, d_model=12, n_q_heads=4, n_kv_heads=hk, head_dim=4, k_seq=3, k_ch=2,
                     flags=flags, causal=causal)
    t = inputs64(sh, scale_w=15.0)
    cfg = cfg_of(sh)
    out, I = O.forward(cfg, t, t["x"])
    G = O.backward(cfg, t, I, t["d_out"])
    names = ["x", "w_qk", "w_v1", "w_v2", "w_o", "conv0_w", "conv1_w", "temp"]
    rng = np.random.default_rng(0)
    for n in names:
        base = t[n]
        flat_idx = rng.choice(base.numel(), size=min(6, base.numel()), replace=False)
        for fi in flat_idx:
            h = 1e-6
            tp, tm = dict(t), dict(t)
            e = torch.zeros(base.numel(), dtype=F64)
            e[fi] = h
            tp[n] = base + e.reshape(base.shape)
            tm[n] = base - e.reshape(base.shape)
            lp = (O.forward(cfg, tp, tp["x"])[0] * t["d_out"]).sum()
            lm = (O.forward(cfg, tm, tm["x"])[0] * t["d_out"]).sum()
            fd = float(lp - lm) / (2 * h)
            an = float(G["d_" + n].reshape(-1)[fi])
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(fd)) + 2e-7, (n, int(fi), fd, an)


@pytest.mark.parametrize("hk", [1, 2, 4])
def test_backward_matches_autograd_of_forward(hk):
    sh = small_shape(B=2, S=10, d_model=24, n_q_heads=4, n_kv_heads=hk, head_dim=6, k_seq=2, k_ch=3)
    t = inputs64(sh, scale_w=12.0)
    cfg = cfg_of(sh)
    names = ["x", "w_qk", "w_v1", "w_v2", "w_o", "conv0_w", "conv1_w", "temp"]
    leaves = [t[n].clone().requires_grad_(True) for n in names]
    u = dict(t)

    class _NoDetach(dict):
        pass
    # run the forward steps on autograd leaves (the step functions are differentiable)
    x, w_qk, w_v1, w_v2, w_o, c0, c1, temp = leaves
    B, S = sh.B, sh.S
    qk0 = O.down_projection(x, w_qk)
    y2 = O.conv2_seq_ch(O.conv1_seq(qk0, c0), c1, sh.n_q_heads + hk, sh.head_dim)
    q0 = qk0[..., : sh.L_q].reshape(B, S, sh.n_q_heads, -1)
    k0 = qk0[..., sh.L_q:].reshape(B, S, hk, -1)
    qh, kh = O.qk_mean(q0, k0, y2[..., : sh.L_q].reshape_as(q0), y2[..., sh.L_q:].reshape_as(k0), cfg.g)
    vflat, _ = O.value_shift(x, w_v1, w_v2, True)
    ang = O.rope_angles(S, sh.head_dim, sh.rope_base)
    q = O.rope(O.l2norm_scale(qh, math.sqrt(sh.head_dim)), ang)
    k = O.rope(O.l2norm_scale(kh, math.sqrt(sh.head_dim) * torch.exp(temp)), ang)
    v = vflat.reshape(B, S, hk, -1)
    # differentiable attention via torch.softmax (independent of O.attention's loop)
    kb = k.repeat_interleave(cfg.g, dim=2)
    vb = v.repeat_interleave(cfg.g, dim=2)
    s = torch.einsum("bthd,buhd->bhtu", q, kb) / math.sqrt(sh.head_dim)
    s = s.masked_fill(torch.ones(S, S, dtype=torch.bool).triu(1), float("-inf"))
    o = torch.einsum("bhtu,buhd->bthd", torch.softmax(s, -1), vb)
    out = O.up_projection(o.reshape(B, S, -1), w_o)
    out_ref, I = O.forward(cfg, t, t["x"])
    assert torch.allclose(out.detach(), out_ref, atol=1e-12)
    (out * t["d_out"]).sum().backward()
    G = O.backward(cfg, t, I, t["d_out"])
    for n, leaf in zip(names, leaves):
        ref = leaf.grad
        got = G["d_" + n]
        assert torch.allclose(got, ref, atol=1e-9 * max(1.0, float(ref.abs().max())), rtol=1e-9), n


def test_backward_adjoint_identity_and_batch_additivity():
    sh = small_shape(B=3, S=24, d_model=32, n_q_heads=4, n_kv_heads=2, head_dim=8)
    t = inputs64(sh)
    cfg = cfg_of(sh)
    out, I = O.forward(cfg, t, t["x"])
    G = O.backward(cfg, t, I, t["d_out"])
    # <d_out, J dx> == <J^T d_out, dx> with J applied by a central difference
    torch.manual_seed(5)
    dx = torch.randn_like(t["x"])
    h = 1e-6
    Jdx = (O.forward(cfg, t, t["x"] + h * dx)[0] - O.forward(cfg, t, t["x"] - h * dx)[0]) / (2 * h)
    lhs = float((t["d_out"] * Jdx).sum())
    rhs = float((G["d_x"] * dx).sum())
    assert abs(lhs - rhs) <= 1e-6 * max(1.0, abs(lhs))
    # sequences are independent: per-sequence runs give the same d_x rows and weight grads that add up
    acc = None
    for b in range(sh.B):
        tb = dict(t)
        xb, db = t["x"][b:b + 1], t["d_out"][b:b + 1]
        _, Ib = O.forward(cfg, tb, xb)
        Gb = O.backward(cfg, tb, Ib, db)
        assert torch.allclose(Gb["d_x"][0], G["d_x"][b], atol=1e-12)
        acc = Gb["d_w_qk"] if acc is None else acc + Gb["d_w_qk"]
    assert torch.allclose(acc, G["d_w_qk"], atol=1e-10)


def test_forward_rows_equals_forward():
    sh = small_shape(S=16)
    t = inputs64(sh)
    cfg = cfg_of(sh)
    out, _ = O.forward(cfg, t, t["x"])
    rows = [0, 3, 15]
    out_r, _, _, _ = O.forward_rows(cfg, t, t["x"], rows)
    assert torch.allclose(out[:, rows], out_r, atol=1e-14)


# ------------------------------------------------------------------ decode with the latent KV cache

@pytest.mark.parametrize("k_seq,k_ch", [(2, 2), (1, 1), (3, 2), (2, 4)])
@pytest.mark.parametrize("flags", [O.ALL_FLAGS, 0, O.ALL_FLAGS & ~O.V_SHIFT, O.ALL_FLAGS & ~O.CONV1,
                                   O.ALL_FLAGS & ~O.CONV2, O.ALL_FLAGS & ~O.QK_MEAN])
def test_decode_token_by_token_equals_whole_sequence_forward(k_seq, k_ch, flags):
    """Feeding the tokens one at a time through the cache must reproduce every row of the causal
    whole-sequence forward, which is pinned above by other means."""
    sh = small_shape(S=9, k_seq=k_seq, k_ch=k_ch, flags=flags)
    cfg, t = cfg_of(sh), inputs64(sh)
    out, I = O.forward(cfg, t, t["x"])
    st = O.decode_init(cfg, sh.B)
    for tok in range(sh.S):
        o_t = O.decode_step(cfg, t, st, t["x"][:, tok])
        assert torch.allclose(o_t, out[:, tok], rtol=1e-10, atol=1e-12), tok
    assert torch.allclose(st["k"], I["k"], rtol=1e-10, atol=1e-12)
    assert torch.allclose(st["v"], I["v"], rtol=1e-10, atol=1e-12)
    assert st["k"].numel() + st["v"].numel() == O.describe(cfg, sh.B, sh.S)["kv_cache_elems"]


@pytest.mark.parametrize("S0", [0, 1, 2, 5])
def test_decode_continues_a_prefill(S0):
    sh = small_shape(S=8, k_seq=3, k_ch=2, n_kv_heads=1)
    cfg, t = cfg_of(sh), inputs64(sh)
    out, I = O.forward(cfg, t, t["x"])
    st = O.decode_state_after_prefill(cfg, I, S0)
    for tok in range(S0, sh.S):
        o_t = O.decode_step(cfg, t, st, t["x"][:, tok])
        assert torch.allclose(o_t, out[:, tok], rtol=1e-10, atol=1e-12), tok


def test_decode_first_token_closed_form_and_planted_mistakes():
    """Position 0: the single key gets probability one, the shifted value half is zero."""
    sh = small_shape(S=3)
    cfg, t = cfg_of(sh), inputs64(sh)
    st = O.decode_init(cfg, sh.B)
    o0 = O.decode_step(cfg, t, st, t["x"][:, 0])
    v = torch.cat([t["x"][:, 0] @ t["w_v1"].T, torch.zeros(sh.B, sh.L_k // 2, dtype=F64)], dim=-1)
    o = v.reshape(sh.B, sh.n_kv_heads, sh.head_dim).repeat_interleave(sh.n_q_heads // sh.n_kv_heads, dim=1)
    assert torch.allclose(o0, o.reshape(sh.B, sh.L_q) @ t["w_o"].T, rtol=1e-10, atol=1e-12)
    # a state that forgot the previous input (value shift) or the conv halo must change the next token
    out, _ = O.forward(cfg, t, t["x"])
    for key in ("x_prev", "qk0_hist"):
        st2 = O.decode_init(cfg, sh.B)
        O.decode_step(cfg, t, st2, t["x"][:, 0])
        st2[key] = torch.zeros_like(st2[key])
        assert not torch.allclose(O.decode_step(cfg, t, st2, t["x"][:, 1]), out[:, 1], rtol=1e-6, atol=1e-8), key
