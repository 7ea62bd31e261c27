"""fp64 CPU oracle for the Compressed Convolutional Attention (CCA / CCGQA) block.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the CUDA
library is checked against.  Only the tests, the smoke check and the benchmark's
cpu-baseline leg may import it; the product path never does, and this file imports
nothing from the product.  All arithmetic is torch CPU float64; inputs are the
bf16-rounded tensors widened exactly, and no intermediate is ever rounded.  There is
no tiling, no online softmax and no fusion: each function is one step of the paper,
in the paper's order, and cites the passage it follows.

Readings taken where the paper is silent (all are runtime parameters):
  * conv kernel sizes default to k_seq = k_ch = 2; no bias in any linear or conv;
  * convs are cross-correlations whose last tap multiplies the current token, with
    zero history before the first token of each sequence;
  * conv2 has h_q + h_k groups of d_h -> d_h channels, q heads first;
  * the value latent is the flat concatenation [W_v1 x_t , W_v2 x_{t-1}] viewed as
    h_k heads (Listing A.1), x_{-1} = 0;
  * softmax scale is 1/sqrt(d_h); beta = exp(temp), one temp per kv head;
  * RoPE rotates the whole head, pairs (c, c + d_h/2), theta_c = base^(-2c/d_h),
    position = token index from 0; order is norm -> sqrt(d_h) -> beta -> RoPE;
  * no epsilon in the L2 norm;
  * q head i reads kv head floor(i / g), g = h_q / h_k;
  * causal = 0 drops only the attention mask; convs and value-shift stay causal.

Pins: see tests/test_oracle_pins.py (brute-force attention, causality and halo,
MHA reduction, CCGQA -> CCA, closed forms, finite differences, autograd, formulas;
the token-by-token decode against the whole-sequence forward and brute force).
The RoPE convention, the conv sizes and the RoPE base are "parity unpinned" against
the authors' kernel (no source or numbers exist); everything else is pinned.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, Optional, Sequence

import torch

F64 = torch.float64

CONV1, CONV2, QK_MEAN, V_SHIFT, QK_NORM, ROPE = 1, 2, 4, 8, 16, 32
ALL_FLAGS = 63


@dataclasses.dataclass(frozen=True)
class OracleConfig:
    """The paper's parameters (notation table): E, h_q, h_k, d_h, kernel sizes."""
    d_model: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    k_seq: int = 2
    k_ch: int = 2
    causal: int = 1
    flags: int = ALL_FLAGS
    rope_base: float = 10000.0

    @property
    def L_q(self):
        return self.n_q_heads * self.head_dim

    @property
    def L_k(self):
        return self.n_kv_heads * self.head_dim

    @property
    def L(self):
        return self.L_q + self.L_k

    @property
    def g(self):
        return self.n_q_heads // self.n_kv_heads


def _f64(t):
    return t.detach().to("cpu").to(F64)


# --------------------------------------------------------------------------------------
# Forward steps
# --------------------------------------------------------------------------------------

def down_projection(x, w_qk):
    """Eq. 7 / packed linear of Listing A.1: latent q (first L_q channels) and k."""
    return x @ w_qk.transpose(0, 1)


def conv1_seq(u, w0):
    """Eq. 8, conv1_seq: depth-wise causal 1-D conv along the sequence.
    u [B,S,L], w0 [L,k]; y[t,c] = sum_j w0[c,j] * u[t-(k-1)+j, c], u[<0] = 0."""
    B, S, L = u.shape
    k = w0.shape[1]
    y = torch.zeros_like(u)
    for j in range(k):
        lag = k - 1 - j
        if lag < S:
            y[:, lag:, :] += u[:, : S - lag, :] * w0[:, j]
    return y


def conv2_seq_ch(u, w1, n_heads, d_h):
    """Eq. 8, conv2_seq+ch: causal conv along the sequence that mixes the d_h channels
    inside each head (one group per q head, then per k head).
    u [B,S,H*d_h], w1 [H*d_h, d_h, k]: (out channel, in channel within head, tap)."""
    B, S, L = u.shape
    k = w1.shape[2]
    uh = u.reshape(B, S, n_heads, d_h)
    wh = w1.reshape(n_heads, d_h, d_h, k)
    y = torch.zeros_like(uh)
    for j in range(k):
        lag = k - 1 - j
        if lag < S:
            y[:, lag:] += torch.einsum("bshi,hoi->bsho", uh[:, : S - lag], wh[..., j])
    return y.reshape(B, S, L)


def qk_mean(q0, k0, yq, yk, g):
    """Eq. 9: mu = (q_pre + B_group(k_pre)) / 2; q += mu; k += E_group(mu).
    All tensors [B,S,h,d_h]; B_group repeats each k head over its g query heads,
    E_group averages over them."""
    B, S, hq, dh = q0.shape
    hk = hq // g
    k_b = k0.unsqueeze(3).expand(B, S, hk, g, dh).reshape(B, S, hq, dh)
    mu = 0.5 * (q0 + k_b)
    mu_k = mu.reshape(B, S, hk, g, dh).mean(dim=3)
    return yq + mu, yk + mu_k


def value_shift(x, w_v1, w_v2, shift):
    """Eq. 10: v = [W_v1 x_t , W_v2 x_{t-1}] on the flat channel axis, x_{-1} = 0."""
    v1 = x @ w_v1.transpose(0, 1)
    if shift:
        xs = torch.zeros_like(x)
        xs[:, 1:] = x[:, :-1]
    else:
        xs = x
    v2 = xs @ w_v2.transpose(0, 1)
    return torch.cat([v1, v2], dim=-1), xs


def l2norm_scale(u, scale):
    """Eq. 11, norm(.)*sqrt(d_h) (times beta for keys): u [B,S,h,d_h], scale [h] or scalar."""
    n = u.norm(p=2, dim=-1, keepdim=True)
    if torch.is_tensor(scale):
        scale = scale.reshape(1, 1, -1, 1)
    return u * scale / n


def rope_angles(S, d_h, base, pos0=0):
    half = d_h // 2
    c = torch.arange(half, dtype=F64)
    theta = torch.pow(torch.tensor(float(base), dtype=F64), -2.0 * c / d_h)
    pos = torch.arange(pos0, pos0 + S, dtype=F64)
    return pos[:, None] * theta[None, :]          # [S, d_h/2]


def rope(u, ang):
    """Eq. 11, RoPE: rotate the pair (c, c + d_h/2) of token t by ang[t,c]."""
    half = u.shape[-1] // 2
    cos = torch.cos(ang)[None, :, None, :]
    sin = torch.sin(ang)[None, :, None, :]
    a, b = u[..., :half], u[..., half:]
    return torch.cat([a * cos - b * sin, b * cos + a * sin], dim=-1)


def attention(q, k, v, g, causal, rows: Optional[Sequence[int]] = None, want_p=False):
    """Eq. 11: o_h = softmax(q_h k_h^T / sqrt(d_h)) v_h with grouped kv heads.
    q [B,S,h_q,d_h], k, v [B,S,h_k,d_h].  Whole score rows are materialised.
    rows: if given, only those query positions are computed (every row is independent).
    Returns o [B,R,h_q,d_h], lse [B,h_q,R] (log-sum-exp of the scaled scores), p or None."""
    B, S, hq, dh = q.shape
    ridx = torch.arange(S) if rows is None else torch.as_tensor(list(rows), dtype=torch.long)
    R = ridx.numel()
    o = torch.zeros(B, R, hq, dh, dtype=F64)
    lse = torch.zeros(B, hq, R, dtype=F64)
    ps = torch.zeros(B, hq, R, S, dtype=F64) if want_p else None
    inv = 1.0 / math.sqrt(dh)
    blk = max(1, (1 << 24) // max(S, 1))            # rows per chunk: memory only, not math
    for b in range(B):
        for i in range(hq):
            j = i // g
            kj, vj = k[b, :, j, :], v[b, :, j, :]
            for r0 in range(0, R, blk):
                rr = ridx[r0:r0 + blk]
                s = (q[b, rr, i, :] @ kj.transpose(0, 1)) * inv
                if causal:
                    s = s.masked_fill(torch.arange(S)[None, :] > rr[:, None], float("-inf"))
                m = s.max(dim=-1, keepdim=True).values
                e = torch.exp(s - m)
                z = e.sum(dim=-1, keepdim=True)
                p = e / z
                o[b, r0:r0 + blk, i, :] = p @ vj
                lse[b, i, r0:r0 + blk] = (m + torch.log(z)).squeeze(-1)
                if want_p:
                    ps[b, i, r0:r0 + blk] = p
    return o, lse, ps


def up_projection(o_flat, w_o):
    """Eq. 11: out = W_o [o_1 .. o_nh]."""
    return o_flat @ w_o.transpose(0, 1)


def pre_attention(cfg: OracleConfig, w: Dict[str, torch.Tensor], x, pos0: int = 0):
    """Steps 1-5 (Eq. 7-11 up to RoPE).  Returns a dict of every intermediate."""
    x = _f64(x)
    B, S, E = x.shape
    hq, hk, dh, g = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.g
    Lq, Lk = cfg.L_q, cfg.L_k
    w_qk, w_v1, w_v2 = _f64(w["w_qk"]), _f64(w["w_v1"]), _f64(w["w_v2"])
    I = {"x": x}
    qk0 = down_projection(x, w_qk)
    I["qk0"] = qk0
    y1 = conv1_seq(qk0, _f64(w["conv0_w"])) if cfg.flags & CONV1 else qk0
    I["y1"] = y1
    y2 = conv2_seq_ch(y1, _f64(w["conv1_w"]), hq + hk, dh) if cfg.flags & CONV2 else y1
    I["y2"] = y2
    q0 = qk0[..., :Lq].reshape(B, S, hq, dh)
    k0 = qk0[..., Lq:].reshape(B, S, hk, dh)
    yq = y2[..., :Lq].reshape(B, S, hq, dh)
    yk = y2[..., Lq:].reshape(B, S, hk, dh)
    if cfg.flags & QK_MEAN:
        qh, kh = qk_mean(q0, k0, yq, yk, g)
    else:
        qh, kh = yq, yk
    I["q_hat"], I["k_hat"] = qh, kh
    v_flat, xs = value_shift(x, w_v1, w_v2, bool(cfg.flags & V_SHIFT))
    I["xs"] = xs
    I["v"] = v_flat.reshape(B, S, hk, dh)
    if cfg.flags & QK_NORM:
        beta = torch.exp(_f64(w["temp"]))
        qn = l2norm_scale(qh, math.sqrt(dh))
        kn = l2norm_scale(kh, math.sqrt(dh) * beta)
    else:
        qn, kn = qh, kh
    I["q_n"], I["k_n"] = qn, kn
    if cfg.flags & ROPE:
        ang = rope_angles(S, dh, cfg.rope_base, pos0)
        I["ang"] = ang
        q, k = rope(qn, ang), rope(kn, ang)
    else:
        q, k = qn, kn
    I["q"], I["k"] = q, k
    return I


def forward(cfg: OracleConfig, w: Dict[str, torch.Tensor], x, want_p=False):
    """The whole block, Eq. 7-11.  Returns (out [B,S,E], intermediates)."""
    I = pre_attention(cfg, w, x)
    B, S, _ = I["x"].shape
    o, lse, p = attention(I["q"], I["k"], I["v"], cfg.g, bool(cfg.causal), want_p=want_p)
    I["o"], I["lse"], I["p"] = o, lse, p
    out = up_projection(o.reshape(B, S, cfg.L_q), _f64(w["w_o"]))
    I["out"] = out
    return out, I


def forward_rows(cfg: OracleConfig, w, x, rows: Sequence[int]):
    """Block output at the given token positions only (projections and latent
    transforms are still computed in full).  Used where the S^2 term is too large to
    compute for every row; every output row equals the corresponding row of forward()."""
    I = pre_attention(cfg, w, x)
    B = I["x"].shape[0]
    o, lse, _ = attention(I["q"], I["k"], I["v"], cfg.g, bool(cfg.causal), rows=rows)
    out = up_projection(o.reshape(B, len(rows), cfg.L_q), _f64(w["w_o"]))
    return out, o, lse, I


# --------------------------------------------------------------------------------------
# Backward (the paper prints none; each step is the adjoint of the forward step above)
# --------------------------------------------------------------------------------------

def conv1_seq_adjoint(dy, u, w0):
    """Adjoint of conv1_seq: du[t,c] = sum_j w0[c,j] dy[t+(k-1)-j, c];
    dw0[c,j] = sum_{b,t} dy[t,c] u[t-(k-1)+j, c]."""
    B, S, L = dy.shape
    k = w0.shape[1]
    du = torch.zeros_like(dy)
    dw = torch.zeros_like(w0)
    for j in range(k):
        lag = k - 1 - j
        if lag < S:
            du[:, : S - lag, :] += dy[:, lag:, :] * w0[:, j]
            dw[:, j] = (dy[:, lag:, :] * u[:, : S - lag, :]).sum(dim=(0, 1))
    return du, dw


def conv2_seq_ch_adjoint(dy, u, w1, n_heads, d_h):
    """Adjoint of conv2_seq_ch."""
    B, S, L = dy.shape
    k = w1.shape[2]
    dyh = dy.reshape(B, S, n_heads, d_h)
    uh = u.reshape(B, S, n_heads, d_h)
    wh = w1.reshape(n_heads, d_h, d_h, k)
    du = torch.zeros_like(uh)
    dw = torch.zeros_like(wh)
    for j in range(k):
        lag = k - 1 - j
        if lag < S:
            du[:, : S - lag] += torch.einsum("bsho,hoi->bshi", dyh[:, lag:], wh[..., j])
            dw[..., j] = torch.einsum("bsho,bshi->hoi", dyh[:, lag:], uh[:, : S - lag])
    return du.reshape(B, S, L), dw.reshape(L, d_h, k)


def l2norm_scale_adjoint(dy, u, scale):
    """y = scale * u / |u|  =>  du = (scale/|u|) (dy - n (n . dy)), n = u/|u|."""
    nrm = u.norm(p=2, dim=-1, keepdim=True)
    n = u / nrm
    if torch.is_tensor(scale):
        scale = scale.reshape(1, 1, -1, 1)
    return (scale / nrm) * (dy - n * (n * dy).sum(dim=-1, keepdim=True))


def rope_adjoint(dy, ang):
    """A rotation's adjoint is the rotation by the negated angle."""
    return rope(dy, -ang)


def attention_adjoint(q, k, v, o, do, g, causal):
    """Adjoint of attention(): dv += p^T do; dp = do v^T; ds = p*(dp - rowsum(do*o));
    dq = ds k / sqrt(d_h); dk += ds^T q / sqrt(d_h), summed over the g heads of a group."""
    B, S, hq, dh = q.shape
    inv = 1.0 / math.sqrt(dh)
    dq = torch.zeros_like(q)
    dk = torch.zeros_like(k)
    dv = torch.zeros_like(v)
    blk = max(1, (1 << 24) // max(S, 1))
    for b in range(B):
        for i in range(hq):
            j = i // g
            kj, vj = k[b, :, j, :], v[b, :, j, :]
            for r0 in range(0, S, blk):
                r1 = min(S, r0 + blk)
                qi = q[b, r0:r1, i, :]
                s = (qi @ kj.transpose(0, 1)) * inv
                if causal:
                    s = s.masked_fill(torch.arange(S)[None, :] > torch.arange(r0, r1)[:, None], float("-inf"))
                p = torch.softmax(s, dim=-1)
                doi = do[b, r0:r1, i, :]
                dp = doi @ vj.transpose(0, 1)
                D = (doi * o[b, r0:r1, i, :]).sum(dim=-1, keepdim=True)
                ds = p * (dp - D)
                dq[b, r0:r1, i, :] = (ds @ kj) * inv
                dk[b, :, j, :] += (ds.transpose(0, 1) @ qi) * inv
                dv[b, :, j, :] += p.transpose(0, 1) @ doi
    return dq, dk, dv


def backward(cfg: OracleConfig, w: Dict[str, torch.Tensor], I: Dict[str, torch.Tensor], d_out):
    """Gradients of <d_out, out> w.r.t. x and every parameter.
    I is the intermediates dict of forward().  Returns a dict of fp64 tensors:
    d_x, d_w_qk, d_w_v1, d_w_v2, d_w_o, d_conv0_w, d_conv1_w, d_temp (+ latent grads)."""
    d_out = _f64(d_out)
    x = I["x"]
    B, S, E = x.shape
    hq, hk, dh, g = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.g
    Lq, Lk, L = cfg.L_q, cfg.L_k, cfg.L
    w_qk, w_v1, w_v2, w_o = (_f64(w[n]) for n in ("w_qk", "w_v1", "w_v2", "w_o"))
    G = {}
    # up-projection
    o_flat = I["o"].reshape(B, S, Lq)
    G["d_w_o"] = torch.einsum("bse,bsc->ec", d_out, o_flat)
    do = (d_out @ w_o).reshape(B, S, hq, dh)
    G["d_o"] = do
    # attention
    dq, dk, dv = attention_adjoint(I["q"], I["k"], I["v"], I["o"], do, g, bool(cfg.causal))
    G["d_q"], G["d_k"], G["d_v"] = dq, dk, dv
    # RoPE
    if cfg.flags & ROPE:
        dqn, dkn = rope_adjoint(dq, I["ang"]), rope_adjoint(dk, I["ang"])
    else:
        dqn, dkn = dq, dk
    # norm, sqrt(d_h), temperature
    if cfg.flags & QK_NORM:
        beta = torch.exp(_f64(w["temp"]))
        G["d_temp"] = (dkn * I["k_n"]).sum(dim=(0, 1, 3))
        dqh = l2norm_scale_adjoint(dqn, I["q_hat"], math.sqrt(dh))
        dkh = l2norm_scale_adjoint(dkn, I["k_hat"], math.sqrt(dh) * beta)
    else:
        G["d_temp"] = torch.zeros(hk, dtype=F64)
        dqh, dkh = dqn, dkn
    # q-k-mean
    dq0 = torch.zeros(B, S, hq, dh, dtype=F64)
    dk0 = torch.zeros(B, S, hk, dh, dtype=F64)
    if cfg.flags & QK_MEAN:
        dmu = dqh + dkh.unsqueeze(3).expand(B, S, hk, g, dh).reshape(B, S, hq, dh) / g
        dq0 += 0.5 * dmu
        dk0 += 0.5 * dmu.reshape(B, S, hk, g, dh).sum(dim=3)
    G["d_q_hat"], G["d_k_hat"] = dqh, dkh
    dy2 = torch.cat([dqh.reshape(B, S, Lq), dkh.reshape(B, S, Lk)], dim=-1)
    # convs
    if cfg.flags & CONV2:
        dy1, G["d_conv1_w"] = conv2_seq_ch_adjoint(dy2, I["y1"], _f64(w["conv1_w"]), hq + hk, dh)
    else:
        dy1, G["d_conv1_w"] = dy2, torch.zeros(L, dh, cfg.k_ch, dtype=F64)
    G["d_y2"], G["d_y1"] = dy2, dy1
    if cfg.flags & CONV1:
        dqk0, G["d_conv0_w"] = conv1_seq_adjoint(dy1, I["qk0"], _f64(w["conv0_w"]))
    else:
        dqk0, G["d_conv0_w"] = dy1, torch.zeros(L, cfg.k_seq, dtype=F64)
    dqk0 = dqk0 + torch.cat([dq0.reshape(B, S, Lq), dk0.reshape(B, S, Lk)], dim=-1)
    G["d_qk0"] = dqk0
    # projections and value-shift
    dvf = dv.reshape(B, S, Lk)
    dv1, dv2 = dvf[..., : Lk // 2], dvf[..., Lk // 2:]
    G["d_w_qk"] = torch.einsum("bsl,bse->le", dqk0, x)
    G["d_w_v1"] = torch.einsum("bsl,bse->le", dv1, x)
    G["d_w_v2"] = torch.einsum("bsl,bse->le", dv2, I["xs"])
    dx = dqk0 @ w_qk + dv1 @ w_v1
    dxs = dv2 @ w_v2
    if cfg.flags & V_SHIFT:
        dx[:, :-1] += dxs[:, 1:]
    else:
        dx += dxs
    G["d_x"] = dx
    return G


# --------------------------------------------------------------------------------------
# Decode: one new token per sequence against the latent KV cache (comparison table of the
# paper, KV-cache and decode columns).  The state is what the block's definition needs of
# the past: the cached latent keys and values (2 L_k numbers per token), the
# pre-convolution q0|k0 of the last k_seq + k_ch - 2 tokens (the convs' halo) and the
# previous token's input (the value shift).
# --------------------------------------------------------------------------------------

def decode_init(cfg: OracleConfig, B: int) -> Dict[str, object]:
    """Empty state: no cached token, zero history (the convs and the value shift see zeros
    before the first token)."""
    pad = cfg.k_seq + cfg.k_ch - 2
    return {
        "k": torch.zeros(B, 0, cfg.n_kv_heads, cfg.head_dim, dtype=F64),
        "v": torch.zeros(B, 0, cfg.n_kv_heads, cfg.head_dim, dtype=F64),
        "qk0_hist": torch.zeros(B, pad, cfg.L, dtype=F64),      # oldest first
        "x_prev": torch.zeros(B, cfg.d_model, dtype=F64),
        "pos": 0,
    }


def decode_step(cfg: OracleConfig, w: Dict[str, torch.Tensor], state: Dict[str, object], x_t):
    """Eq. 7-11 for the single token x_t [B,E] at position state["pos"], every sequence at the
    same position.  Returns out [B,E]; the state is advanced in place.  The attention is causal by
    construction: the new query sees the cached tokens and itself."""
    x_t = _f64(x_t)
    B, E = x_t.shape
    hq, hk, dh, g = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.g
    Lq, Lk, L = cfg.L_q, cfg.L_k, cfg.L
    ks = cfg.k_seq if cfg.flags & CONV1 else 1
    kc = cfg.k_ch if cfg.flags & CONV2 else 1
    pad = cfg.k_seq + cfg.k_ch - 2
    pos = int(state["pos"])
    qk0_t = x_t @ _f64(w["w_qk"]).transpose(0, 1)                                   # Eq. 7
    win = torch.cat([state["qk0_hist"], qk0_t[:, None, :]], dim=1)                  # tokens pos-pad .. pos
    # Eq. 8, conv1 at the kc tokens conv2 looks at, then conv2 at the new token
    y1 = []
    for r in range(kc):                                   # token pos - (kc-1) + r  = window row pad - (kc-1) + r
        row = pad - (kc - 1) + r
        if cfg.flags & CONV1:
            w0 = _f64(w["conv0_w"])
            acc = torch.zeros(B, L, dtype=F64)
            for j in range(ks):
                acc = acc + win[:, row - (ks - 1) + j, :] * w0[:, j]
            y1.append(acc)
        else:
            y1.append(win[:, row, :])
    if cfg.flags & CONV2:
        w1 = _f64(w["conv1_w"]).reshape(hq + hk, dh, dh, kc)
        y2 = torch.zeros(B, hq + hk, dh, dtype=F64)
        for r in range(kc):
            y2 = y2 + torch.einsum("bhi,hoi->bho", y1[r].reshape(B, hq + hk, dh), w1[..., r])
        y2 = y2.reshape(B, L)
    else:
        y2 = y1[-1]
    q0 = qk0_t[:, :Lq].reshape(B, hq, dh)
    k0 = qk0_t[:, Lq:].reshape(B, hk, dh)
    qh = y2[:, :Lq].reshape(B, hq, dh)
    kh = y2[:, Lq:].reshape(B, hk, dh)
    if cfg.flags & QK_MEAN:                                                          # Eq. 9
        mu = 0.5 * (q0 + k0.repeat_interleave(g, dim=1))
        qh = qh + mu
        kh = kh + mu.reshape(B, hk, g, dh).mean(dim=2)
    xs = state["x_prev"] if cfg.flags & V_SHIFT else x_t                             # Eq. 10
    v_t = torch.cat([x_t @ _f64(w["w_v1"]).transpose(0, 1), xs @ _f64(w["w_v2"]).transpose(0, 1)], dim=-1)
    v_t = v_t.reshape(B, hk, dh)
    if cfg.flags & QK_NORM:                                                          # Eq. 11
        beta = torch.exp(_f64(w["temp"]))
        qh = qh * math.sqrt(dh) / qh.norm(dim=-1, keepdim=True)
        kh = kh * (math.sqrt(dh) * beta)[None, :, None] / kh.norm(dim=-1, keepdim=True)
    if cfg.flags & ROPE:
        half = dh // 2
        c = torch.arange(half, dtype=F64)
        ang = pos * torch.pow(torch.tensor(float(cfg.rope_base), dtype=F64), -2.0 * c / dh)
        cs, sn = torch.cos(ang), torch.sin(ang)

        def rot(u):
            a, b = u[..., :half], u[..., half:]
            return torch.cat([a * cs - b * sn, b * cs + a * sn], dim=-1)
        qh, kh = rot(qh), rot(kh)
    state["k"] = torch.cat([state["k"], kh[:, None]], dim=1)
    state["v"] = torch.cat([state["v"], v_t[:, None]], dim=1)
    o = torch.zeros(B, hq, dh, dtype=F64)
    for i in range(hq):
        j = i // g
        s = torch.einsum("bd,bsd->bs", qh[:, i], state["k"][:, :, j]) / math.sqrt(dh)
        p = torch.softmax(s, dim=-1)
        o[:, i] = torch.einsum("bs,bsd->bd", p, state["v"][:, :, j])
    out = o.reshape(B, Lq) @ _f64(w["w_o"]).transpose(0, 1)
    if pad > 0:
        state["qk0_hist"] = win[:, 1:, :].clone()
    state["x_prev"] = x_t.clone()
    state["pos"] = pos + 1
    state["q_last"], state["o_last"] = qh, o
    return out


def decode_state_after_prefill(cfg: OracleConfig, I: Dict[str, torch.Tensor], S0: int) -> Dict[str, object]:
    """The decode state after the first S0 tokens of a prefill whose intermediates are I
    (from pre_attention / forward): cached k, v, the q0|k0 halo and the last input."""
    pad = cfg.k_seq + cfg.k_ch - 2
    B = I["x"].shape[0]
    hist = torch.zeros(B, pad, cfg.L, dtype=F64)
    n = min(pad, S0)
    if n > 0:
        hist[:, pad - n:, :] = I["qk0"][:, S0 - n:S0, :]
    return {
        "k": I["k"][:, :S0].clone(), "v": I["v"][:, :S0].clone(), "qk0_hist": hist,
        "x_prev": I["x"][:, S0 - 1, :].clone() if S0 > 0 else torch.zeros(B, cfg.d_model, dtype=F64),
        "pos": S0,
    }


# --------------------------------------------------------------------------------------
# Closed-form counts (comparison table of the paper, CCGQA row, and its Conv footnote)
# --------------------------------------------------------------------------------------

def describe(cfg: OracleConfig, B: int, S: int) -> Dict[str, int]:
    """Integer metadata: latent widths, group size, padding, and the paper's parameter,
    KV-cache and FLOP counts.  The conv term follows the structure of the two convs
    (depth-wise over all L channels, grouped d_h x d_h per head), which is what the
    footnote's CCGQA substitution gives for the grouped term."""
    E, dh = cfg.d_model, cfg.head_dim
    Lq, Lk, L = cfg.L_q, cfg.L_k, cfg.L
    conv_params = L * cfg.k_seq + L * dh * cfg.k_ch
    T = B * S
    proj = 2 * T * E * (Lq + 2 * Lk) + 2 * T * Lq * E
    return {
        "L_q": Lq, "L_k": Lk, "g": cfg.g,
        "total_padding": cfg.k_seq + cfg.k_ch - 2,
        "v_shift_split": Lk // 2,
        "conv_params": conv_params,
        "params": E * Lq + 2 * E * Lk + Lq * E + conv_params,
        "kv_cache_elems": 2 * B * S * Lk,
        "fwd_flops": proj + 4 * B * S * S * Lq + 2 * T * conv_params,
        "fwd_flops_causal": proj + 2 * B * S * S * Lq + 2 * T * conv_params,
        "decode_flops": 2 * B * E * (Lq + 2 * Lk) + 2 * B * Lq * E + 4 * B * S * Lq + 2 * B * conv_params,
    }
