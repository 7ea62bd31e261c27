"""Pins of the MLA oracle (paper Section 2.1, Eq. 3-6) against things it does not define itself: scalar brute-force
attention, the paper's own absorbed form (Eq. 5), the CCA oracle's plain-MHA reduction (Eq. 1-2) with the low-rank
products as full weights, closed forms, causality, and the comparison table's MLA row evaluated by hand."""
import math

import pytest
import torch

from oracle import cca_oracle as O
from oracle import mla_oracle as M

F64 = torch.float64


def make(cfg, B, S, seed=0, std=0.2):
    g = torch.Generator().manual_seed(seed)
    r = lambda *s: torch.randn(*s, generator=g, dtype=F64) * std
    E, nh = cfg.d_model, cfg.n_heads
    w = {"w_dq": r(cfg.d_cq, E), "w_dkv": r(cfg.d_ckv, E), "w_uq": r(nh * cfg.d_nope, cfg.d_cq),
         "w_uqr": r(nh * cfg.d_rope, cfg.d_cq), "w_uk": r(nh * cfg.d_nope, cfg.d_ckv), "w_uv": r(nh * cfg.d_v, cfg.d_ckv),
         "w_kr": r(cfg.d_rope, E), "w_o": r(E, nh * cfg.d_v)}
    x = torch.randn(B, S, E, generator=g, dtype=F64)
    return w, x


def test_attention_matches_scalar_brute_force():
    g = torch.Generator().manual_seed(1)
    B, S, nh, dqk, dv = 1, 7, 2, 6, 4
    q, k, v = (torch.randn(B, S, nh, d, generator=g, dtype=F64) for d in (dqk, dqk, dv))
    o, lse = M.attention_mha(q, k, v, True)
    for i in range(nh):
        for t in range(S):
            s = [sum(float(q[0, t, i, c]) * float(k[0, u, i, c]) for c in range(dqk)) / math.sqrt(dqk) for u in range(t + 1)]
            m = max(s)
            e = [math.exp(a - m) for a in s]
            z = sum(e)
            for c in range(dv):
                ref = sum(e[u] / z * float(v[0, u, i, c]) for u in range(t + 1))
                assert abs(float(o[0, t, i, c]) - ref) < 1e-12
            assert abs(float(lse[0, i, t]) - (m + math.log(z))) < 1e-12


@pytest.mark.parametrize("causal", [1, 0])
def test_absorbed_form_of_eq5_equals_the_up_projected_form(causal):
    cfg = M.MlaConfig(d_model=48, n_heads=3, d_nope=8, d_rope=0, d_v=10, d_ckv=12, d_cq=20, causal=causal)
    w, x = make(cfg, 2, 9, seed=2)
    out, _ = M.forward(cfg, w, x)
    ref = M.forward_absorbed_nope(cfg, w, x)
    assert torch.allclose(out, ref, rtol=1e-10, atol=1e-12)


def test_without_rope_it_is_mha_with_low_rank_weights():
    """d_rope = 0: Eq. 3-4 followed by attention is Eq. 1-2 with W_Q = W_UQ W_DQ, W_K = W_UK W_DKV, W_V = W_UV W_DKV,
    which the CCA oracle computes with every latent transform off and no compression."""
    nh, d = 4, 8
    E = nh * d
    cfg = M.MlaConfig(d_model=E, n_heads=nh, d_nope=d, d_rope=0, d_v=d, d_ckv=12, d_cq=20)
    w, x = make(cfg, 2, 11, seed=3)
    out, I = M.forward(cfg, w, x)
    wq, wk, wv = w["w_uq"] @ w["w_dq"], w["w_uk"] @ w["w_dkv"], w["w_uv"] @ w["w_dkv"]
    ccfg = O.OracleConfig(E, nh, nh, d, 1, 1, 1, 0)
    cw = {"w_qk": torch.cat([wq, wk]), "w_v1": wv[: E // 2], "w_v2": wv[E // 2:], "w_o": w["w_o"],
          "conv0_w": torch.zeros(2 * E, 1, dtype=F64), "conv1_w": torch.zeros(2 * E, d, 1, dtype=F64),
          "temp": torch.zeros(nh)}
    ref, J = O.forward(ccfg, cw, x)
    assert torch.allclose(out, ref, rtol=1e-10, atol=1e-12)
    assert torch.allclose(I["lse"], J["lse"], rtol=1e-10, atol=1e-12)


def test_rope_part_is_shared_across_heads_and_identity_at_position_zero():
    cfg = M.MlaConfig(d_model=32, n_heads=4, d_nope=4, d_rope=4, d_v=8, d_ckv=8, d_cq=16)
    w, x = make(cfg, 1, 6, seed=4)
    _, I = M.forward(cfg, w, x)
    k = I["k"]
    for i in range(1, cfg.n_heads):
        assert torch.equal(k[:, :, i, cfg.d_nope:], k[:, :, 0, cfg.d_nope:])
    assert torch.allclose(k[0, 0, 0, cfg.d_nope:], x[0, 0] @ w["w_kr"].T, rtol=1e-12, atol=1e-14)   # angle 0 at t = 0
    q_pre = (I["c_q"] @ w["w_uqr"].T).reshape(1, 6, cfg.n_heads, cfg.d_rope)
    assert torch.allclose(I["q"][0, 0, :, cfg.d_nope:], q_pre[0, 0], rtol=1e-12, atol=1e-14)
    # a rotation: norms of the rope parts are those of the un-rotated projections
    assert torch.allclose(I["q"][..., cfg.d_nope:].norm(dim=-1), q_pre.norm(dim=-1), rtol=1e-12)


def test_single_token_closed_form_and_causality():
    cfg = M.MlaConfig(d_model=32, n_heads=4, d_nope=4, d_rope=4, d_v=8, d_ckv=8, d_cq=16)
    w, x = make(cfg, 2, 8, seed=5)
    out, _ = M.forward(cfg, w, x)
    one, _ = M.forward(cfg, w, x[:, :1])
    ref = (x[:, :1] @ w["w_dkv"].T @ w["w_uv"].T) @ w["w_o"].T        # the only key gets weight 1
    assert torch.allclose(one, ref, rtol=1e-10, atol=1e-12)
    x2 = x.clone()
    x2[:, 5:] += 1.0
    out2, _ = M.forward(cfg, w, x2)
    assert torch.equal(out[:, :5], out2[:, :5])                       # the future does not reach back


def test_counts_match_the_comparison_table_mla_row():
    """E = 2048, c_q = 2, c_kv = 4, 16 heads of 128 (n_h d_nope = n_h d_v = E as the table assumes), E_r = 64, B = 2,
    S = 4096, by hand:  params E^2 + 3 E^2/c_kv + 2 E^2/c_q = 4194304 (1 + 3/4 + 1) = 11534336;
    cache B S E / c_kv + B S E_r = 8192 (512 + 64) = 4718592;
    FLOPs 2 B S E^2 + 4 B S E^2 / c_q + 6 B S E^2 / c_kv + 4 B E S^2
          = 8192 * 4194304 * (2 + 2 + 1.5) + 4 * 2 * 2048 * 4096^2 = 188978561024 + 274877906944 = 463856467968."""
    cfg = M.MlaConfig(d_model=2048, n_heads=16, d_nope=128, d_rope=64, d_v=128, d_ckv=512, d_cq=1024)
    d = M.describe(cfg, 2, 4096)
    assert d["params"] == 11534336
    assert d["kv_cache_elems"] == 4718592
    assert d["fwd_flops"] == 463856467968
    assert d["rope_params"] == 64 * 2048 + 16 * 64 * 1024
