"""Softmax edge cases of the latent attention (Eq. 11) on the GPU against the oracle, all with the q/k
normalisation on.  With random inputs the normalised logits are small and every row is nearly uniform, which
exercises one corner of the kernels only.  Here:

  * the key temperature puts the logit bound sqrt(d_h) * beta * log2(e) just under and just over the value at
    which the kernels switch from a fixed row maximum to the online form, and far to either side (temp = +1.5, -3);
  * keys exactly aligned and exactly anti-aligned with the queries (w_k = w_q, tokens +a / -a, no convs, no RoPE):
    the logits sit on +bound and -bound, so a row holds probabilities 2^(-2 bound) below its largest one, and a
    row whose keys are all anti-aligned has every probability that far below the fixed maximum;
  * repeated tokens with the whole method on (peaked rows whose logits follow the RoPE phase).

Forward, backward and the decode step.  Tolerance as everywhere: 1e-2 + 1e-2 |ref| on outputs, saved activations
and d_x; parameter gradients by tests/util.py::check_param_grads."""
import math

import pytest
import torch

from oracle import cca_oracle as O
from paper_2510_04476_b200 import synth
from tests.util import check_close, check_param_grads, oracle_cfg, to_device

pytestmark = pytest.mark.gpu
LOG2E = 1.4426950408889634
SWITCH = 56.0                       # the kernels use the fixed maximum while sqrt(d_h) beta log2(e) * 1.01 <= 56


def temp_at(dh, bound):
    """temp such that sqrt(d_h) * exp(temp) * log2(e) * 1.01 equals `bound`."""
    return math.log(bound / (math.sqrt(dh) * LOG2E * 1.01))


def _cca(sh):
    from paper_2510_04476_b200.binding import CCA
    return CCA.from_shape(sh)


def run(sh, t, backward=True, decode_tail=2):
    cfg = oracle_cfg(sh)
    out_ref, I = O.forward(cfg, t, t["x"])
    dev = to_device(t)
    cca = _cca(sh)
    ws = cca.alloc_workspace(sh.B, sh.S, True)
    out = cca.forward(dev, dev["x"], ws)
    torch.cuda.synchronize()
    assert cca.last_status() == 0
    sv = cca.saved(ws, sh.B, sh.S)
    # a key carries the factor beta = exp(temp), and so does its rounding noise: compared at unit temperature
    beta = torch.exp(t["temp"].double()).clamp(min=1.0)[None, None, :, None]
    check_close("k", sv["k"].reshape(I["k"].shape).double().cpu() / beta, I["k"] / beta)
    for n in ("q", "v", "o"):
        check_close(n, sv[n].reshape(I[n].shape), I[n])
    check_close("lse", sv["lse"], I["lse"])
    check_close("out", out, out_ref)
    if backward:
        G = O.backward(cfg, t, I, t["d_out"])
        d_x, grads = cca.backward(dev, dev["x"], dev["d_out"], ws)
        torch.cuda.synchronize()
        assert cca.last_status() == 0
        check_close("d_x", d_x, G["d_x"])
        check_param_grads(cfg, t, I, G, grads)
    if decode_tail and sh.causal and sh.S > decode_tail:
        S0 = sh.S - decode_tail
        x0 = dev["x"][:, :S0].contiguous()
        ws2 = cca.alloc_workspace(sh.B, S0, False)
        cca.forward(dev, x0, ws2)
        st = cca.new_decode_state(sh.B, sh.S)
        cca.decode_state_from_prefill(x0, ws2, st)
        st["pos"].fill_(S0)
        dws = cca.alloc_decode_workspace(sh.B, sh.S)
        for tok in range(S0, sh.S):
            o = cca.decode_step(dev, dev["x"][:, tok].contiguous(), st, sh.S, dws)
            st["pos"] += 1
            check_close(f"decode[{tok}]", o, out_ref[:, tok])
        torch.cuda.synchronize()
        assert cca.last_status() == 0
    cca.close()


def shape(dh, S=300, **kw):
    hq, hk = (8, 2) if dh == 64 else (4, 2)
    return synth.Shape(f"edge_dh{dh}", kw.pop("B", 1), S, 512 if dh == 64 else 1024, hq, hk, dh, seed=kw.pop("seed", 21), **kw)


@pytest.mark.parametrize("dh", [64, 128])
@pytest.mark.parametrize("bound", [SWITCH * 0.995, SWITCH * 1.005, SWITCH * 0.9, SWITCH * 1.3],
                         ids=["just_under_switch", "just_over_switch", "under", "well_over"])
def test_temperature_around_the_fixed_maximum_switch(dh, bound):
    sh = shape(dh)
    t = synth.make_inputs(sh)
    t["temp"] = torch.full_like(t["temp"], temp_at(dh, bound))
    t["temp"][-1] = temp_at(dh, SWITCH * 0.5)          # kv heads on both sides of the switch in one launch
    run(sh, t)


@pytest.mark.parametrize("dh", [64, 128])
@pytest.mark.parametrize("temp", [1.5, -3.0])
def test_extreme_temperatures(dh, temp):
    sh = shape(dh, S=420, B=2)
    t = synth.make_inputs(sh)
    t["temp"] = torch.full_like(t["temp"], temp)
    run(sh, t)


def aligned_inputs(dh, S, pattern, temp):
    """q head i and kv head i share their projection rows (h_q = h_k), no convs, no q-k-mean, no RoPE: q and k of a
    token are parallel.  Tokens are +a or -a by `pattern` (one entry per token), so every logit is exactly
    +sqrt(d_h) beta (same sign) or -sqrt(d_h) beta (opposite sign)."""
    sh = synth.Shape(f"aligned_dh{dh}", 1, S, 2 * dh * 2, 2, 2, dh, seed=33, flags=8 | 16)     # value-shift + norm only
    t = synth.make_inputs(sh)
    Lq = sh.L_q
    t["w_qk"][Lq:] = t["w_qk"][:Lq]
    a = t["x"][0, 0].clone()
    sign = torch.tensor(pattern, dtype=torch.float32)[:, None]
    t["x"] = (sign * a.float()[None, :]).to(torch.bfloat16)[None]
    t["temp"] = torch.full_like(t["temp"], temp)
    return sh, t


@pytest.mark.parametrize("dh", [64, 128])
@pytest.mark.parametrize("kind", ["all_aligned", "all_anti_aligned_past", "alternating", "one_aligned_key_far_back"])
@pytest.mark.parametrize("where", ["under_switch", "over_switch"])
def test_aligned_and_anti_aligned_keys(dh, kind, where):
    S = 300
    if kind == "all_aligned":
        pattern = [1.0] * S
    elif kind == "all_anti_aligned_past":
        pattern = [1.0] * (S - 40) + [-1.0] * 40        # the last 40 queries see 260 anti-aligned keys and a few aligned
    elif kind == "alternating":
        pattern = [1.0 if i % 2 == 0 else -1.0 for i in range(S)]
    else:
        pattern = [-1.0] * S
        pattern[3] = 1.0
        pattern[S - 1] = 1.0                            # the last query: one aligned key 296 tokens back, itself, rest anti
    temp = temp_at(dh, SWITCH * (0.98 if where == "under_switch" else 1.1))
    sh, t = aligned_inputs(dh, S, pattern, temp)
    run(sh, t)


@pytest.mark.parametrize("dh", [64, 128])
def test_repeated_tokens_with_every_stage_on(dh):
    """All tokens equal: after the convs' halo every pre-RoPE q and k is the same vector, the logits follow the RoPE
    phase of the distance only, and with temp = 1.2 the rows are sharply peaked on the nearest keys."""
    sh = shape(dh, S=500)
    t = synth.make_inputs(sh)
    t["x"] = t["x"][:, :1].expand(-1, sh.S, -1).contiguous()
    t["temp"] = torch.full_like(t["temp"], 1.2)
    run(sh, t)


def test_non_causal_rows_with_anti_aligned_keys():
    sh, t = aligned_inputs(64, 260, [1.0 if i % 3 else -1.0 for i in range(260)], temp_at(64, SWITCH * 0.98))
    sh = sh.replace(causal=0)
    run(sh, t, decode_tail=0)
