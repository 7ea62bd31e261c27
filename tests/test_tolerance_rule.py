"""The parameter-gradient rule of tests/util.py, exercised on the CPU: gradients that carry only the rounding
noise of a bf16-storage pipeline pass; planted mistakes (in copies of the oracle's results) fail."""
import pytest
import torch

from oracle import cca_oracle as O
from paper_2510_04476_b200 import synth
from tests import noise_model as NM
from tests.util import PARAM_NAMES, check_param_grads, oracle_cfg


@pytest.fixture(scope="module")
def case():
    sh = synth.Shape("tol", 2, 384, 512, 8, 2, 64, seed=11)
    t = synth.make_inputs(sh)
    cfg = oracle_cfg(sh)
    _, I = O.forward(cfg, t, t["x"])
    G = O.backward(cfg, t, I, t["d_out"])
    M = NM.storage_model_gradients(cfg, t)
    return cfg, t, I, G, M


def _as_grads(G):
    return {"d_" + n: G["d_" + n].clone() for n in PARAM_NAMES}


def test_bf16_storage_noise_alone_passes(case):
    cfg, t, I, G, M = case
    rep = check_param_grads(cfg, t, I, G, _as_grads(M))
    for n in ("w_qk", "w_v1", "w_v2", "w_o", "conv0_w", "conv1_w"):
        assert 1.0 <= rep[n]["kappa"] < 4.0           # a handful of roundings per term, not tens


def test_exact_gradients_pass(case):
    cfg, t, I, G, M = case
    check_param_grads(cfg, t, I, G, _as_grads(G))


def test_threefold_error_on_one_temperature_gradient_fails(case):
    cfg, t, I, G, M = case
    for j in range(cfg.n_kv_heads):
        g = _as_grads(G)
        g["d_temp"][j] *= 3.0
        with pytest.raises(AssertionError, match="d_temp"):
            check_param_grads(cfg, t, I, G, g)


def test_systematic_three_percent_error_fails(case):
    cfg, t, I, G, M = case
    for n in ("w_qk", "w_v1", "w_o", "conv0_w", "conv1_w"):
        g = _as_grads(M)
        g["d_" + n] = g["d_" + n] * 1.03
        with pytest.raises(AssertionError, match="d_" + n):
            check_param_grads(cfg, t, I, G, g)


def test_value_shift_dropped_from_a_weight_gradient_fails(case):
    cfg, t, I, G, M = case
    g = _as_grads(G)
    Lk = cfg.L_k
    dv2 = G["d_v"].reshape(*I["x"].shape[:2], Lk)[..., Lk // 2:]
    g["d_w_v2"] = torch.einsum("bsl,bse->le", dv2, I["x"])          # x_t where x_{t-1} belongs
    with pytest.raises(AssertionError, match="d_w_v2"):
        check_param_grads(cfg, t, I, G, g)


def test_single_wrong_element_fails(case):
    cfg, t, I, G, M = case
    g = _as_grads(M)
    rss = NM.term_rss(cfg, t, I, G)["w_qk"]
    g["d_w_qk"][3, 5] += 0.1 * rss[3, 5] + 0.05 * G["d_w_qk"][3, 5].abs() + 0.05     # 50 roundings' worth
    with pytest.raises(AssertionError, match="d_w_qk"):
        check_param_grads(cfg, t, I, G, g)
