"""Stored expected values: the paper's comparison-table formulas evaluated by hand at the benchmark shapes, and the
oracle's own output on a tiny input (a regression guard written by tests/golden/make_oracle_golden.py)."""
import ctypes as C
import importlib.util
import os

import torch

from oracle import cca_oracle as O

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _table():
    rows = []
    for line in open(os.path.join(GOLDEN, "comparison_table_ccgqa.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        rows.append((f[0], *[int(v) for v in f[1:]]))
    return rows


def test_oracle_counts_match_the_comparison_table():
    for name, B, S, E, hq, hk, dh, params, kv, fwd, dec in _table():
        cfg = O.OracleConfig(E, hq, hk, dh, 2, 2)
        d = O.describe(cfg, B, S)
        conv = d["conv_params"]
        assert d["params"] - conv == params, name
        assert d["kv_cache_elems"] == kv, name
        assert d["fwd_flops"] - 2 * B * S * conv == fwd, name
        assert d["decode_flops"] - 2 * B * conv == dec, name


def test_library_counts_match_the_comparison_table():
    from paper_2510_04476_b200 import binding
    lib = binding.load_library()
    for name, B, S, E, hq, hk, dh, params, kv, fwd, dec in _table():
        cfg = binding.cca_config(E, hq, hk, dh, E // (hq * dh), 2, 2, 1, 63, 10000.0)
        h = C.c_void_p()
        assert lib.cca_init(C.byref(cfg), -1, C.byref(h)) == 0          # host-only handle
        lay = binding.cca_layout()
        assert lib.cca_describe(h, B, S, C.byref(lay)) == 0
        conv = lay.conv_params
        assert lay.params - conv == params, name
        assert lay.kv_cache_elems == kv, name
        assert lay.fwd_flops - 2 * B * S * conv == fwd, name
        assert lay.decode_flops - 2 * B * conv == dec, name
        lib.cca_destroy(h)


def test_oracle_reproduces_its_stored_output():
    spec = importlib.util.spec_from_file_location("make_oracle_golden", os.path.join(GOLDEN, "make_oracle_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    vals = mod.compute()
    lines = [l for l in open(os.path.join(GOLDEN, "oracle_tiny_forward.txt")) if not l.startswith("#")]
    assert len(lines) == 2 * len(vals)
    for i in range(0, len(lines), 2):
        head = lines[i].split()
        name, shape = head[0], [int(v) for v in head[1:]]
        ref = torch.tensor([float(v) for v in lines[i + 1].split()], dtype=torch.float64).reshape(shape)
        assert torch.allclose(vals[name], ref, rtol=1e-12, atol=1e-14), name


def test_causal_flop_count_matches_hand_evaluation():
    """fwd_flops_causal is fwd_flops with the S^2 term halved; the three terms are stored evaluated by hand."""
    for line in open(os.path.join(GOLDEN, "causal_flops.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        name, (B, S, E, hq, hk, dh, proj, conv, attn, total) = f[0], [int(v) for v in f[1:]]
        assert proj + conv + attn == total, name
        d = O.describe(O.OracleConfig(E, hq, hk, dh, 2, 2), B, S)
        assert d["fwd_flops_causal"] == total, name
        assert d["fwd_flops"] - d["fwd_flops_causal"] == 2 * B * S * S * hq * dh == attn, name
        assert d["fwd_flops"] == proj + conv + 2 * attn, name
