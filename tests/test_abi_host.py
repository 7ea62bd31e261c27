"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, validates
configurations, and its integer metadata equals the oracle's closed forms bit for bit."""
import ctypes as C
import os
import re

import pytest

from oracle import cca_oracle as O
from paper_2510_04476_b200 import binding, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "cca.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cca_[a-z_]+)\s*\(", text)))


def test_library_loads_and_exports_every_declared_symbol():
    lib = binding.load_library()
    names = declared_symbols()
    assert "cca_init" in names and "cca_forward" in names and "cca_backward" in names
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(binding.SYMBOLS), set(names) ^ set(binding.SYMBOLS)


def host_handle(lib, **kw):
    d = dict(d_model=2048, n_q_heads=16, n_kv_heads=4, head_dim=64, compression=2, k_seq=2, k_ch=2, causal=1,
             flags=63, rope_base=10000.0)
    d.update(kw)
    cfg = binding.cca_config(**d)
    h = C.c_void_p()
    return lib.cca_init(C.byref(cfg), -1, C.byref(h)), h


@pytest.mark.parametrize("kw,code", [
    ({}, 0),
    ({"compression": 3}, 1),                       # E != C * h_q * d_h
    ({"n_kv_heads": 3}, 1),                        # h_q % h_k
    ({"k_seq": 0}, 1),
    ({"flags": 64}, 1),
    ({"head_dim": 16, "n_q_heads": 64, "n_kv_heads": 16}, 2),
    ({"k_ch": 5}, 2),
    ({"rope_base": 0.0}, 1),
])
def test_config_validation(kw, code):
    lib = binding.load_library()
    rc, h = host_handle(lib, **kw)
    assert rc == code
    if rc == 0:
        assert lib.cca_destroy(h) == 0


def test_host_only_handle_refuses_compute_and_bad_sizes():
    lib = binding.load_library()
    rc, h = host_handle(lib)
    assert rc == 0
    n = C.c_size_t()
    assert lib.cca_workspace_size(h, 0, 128, 1, C.byref(n)) == 1
    assert lib.cca_workspace_size(h, 1, 128, 1, None) == 1
    assert lib.cca_workspace_size(h, 2, 128, 0, C.byref(n)) == 0
    fwd_only = n.value
    assert lib.cca_workspace_size(h, 2, 128, 1, C.byref(n)) == 0
    assert n.value > fwd_only > 0
    w = binding.cca_weights()
    assert lib.cca_forward(h, C.byref(w), None, None, None, 0, 1, 128, 0, None) == 1
    assert lib.cca_set_wait_limit(h, 1 << 22) == 1          # a host-only handle has no device status block
    assert lib.cca_wait_selftest(h, None) == 1
    assert lib.cca_status_string(4) == b"workspace too small"
    lib.cca_destroy(h)


@pytest.mark.parametrize("sh,B,S", [(s, s.B, s.S) for s in synth.CONFIGS.values()] +
                         [(synth.sweep_shape(S, Cc), 65536 // S, S) for S in (1024, 65536) for Cc in (1, 2, 4, 8)])
def test_metadata_is_bit_exact_against_oracle(sh, B, S):
    lib = binding.load_library()
    rc, h = host_handle(lib, d_model=sh.d_model, n_q_heads=sh.n_q_heads, n_kv_heads=sh.n_kv_heads,
                        head_dim=sh.head_dim, compression=sh.compression, k_seq=sh.k_seq, k_ch=sh.k_ch)
    assert rc == 0
    lay = binding.cca_layout()
    assert lib.cca_describe(h, B, S, C.byref(lay)) == 0
    ref = O.describe(O.OracleConfig(sh.d_model, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.k_seq, sh.k_ch), B, S)
    for k, v in ref.items():
        assert int(getattr(lay, k)) == v, k
    g = sh.n_q_heads // sh.n_kv_heads
    assert list(lay.q_to_kv_head)[: sh.n_q_heads] == [i // g for i in range(sh.n_q_heads)]
    assert all(x == -1 for x in list(lay.q_to_kv_head)[sh.n_q_heads:])
    offs = [lay.off_qk0, lay.off_q, lay.off_k, lay.off_v, lay.off_o, lay.off_lse, lay.off_rope, lay.saved_bytes]
    assert offs == sorted(offs) and all(o % 256 == 0 for o in offs)
    assert lay.off_q - lay.off_qk0 >= B * S * (sh.L) * 4
    lib.cca_destroy(h)
