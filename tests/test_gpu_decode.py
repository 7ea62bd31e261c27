"""GPU parity of the decode step (one new token per sequence against the latent KV cache) with the fp64
oracle's token-by-token decode and, after a prefill on the GPU, with rows of the oracle's whole-sequence
forward.  Tolerance as everywhere: max |err| <= 1e-2 + 1e-2 |ref|."""
import pytest
import torch

from oracle import cca_oracle as O
from paper_2510_04476_b200 import synth
from tests.util import check_close, oracle_cfg, to_device

pytestmark = pytest.mark.gpu


def _cca(sh):
    from paper_2510_04476_b200.binding import CCA
    return CCA.from_shape(sh)


def S_(name, B, S, E, hq, hk, dh, **kw):
    return synth.Shape(name, B, S, E, hq, hk, dh, seed=sum(map(ord, name)) % 1000, **kw)


EMPTY_START = [
    S_("dec_dh32", 3, 20, 256, 4, 2, 32),
    S_("dec_dh64_g4", 2, 40, 512, 8, 2, 64),
    S_("dec_dh128_g4", 2, 33, 1024, 4, 1, 128),
    S_("dec_mha_g1", 2, 17, 256, 4, 4, 64, flags=0),
    S_("dec_g2", 2, 17, 512, 4, 2, 64),
    S_("dec_g8", 1, 19, 512, 8, 1, 64),
    S_("dec_g16", 1, 37, 1024, 16, 1, 64),
    S_("dec_g12_dh128", 2, 21, 1536, 12, 1, 128, flags=63 & ~16),
    S_("dec_k3_k4", 2, 15, 512, 8, 2, 64, k_seq=3, k_ch=4),
    S_("dec_k1_k1", 2, 9, 512, 8, 2, 64, k_seq=1, k_ch=1),
    S_("dec_no_shift", 2, 9, 512, 8, 2, 64, flags=63 & ~8),
    S_("dec_no_conv2", 2, 9, 512, 8, 2, 64, flags=63 & ~2),
    S_("dec_no_norm", 2, 9, 512, 8, 2, 64, flags=63 & ~16),
    S_("dec_no_mean_no_rope", 2, 9, 512, 8, 2, 64, flags=63 & ~4 & ~32),
    S_("dec_batch_over_16", 19, 6, 256, 4, 2, 64),
    S_("dec_dh256_g2", 2, 25, 1024, 4, 2, 256),
    S_("dec_dh256_g4_no_norm", 1, 37, 1024, 4, 1, 256, flags=63 & ~16),
]


@pytest.mark.parametrize("sh", EMPTY_START, ids=lambda s: s.name)
def test_decode_from_empty_state_matches_oracle(sh):
    t = synth.make_inputs(sh, want_dout=False)
    cfg = oracle_cfg(sh)
    dev = to_device(t)
    cca = _cca(sh)
    S_max = sh.S + 3
    st = cca.new_decode_state(sh.B, S_max)
    ws = cca.alloc_decode_workspace(sh.B, S_max)
    ost = O.decode_init(cfg, sh.B)
    for tok in range(sh.S):
        ref = O.decode_step(cfg, t, ost, t["x"][:, tok])
        out = cca.decode_step(dev, dev["x"][:, tok].contiguous(), st, tok + 1, ws)
        st["pos"] += 1
        check_close(f"out[{tok}]", out, ref)
    torch.cuda.synchronize()
    assert cca.last_status() == 0
    check_close("k_cache", st["k_cache"][:, :sh.S].reshape(ost["k"].shape), ost["k"])
    check_close("v_cache", st["v_cache"][:, :sh.S].reshape(ost["v"].shape), ost["v"])
    if st["qk0_hist"].numel():
        check_close("qk0_hist", st["qk0_hist"], ost["qk0_hist"])
    assert torch.equal(st["x_prev"].cpu(), t["x"][:, sh.S - 1])
    assert (st["k_cache"][:, sh.S:] == 0).all() and (st["v_cache"][:, sh.S:] == 0).all()     # nothing past the end
    cca.close()


@pytest.mark.parametrize("sh,S0", [(S_("dec_prefill_dh64", 2, 712, 512, 8, 2, 64), 700),
                                   (S_("dec_prefill_dh128", 1, 1300, 1024, 8, 2, 128), 1290),
                                   (S_("dec_prefill_one", 2, 6, 512, 8, 2, 64, k_seq=3, k_ch=3), 1),
                                   (S_("dec_prefill_dh256", 1, 1034, 1024, 4, 1, 256), 1024)],
                         ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_decode_continues_a_gpu_prefill(sh, S0):
    """Prefill S0 tokens with cca_forward, hand the workspace over, decode the rest: every decoded row must
    equal the oracle's whole-sequence forward at that position (several key chunks per sequence)."""
    t = synth.make_inputs(sh, want_dout=False)
    rows = list(range(S0, sh.S))
    out_ref, _, _, I = O.forward_rows(oracle_cfg(sh), t, t["x"], rows)
    dev = to_device(t)
    cca = _cca(sh)
    ws = cca.alloc_workspace(sh.B, S0, False)
    cca.forward(dev, dev["x"][:, :S0].contiguous(), ws)
    st = cca.new_decode_state(sh.B, sh.S)
    cca.decode_state_from_prefill(dev["x"][:, :S0].contiguous(), ws, st)
    st["pos"].fill_(S0)
    dws = cca.alloc_decode_workspace(sh.B, sh.S)
    for i, tok in enumerate(rows):
        out = cca.decode_step(dev, dev["x"][:, tok].contiguous(), st, sh.S, dws)
        st["pos"] += 1
        check_close(f"out[{tok}]", out, out_ref[:, i])
    torch.cuda.synchronize()
    assert cca.last_status() == 0
    check_close("k_cache", st["k_cache"].reshape(I["k"].shape), I["k"])
    check_close("v_cache", st["v_cache"].reshape(I["v"].shape), I["v"])
    cca.close()


def test_decode_ragged_positions():
    """Sequences of different lengths in one batch: each follows its own positions (RoPE angle, cache row,
    number of keys)."""
    lens = [5, 131, 300]
    n_new = 4
    base = S_("dec_ragged", 1, max(lens) + n_new, 512, 8, 2, 64)
    cca = _cca(base)
    S_max = max(lens) + n_new
    batch = cca.new_decode_state(len(lens), S_max)
    seqs, refs = [], []
    w = None
    for b, n in enumerate(lens):
        sh = base.replace(S=n + n_new, seed=base.seed)          # same weights (same seed, drawn after x) ...
        t = synth.make_inputs(sh, want_dout=False)
        if w is None:
            w = {k: v for k, v in t.items() if k != "x"}
        t = {**w, "x": t["x"]}                                      # ... made identical explicitly
        out_ref, _, _, _ = O.forward_rows(oracle_cfg(sh), t, t["x"], list(range(n, n + n_new)))
        refs.append(out_ref[0])
        seqs.append(t["x"][0])
        dev1 = to_device(t)
        ws = cca.alloc_workspace(1, n, False)
        cca.forward(dev1, dev1["x"][:, :n].contiguous(), ws)
        one = cca.new_decode_state(1, S_max)
        cca.decode_state_from_prefill(dev1["x"][:, :n].contiguous(), ws, one)
        for name in ("k_cache", "v_cache", "qk0_hist", "x_prev"):
            batch[name][b].copy_(one[name][0])
    devw = to_device(w)
    batch["pos"].copy_(torch.tensor(lens, dtype=torch.int32))
    dws = cca.alloc_decode_workspace(len(lens), S_max)
    for i in range(n_new):
        x = torch.stack([seqs[b][lens[b] + i] for b in range(len(lens))]).cuda()
        out = cca.decode_step(devw, x, batch, S_max, dws)
        batch["pos"] += 1
        check_close(f"step {i}", out, torch.stack([refs[b][i] for b in range(len(lens))]))
    torch.cuda.synchronize()
    assert cca.last_status() == 0
    cca.close()


def test_decode_position_outside_cache_is_reported_not_written():
    sh = S_("dec_bad_pos", 2, 4, 256, 4, 2, 64)
    t = synth.make_inputs(sh, want_dout=False)
    dev = to_device(t)
    cca = _cca(sh)
    st = cca.new_decode_state(sh.B, 8)
    ws = cca.alloc_decode_workspace(sh.B, 8)
    st["pos"].copy_(torch.tensor([0, 8], dtype=torch.int32))       # second sequence: one past the capacity
    cca.decode_step(dev, dev["x"][:, 0].contiguous(), st, 8, ws)
    torch.cuda.synchronize()
    assert cca.last_status() == 120
    assert (st["k_cache"][1] == 0).all() and (st["v_cache"][1] == 0).all()
    assert cca.last_status() == 0                                   # reading the status clears it
    cca.close()


def test_decode_host_side_argument_checks():
    from paper_2510_04476_b200.binding import CcaError
    sh = S_("dec_args", 2, 4, 256, 4, 2, 64)
    t = synth.make_inputs(sh, want_dout=False)
    dev = to_device(t)
    cca = _cca(sh)
    st = cca.new_decode_state(sh.B, 8)
    ws = cca.alloc_decode_workspace(sh.B, 8)
    with pytest.raises(CcaError):                                   # max_len beyond the cache capacity
        cca.decode_step(dev, dev["x"][:, 0].contiguous(), st, 9, ws)
    with pytest.raises(CcaError):                                   # workspace too small
        cca.decode_step(dev, dev["x"][:, 0].contiguous(), st, 8, ws[:300])
    nc = _cca(sh.replace(causal=0))
    with pytest.raises(CcaError):                                   # decode is causal by construction
        nc.decode_step(dev, dev["x"][:, 0].contiguous(), st, 8, ws)
    nc.close()
    cca.close()


def test_decode_at_16k_context_of_the_prefill_shape():
    """The 16k prefill shape: prefill on the GPU, then two decode steps against the 16384-token cache."""
    base = synth.CONFIGS["cfg3_prefill16k"]
    S0, n_new = base.S, 2
    sh = base.replace(S=S0 + n_new)
    t = synth.make_inputs(sh, want_dout=False)
    rows = list(range(S0, S0 + n_new))
    out_ref, _, _, _ = O.forward_rows(oracle_cfg(sh), t, t["x"], rows)
    dev = to_device(t)
    cca = _cca(sh)
    ws = cca.alloc_workspace(1, S0, False)
    x0 = dev["x"][:, :S0].contiguous()
    cca.forward(dev, x0, ws)
    st = cca.new_decode_state(1, S0 + n_new)
    cca.decode_state_from_prefill(x0, ws, st)
    st["pos"].fill_(S0)
    dws = cca.alloc_decode_workspace(1, S0 + n_new)
    for i, tok in enumerate(rows):
        out = cca.decode_step(dev, dev["x"][:, tok].contiguous(), st, S0 + n_new, dws)
        st["pos"] += 1
        check_close(f"out[{tok}]", out, out_ref[:, i])
    torch.cuda.synchronize()
    assert cca.last_status() == 0
    cca.close()
