"""Random shapes outside the benchmark configurations: forward, backward, decode continuation and chunked prefill
against the oracle.  A guard against logic errors (indexing, tails, flag combinations).  Outputs (prefill and
decode) get no tail allowance: every element is within 1e-2 + 1e-2 |ref| plus six standard deviations of the
rounding noise of its own sum (tests/util.py::check_out_wide; the widest shapes drawn here, d_model 4096 against
65 keys, have outputs of rms 1.1, where the bf16 rounding of o alone is a third of the absolute 1e-2).  The input
gradient gets a tail allowance:
at the widest shapes drawn here (E = 4096, 16 query heads) the bf16-operand pipeline leaves up to 0.03 % of its
elements above the bound, by a factor of at most 2.2 (rms error 0.3-0.6 % of the rms value); a wrong index or a
dropped term is off by orders of magnitude more.  Parameter gradients: tests/util.py::check_param_grads."""
import random

import pytest
import torch

from oracle import cca_oracle as O
from paper_2510_04476_b200 import synth
from tests.util import check_close, check_out_wide, check_param_grads, oracle_cfg, to_device

pytestmark = pytest.mark.gpu
DX_TAIL = (1e-3, 3.0)       # input gradient only


def draw(seed):
    rng = random.Random(seed)
    while True:
        dh = rng.choice([32, 64, 64, 128, 128])
        hk = rng.choice([1, 2, 4])
        g = rng.choice([1, 2, 4, 8])
        hq = hk * g
        if hq > 16:
            hq = hk * 2
        C = rng.choice([1, 2, 4])
        E = C * hq * dh
        if E > 4096:
            E = hq * dh
        B = rng.choice([1, 1, 2, 3])
        S = rng.choice([1, 2, 5, 63, 64, 65, 127, 128, 129, 255, 256, 257, 300, 511, 513, 700, 1000, 1025, 1537, 2049])
        ks, kc = rng.choice([1, 2, 2, 3, 4]), rng.choice([1, 2, 2, 3, 4])
        flags = rng.choice([63, 63, 63, 63 & ~4, 63 & ~8, 63 & ~16, 63 & ~32, 63 & ~1, 63 & ~2, 0, 16 | 32])
        causal = rng.choice([1, 1, 1, 0])
        if (hk * dh) % 2 == 0:
            return synth.Shape(f"random{seed}", B, S, E, hq, hk, dh, k_seq=ks, k_ch=kc, causal=causal, flags=flags,
                               seed=4000 + seed)


@pytest.mark.parametrize("seed", range(24))
def test_random_shape(seed):
    from paper_2510_04476_b200.binding import CCA
    sh = draw(seed)
    t = synth.make_inputs(sh)
    cfg = oracle_cfg(sh)
    out_ref, I = O.forward(cfg, t, t["x"])
    G = O.backward(cfg, t, I, t["d_out"])
    dev = to_device(t)
    cca = CCA.from_shape(sh)
    ws = cca.alloc_workspace(sh.B, sh.S, True)
    out = cca.forward(dev, dev["x"], ws)
    d_x, grads = cca.backward(dev, dev["x"], dev["d_out"], ws)
    torch.cuda.synchronize()
    assert cca.last_status() == 0
    model = check_out_wide(cfg, t, I, "out", out, out_ref)
    check_close("d_x", d_x, G["d_x"], tail=DX_TAIL)
    check_param_grads(cfg, t, I, G, grads, model=model)
    if sh.causal and sh.S >= 2:
        # the last three tokens again, one at a time against the cache of a shorter prefill
        S0 = max(1, sh.S - 3)
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
            check_out_wide(cfg, t, I, f"decode[{tok}]", o, out_ref[:, tok], rows=tok, model=model)
    if sh.causal and sh.B == 1 and (sh.flags & 2) and (sh.head_dim == 64 or (sh.head_dim == 128 and sh.k_ch <= 2)):
        cut = (sh.S // 2) // 256 * 256
        if cut >= 512 and sh.S - cut >= 512:
            ws3 = cca.alloc_workspace(1, sh.S, False)
            a = cca.forward_chunk(dev, dev["x"][0, :cut].contiguous(), ws3, sh.S, 0)
            b = cca.forward_chunk(dev, dev["x"][0, cut:].contiguous(), ws3, sh.S, cut)
            assert torch.equal(torch.cat([a, b])[None], out)
    torch.cuda.synchronize()
    assert cca.last_status() == 0
    cca.close()
