"""GPU parity of the MLA baseline (paper Section 2.1, Eq. 3-6) run on the library's GEMM and attention kernels,
against the fp64 MLA oracle: latents, attention operands, attention output and block output, element by element."""
import pytest
import torch

from oracle import mla_oracle as M
from paper_2510_04476_b200 import synth
from tests.util import check_close

pytestmark = pytest.mark.gpu


def run(m, impl=1, scale=4.0):
    from paper_2510_04476_b200.binding import CCA
    t = synth.make_mla_inputs(m)
    for n in ("w_uq", "w_uqr", "w_uk", "w_uv", "w_kr"):        # larger logits and outputs than the N(0, 0.02) recipe gives:
        t[n] = (t[n].float() * scale).to(torch.bfloat16)       # peaked rows, outputs well above the absolute tolerance
    cfg = M.MlaConfig(m.d_model, m.n_heads, m.d_nope, m.d_rope, m.head_dim, m.d_ckv, m.d_cq, m.causal, m.rope_base)
    out_ref, I = M.forward(cfg, t, t["x"])
    dev = {k: v.cuda().contiguous() for k, v in t.items()}
    cca = CCA(m.d_model, m.n_heads, m.n_heads, m.head_dim, causal=m.causal, flags=0, rope_base=m.rope_base)
    cca.set_impl(impl)
    out, ws = cca.mla_forward((m.d_nope, m.d_rope, m.d_ckv, m.d_cq), dev, dev["x"])
    torch.cuda.synchronize()
    assert cca.last_status() == 0
    check_close("out", out, out_ref)
    cca.close()


CASES = [
    synth.MlaShape("mla_dh64", 2, 300, 512, 8, 32, 32, 128, 256, seed=5),
    synth.MlaShape("mla_dh128_ragged", 1, 777, 1024, 8, 64, 64, 256, 512, seed=6),
    synth.MlaShape("mla_uneven_parts", 1, 260, 1024, 8, 96, 32, 256, 512, seed=7),
    synth.MlaShape("mla_noncausal", 2, 200, 512, 4, 64, 64, 128, 256, causal=0, seed=8),
    synth.MlaShape("mla_one_token", 3, 1, 512, 8, 32, 32, 128, 256, seed=9),
]


@pytest.mark.parametrize("impl", [1, 0])
@pytest.mark.parametrize("m", CASES, ids=lambda m: m.name)
def test_mla_forward_matches_oracle(m, impl):
    run(m, impl)


def test_mla_baseline_of_the_kernel_grid_shape():
    run(synth.mla_like(synth.Shape("grid", 1, 2048, 2048, 4, 1, 128, seed=3)), scale=1.0)     # the grid's own recipe


def test_mla_argument_checks():
    from paper_2510_04476_b200.binding import CCA, CcaError
    m = CASES[0]
    dev = {k: v.cuda().contiguous() for k, v in synth.make_mla_inputs(m).items()}
    cca = CCA(m.d_model, m.n_heads, m.n_heads, m.head_dim, flags=0)
    with pytest.raises(CcaError, match="invalid argument"):
        cca.mla_forward((m.d_nope, m.d_rope + 16, m.d_ckv, m.d_cq), dev, dev["x"])        # parts do not add up to d_h
    gq = CCA(m.d_model, m.n_heads, m.n_heads // 2, m.head_dim, flags=0)
    with pytest.raises(CcaError, match="invalid argument"):
        gq.mla_forward((m.d_nope, m.d_rope, m.d_ckv, m.d_cq), dev, dev["x"])             # MLA has one k, v per query head
    cca.close()
    gq.close()
