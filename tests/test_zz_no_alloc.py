"""cca_forward_static: the forward for callers that may not allocate device memory (a process whose GPU memory
belongs to another allocator, a plug-in that is lent only a stream and its buffers).  Its scratch is a fixed
array inside the library, shared by all calls, so the checks are: same result as cca_forward, twice in a row
(the second call starts from the first call's leftovers), no change in the device's free memory across the calls
(nothing was allocated, by the library or by the binding), and a clear refusal beyond the built-in size.
This file is named to be collected last."""
import pytest
import torch

from paper_2510_04476_b200 import synth
from tests.util import check_close, to_device

pytestmark = pytest.mark.gpu


def test_static_workspace_forward_matches_forward_twice_in_a_row():
    from paper_2510_04476_b200.binding import CCA
    shapes = [synth.Shape("static_a", 2, 300, 512, 8, 2, 64, seed=11),
              synth.Shape("static_b", 1, 130, 1024, 4, 2, 128, seed=12)]
    for sh in shapes:
        t = to_device(synth.make_inputs(sh, want_dout=False))
        cca = CCA.from_shape(sh)
        ws = cca.alloc_workspace(sh.B, sh.S, False)
        ref = cca.forward(t, t["x"], ws).clone()
        torch.cuda.synchronize()
        out = torch.empty_like(t["x"])
        free_before = None
        for call in range(3):
            out.fill_(float("nan"))
            torch.cuda.synchronize()
            if call == 1:
                # after the warm-up call (which may load the kernels' code onto the device): the next two calls
                # must leave the device's free memory exactly where it is
                free_before = torch.cuda.mem_get_info()[0]
            cca.forward_static(t, t["x"], out)
            torch.cuda.synchronize()
            assert cca.last_status() == 0
            if call >= 1:
                assert torch.cuda.mem_get_info()[0] == free_before, "cca_forward_static changed the free device memory"
            check_close(f"{sh.name} call {call}", out, ref.double())
            assert torch.equal(out, ref), "same kernels on the same inputs: the bits should agree too"
        cca.close()


def test_static_workspace_rejects_sizes_beyond_its_maximum():
    from paper_2510_04476_b200.binding import CCA, CcaError
    sh = synth.CONFIGS["cfg2_small"]          # 4096 tokens of a 1280-wide latent: more than 32 MiB
    cca = CCA.from_shape(sh)
    assert cca.workspace_size(sh.B, sh.S, False) > (32 << 20)
    x = torch.zeros(sh.B, sh.S, sh.d_model, dtype=torch.bfloat16, device="cuda")
    w = {n: torch.zeros(1, dtype=torch.float32 if n == "temp" else torch.bfloat16, device="cuda")
         for n in ("w_qk", "w_v1", "w_v2", "w_o", "conv0_w", "conv1_w", "temp")}
    with pytest.raises(CcaError, match="built-in static workspace"):
        cca.forward_static(w, x, torch.empty_like(x))
    cca.close()
