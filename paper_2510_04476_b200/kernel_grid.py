"""Latency grid of the block's kernels, after the paper's kernel study (Appendix D.1): d_model 2048, latent
head size 64 or 128, sequence lengths 512 ... 16384, forward causal and non-causal, forward + backward
non-causal, for CCGQA (C = 4, four query heads per kv head) and for the same kernels configured as GQA
(no compression, four query heads per kv head, latent transforms off) and as MHA.

    python -m paper_2510_04476_b200.kernel_grid [--tokens 32768] [--steps 5] [--head-dims 64,128]

Prints one JSON line per (method, head size, sequence length) and a markdown table at the end.  Every number
is a CUDA-event time on the launching stream after three warm-up steps; the batch is tokens / S sequences.
"""
from __future__ import annotations

import argparse
import json
import sys

import torch

from . import synth
from .binding import CCA


def shapes_for(dh: int, S: int, tokens: int):
    E = 2048
    B = max(1, tokens // S)
    h = E // dh
    seed = 7000 + dh + S
    ccgqa = synth.Shape(f"grid_ccgqa_d{dh}_S{S}", B, S, E, h // 4, max(1, h // 16), dh, seed=seed)
    gqa = synth.Shape(f"grid_gqa_d{dh}_S{S}", B, S, E, h, h // 4, dh, flags=0, seed=seed)
    mha = synth.Shape(f"grid_mha_d{dh}_S{S}", B, S, E, h, h, dh, flags=0, seed=seed)
    return {"ccgqa": ccgqa, "gqa": gqa, "mha": mha}


def time_shape(sh: synth.Shape, steps: int, device: int):
    """ms of: forward causal (block, attention kernel), forward non-causal (same), forward + backward non-causal."""
    res = {}
    t = synth.make_inputs(sh, want_dout=True)
    dev = {k: v.cuda(device).contiguous() for k, v in t.items()}
    out = torch.empty_like(dev["x"])
    for causal in (1, 0):
        s = sh.replace(causal=causal)
        cca = CCA.from_shape(s, device=device)
        ws = cca.alloc_workspace(s.B, s.S, True)
        for _ in range(3):
            cca.forward(dev, dev["x"], ws, out)
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in ev:
            a.record(); b.record()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for i in range(steps):
            cca.set_attention_events(*ev[i])
            cca.forward(dev, dev["x"], ws, out)
        e1.record()
        torch.cuda.synchronize()
        cca.set_attention_events(None, None)
        key = "causal" if causal else "noncausal"
        res[f"fwd_{key}_ms"] = e0.elapsed_time(e1) / steps
        res[f"attn_fwd_{key}_ms"] = sum(a.elapsed_time(b) for a, b in ev) / steps
        if not causal and sh.head_dim <= 128:          # head size 256 has no backward
            for _ in range(2):
                cca.forward(dev, dev["x"], ws, out)
                cca.backward(dev, dev["x"], dev["d_out"], ws)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(steps):
                cca.forward(dev, dev["x"], ws, out)
                cca.backward(dev, dev["x"], dev["d_out"], ws)
            e1.record()
            torch.cuda.synchronize()
            res["fwd_bwd_noncausal_ms"] = e0.elapsed_time(e1) / steps
        st = cca.last_status()
        cca.close()
        if st != 0:
            raise RuntimeError(f"device status {st} at {s.name}")
        del ws
    return res


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--tokens", type=int, default=32768)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--head-dims", default="64,128")
    ap.add_argument("--seq-lens", default="512,1024,2048,4096,8192,16384")
    ap.add_argument("--device", type=int, default=0)
    a = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("kernel_grid needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(a.device)
    rows = []
    for dh in [int(v) for v in a.head_dims.split(",")]:
        for S in [int(v) for v in a.seq_lens.split(",")]:
            rec = {"head_dim": dh, "S": S, "B": max(1, a.tokens // S)}
            for name, sh in shapes_for(dh, S, a.tokens).items():
                r = time_shape(sh, a.steps, a.device)
                rec[name] = r
                print(json.dumps({"method": name, "head_dim": dh, "S": S, "B": sh.B, "heads": [sh.n_q_heads, sh.n_kv_heads],
                                  **{k: round(v, 4) for k, v in r.items()}}), flush=True)
            rows.append(rec)
    cols = ["fwd_causal_ms", "fwd_noncausal_ms", "fwd_bwd_noncausal_ms"]
    print("\n| d_h | S | B | " + " | ".join(f"{c[:-3]}: CCGQA / GQA / MHA (ms), MHA/CCGQA" for c in cols) + " |")
    print("|---|---|---|" + "---|" * len(cols))
    for r in rows:
        cells = []
        for c in cols:
            if c not in r["ccgqa"]:
                cells.append("-")
                continue
            v = [r[m][c] for m in ("ccgqa", "gqa", "mha")]
            cells.append(f"{v[0]:.3f} / {v[1]:.3f} / {v[2]:.3f}, {v[2] / v[0]:.2f}x")
        print(f"| {r['head_dim']} | {r['S']} | {r['B']} | " + " | ".join(cells) + " |")
    return 0


if __name__ == "__main__":
    sys.exit(main())
