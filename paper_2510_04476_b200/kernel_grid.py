"""Latency grid of the block's kernels, after the paper's kernel study (Appendix D.1): d_model 2048, latent
head size 64 or 128, sequence lengths 512 ... 16384, forward causal and non-causal, forward + backward
non-causal, for CCGQA (C = 4, four query heads per kv head) and for the same kernels configured as GQA
(no compression, four query heads per kv head, latent transforms off), as MHA, and as MLA (Section 2.1 of the paper,
Eq. 3-6: E / d_h heads, half of each head RoPE with one shared RoPE key, KV latent E / 4, query latent E / 2; forward only).

    python -m paper_2510_04476_b200.kernel_grid [--tokens 32768] [--steps 5] [--head-dims 64,128]
    python -m paper_2510_04476_b200.kernel_grid --sweep          # context x compression sweep, forward and backward

Prints one JSON line per (method, head size, sequence length) and a markdown table at the end.  Every number
is a CUDA-event time on the launching stream after three warm-up steps; the batch is tokens / S sequences.
"""
from __future__ import annotations

import argparse
import json
import sys

import torch

from . import synth
from .binding import CCA, stack_down_projection


def shapes_for(dh: int, S: int, tokens: int):
    E = 2048
    B = max(1, tokens // S)
    h = E // dh
    seed = 7000 + dh + S
    ccgqa = synth.Shape(f"grid_ccgqa_d{dh}_S{S}", B, S, E, h // 4, max(1, h // 16), dh, seed=seed)
    gqa = synth.Shape(f"grid_gqa_d{dh}_S{S}", B, S, E, h, h // 4, dh, flags=0, seed=seed)
    mha = synth.Shape(f"grid_mha_d{dh}_S{S}", B, S, E, h, h, dh, flags=0, seed=seed)
    return {"ccgqa": ccgqa, "gqa": gqa, "mha": mha, "mla": synth.mla_like(mha)}


def time_mla(m: synth.MlaShape, steps: int, device: int):
    """ms of the MLA baseline's forward, causal and non-causal (block, attention kernel)."""
    res = {}
    dev = {k: v.cuda(device).contiguous() for k, v in synth.make_mla_inputs(m).items()}
    out = torch.empty_like(dev["x"])
    dims = (m.d_nope, m.d_rope, m.d_ckv, m.d_cq)
    for causal in (1, 0):
        cca = CCA(m.d_model, m.n_heads, m.n_heads, m.head_dim, causal=causal, flags=0, device=device)
        for _ in range(3):
            cca.mla_forward(dims, dev, dev["x"], out)
        torch.cuda.synchronize()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in ev:
            a.record(); b.record()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for i in range(steps):
            cca.set_attention_events(*ev[i])
            cca.mla_forward(dims, dev, dev["x"], out)
        e1.record()
        torch.cuda.synchronize()
        cca.set_attention_events(None, None)
        key = "causal" if causal else "noncausal"
        res[f"fwd_{key}_ms"] = e0.elapsed_time(e1) / steps
        res[f"attn_fwd_{key}_ms"] = sum(a.elapsed_time(b) for a, b in ev) / steps
        st = cca.last_status()
        cca.close()
        if st != 0:
            raise RuntimeError(f"device status {st} at {m.name}")
    return res


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
        if not causal:
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


def sweep(steps: int, device: int):
    """Context x compression sweep of the benchmark (d_model 2048, latent head size 64, 32 / C query heads, a quarter as
    many kv heads, 65536 tokens per point): forward and forward + backward, causal, ms and algorithmic TFLOP/s."""
    rows = []
    for C in (1, 2, 4, 8):
        for S in (1024, 4096, 16384, 32768, 65536):
            sh = synth.sweep_shape(S, C)
            t = synth.make_inputs(sh, want_dout=True)
            dev = stack_down_projection({k: v.cuda(device).contiguous() for k, v in t.items()})
            out = torch.empty_like(dev["x"])
            cca = CCA.from_shape(sh, device=device)
            ws = cca.alloc_workspace(sh.B, sh.S, True)
            for _ in range(2):
                cca.forward(dev, dev["x"], ws, out)
                cca.backward(dev, dev["x"], dev["d_out"], ws)
            torch.cuda.synchronize()
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            fwd = bwd = 0.0
            for _ in range(steps):
                e0.record()
                cca.forward(dev, dev["x"], ws, out)
                e1.record()
                cca.backward(dev, dev["x"], dev["d_out"], ws)
                e2.record()
                torch.cuda.synchronize()
                fwd += e0.elapsed_time(e1) / steps
                bwd += e1.elapsed_time(e2) / steps
            st = cca.last_status()
            cca.close()
            if st != 0:
                raise RuntimeError(f"device status {st} at {sh.name}")
            T = sh.B * sh.S
            proj = 2 * T * sh.d_model * (sh.L_q + 2 * sh.L_k) + 2 * T * sh.L_q * sh.d_model
            conv = 2 * T * (sh.L * sh.k_seq + sh.L * sh.head_dim * sh.k_ch)
            attn = 2 * sh.B * sh.S * sh.S * sh.L_q
            f_fwd, f_all = proj + conv + attn, 3 * (proj + conv) + 3.5 * attn
            rec = {"C": C, "S": S, "B": sh.B, "heads": [sh.n_q_heads, sh.n_kv_heads], "fwd_ms": round(fwd, 4),
                   "fwd_bwd_ms": round(fwd + bwd, 4), "fwd_tflops": round(f_fwd / fwd / 1e9, 1),
                   "fwd_bwd_tflops": round(f_all / (fwd + bwd) / 1e9, 1)}
            print(json.dumps(rec), flush=True)
            rows.append(rec)
            del ws, dev, out
            torch.cuda.empty_cache()
    print("\n| C | S | B | forward ms (TFLOP/s) | forward + backward ms (TFLOP/s) |")
    print("|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['C']} | {r['S']} | {r['B']} | {r['fwd_ms']:.3f} ({r['fwd_tflops']:.0f}) | {r['fwd_bwd_ms']:.3f} ({r['fwd_bwd_tflops']:.0f}) |")
    return 0


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--tokens", type=int, default=32768)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--head-dims", default="64,128")
    ap.add_argument("--seq-lens", default="512,1024,2048,4096,8192,16384")
    ap.add_argument("--device", type=int, default=0)
    ap.add_argument("--sweep", action="store_true", help="the context x compression sweep instead of the head-size grid")
    a = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise SystemExit("kernel_grid needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(a.device)
    if a.sweep:
        return sweep(a.steps, a.device)
    rows = []
    for dh in [int(v) for v in a.head_dims.split(",")]:
        for S in [int(v) for v in a.seq_lens.split(",")]:
            rec = {"head_dim": dh, "S": S, "B": max(1, a.tokens // S)}
            for name, sh in shapes_for(dh, S, a.tokens).items():
                r = time_mla(sh, a.steps, a.device) if name == "mla" else time_shape(sh, a.steps, a.device)
                rec[name] = r
                heads = [sh.n_heads, sh.n_heads] if name == "mla" else [sh.n_q_heads, sh.n_kv_heads]
                print(json.dumps({"method": name, "head_dim": dh, "S": S, "B": sh.B, "heads": heads,
                                  **{k: round(v, 4) for k, v in r.items()}}), flush=True)
            rows.append(rec)
    cols = ["fwd_causal_ms", "fwd_noncausal_ms", "fwd_bwd_noncausal_ms"]
    print("\n| d_h | S | B | " + " | ".join(f"{c[:-3]}: CCGQA / GQA / MLA / MHA (ms), MHA/CCGQA" for c in cols) + " |")
    print("|---|---|---|" + "---|" * len(cols))
    for r in rows:
        cells = []
        for c in cols:
            if c not in r["ccgqa"]:
                cells.append("-")
                continue
            v = [r[m][c] for m in ("ccgqa", "gqa", "mha")]
            mla = f"{r['mla'][c]:.3f}" if c in r["mla"] else "-"
            cells.append(f"{v[0]:.3f} / {v[1]:.3f} / {mla} / {v[2]:.3f}, {v[2] / v[0]:.2f}x")
        print(f"| {r['head_dim']} | {r['S']} | {r['B']} | " + " | ".join(cells) + " |")
    return 0


if __name__ == "__main__":
    sys.exit(main())
