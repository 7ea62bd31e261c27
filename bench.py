#!/usr/bin/env python
"""Benchmark of the CCA / CCGQA block on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One "step" is one pass of the whole hot path over one batch of seeded synthetic input: the forward
of the block for the forward-only workloads (the 16k-context prefill headline), forward + backward
for the training workloads.  Prints ONE JSON line (rank 0).  N > 1 runs N independent replicas of the
same workload (the block has no exchange step), launched by torch.distributed.run.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch

from paper_2510_04476_b200 import synth
from paper_2510_04476_b200.replicas import max_over_ranks

METRIC = "CCGQA block throughput at 16k context (algorithmic causal FLOPs / device time)"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAK_TFLOPS = 1590.0
TRAIN_WORKLOADS = {"cfg2_small", "cfg4_train"}


def dram_traffic(kernel: str, workload: str):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of `kernel` at `workload`, from the ncu captures
    recorded in profiles/dram_traffic.json.  An entry names the source file of its kernel and that file's sha256 at
    capture time: once the file has changed the figure is stale and None is returned."""
    import hashlib
    try:
        entries = json.load(open(os.path.join(ROOT, "profiles", "dram_traffic.json")))["entries"]
    except Exception:
        return None
    for e in entries:
        if e.get("kernel") == kernel and e.get("workload") == workload:
            try:
                cur = hashlib.sha256(open(os.path.join(ROOT, e["source"]), "rb").read()).hexdigest()
            except Exception:
                return None
            return int(e["bytes"]) if cur == e.get("source_sha256") else None
    return None


def flops_of(sh, backward: bool):
    T = sh.B * sh.S
    proj = 2 * T * sh.d_model * (sh.L_q + 2 * sh.L_k) + 2 * T * sh.L_q * sh.d_model
    conv = 2 * T * (sh.L * sh.k_seq + sh.L * sh.head_dim * sh.k_ch)
    attn = (2 if sh.causal else 4) * sh.B * sh.S * sh.S * sh.L_q
    fwd = proj + conv + attn
    total = fwd + (2 * (proj + conv) + 2.5 * attn if backward else 0)
    return {"total": total, "fwd": fwd, "attn_fwd": attn, "attn_bwd": 2.5 * attn, "proj": proj, "conv": conv}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["bf16_tflops"]), "measured (cuBLAS bf16 burst)", d
        except Exception:
            pass
    return FALLBACK_PEAK_TFLOPS, "fallback", {}


def stage_table(sh, backward):
    """(name, first event, last event, bound, algorithmic work per launch) of every stage between two stage events.
    Tensor stages: FLOPs of the contraction.  HBM stages: the bytes the stage must move if nothing is re-read
    (latents in the precision they are kept in)."""
    T, E, L, Lq, Lk, dh = sh.B * sh.S, sh.d_model, sh.L, sh.L_q, sh.L_k, sh.head_dim
    attn = (2 if sh.causal else 4) * sh.B * sh.S * sh.S * Lq
    H = sh.n_q_heads + sh.n_kv_heads
    rows = [
        ("down-projection (q|k|v in one contraction)", "fwd_begin", "fwd_proj", "tensor", 2 * T * E * (L + Lk)),
        ("latent transforms (convs, q-k-mean, norm, RoPE)", "fwd_proj", "fwd_transform", "hbm", 2 * T * L + 2 * T * L),
        ("latent attention forward", "fwd_transform", "fwd_attn", "tensor", attn),
        ("up-projection", "fwd_attn", "fwd_end", "tensor", 2 * T * Lq * E),
    ]
    if backward:
        rows += [
            ("d_o = d_out W_o", "bwd_begin", "bwd_do", "tensor", 2 * T * E * Lq),
            ("d_W_o = d_out^T o", "bwd_do", "bwd_dwo", "tensor", 2 * T * E * Lq),
            ("delta = rowsum(dO o O)", "bwd_dwo", "bwd_delta", "hbm", 4 * T * Lq + 2 * T * Lq + 4 * T * sh.n_q_heads),
            ("latent attention backward", "bwd_delta", "bwd_attn", "tensor", 2.5 * attn),
            ("norm / RoPE adjoint, d_temp", "bwd_attn", "bwd_norm", "hbm", 2 * (4 * T * L) + 2 * T * L + 4 * T * H),
            ("conv2 adjoint, d_conv1_w", "bwd_norm", "bwd_conv2", "hbm", 4 * T * L + 4 * T * L + 4 * T * L),
            ("conv1 and q-k-mean adjoint, d_conv0_w", "bwd_conv2", "bwd_conv1", "hbm", 3 * (4 * T * L) + 2 * T * L),
            ("value-unshift", "bwd_conv1", "bwd_pack", "hbm", 4 * T * Lk + 2 * T * Lk),
            ("down-projection weight gradients", "bwd_pack", "bwd_dw", "tensor", 2 * T * (L + Lk) * E),
            ("d_x", "bwd_dw", "bwd_end", "tensor", 2 * T * (L + Lk) * E),
        ]
    return rows


def per_kernel_roofline(cca, step, sh, backward, n=5):
    """Every stage of the step bracketed by CUDA events the library records on the launching stream
    (cca_set_stage_events); a few extra steps outside the timed region.  Fractions are of the measured peaks."""
    from paper_2510_04476_b200.binding import CCA
    names = CCA.STAGE_EVENTS
    sets = [[torch.cuda.Event(enable_timing=True) for _ in names] for _ in range(n)]
    torch.cuda.synchronize()
    for evs in sets:
        for e in evs:
            e.record()
    torch.cuda.synchronize()
    for evs in sets:
        cca.set_stage_events(evs)
        step()
    torch.cuda.synchronize()
    cca.set_stage_events(None)
    tf_peak, tf_kind, _ = measured_peak()
    hbm, hbm_kind = hbm_peak()
    idx = {nm: i for i, nm in enumerate(names)}
    out = []
    for name, a, b, bound, work in stage_table(sh, backward):
        try:
            ms = sum(evs[idx[a]].elapsed_time(evs[idx[b]]) for evs in sets) / n
        except Exception:
            continue
        if ms <= 0:
            continue
        if bound == "tensor":
            ach, peak, unit, kind = work / (ms * 1e-3) / 1e12, tf_peak, "TFLOP/s", tf_kind
        else:
            ach, peak, unit, kind = work / (ms * 1e-3) / 1e9, hbm, "GB/s", hbm_kind
        out.append({"kernel": name, "bound": bound, "ms": ms, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak,
                    "peak_kind": kind, "work_per_launch": work})
    return out


def sustained(step, barrier, fl_total, seconds, index):
    """The step back to back for `seconds`: throughput under the power cap, with the SM clock sampled meanwhile,
    against the measured sustained GEMM rate."""
    sampler = ClockSampler(index)
    sampler.start()
    time.sleep(0.15)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0 = time.time()
    e0.record()
    n = 0
    while time.time() - w0 < seconds:
        for _ in range(50):
            step()
        n += 50
        if n % 500 == 0:
            torch.cuda.synchronize()             # keep the launch queue bounded
    e1.record()
    barrier()
    w1 = time.time()
    clocks = sampler.stop(w0, w1)
    ms = e0.elapsed_time(e1) / n
    tf = fl_total / (ms * 1e-3) / 1e12
    try:
        peak = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops_sustained"])
        kind = "measured (cuBLAS bf16, seconds-long loop)"
    except Exception:
        peak, kind = 1400.0, "fallback"
    return {"seconds": w1 - w0, "steps": n, "ms_per_step": ms, "tflops": tf, "peak": peak, "peak_kind": kind,
            "frac": tf / peak, "clocks": clocks}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: str):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0=None, t1=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.06)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        clocks, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.lines:
            if t0 is not None and not (t0 - 0.05 <= ts <= t1 + 0.1):
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                clocks.append(float(parts[0]))
                mx = float(parts[1])
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        clocks.sort()
        med = clocks[len(clocks) // 2] if clocks else None
        return {"sm_mhz": med, "sm_max_mhz": mx, "reasons": sorted(reasons), "samples": len(clocks)}


def oracle_sample(sh, n_rows=16384, backward=False):
    """The oracle, as it stands, on a bounded sample of the workload.  Forward workloads: projections and
    latent transforms in full, the S^2 stage and the up-projection on n_rows sampled query positions per
    sequence (every position if n_rows >= S).  Training workloads: the whole forward and backward."""
    from oracle import cca_oracle as O
    t = synth.make_inputs(sh, want_dout=backward)
    cfg = O.OracleConfig(sh.d_model, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.k_seq, sh.k_ch, sh.causal, sh.flags,
                         sh.rope_base)
    if backward:
        t0 = time.perf_counter()
        _, I = O.forward(cfg, t, t["x"])
        O.backward(cfg, t, I, t["d_out"])
        dt = time.perf_counter() - t0
        return flops_of(sh, True)["total"] / dt / 1e12, dt, "whole workload: forward and backward of every sequence"
    g = torch.Generator().manual_seed(123)
    if n_rows >= sh.S:
        rows = list(range(sh.S))
    else:
        rows = sorted(set(int(r) for r in torch.randint(0, sh.S, (n_rows,), generator=g)))
    t0 = time.perf_counter()
    O.forward_rows(cfg, t, t["x"], rows)
    dt = time.perf_counter() - t0
    T = sh.B * sh.S
    fl = 2 * T * sh.d_model * (sh.L_q + 2 * sh.L_k) + 2 * T * (sh.L * sh.k_seq + sh.L * sh.head_dim * sh.k_ch)
    fl += sum((2 if sh.causal else 4) * sh.B * (2 * (r + 1) if sh.causal else sh.S) * sh.L_q for r in rows)
    fl += 2 * sh.B * len(rows) * sh.L_q * sh.d_model
    return fl / dt / 1e12, dt, (f"down-projections and latent transforms in full; attention and up-projection on "
                                f"{len(rows)} of {sh.S} query rows per sequence")


def run_reference(args, rank, world):
    if rank != 0:
        return
    sh = synth.CONFIGS[args.workload]
    vals = []
    for _ in range(args.warmup):
        pass                                   # the oracle has no warm-up state; keep the run short
    t_all = time.perf_counter()
    sample = ""
    for _ in range(max(1, args.steps)):
        v, dt, sample = oracle_sample(sh, n_rows=512, backward=False)
        vals.append((v, dt))
        if time.perf_counter() - t_all > 150:
            break
    v = sum(x for x, _ in vals) / len(vals)
    ms = 1e3 * sum(d for _, d in vals) / len(vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": len(vals),
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": sh.name, "B": sh.B, "S": sh.S, "d_model": sh.d_model, "n_q_heads": sh.n_q_heads,
                   "n_kv_heads": sh.n_kv_heads, "head_dim": sh.head_dim, "note": "fp64 CPU oracle on a bounded sample"},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, rank, world, local_rank):
    from paper_2510_04476_b200.binding import CCA, stack_down_projection
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    sh = synth.CONFIGS[args.workload]
    backward = args.workload in TRAIN_WORKLOADS or args.backward
    t = synth.make_inputs(sh, want_dout=backward)
    dev = stack_down_projection({k: v.cuda(local_rank).contiguous() for k, v in t.items()})
    cca = CCA.from_shape(sh, device=local_rank)
    cca.set_impl(args.kernels)
    act_bytes = sh.B * sh.S * sh.d_model * 2
    ws = cca.alloc_workspace(sh.B, sh.S, backward, extra=2 * act_bytes + 1024)
    out = torch.empty_like(dev["x"])

    def step():
        cca.forward(dev, dev["x"], ws, out)
        if backward:
            return cca.backward(dev, dev["x"], dev["d_out"], ws)
        return None

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, b in ev:
        a.record(); b.record()
    torch.cuda.synchronize()
    vis = [v for v in os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",") if v]
    sampler = ClockSampler(vis[local_rank] if local_rank < len(vis) else str(local_rank))
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    barrier()
    l0 = cca.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0 = time.time()
    e0.record()
    for i in range(args.steps):
        cca.set_attention_events(*ev[i])
        step()
    e1.record()
    barrier()
    w1 = time.time()
    cca.set_attention_events(None, None)
    launches = cca.launch_count() - l0
    clocks = sampler.stop(w0, w1) if rank == 0 else None
    ms_total = e0.elapsed_time(e1)
    ms_step = max_over_ranks(ms_total, dist, "cuda") / args.steps
    status = cca.last_status()
    fl = flops_of(sh, backward)
    value = world * fl["total"] / (ms_step * 1e-3) / 1e12
    attn_ms = sum(a.elapsed_time(b) for a, b in ev) / args.steps

    # end to end through the C ABI with host buffers (forward workloads) / pinned copies (training)
    xh = t["x"].pin_memory()
    oh = torch.empty_like(t["x"]).pin_memory()
    if backward:
        dh_ = t["d_out"].pin_memory()
        xd, dd = torch.empty_like(dev["x"]), torch.empty_like(dev["d_out"])

    def e2e_step():
        if not backward:
            cca.forward_host(dev, xh, oh, ws)
        else:
            xd.copy_(xh, non_blocking=True)
            dd.copy_(dh_, non_blocking=True)
            cca.forward(dev, xd, ws, out)
            d_x, _ = cca.backward(dev, xd, dd, ws)
            oh.copy_(d_x, non_blocking=True)
            torch.cuda.synchronize()

    e2e_step()
    barrier()
    n_e2e = min(args.steps, 10)
    t0 = time.perf_counter()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()
    for _ in range(n_e2e):
        e2e_step()
    g1.record()
    barrier()
    e2e_ms = max_over_ranks(g0.elapsed_time(g1) / n_e2e, dist, "cuda")
    e2e_val = world * fl["total"] / (e2e_ms * 1e-3) / 1e12
    h2d = act_bytes * (2 if backward else 1)
    d2h = act_bytes

    peak, peak_kind, _ = measured_peak()
    # the events bracket the last attention stage of a step: the forward kernel, or the two adjoint kernels of a
    # training step (2.5 x the forward's FLOPs: five contractions against two)
    attn_key = "attn_bwd" if backward else "attn_fwd"
    attn_tflops = fl[attn_key] / (attn_ms * 1e-3) / 1e12
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": sh.name, "step": "forward+backward" if backward else "forward", "B": sh.B, "S": sh.S,
                   "d_model": sh.d_model, "n_q_heads": sh.n_q_heads, "n_kv_heads": sh.n_kv_heads,
                   "head_dim": sh.head_dim, "k_seq": sh.k_seq, "k_ch": sh.k_ch, "causal": sh.causal,
                   "parallelism": f"replicas x{world}" if world > 1 else "1 gpu",
                   "l2": "no flush: each step streams x, out and the latents (>= 0.4 GB), more than the 126 MB L2",
                   "kernels": "tcgen05+simt" if args.kernels else "simt"},
        "clocks": clocks,
        "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms},
        "gpu_launches": int(launches),
        "roofline": {"bound": "tensor",
                     "kernel": "latent attention backward" if backward else "latent attention forward",
                     "achieved": attn_tflops, "peak": peak,
                     "unit": "TFLOP/s", "frac": attn_tflops / peak, "peak_kind": peak_kind,
                     "frac_of_nominal_2250": attn_tflops / NOMINAL_BF16_TFLOPS, "ms_per_launch": attn_ms,
                     "flops_per_launch": fl[attn_key],
                     "traffic": (dram_traffic("attention_backward" if backward else "attention_forward", sh.name)
                                 if args.kernels else None)},
        "pct_of_nominal_bf16_peak": 100.0 * value / world / NOMINAL_BF16_TFLOPS,
        "device_status": status,
    }
    if rank == 0 and args.kernels:
        line["roofline_per_kernel"] = per_kernel_roofline(cca, step, sh, backward)
    if rank == 0 and world == 1 and args.sustain > 0:
        line["sustained"] = sustained(step, barrier, fl["total"], args.sustain,
                                      vis[local_rank] if local_rank < len(vis) else str(local_rank))
    if rank == 0 and world == 1 and not args.no_mha and not backward:
        line["mha_same_shape"] = mha_compare(sh, args, ms_step, attn_ms, local_rank)
        line["forward_backward_same_shape"] = fwd_bwd_same_shape(sh, args, local_rank)
    if rank == 0 and world == 1 and not args.no_cpu:
        v, dt, sample = oracle_sample(sh, backward=backward)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
                                "sample": sample, "seconds": dt}
    if rank == 0:
        print(json.dumps(line), flush=True)
    cca.close()
    if dist is not None:
        dist.destroy_process_group()


DECODE_WORKLOADS = {
    # model of the 16k prefill shape; 32 sequences, each with 16384 cached tokens
    "decode16k": dict(model="cfg3_prefill16k", B=32, context=16384),
}


def decode_bytes(sh, B, context):
    """Algorithmic HBM bytes of one decode step: every cached key and value row of every sequence once, every
    weight once, the new token's input and output."""
    cache = 2 * B * (context + 1) * sh.L_k * 2
    weights = 2 * (sh.L + sh.L_k) * sh.d_model + 2 * sh.d_model * sh.L_q + 2 * sh.L * (sh.k_seq + sh.head_dim * sh.k_ch)
    io = 2 * 2 * B * sh.d_model
    return {"cache": cache, "weights": weights, "io": io, "total": cache + weights + io}


def hbm_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (copy)"
    except Exception:
        return 6650.0, "fallback"


def run_decode(args, rank, world, local_rank):
    """One decode step per timed step: B new tokens against caches of `context` tokens per sequence.  The cache of
    one really prefilled sequence is replicated over the batch (the step's work does not depend on the values)."""
    from paper_2510_04476_b200.binding import CCA
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    wl = DECODE_WORKLOADS[args.workload]
    sh = synth.CONFIGS[wl["model"]]
    B, ctx = wl["B"], wl["context"]
    n_steps = max(3, args.warmup) + args.steps + 12
    S_max = ctx + n_steps + 1
    t = synth.make_inputs(sh.replace(B=1, S=ctx), want_dout=False)
    dev = {k: v.cuda(local_rank).contiguous() for k, v in t.items()}
    cca = CCA.from_shape(sh, device=local_rank)
    ws = cca.alloc_workspace(1, ctx, False)
    cca.forward(dev, dev["x"], ws)
    one = cca.new_decode_state(1, S_max)
    cca.decode_state_from_prefill(dev["x"], ws, one)
    st = cca.new_decode_state(B, S_max)
    for n in ("k_cache", "v_cache", "qk0_hist", "x_prev"):
        st[n].copy_(one[n].expand_as(st[n]))
    del ws, one
    g = torch.Generator().manual_seed(99)
    xs_host = torch.randn(n_steps, B, sh.d_model, generator=g).to(torch.bfloat16).pin_memory()
    xs = xs_host.cuda(local_rank)
    pos_table = (ctx + torch.arange(n_steps, dtype=torch.int32)[:, None].expand(n_steps, B)).contiguous().cuda(local_rank)
    dws = cca.alloc_decode_workspace(B, S_max)
    out = torch.empty(B, sh.d_model, dtype=torch.bfloat16, device=dev["x"].device)
    it = [0]

    def step(x=None):
        i = it[0]
        it[0] += 1
        st["pos"] = pos_table[i]
        cca.decode_step(dev, xs[i] if x is None else x, st, S_max, dws, out)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    barrier()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    for a, b in ev:
        a.record(); b.record()
    torch.cuda.synchronize()
    vis = [v for v in os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",") if v]
    sampler = ClockSampler(vis[local_rank] if local_rank < len(vis) else str(local_rank))
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    barrier()
    l0 = cca.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    w0 = time.time()
    e0.record()
    for i in range(args.steps):
        cca.set_attention_events(*ev[i])
        step()
    e1.record()
    barrier()
    w1 = time.time()
    cca.set_attention_events(None, None)
    launches = cca.launch_count() - l0
    clocks = sampler.stop(w0, w1) if rank == 0 else None
    ms_step = max_over_ranks(e0.elapsed_time(e1), dist, "cuda") / args.steps
    attn_ms = sum(a.elapsed_time(b) for a, b in ev) / args.steps
    status = cca.last_status()
    # end to end: the new tokens come from pinned host memory, the outputs go back to it
    oh = torch.empty(B, sh.d_model, dtype=torch.bfloat16).pin_memory()
    xd = torch.empty(B, sh.d_model, dtype=torch.bfloat16, device=out.device)
    n_e2e = min(args.steps, 10)
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    g0.record()
    for i in range(n_e2e):
        xd.copy_(xs_host[it[0]], non_blocking=True)
        step(xd)
        oh.copy_(out, non_blocking=True)
        torch.cuda.synchronize()
    g1.record()
    barrier()
    e2e_ms = max_over_ranks(g0.elapsed_time(g1) / n_e2e, dist, "cuda")
    by = decode_bytes(sh, B, ctx)
    peak, peak_kind = hbm_peak()
    attn_gbs = by["cache"] / (attn_ms * 1e-3) / 1e9
    line = {
        "metric": "CCGQA decode throughput at 16k context (new tokens / device time)", "value": world * B / (ms_step * 1e-3),
        "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "step": "decode", "B": B, "context": ctx, "d_model": sh.d_model,
                   "n_q_heads": sh.n_q_heads, "n_kv_heads": sh.n_kv_heads, "head_dim": sh.head_dim, "k_seq": sh.k_seq,
                   "k_ch": sh.k_ch, "parallelism": f"replicas x{world}" if world > 1 else "1 gpu",
                   "l2": f"no flush: each step streams {by['cache'] / 1e6:.0f} MB of cache, more than the 126 MB L2"},
        "clocks": clocks,
        "e2e": {"value": world * B / (e2e_ms * 1e-3), "unit": "tokens/s",
                "h2d_bytes_per_step": B * sh.d_model * 2, "d2h_bytes_per_step": B * sh.d_model * 2,
                "ms_per_step": e2e_ms},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "decode attention over the latent cache", "achieved": attn_gbs, "peak": peak,
                     "unit": "GB/s", "frac": attn_gbs / peak, "peak_kind": peak_kind, "ms_per_launch": attn_ms,
                     "bytes_per_launch": by["cache"], "traffic": dram_traffic("decode_attention", args.workload)},
        "step_gbs": by["total"] / (ms_step * 1e-3) / 1e9, "step_bytes": by,
        "device_status": status,
    }
    if rank == 0 and world == 1 and not args.no_cpu:
        v, dt, sample = oracle_decode_sample(sh, ctx)
        line["cpu_baseline"] = {"value": v, "unit": "tokens/s", "cores": torch.get_num_threads(), "kind": "oracle",
                                "sample": sample, "seconds": dt}
    if rank == 0:
        print(json.dumps(line), flush=True)
    cca.close()
    if dist is not None:
        dist.destroy_process_group()


def oracle_decode_sample(sh, ctx):
    """The oracle's decode step, as it stands, for one sequence with `ctx` cached tokens (the prefill that fills
    the cache is not timed)."""
    from oracle import cca_oracle as O
    n_new = 2048
    s1 = sh.replace(B=1, S=ctx + n_new)
    t = synth.make_inputs(s1, want_dout=False)
    cfg = O.OracleConfig(sh.d_model, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.k_seq, sh.k_ch, sh.causal, sh.flags,
                         sh.rope_base)
    I = O.pre_attention(cfg, t, t["x"][:, :ctx])
    st = O.decode_state_after_prefill(cfg, I, ctx)
    t0 = time.perf_counter()
    n = 0
    while n < n_new and (n < 4 or time.perf_counter() - t0 < 10.0):
        O.decode_step(cfg, t, st, t["x"][:, ctx + n])
        n += 1
    dt = time.perf_counter() - t0
    return n / dt, dt, f"{n} consecutive tokens of one sequence with {ctx} cached tokens"


def fwd_bwd_same_shape(sh, args, local_rank):
    """The headline shape with the backward as well (the metric asks for forward and forward + backward at
    16k context).  Reported beside the forward-only line; not part of the timed region above."""
    from paper_2510_04476_b200.binding import CCA, stack_down_projection
    t = synth.make_inputs(sh, want_dout=True)
    dev = stack_down_projection({k: v.cuda(local_rank).contiguous() for k, v in t.items()})
    cca = CCA.from_shape(sh, device=local_rank)
    cca.set_impl(args.kernels)
    ws = cca.alloc_workspace(sh.B, sh.S, True)
    out = torch.empty_like(dev["x"])
    n = min(args.steps, 10)
    for _ in range(3):
        cca.forward(dev, dev["x"], ws, out)
        cca.backward(dev, dev["x"], dev["d_out"], ws)
    torch.cuda.synchronize()
    e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    fwd = bwd = 0.0
    for _ in range(n):
        e0.record()
        cca.forward(dev, dev["x"], ws, out)
        e1.record()
        cca.backward(dev, dev["x"], dev["d_out"], ws)
        e2.record()
        torch.cuda.synchronize()
        fwd += e0.elapsed_time(e1)
        bwd += e1.elapsed_time(e2)
    status = cca.last_status()
    cca.close()
    fl = flops_of(sh, True)
    ms = (fwd + bwd) / n
    return {"ms_per_step": ms, "forward_ms": fwd / n, "backward_ms": bwd / n, "tflops": fl["total"] / (ms * 1e-3) / 1e12,
            "pct_of_nominal_bf16_peak": 100.0 * fl["total"] / (ms * 1e-3) / 1e12 / NOMINAL_BF16_TFLOPS,
            "device_status": status}


def mha_compare(sh, args, cca_ms, cca_attn_ms, local_rank):
    """Same kernels configured as plain multi-head attention of equal d_model (no compression, no
    latent transforms): reproduces the paper's speed-up ratio on this machine."""
    from paper_2510_04476_b200.binding import CCA
    m = synth.mha_like(sh)
    t = synth.make_inputs(m, want_dout=False)
    dev = {k: v.cuda(local_rank).contiguous() for k, v in t.items()}
    cca = CCA.from_shape(m, device=local_rank)
    cca.set_impl(args.kernels)
    ws = cca.alloc_workspace(m.B, m.S, False)
    out = torch.empty_like(dev["x"])
    n = min(args.steps, 5)
    for _ in range(2):
        cca.forward(dev, dev["x"], ws, out)
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
    for a, b in ev:
        a.record(); b.record()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(n):
        cca.set_attention_events(*ev[i])
        cca.forward(dev, dev["x"], ws, out)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / n
    attn = sum(a.elapsed_time(b) for a, b in ev) / n
    cca.close()
    return {"config": f"{m.n_q_heads} heads x {m.head_dim}, C=1, transforms off", "block_ms": ms, "attention_ms": attn,
            "block_speedup_of_ccgqa": ms / cca_ms, "attention_speedup_of_ccgqa": attn / cca_attn_ms}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3_prefill16k", choices=sorted(synth.CONFIGS) + sorted(DECODE_WORKLOADS))
    ap.add_argument("--kernels", type=int, default=1, help="0 = SIMT kernels only, 1 = tcgen05 kernels where available")
    ap.add_argument("--backward", action="store_true", help="time forward + backward on a forward-only workload too")
    ap.add_argument("--no-mha", action="store_true")
    ap.add_argument("--sustain", type=float, default=3.0,
                    help="seconds of back-to-back steps for the sustained (power-capped) figure; 0 = skip")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference" and args.workload in DECODE_WORKLOADS:
        raise SystemExit("the reference arm times the prefill workloads; the decode line carries its own cpu_baseline")
    if args.impl == "reference":
        run_reference(args, rank, world)
    elif args.workload in DECODE_WORKLOADS:
        run_decode(args, rank, world, local_rank)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
