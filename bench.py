#!/usr/bin/env python
"""Benchmark of the LAGA per-rank attention hot path on B200.

One "step" is one pass of the whole hot path over one batch of synthetic input: laga_fwd followed
by laga_bwd on the DeepSeek-V3 per-rank shard (h=16 heads, S=16384, causal, bf16) -- Algorithm 1
steps 4-5 of the paper and the backward of its Section 5.2.  The metric is algorithmic TFLOP/s
(causal pairs only, recomputation not counted) of forward+backward.

  python bench.py [--gpus N --steps K --warmup W]        the CUDA path (rank r runs its own shard)
  python bench.py --impl reference [...]                  the fp64 CPU oracle on a bounded sample

Under torchrun (N > 1) every rank is one sequence-parallel rank's shard: the path has no collective
between ranks, so this is weak scaling over independent replicas; time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2607_17644_b200.inputs import CONFIGS, CONFIG_SEEDS, LagaShape, make_inputs  # noqa: E402

METRIC = "laga_attention_block_fwd_bwd_tflops"
UNIT = "TFLOP/s"
WORKLOAD = "c2"
KERNELS_PER_STEP = 9   # fwd: up_project, attn_fwd; bwd: up_project, delta, dkv, dq, dkpe_convert, dckv, dw
# DRAM bytes (read + write) per launch of attn_bwd_dkv, from the ncu capture summarised in
# profiles/ncu_full_c3_sp8_kernels.txt (S=8192, h=16: 155.5 MB read + 43.3 MB written), expressed per
# (token, head).  The kernel's traffic is its inputs and outputs once each (K/V, Q and dO tiles are
# re-read from L2, not DRAM), so it grows in proportion to S*h and is scaled that way to the workload.
DKV_DRAM_BYTES_PER_TOKEN_HEAD = (155.500800e6 + 43.290624e6) / (8192 * 16)


def flops(sh: LagaShape):
    """Algorithmic FLOPs: causal pairs only; the recomputed up-projection and P are not counted."""
    pairs = sh.S * (sh.S + 1) // 2
    f_attn_fwd = 2 * sh.h * pairs * (sh.d_qk + sh.d_v)
    f_up = 2 * sh.S * sh.d_c * sh.n_cols
    f_attn_bwd = 2 * sh.h * pairs * (3 * sh.d_qk + 2 * sh.d_v)
    return {"fwd": f_attn_fwd + f_up, "bwd": f_attn_bwd + 2 * f_up, "attn_bwd_dkv": 2 * sh.h * pairs * (2 * sh.d_qk + 2 * sh.d_v)}


def activation_memory(sh: LagaShape, ws_fwd: int, ws_bwd: int, allocated_in_step: int):
    """Bytes alive at the backward's peak beyond the inputs (q, c_kv, k_pe, W, dO) and the gradient
    outputs, for this path and for the explicit form with a fused attention kernel (per-head
    K[S,h,192] and V[S,h,128] saved in bf16 by the forward; dK, dV in bf16; delta in fp32)."""
    tok_head = sh.S * sh.h
    saved = tok_head * sh.d_v * 2 + tok_head * 4                    # out bf16 + lse fp32 (both forms)
    ours = saved + max(ws_fwd, ws_bwd) + allocated_in_step
    explicit = saved + tok_head * (sh.d_qk + sh.d_v) * 2 * 2 + tok_head * 4
    return {"laga_bytes": ours, "explicit_form_bytes": explicit, "ratio": ours / explicit,
            "workspace_bytes": {"fwd": ws_fwd, "bwd": ws_bwd}, "allocated_inside_step": allocated_in_step}


def compare_eager(sh: LagaShape, inputs, cuda_results, laga_ms: float, laga_peak_bytes: dict, reps: int = 2):
    """Time the explicit (B1) and absorbed (B2) forms of the same block written in eager PyTorch ops
    with the full S x S score matrix, as the paper's memory study ran them (Section 6, memory table),
    and record what each keeps alive beyond its inputs.  Library kernels, comparison only."""
    from paper_2607_17644_b200 import eager_forms
    q, c_kv, k_pe, w, dout = inputs
    res = {"how": "eager PyTorch bf16 (cuBLAS + ATen) with autograd, full S x S scores per head; peak_bytes = "
                  "torch.cuda.max_memory_allocated above the inputs, over one forward+backward",
           "laga_cuda": {"ms_per_step": laga_ms, "peak_bytes": laga_peak_bytes["laga_bytes"]}}
    names = ("out", "dq", "dc_kv", "dk_pe", "dw_kv_b")
    for name, form in (("explicit", eager_forms.explicit_form), ("absorbed", eager_forms.absorbed_form)):
        torch.cuda.synchronize()
        torch.cuda.empty_cache()
        got = eager_forms.run_form(form, q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale)   # warm-up + check
        err = {n: float((g.float() - r.float()).abs().max()) for n, g, r in zip(names, got, cuda_results)}
        del got
        torch.cuda.synchronize()
        torch.cuda.empty_cache()
        base = torch.cuda.memory_allocated()
        torch.cuda.reset_peak_memory_stats()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            eager_forms.run_form(form, q, c_kv, k_pe, w, dout, sh.d_v, sh.softmax_scale)
        e1.record()
        torch.cuda.synchronize()
        res[name] = {"ms_per_step": e0.elapsed_time(e1) / reps, "peak_bytes": torch.cuda.max_memory_allocated() - base,
                     "max_abs_diff_vs_laga_cuda": err}
    res["absorbed_minus_explicit_bytes"] = res["absorbed"]["peak_bytes"] - res["explicit"]["peak_bytes"]
    return res


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p["bf16_tflops_sustained"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while a region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, sm_max, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                sm_max.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(sm_max) if sm_max else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def dist_setup(n_gpus: int):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group(backend="nccl", device_id=torch.device("cuda", local_rank))
    else:
        torch.cuda.set_device(0)
    if world != n_gpus and rank == 0:
        print(f"[bench] note: --gpus {n_gpus} but WORLD_SIZE={world}; using WORLD_SIZE", file=sys.stderr)
    return world, rank, local_rank


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    torch.cuda.synchronize()


def max_over_ranks(value: float, world: int, device: str = "cuda") -> float:
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([value], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())
    return value


def run_cuda(args):
    from paper_2607_17644_b200 import laga
    laga.lib()
    world, rank, local_rank = dist_setup(args.gpus)
    dev = torch.device("cuda", torch.cuda.current_device())
    sh = CONFIGS[args.workload]
    fl = flops(sh)
    # each rank is one SP rank's shard of the same layer: its own draw of the shard's tensors
    host = make_inputs(sh, CONFIG_SEEDS[args.workload] + 7919 * rank, pin_memory=True)
    q, c_kv, k_pe, w, dout = (t.to(dev, non_blocking=True) for t in host)
    out = torch.empty(sh.S, sh.h, sh.d_v, dtype=torch.bfloat16, device=dev)
    lse = torch.empty(sh.S, sh.h, dtype=torch.float32, device=dev)
    dq, dc_kv, dk_pe = torch.empty_like(q), torch.empty_like(c_kv), torch.empty_like(k_pe)
    dw = torch.empty(sh.d_c, sh.n_cols, dtype=torch.float32, device=dev)
    ws_f = laga.alloc_workspace(laga.fwd_workspace_bytes(sh.S, sh.h), dev)
    ws_b = laga.alloc_workspace(laga.bwd_workspace_bytes(sh.S, sh.h), dev)
    torch.cuda.synchronize()
    torch.cuda.reset_peak_memory_stats()
    base_mem = torch.cuda.memory_allocated()

    def step():
        laga.fwd(q, c_kv, k_pe, w, out=out, lse=lse, workspace=ws_f)
        laga.bwd(q, c_kv, k_pe, w, out, lse, dout, dq=dq, dc_kv=dc_kv, dk_pe=dk_pe, dw_kv_b=dw, workspace=ws_b)

    def fwd_only():
        laga.fwd(q, c_kv, k_pe, w, out=out, lse=lse, workspace=ws_f)

    for _ in range(max(args.warmup, 3)):
        step()
    laga.check_status(ws_f, where="warm-up laga_fwd")
    laga.check_status(ws_b, where="warm-up laga_bwd")

    # ---- timed region: exactly K steps, device-timed, events around the dominant kernel -------------
    K = args.steps
    dom = "attn_bwd_dkv"
    k_starts = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
    k_stops = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
    for e in k_starts + k_stops:
        e.record()
    laga.profile_kernel(dom, k_starts, k_stops)
    d_starts = [torch.cuda.Event(enable_timing=True) for _ in range(K)]     # the one HBM-bound kernel of weight: delta
    d_stops = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
    for e in d_starts + d_stops:
        e.record()
    laga.profile_kernel("bwd_delta", d_starts, d_stops)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    barrier(world)
    ev0.record()
    for _ in range(K):
        step()
    ev1.record()
    barrier(world)
    clocks = sampler.stop()
    laga.profile_kernel(dom)
    laga.profile_kernel("bwd_delta")
    delta_ms = statistics.mean(a.elapsed_time(b) for a, b in zip(d_starts, d_stops))
    s_pad = (sh.S + 127) // 128 * 128
    delta_bytes = 2 * sh.S * sh.h * sh.d_v * 2 + sh.S * sh.h * 4 + 2 * s_pad * sh.h * 4   # O, dO, LSE in; two statistics out
    total_ms = max_over_ranks(ev0.elapsed_time(ev1), world)
    ms_per_step = total_ms / K
    dom_ms = statistics.mean(a.elapsed_time(b) for a, b in zip(k_starts, k_stops))
    laga.check_status(ws_f, where="timed laga_fwd")
    laga.check_status(ws_b, where="timed laga_bwd")

    # ---- forward alone (reported beside the headline) ---------------------------------------------
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    f0.record()
    for _ in range(K):
        fwd_only()
    f1.record()
    barrier(world)
    fwd_ms = max_over_ranks(f0.elapsed_time(f1), world) / K
    peak_act = torch.cuda.max_memory_allocated() - base_mem   # nothing is allocated inside a step

    # ---- end to end: pinned host buffers in, results out, every step ------------------------------
    host_out = [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in (out, lse, dq, dc_kv, dk_pe, dw)]
    h2d = sum(t.numel() * t.element_size() for t in host)
    d2h = sum(t.numel() * t.element_size() for t in host_out)

    def e2e_step():
        for d, s in zip((q, c_kv, k_pe, w, dout), host):
            d.copy_(s, non_blocking=True)
        step()
        for d, s in zip(host_out, (out, lse, dq, dc_kv, dk_pe, dw)):
            d.copy_(s, non_blocking=True)

    Ke = max(3, min(K, 10))
    for _ in range(2):
        e2e_step()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    g0.record()
    for _ in range(Ke):
        e2e_step()
    g1.record()
    barrier(world)
    e2e_serial_ms = max_over_ranks(g0.elapsed_time(g1), world) / Ke

    # The same, as a training loop would run it: the copy-in of step i+1 and the copy-out of step i-1
    # overlap the kernels of step i (three streams, two sets of device and pinned host buffers).  Every
    # step still moves all of its inputs from pinned host memory and all of its results back.
    in_dev = [(q, c_kv, k_pe, w, dout), tuple(torch.empty_like(t) for t in (q, c_kv, k_pe, w, dout))]
    out_dev = [(out, lse, dq, dc_kv, dk_pe, dw), tuple(torch.empty_like(t) for t in (out, lse, dq, dc_kv, dk_pe, dw))]
    host_outs = [host_out, [torch.empty(t.shape, dtype=t.dtype, pin_memory=True) for t in host_out]]
    s_in, s_c, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()

    def pipelined(n_steps, first_event=None, last_event=None):
        in_ready = [None, None]
        compute_done = [None, None]
        out_done = [None, None]
        for i in range(n_steps):
            b = i & 1
            with torch.cuda.stream(s_in):
                if i == 0 and first_event is not None:
                    first_event.record()
                if compute_done[b] is not None:
                    s_in.wait_event(compute_done[b])          # step i-2 has finished reading these inputs
                for d, s in zip(in_dev[b], host):
                    d.copy_(s, non_blocking=True)
                in_ready[b] = torch.cuda.Event()
                in_ready[b].record()
            with torch.cuda.stream(s_c):
                s_c.wait_event(in_ready[b])
                if out_done[b] is not None:
                    s_c.wait_event(out_done[b])               # step i-2's results have left these buffers
                qi, ci, ki, wi, doi = in_dev[b]
                oo, ll, dqo, dco, dko, dwo = out_dev[b]
                laga.fwd(qi, ci, ki, wi, out=oo, lse=ll, workspace=ws_f)
                laga.bwd(qi, ci, ki, wi, oo, ll, doi, dq=dqo, dc_kv=dco, dk_pe=dko, dw_kv_b=dwo, workspace=ws_b)
                compute_done[b] = torch.cuda.Event()
                compute_done[b].record()
            with torch.cuda.stream(s_out):
                s_out.wait_event(compute_done[b])
                for d, s in zip(host_outs[b], out_dev[b]):
                    d.copy_(s, non_blocking=True)
                out_done[b] = torch.cuda.Event()
                out_done[b].record()
                if i == n_steps - 1 and last_event is not None:
                    last_event.record()

    torch.cuda.synchronize()
    pipelined(3)
    torch.cuda.synchronize()
    Kp = max(6, min(2 * K, 20))
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    pipelined(Kp, p0, p1)
    barrier(world)
    e2e_ms = max_over_ranks(p0.elapsed_time(p1), world) / Kp     # includes the pipeline's fill and drain
    laga.check_status(ws_f, where="e2e laga_fwd")
    laga.check_status(ws_b, where="e2e laga_bwd")
    assert math.isfinite(float(host_outs[1][1].sum())), "LSE read back from the device is not finite"
    assert math.isfinite(float(host_out[1].sum())), "LSE read back from the device is not finite"

    peaks = measured_peaks()
    total_flops = fl["fwd"] + fl["bwd"]
    value = world * total_flops / (ms_per_step * 1e-3) / 1e12
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{args.workload}: DeepSeek-V3 per-rank shard, S={sh.S}, h_local={sh.h}, d_c=512, "
                               "d_nope=128, d_rope=64, d_v=128, causal, forward+backward", "S": sh.S, "h_local": sh.h,
                   "parallelism": f"{world} independent SP-rank shards (no collective on this path)",
                   "l2_policy": f"inputs larger than L2 ({h2d / 1e6:.0f} MB of inputs plus "
                                f"{ws_b.numel() / 1e6:.0f} MB of K/V and dK/dV per step vs 126 MB L2)",
                   "flops_per_step": total_flops},
        "fwd_ms": fwd_ms, "fwd_tflops": world * fl["fwd"] / (fwd_ms * 1e-3) / 1e12,
        "frac_of_bf16_peak": value / world / peaks["bf16_tflops"],
        "frac_of_bf16_sustained": value / world / peaks["bf16_tflops_sustained"],
        "activation_memory": activation_memory(sh, ws_f.numel(), ws_b.numel(), int(peak_act)),
        "clocks": clocks,
        "e2e": {"value": world * total_flops / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": Kp,
                "how": "public API (laga.fwd + laga.bwd) with pinned host buffers; copy-in of step i+1 and copy-out of "
                       "step i-1 overlap the kernels of step i (3 streams, double buffers); fill and drain included",
                "serial_ms_per_step": e2e_serial_ms,
                "serial_value": world * total_flops / (e2e_serial_ms * 1e-3) / 1e12},
        "gpu_launches": KERNELS_PER_STEP * K,
        "roofline": {"bound": "tensor", "kernel": dom, "achieved": fl["attn_bwd_dkv"] / (dom_ms * 1e-3) / 1e12,
                     "peak": peaks["bf16_tflops_sustained"], "unit": UNIT,
                     "frac": fl["attn_bwd_dkv"] / (dom_ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                     "peak_source": peaks["source"] + " sustained cuBLAS bf16 (kernel timed inside a long step)",
                     "kernel_ms": dom_ms, "flops_per_launch": fl["attn_bwd_dkv"],
                     "traffic": DKV_DRAM_BYTES_PER_TOKEN_HEAD * sh.S * sh.h,
                     "traffic_note": "bytes per launch, ncu dram read+write at S=8192,h=16 scaled by S*h"},
    }
    if args.compare_eager and world == 1:
        del in_dev, out_dev, host_outs
        line["eager_forms"] = compare_eager(sh, (q, c_kv, k_pe, w, dout), (out, dq, dc_kv, dk_pe, dw),
                                            laga_ms=ms_per_step, laga_peak_bytes=line["activation_memory"])
    line["hbm_kernels"] = {"bwd_delta": {"kernel_ms": delta_ms, "bytes_per_launch": delta_bytes,
                                         "achieved": delta_bytes / (delta_ms * 1e-3) / 1e9, "unit": "GB/s",
                                         "peak": peaks["hbm_gbs"], "frac": delta_bytes / (delta_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                         "share_of_step": delta_ms / ms_per_step}}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(sample_tokens=args.cpu_sample_tokens)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def oracle_sample(sample_tokens: int):
    """The bounded sample both CPU legs run: head 0 of the c2 shard restricted to its first
    `sample_tokens` tokens (a causal prefix is a self-contained sub-problem of the same workload)."""
    sh = CONFIGS[WORKLOAD]
    q, c_kv, k_pe, w, dout = make_inputs(sh, CONFIG_SEEDS[WORKLOAD])
    n = sample_tokens
    sub = LagaShape(S=n, h=1)
    tensors = (q[:n, :1].contiguous(), c_kv[:n].contiguous(), k_pe[:n].contiguous(), w[:, :256].contiguous(),
               dout[:n, :1].contiguous())
    return sub, tensors


def cpu_baseline(sample_tokens: int):
    import oracle
    sub, (q, c_kv, k_pe, w, dout) = oracle_sample(sample_tokens)
    fl = flops(sub)
    t0 = time.perf_counter()
    oracle.bwd(q, c_kv, k_pe, w, dout, sub.d_v, sub.softmax_scale, causal=True)   # computes forward and backward
    dt = time.perf_counter() - t0
    return {"value": (fl["fwd"] + fl["bwd"]) / dt / 1e12, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "seconds": dt, "sample": f"head 0, first {sample_tokens} tokens of the c2 shard (causal prefix), "
                                      "forward+backward in fp64, one pass"}


def run_reference(args):
    """Reference arm: the fp64 CPU oracle as it stands, on the host cores; each step is one pass over a
    bounded sample of the c2 workload.  Rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    oracle.build()
    sub, (q, c_kv, k_pe, w, dout) = oracle_sample(args.ref_sample_tokens)
    fl = flops(sub)
    total = fl["fwd"] + fl["bwd"]

    def step():
        oracle.bwd(q, c_kv, k_pe, w, dout, sub.d_v, sub.softmax_scale, causal=True)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    value = total / dt / 1e12
    sample = (f"head 0, first {args.ref_sample_tokens} tokens of the c2 shard (causal prefix), forward+backward "
              "in fp64 per step")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "c2: DeepSeek-V3 per-rank shard, S=16384, h_local=16 (bounded sample per step)",
                       "sample": sample, "flops_per_step": total},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["cuda", "reference"], default="cuda")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing leg")
    ap.add_argument("--workload", choices=sorted(CONFIGS), default=WORKLOAD,
                    help="benchmark configuration (default c2, the headline; others are for profiling)")
    ap.add_argument("--compare-eager", action="store_true",
                    help="also time the explicit and absorbed forms in eager PyTorch (N=1; tens of GB at c2)")
    ap.add_argument("--cpu-sample-tokens", type=int, default=16384,
                    help="tokens of head 0 the cpu_baseline leg runs (16384 = the whole head: ~10 s on 16 cores)")
    ap.add_argument("--ref-sample-tokens", type=int, default=2048,
                    help="tokens of head 0 per step in --impl reference (2048: well under a second per step)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py: no CUDA device; the CUDA path has no fallback")
        run_cuda(args)


if __name__ == "__main__":
    main()
