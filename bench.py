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
# DRAM bytes (read + write) of ONE launch of attn_bwd_dkv at the headline workload (c2), from the ncu
# capture summarised in profiles/ncu_dram_c2_attn_bwd_dkv.txt.  For other workloads the figure is scaled
# by S*h (the kernel reads its inputs and writes its outputs once; tiles are re-read from L2, not DRAM)
# and flagged as scaled.
DKV_DRAM_BYTES_C2 = 337137408 + 112096000          # dram__bytes_read.sum + dram__bytes_write.sum of one launch
DKV_DRAM_C2_TOKEN_HEADS = 16384 * 16


def flops(sh: LagaShape):
    """Algorithmic FLOPs: causal pairs only; the recomputed up-projection and P are not counted."""
    pairs = sh.S * (sh.S + 1) // 2
    f_attn_fwd = 2 * sh.h * pairs * (sh.d_qk + sh.d_v)
    f_up = 2 * sh.S * sh.d_c * sh.n_cols
    f_attn_bwd = 2 * sh.h * pairs * (3 * sh.d_qk + 2 * sh.d_v)
    return {"fwd": f_attn_fwd + f_up, "bwd": f_attn_bwd + 2 * f_up, "attn_fwd": f_attn_fwd, "attn_bwd": f_attn_bwd,
            # executed by each backward kernel (S and dP are recomputed in both): dkv = S^T, dP^T, dV, dK; dq = S, dP, dQ
            "attn_bwd_dkv": 2 * sh.h * pairs * (2 * sh.d_qk + 2 * sh.d_v),
            "attn_bwd_dq": 2 * sh.h * pairs * (2 * sh.d_qk + sh.d_v)}


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
    with the full S x S score matrix, as the paper's memory study ran them (Section 4, activation-memory table),
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
    """Samples SM clock and throttle reasons of one GPU with nvidia-smi while a region runs.  The period
    is 20 ms; the timed region of the default run lasts about 0.1 s, so this is a coarse record (and
    nvidia-smi's clock reading lags the power controller): the clock the kernels really ran at is taken
    inside the kernels themselves (laga_query_kernel_clocks) and reported beside it."""
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
                                          "--format=csv,noheader,nounits", "-lms", "20"],
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
        sm, sm_max, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                sm_max.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(sm_max) if sm_max else None,
                "samples": len(sm), "power_w_max": max(power) if power else None, "reasons": sorted(reasons)}


def self_launch(n_gpus: int) -> int:
    """`python bench.py --gpus N` without a launcher: start N ranks of this script under torch.distributed.run
    on one node (127.0.0.1, a free port) and hand back its exit code.  Rank 0 of that job prints the line."""
    import socket
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.run(cmd).returncode


def dist_setup(n_gpus: int, backend: str = "nccl"):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if backend == "nccl":
        torch.cuda.set_device(local_rank if world > 1 else 0)
    if world > 1:
        import torch.distributed as dist
        if backend == "nccl":
            dist.init_process_group(backend="nccl", device_id=torch.device("cuda", local_rank))
        else:
            dist.init_process_group(backend=backend)
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


def run_dry(args):
    """The launch and reduction plumbing of the N-rank run with no GPU work (gloo): every rank contributes a
    made-up step time and rank 0 prints the line's skeleton.  Used by the CPU test of the launcher."""
    world, rank, _ = dist_setup(args.gpus, backend="gloo")
    fake_ms = 10.0 + 5.0 * rank
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
    total_ms = max_over_ranks(fake_ms, world, device="cpu")
    if rank == 0:
        print(json.dumps({"impl": "dry-run", "n_gpus": world, "ms_per_step": total_ms, "scaling": "weak"}), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_c4(args):
    """Benchmark configuration 4: the absorbed form (Section 3.2, baseline B2) on configuration 2's inputs,
    forward, as hand-written kernels (laga_absorbed_fwd), beside the LAGA forward on the same inputs: time,
    useful TFLOP/s (the explicit form's 640 FLOP per causal pair and head plus one up-projection -- the work
    the result needs), executed TFLOP/s (what the absorbed kernels actually run) and the scratch each form
    keeps alive.  One GPU; the absorbed form has no backward here."""
    from paper_2607_17644_b200 import laga
    laga.lib()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    sh = CONFIGS["c4"]
    fl = flops(sh)
    pairs = sh.S * (sh.S + 1) // 2
    q, c_kv, k_pe, w, _ = (t.to(dev) if t is not None else None for t in make_inputs(sh, CONFIG_SEEDS["c4"], with_dout=False))
    out = torch.empty(sh.S, sh.h, sh.d_v, dtype=torch.bfloat16, device=dev)
    lse = torch.empty(sh.S, sh.h, dtype=torch.float32, device=dev)
    out_l, lse_l = torch.empty_like(out), torch.empty_like(lse)
    ws_a = laga.alloc_workspace(laga.absorbed_fwd_workspace_bytes(sh.S, sh.h), dev)
    ws_l = laga.alloc_workspace(laga.fwd_workspace_bytes(sh.S, sh.h), dev)
    K, W = args.steps, max(args.warmup, 3)

    def timed(fn):
        for _ in range(W):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(K):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / K

    abs_ms = timed(lambda: laga.absorbed_fwd(q, c_kv, k_pe, w, out=out, lse=lse, workspace=ws_a))
    laga_ms = timed(lambda: laga.fwd(q, c_kv, k_pe, w, out=out_l, lse=lse_l, workspace=ws_l))
    laga.check_status(ws_a, where="laga_absorbed_fwd")
    laga.check_status(ws_l, where="laga_fwd")
    executed = 2 * sh.h * pairs * (2 * (sh.d_c + sh.d_rope) + sh.d_c) + 2 * 2 * sh.S * sh.h * sh.d_nope * sh.d_c   # both halves' scores + P V, two batched GEMMs
    nominal = 2 * sh.h * pairs * ((sh.d_c + sh.d_rope) + sh.d_c) + 2 * 2 * sh.S * sh.h * sh.d_nope * sh.d_c
    peaks = measured_peaks()
    line = {"metric": "absorbed_form_fwd_useful_tflops", "value": fl["fwd"] / (abs_ms * 1e-3) / 1e12, "unit": UNIT,
            "n_gpus": 1, "steps": K, "warmup": W, "ms_per_step": abs_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "c4: absorbed form on c2's inputs (S=16384, h_local=16, causal), forward",
                       "l2_policy": "inputs and scratch larger than L2 (q_abs and the latent accumulator alone are 537 MB)"},
            "absorbed": {"ms": abs_ms, "useful_tflops": fl["fwd"] / (abs_ms * 1e-3) / 1e12,
                         "executed_tflops": executed / (abs_ms * 1e-3) / 1e12,
                         "executed_flops": executed, "nominal_flops_of_the_form": nominal, "useful_flops": fl["fwd"],
                         "executed_frac_of_burst_peak": executed / (abs_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                         "scratch_bytes": ws_a.numel()},
            "laga": {"ms": laga_ms, "tflops": fl["fwd"] / (laga_ms * 1e-3) / 1e12, "scratch_bytes": ws_l.numel()},
            "absorbed_over_laga": {"time": abs_ms / laga_ms, "scratch": ws_a.numel() / ws_l.numel(),
                                   "extra_scratch_bytes": ws_a.numel() - ws_l.numel()},
            "max_abs_diff_between_forms": {"out": float((out.float() - out_l.float()).abs().max()),
                                           "lse": float((lse - lse_l).abs().max())},
            "gpu_launches": 3 * K}
    print(json.dumps(line), flush=True)


PACKED_MIXES = {
    # 16384 tokens of a 16-head shard each, packed in different ways (lengths in tokens)
    "1x16384": [16384],
    "4x4096": [4096] * 4,
    "ragged_8": [8192, 4096, 2048, 1024, 512, 256, 128, 128],
    "64x256": [256] * 64,
}


SWEEP_LENGTHS = (1024, 2048, 4096, 8192, 16384, 32768, 65536)


def run_sweep(args):
    """Sequence-length sweep at the headline head count (h_local = 16): forward and forward+backward of one
    rank's shard from 1 K to 64 K tokens (the paper evaluates 4 K, 8 K and 16 K; the longer ones show where the
    path settles once per-item and per-launch costs are amortised).  Device-timed, no per-kernel events."""
    from paper_2607_17644_b200 import laga
    laga.lib()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    peaks = measured_peaks()
    K, W = args.steps, max(args.warmup, 3)
    rows = {}
    for S in SWEEP_LENGTHS:
        sh = LagaShape(S=S, h=16)
        q, c_kv, k_pe, w, dout = (t.to(dev) for t in make_inputs(sh, 5000 + S))
        out = torch.empty(sh.S, sh.h, sh.d_v, dtype=torch.bfloat16, device=dev)
        lse = torch.empty(sh.S, sh.h, dtype=torch.float32, device=dev)
        dq, dc_kv, dk_pe = torch.empty_like(q), torch.empty_like(c_kv), torch.empty_like(k_pe)
        dw = torch.empty(sh.d_c, sh.n_cols, dtype=torch.float32, device=dev)
        ws_f = laga.alloc_workspace(laga.fwd_workspace_bytes(sh.S, sh.h), dev)
        ws_b = laga.alloc_workspace(laga.bwd_workspace_bytes(sh.S, sh.h), dev)

        def fwd_only():
            laga.fwd(q, c_kv, k_pe, w, out=out, lse=lse, workspace=ws_f)

        def step():
            fwd_only()
            laga.bwd(q, c_kv, k_pe, w, out, lse, dout, dq=dq, dc_kv=dc_kv, dk_pe=dk_pe, dw_kv_b=dw, workspace=ws_b)

        def timed(fn):
            for _ in range(W):
                fn()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(K):
                fn()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / K

        step_ms, fwd_ms = timed(step), timed(fwd_only)
        laga.check_status(ws_f, where=f"sweep S={S} laga_fwd")
        laga.check_status(ws_b, where=f"sweep S={S} laga_bwd")
        fl = flops(sh)
        total = fl["fwd"] + fl["bwd"]
        rows[str(S)] = {"S": S, "h_local": 16, "ms_per_step": step_ms, "tflops": total / (step_ms * 1e-3) / 1e12,
                        "frac_of_bf16_peak": total / (step_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                        "fwd_ms": fwd_ms, "fwd_tflops": fl["fwd"] / (fwd_ms * 1e-3) / 1e12, "flops_per_step": total}
        del q, c_kv, k_pe, w, dout, out, lse, dq, dc_kv, dk_pe, dw, ws_f, ws_b
        torch.cuda.empty_cache()
    head = rows["16384"]
    line = {"metric": METRIC, "value": head["tflops"], "unit": UNIT, "n_gpus": 1, "steps": K, "warmup": W,
            "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "sweep: one rank's DeepSeek-V3 shard, h_local=16, causal, forward+backward, S from 1024 to 65536 "
                                   "(the line's value is the S=16384 row)",
                       "l2_policy": "inputs and workspaces larger than L2 from S=8192 on; the shorter rows fit in L2 (as they would "
                                    "between the layers of a model this small)"},
            "peak_source": peaks["source"] + " cuBLAS bf16, burst", "sweep": rows, "gpu_launches": 9 * K}
    print(json.dumps(line), flush=True)


def run_packed(args):
    """Batches and variable-length sequences (laga_fwd_varlen / laga_bwd_varlen): the same 16384 tokens of a
    16-head shard packed as one sequence, as a batch of four, as a ragged mix and as 64 short sequences.  Each
    mix is timed through one packed call per direction and, for comparison, as a loop of single-sequence calls
    over the same rows.  FLOPs are algorithmic: causal pairs inside each sequence plus the token-wise GEMMs."""
    from paper_2607_17644_b200 import laga
    laga.lib()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    sh = CONFIGS["c2"]
    q, c_kv, k_pe, w, dout = (t.to(dev) for t in make_inputs(sh, CONFIG_SEEDS["c2"]))
    out = torch.empty(sh.S, sh.h, sh.d_v, dtype=torch.bfloat16, device=dev)
    lse = torch.empty(sh.S, sh.h, dtype=torch.float32, device=dev)
    dq, dc_kv, dk_pe = torch.empty_like(q), torch.empty_like(c_kv), torch.empty_like(k_pe)
    dw = torch.empty(sh.d_c, sh.n_cols, dtype=torch.float32, device=dev)
    K, W = args.steps, max(args.warmup, 3)

    def timed(fn):
        for _ in range(W):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(K):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / K

    results = {}
    for name, lengths in PACKED_MIXES.items():
        cu = [0]
        for n in lengths:
            cu.append(cu[-1] + n)
        pairs = sum(n * (n + 1) // 2 for n in lengths)
        total = 2 * sh.h * pairs * (sh.d_qk + sh.d_v) + 2 * sh.h * pairs * (3 * sh.d_qk + 2 * sh.d_v) \
            + 3 * 2 * sh.S * sh.d_c * sh.n_cols
        ws_f = laga.alloc_workspace(laga.fwd_varlen_workspace_bytes(sh.S, len(lengths), sh.h), dev)
        ws_b = laga.alloc_workspace(laga.bwd_varlen_workspace_bytes(sh.S, len(lengths), sh.h), dev)

        def packed_step():
            laga.fwd(q, c_kv, k_pe, w, out=out, lse=lse, workspace=ws_f, cu_seqlens=cu)
            laga.bwd(q, c_kv, k_pe, w, out, lse, dout, dq=dq, dc_kv=dc_kv, dk_pe=dk_pe, dw_kv_b=dw, workspace=ws_b,
                     cu_seqlens=cu)

        packed_ms = timed(packed_step)
        laga.check_status(ws_f, where=f"{name} laga_fwd_varlen")
        laga.check_status(ws_b, where=f"{name} laga_bwd_varlen")
        n_max = max(lengths)
        ws_f1 = laga.alloc_workspace(laga.fwd_workspace_bytes(n_max, sh.h), dev)
        ws_b1 = laga.alloc_workspace(laga.bwd_workspace_bytes(n_max, sh.h), dev)
        dw1 = torch.empty_like(dw)

        def loop_step():
            for i, (a, b) in enumerate(zip(cu[:-1], cu[1:])):
                laga.fwd(q[a:b], c_kv[a:b], k_pe[a:b], w, out=out[a:b], lse=lse[a:b], workspace=ws_f1)
                laga.bwd(q[a:b], c_kv[a:b], k_pe[a:b], w, out[a:b], lse[a:b], dout[a:b], dq=dq[a:b], dc_kv=dc_kv[a:b],
                         dk_pe=dk_pe[a:b], dw_kv_b=dw1, workspace=ws_b1, flags=laga.FLAG_ACCUM_DW if i else 0)

        loop_ms = timed(loop_step)
        laga.check_status(ws_b1, where=f"{name} loop of laga_bwd")
        results[name] = {"sequences": len(lengths), "longest": n_max, "algorithmic_flops": total,
                         "packed_ms": packed_ms, "packed_tflops": total / (packed_ms * 1e-3) / 1e12,
                         "one_call_per_sequence_ms": loop_ms, "one_call_per_sequence_tflops": total / (loop_ms * 1e-3) / 1e12,
                         "launches_packed": 11, "launches_looped": 11 * len(lengths)}
        del ws_f, ws_b, ws_f1, ws_b1
    head = results["4x4096"]
    line = {"metric": "packed_batch_fwd_bwd_tflops", "value": head["packed_tflops"], "unit": UNIT, "n_gpus": 1, "steps": K,
            "warmup": W, "ms_per_step": head["packed_ms"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "packed: 16384 tokens of a 16-head DeepSeek-V3 shard as a batch of 4 x 4096 (headline of "
                                   "this line) and three other packings; causal within each sequence",
                       "l2_policy": "inputs and workspaces larger than L2"},
            "mixes": results, "gpu_launches": 11 * K}
    print(json.dumps(line), flush=True)


LINEAR_SHAPES = {
    # name: (K, N) for M = 16384 tokens and a 16-head shard of DeepSeek-V3 (hidden 7168, q_lora 1536)
    "W_kv_a (step 1: hidden -> latent + rope key)": (7168, 576),
    "W_q_b (step 1: low-rank query -> 16 heads x 192)": (1536, 3072),
    "W_kv_b (step 4: latent -> 16 heads x 256)": (512, 4096),
    "W_o (step 7: 16 heads x 128 -> hidden)": (2048, 7168),
}


def run_linear(args):
    """The dense projections around the path (Algorithm 1 steps 1, 4 and 7) through laga_linear /
    laga_linear_backward on 16384 tokens, with the same products through torch.matmul (cuBLAS) beside them."""
    from paper_2607_17644_b200 import laga
    laga.lib()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    M, K_steps, W = 16384, args.steps, max(args.warmup, 3)
    g = torch.Generator().manual_seed(1234)

    def timed(fn):
        for _ in range(W):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(K_steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / K_steps

    rows = {}
    for name, (K, N) in LINEAR_SHAPES.items():
        x = torch.randn(M, K, generator=g).to(torch.bfloat16).to(dev)
        w = (torch.randn(K, N, generator=g) * K ** -0.5).to(torch.bfloat16).to(dev)
        dy = torch.randn(M, N, generator=g).to(torch.bfloat16).to(dev)
        y = torch.empty(M, N, dtype=torch.bfloat16, device=dev)
        dx = torch.empty(M, K, dtype=torch.bfloat16, device=dev)
        dw = torch.empty(K, N, dtype=torch.float32, device=dev)
        st = torch.zeros(1, dtype=torch.int32, device=dev)
        fwd_ms = timed(lambda: laga.linear(x, w, y=y, status_word=st))
        bwd_ms = timed(lambda: laga.linear_backward(dy, x, w, dx=dx, dw=dw, status_word=st))
        assert laga.query_status(st)[0] == laga.OK
        lib_fwd_ms = timed(lambda: torch.matmul(x, w, out=y))
        wt = w.t().contiguous()

        def lib_bwd():
            torch.matmul(dy, wt, out=dx)
            torch.matmul(x.t(), dy)

        lib_bwd_ms = timed(lib_bwd)
        fl = 2.0 * M * K * N
        rows[name] = {"K": K, "N": N, "fwd_ms": fwd_ms, "fwd_tflops": fl / (fwd_ms * 1e-3) / 1e12,
                      "bwd_ms": bwd_ms, "bwd_tflops": 2 * fl / (bwd_ms * 1e-3) / 1e12,
                      "torch_matmul_fwd_ms": lib_fwd_ms, "torch_matmul_bwd_ms": lib_bwd_ms}
        del x, w, dy, y, dx, dw, wt
    # LayerNorm of the latent (step 1): HBM-bound, reported against the measured copy bandwidth.  262144 tokens so
    # that one tensor (268 MB) is larger than L2; the timed calls then really stream from and to HBM.
    D, M_ln = 512, 262144
    x = torch.randn(M_ln, D, generator=g).to(torch.bfloat16).to(dev)
    gamma = (1 + 0.2 * torch.randn(D, generator=g)).to(torch.bfloat16).to(dev)
    beta = (0.1 * torch.randn(D, generator=g)).to(torch.bfloat16).to(dev)
    dy = torch.randn(M_ln, D, generator=g).to(torch.bfloat16).to(dev)
    y, dx = torch.empty_like(x), torch.empty_like(x)
    _, mean, rstd = laga.layernorm(x, gamma, beta, y=y)
    ln_fwd_ms = timed(lambda: laga.layernorm(x, gamma, beta, y=y))
    ln_bwd_ms = timed(lambda: laga.layernorm_backward(dy, x, gamma, mean, rstd, dx=dx))
    peaks = measured_peaks()
    fwd_bytes, bwd_bytes = 2 * M_ln * D * 2 + 2 * M_ln * 4, 3 * M_ln * D * 2 + 2 * M_ln * 4
    layernorm = {"M": M_ln, "D": D, "fwd_ms": ln_fwd_ms, "fwd_bytes": fwd_bytes, "fwd_gbs": fwd_bytes / (ln_fwd_ms * 1e-3) / 1e9,
                 "bwd_ms": ln_bwd_ms, "bwd_bytes": bwd_bytes, "bwd_gbs": bwd_bytes / (ln_bwd_ms * 1e-3) / 1e9,
                 "hbm_peak_gbs": peaks["hbm_gbs"], "fwd_frac": fwd_bytes / (ln_fwd_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                 "bwd_frac": bwd_bytes / (ln_bwd_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                 "note": "algorithmic bytes: x in, y out (+ the two statistics) forward; dy and x in, dx out backward"}
    del x, dy, y, dx
    head = rows["W_o (step 7: 16 heads x 128 -> hidden)"]
    line = {"metric": "linear_projection_fwd_tflops", "value": head["fwd_tflops"], "unit": UNIT, "n_gpus": 1, "steps": K_steps,
            "warmup": W, "ms_per_step": head["fwd_ms"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "linear: the dense projections of Algorithm 1 steps 1, 4 and 7 at 16384 tokens, 16-head shard "
                                   "(headline of this line: W_o forward)",
                       "l2_policy": "operands larger than L2 except W"},
            "shapes": rows, "layernorm_of_the_latent": layernorm, "gpu_launches": K_steps}
    print(json.dumps(line), flush=True)


def run_cuda(args):
    from paper_2607_17644_b200 import laga
    laga.lib()
    if args.workload == "c4":
        return run_c4(args)
    if args.workload == "linear":
        return run_linear(args)
    if args.workload == "packed":
        return run_packed(args)
    if args.workload == "sweep":
        return run_sweep(args)
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

    def step_kv_saved():   # variant: the backward reuses the forward's K_nope/V from a workspace both calls share
        laga.fwd(q, c_kv, k_pe, w, out=out, lse=lse, workspace=ws_b)
        laga.bwd(q, c_kv, k_pe, w, out, lse, dout, dq=dq, dc_kv=dc_kv, dk_pe=dk_pe, dw_kv_b=dw, workspace=ws_b,
                 flags=laga.FLAG_KV_SAVED)

    for _ in range(max(args.warmup, 3)):
        step()
    laga.check_status(ws_f, where="warm-up laga_fwd")
    laga.check_status(ws_b, where="warm-up laga_bwd")

    # ---- timed region: exactly K steps, device-timed, events around the three attention kernels ----
    # (The delta kernel is timed after the region, in steps of its own: an event record in front of it would
    # serialise it behind the recomputed up-projection, beside which it otherwise runs.)
    K = args.steps
    dom = "attn_bwd_dkv"
    timed = ("attn_bwd_dkv", "attn_bwd_dq", "attn_fwd")
    kernel_events = {}
    for name in timed:
        starts = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
        stops = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
        for e in starts + stops:
            e.record()
        laga.profile_kernel(name, starts, stops)
        kernel_events[name] = (starts, stops)
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
    for name in timed:
        laga.profile_kernel(name)
    kernel_ms = {name: statistics.mean(a.elapsed_time(b) for a, b in zip(*kernel_events[name])) for name in timed}
    # the SM clock the attention kernels of the LAST timed step ran at, measured inside the kernels
    in_kernel = {**laga.query_kernel_clocks(ws_f), **laga.query_kernel_clocks(ws_b)}
    clocks["in_kernel_sm_mhz"] = {k: round(v[0], 1) for k, v in in_kernel.items()}
    Kd = max(3, min(K, 5))
    d_starts = [torch.cuda.Event(enable_timing=True) for _ in range(Kd)]
    d_stops = [torch.cuda.Event(enable_timing=True) for _ in range(Kd)]
    for e in d_starts + d_stops:
        e.record()
    laga.profile_kernel("bwd_delta", d_starts, d_stops)
    for _ in range(Kd):
        step()
    torch.cuda.synchronize()
    laga.profile_kernel("bwd_delta")
    delta_ms = statistics.mean(a.elapsed_time(b) for a, b in zip(d_starts, d_stops))
    s_pad = (sh.S + 127) // 128 * 128
    delta_bytes = 2 * sh.S * sh.h * sh.d_v * 2 + sh.S * sh.h * 4 + 2 * s_pad * sh.h * 4 + sh.S * sh.d_rope * 4   # O, dO, LSE in; two statistics out; rope-gradient accumulator cleared
    total_ms = max_over_ranks(ev0.elapsed_time(ev1), world)
    ms_per_step = total_ms / K
    dom_ms = kernel_ms[dom]
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

    # ---- the same default step without the per-kernel events of the timed region (what a caller sees: the event
    #      records sit between launches that otherwise overlap their set-up with the previous kernel's tail) ----
    for _ in range(2):
        step()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    p0.record()
    for _ in range(K):
        step()
    p1.record()
    barrier(world)
    plain_ms = max_over_ranks(p0.elapsed_time(p1), world) / K

    # ---- variant: LAGA_FLAG_KV_SAVED (reported, not the headline) ------------------------------------
    for _ in range(2):
        step_kv_saved()
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    s0.record()
    for _ in range(K):
        step_kv_saved()
    s1.record()
    barrier(world)
    kv_saved_ms = max_over_ranks(s0.elapsed_time(s1), world) / K
    laga.check_status(ws_b, where="kv-saved step")

    # ---- variant: LAGA_FLAG_FUSED_KV_REBUILD, step 4 rebuilt inside the dK/dV kernel (reported, not the headline) ----
    def step_kv_rebuild():
        laga.fwd(q, c_kv, k_pe, w, out=out, lse=lse, workspace=ws_f)
        laga.bwd(q, c_kv, k_pe, w, out, lse, dout, dq=dq, dc_kv=dc_kv, dk_pe=dk_pe, dw_kv_b=dw, workspace=ws_b,
                 flags=laga.FLAG_FUSED_KV_REBUILD)

    for _ in range(2):
        step_kv_rebuild()
    # default and rebuilt steps alternate in blocks of K (the clock drifts over a long run: only neighbours compare)
    ab = {"default": [], "rebuild": []}
    for _ in range(3):
        for key, fn in (("default", step), ("rebuild", step_kv_rebuild)):
            r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier(world)
            r0.record()
            for _ in range(K):
                fn()
            r1.record()
            barrier(world)
            ab[key].append(max_over_ranks(r0.elapsed_time(r1), world) / K)
    kv_rebuild_ms = statistics.median(ab["rebuild"])
    kv_rebuild_default_ms = statistics.median(ab["default"])
    laga.check_status(ws_b, where="kv-rebuild step")

    # ---- variant: LAGA_FLAG_FUSED_BWD, the one-pass CTA-pair backward (reported, not the headline) ---------
    one_pass_ms = None
    try:
        ws_1 = laga.alloc_workspace(laga.bwd_workspace_bytes(sh.S, sh.h, flags=laga.FLAG_FUSED_BWD), dev)

        def step_one_pass():
            laga.fwd(q, c_kv, k_pe, w, out=out, lse=lse, workspace=ws_f)
            laga.bwd(q, c_kv, k_pe, w, out, lse, dout, dq=dq, dc_kv=dc_kv, dk_pe=dk_pe, dw_kv_b=dw, workspace=ws_1,
                     flags=laga.FLAG_FUSED_BWD)

        for _ in range(2):
            step_one_pass()
        o0, o1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier(world)
        o0.record()
        for _ in range(K):
            step_one_pass()
        o1.record()
        barrier(world)
        one_pass_ms = max_over_ranks(o0.elapsed_time(o1), world) / K
        laga.check_status(ws_1, where="one-pass backward step")
        del ws_1
        step()                                               # leave the default path's gradients in the output buffers
    except Exception as exc:
        one_pass_ms = f"unavailable: {type(exc).__name__}: {exc}"

    # ---- variant: the same step replayed from a CUDA graph (launch overhead off the critical path) -------
    graph_ms = None
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step()                                           # warm this stream's view of everything
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):                        # the library only enqueues on the current stream
            step()
        for _ in range(2):
            graph.replay()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier(world)
        c0.record()
        for _ in range(K):
            graph.replay()
        c1.record()
        barrier(world)
        graph_ms = max_over_ranks(c0.elapsed_time(c1), world) / K
        laga.check_status(ws_b, where="graph replay")
    except Exception as exc:                                 # reported, never fatal: the headline does not depend on it
        graph_ms = f"unavailable: {type(exc).__name__}: {exc}"

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
    dom_tflops = fl[dom] / (dom_ms * 1e-3) / 1e12
    bwd_attn_ms = kernel_ms["attn_bwd_dkv"] + kernel_ms["attn_bwd_dq"]
    token_heads = sh.S * sh.h
    if DKV_DRAM_BYTES_C2 is None:
        traffic, traffic_note = None, "no ncu capture of this kernel yet"
    elif token_heads == DKV_DRAM_C2_TOKEN_HEADS:
        traffic, traffic_note = DKV_DRAM_BYTES_C2, "ncu dram read+write of one launch at this workload (profiles/ncu_dram_c2_attn_bwd_dkv.txt)"
    else:
        traffic = DKV_DRAM_BYTES_C2 * token_heads / DKV_DRAM_C2_TOKEN_HEADS
        traffic_note = "ncu dram read+write of one launch at S=16384,h=16, scaled by S*h"
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
        # Dominant kernel.  `achieved` = FLOPs this kernel executes per launch (S^T, dP^T, dV, dK: 1280 per causal
        # pair and head) / its mean CUDA-event time over the K timed launches.  `peak` is the measured cuBLAS bf16
        # BURST figure; the same kernel against the sustained figure, the clock it ran at (stamped inside the
        # kernel) and the whole backward attention on algorithmic FLOPs are given beside it.
        "roofline": {"bound": "tensor", "kernel": dom, "achieved": dom_tflops, "peak": peaks["bf16_tflops"], "unit": UNIT,
                     "frac": dom_tflops / peaks["bf16_tflops"],
                     "frac_of_sustained_peak": dom_tflops / peaks["bf16_tflops_sustained"],
                     "peak_source": peaks["source"] + " cuBLAS bf16, burst (sustained: "
                                    f"{peaks['bf16_tflops_sustained']})",
                     "kernel_ms": dom_ms, "flops_per_launch": fl[dom],
                     "sm_mhz_in_kernel": clocks["in_kernel_sm_mhz"].get(dom),
                     "kernel_ms_x_sm_mhz": dom_ms * clocks["in_kernel_sm_mhz"].get(dom, 0.0),
                     "traffic": traffic, "traffic_note": traffic_note,
                     "other_kernels": {
                         "attn_bwd_dq": {"kernel_ms": kernel_ms["attn_bwd_dq"], "executed_tflops": fl["attn_bwd_dq"] / (kernel_ms["attn_bwd_dq"] * 1e-3) / 1e12},
                         "attn_fwd": {"kernel_ms": kernel_ms["attn_fwd"], "executed_tflops": fl["attn_fwd"] / (kernel_ms["attn_fwd"] * 1e-3) / 1e12}},
                     "backward_attention": {"ms": bwd_attn_ms, "algorithmic_flops": fl["attn_bwd"],
                                            "algorithmic_tflops": fl["attn_bwd"] / (bwd_attn_ms * 1e-3) / 1e12,
                                            "frac_of_burst_peak": fl["attn_bwd"] / (bwd_attn_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                            "note": "dkv + dq kernels; S and dP are recomputed in both (2304 executed vs 1664 algorithmic FLOP per pair)"}},
        "variants": {"no_kernel_events": {"ms_per_step": plain_ms, "value": world * total_flops / (plain_ms * 1e-3) / 1e12,
                                          "note": "the headline step again, without the CUDA events the timed region records "
                                                  "around three kernels for the roofline figures"},
                     "kv_saved": {"ms_per_step": kv_saved_ms, "value": world * total_flops / (kv_saved_ms * 1e-3) / 1e12,
                                  "note": "LAGA_FLAG_KV_SAVED: the backward reads the forward's K_nope/V from a shared "
                                          "workspace instead of recomputing step 4 (one launch less); not the headline"},
                     "kv_rebuild": {"ms_per_step": kv_rebuild_ms, "value": world * total_flops / (kv_rebuild_ms * 1e-3) / 1e12,
                                    "default_ms_per_step_alternating": kv_rebuild_default_ms,
                                    "ratio_to_default": kv_rebuild_ms / kv_rebuild_default_ms,
                                    "note": "LAGA_FLAG_FUSED_KV_REBUILD: the recomputation of step 4 fused into the dK/dV kernel's item "
                                            "prologue (one launch less, K/V tiles built once per item); medians of three blocks of "
                                            "K steps alternating with blocks of the default step (no kernel events); not the headline"},
                     "one_pass_bwd": {"ms_per_step": one_pass_ms,
                                      "note": "LAGA_FLAG_FUSED_BWD: backward attention that computes every score tile once on CTA "
                                              "pairs (1664 instead of 2304 executed FLOP per pair) with dQ summed by fp32 atomics; "
                                              "slower as measured, kept as the opt-in alternative; not the headline"},
                     "cuda_graph": {"ms_per_step": graph_ms,
                                    "note": "the same forward+backward step captured once and replayed (11 launches per step: "
                                            "what short sequences are bound by); not the headline"}},
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
        step()                                                    # the results the parity figures are taken from
        torch.cuda.synchronize()
        gpu_results = {"out": out, "lse": lse, "dq": dq, "dw": dw}
        line["cpu_baseline"], line["parity"] = cpu_baseline(args.cpu_sample_tokens, args.workload, gpu_results,
                                                            lambda t: head0_shard_gradients(laga, sh, t, dev))
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def head0_shard_gradients(laga, sh, tensors, dev):
    """dc_kv and dk_pe are sums over the shard's heads, so head 0's share is not visible in the full run:
    run the CUDA path once more on the one-head shard the oracle sample is (outside any timed region)."""
    q, c_kv, k_pe, w, dout = (t.to(dev) for t in tensors)
    out, lse, ws = laga.fwd(q, c_kv, k_pe, w)
    _, dc_kv, dk_pe, _, ws2 = laga.bwd(q, c_kv, k_pe, w, out, lse, dout)
    laga.check_status(ws, where="parity laga_fwd")
    laga.check_status(ws2, where="parity laga_bwd")
    return {"dc_kv": dc_kv, "dk_pe": dk_pe}


def oracle_sample(sample_tokens: int, workload: str = WORKLOAD):
    """The bounded sample both CPU legs run: head 0 of the workload's shard restricted to its first
    `sample_tokens` tokens (a causal prefix is a self-contained sub-problem of the same workload)."""
    sh = CONFIGS[workload]
    q, c_kv, k_pe, w, dout = make_inputs(sh, CONFIG_SEEDS[workload])
    n = min(sample_tokens, sh.S)
    sub = LagaShape(S=n, h=1)
    tensors = (q[:n, :1].contiguous(), c_kv[:n].contiguous(), k_pe[:n].contiguous(), w[:, :256].contiguous(),
               dout[:n, :1].contiguous())
    return sub, tensors


def error_metrics(g, r):
    g, r = g.detach().to("cpu", torch.float64), r.to(torch.float64)
    diff = (g - r).abs()
    rms = float(r.pow(2).mean().sqrt())
    return {"max_abs": float(diff.max()), "rel_l2": float((g - r).norm() / r.norm().clamp_min(1e-300)),
            "scaled_max_abs": float(diff.max()) / max(1.0, rms), "ref_rms": rms, "ref_max": float(r.abs().max())}


def cpu_baseline(sample_tokens: int, workload: str = WORKLOAD, gpu_results=None, one_head_gradients=None):
    """The oracle as it stands, timed on the host cores on a bounded sample of the workload.  When the GPU
    results of the same workload are passed in, the oracle's numbers double as the parity record: raw
    max-abs, relative L2 and max-abs scaled by the reference's rms for every tensor, against the plain oracle
    (the timed call) and against the oracle that rounds K_nope/V to bf16 (a second, untimed call).  out, lse
    and dq are the head-0 rows of the timed configuration's own results; dc_kv and dk_pe (sums over heads)
    come from one more run of the CUDA path on the one-head sample."""
    import oracle
    sub, tensors = oracle_sample(sample_tokens, workload)
    q, c_kv, k_pe, w, dout = tensors
    fl = flops(sub)
    t0 = time.perf_counter()
    ref = oracle.bwd(q, c_kv, k_pe, w, dout, sub.d_v, sub.softmax_scale, causal=True, return_fwd=True)   # forward and backward
    dt = time.perf_counter() - t0
    base = {"value": (fl["fwd"] + fl["bwd"]) / dt / 1e12, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "seconds": dt, "sample": f"head 0, first {sub.S} tokens of the {workload} shard (causal prefix), "
                                      "forward+backward in fp64, one pass"}
    if gpu_results is None:
        return base, None
    n, full = sub.S, sub.S == CONFIGS[workload].S
    shard = one_head_gradients(tensors)
    # (dW sums over every token: the full run's head-0 columns match only a full-length sample)
    got = {"out": gpu_results["out"][:n, :1], "dq": gpu_results["dq"][:n, :1], "dc_kv": shard["dc_kv"],
           "dk_pe": shard["dk_pe"]}
    if full:
        got["dw"] = gpu_results["dw"][:, :256]
    refs = {"unrounded": ref,
            "kv_round_bf16": oracle.bwd(q, c_kv, k_pe, w, dout, sub.d_v, sub.softmax_scale, causal=True,
                                        kv_round_bf16=True, return_fwd=True)}
    parity = {"sample": base["sample"], "tolerances": {"max_abs": 2e-2, "rel_l2": 5e-3, "lse_vs_kv_round_bf16": 1e-3,
                                                       "note": "dw, and the early-key rows of dc_kv / dk_pe, are bound on "
                                                               "the scaled max-abs (their entries reach 5..35)"}}
    for mode, r in refs.items():
        parity[mode] = {name: error_metrics(t, r[name]) for name, t in got.items()}
        parity[mode]["lse"] = {"max_abs": float((gpu_results["lse"][:n, :1].detach().to("cpu", torch.float64) - r["lse"]).abs().max())}
    return base, parity


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
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing and parity leg")
    ap.add_argument("--workload", choices=sorted(CONFIGS) + ["packed", "linear", "sweep"], default=WORKLOAD,
                    help="benchmark configuration (default c2, the headline; c4 = the absorbed form beside the LAGA "
                         "forward on c2's inputs; packed = batches / variable-length sequences through the varlen "
                         "entry points; linear = the dense projections of steps 1, 4 and 7; others are for profiling)")
    ap.add_argument("--compare-eager", action="store_true",
                    help="also time the explicit and absorbed forms in eager PyTorch (N=1; tens of GB at c2)")
    ap.add_argument("--cpu-sample-tokens", type=int, default=16384,
                    help="tokens of head 0 the cpu_baseline leg runs (16384 = the whole head: ~10 s on 16 cores)")
    ap.add_argument("--ref-sample-tokens", type=int, default=2048,
                    help="tokens of head 0 per step in --impl reference (2048: well under a second per step)")
    ap.add_argument("--dry-run", action="store_true",
                    help="exercise the N-rank launch and the max-over-ranks reduction on the CPU (gloo), no GPU work")
    args = ap.parse_args()
    # `python bench.py --gpus N` outside a launcher: start the N ranks ourselves (one per GPU)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "cuda":
        raise SystemExit(self_launch(args.gpus))
    if args.dry_run:
        run_dry(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py: no CUDA device; the CUDA path has no fallback")
        run_cuda(args)


if __name__ == "__main__":
    main()
