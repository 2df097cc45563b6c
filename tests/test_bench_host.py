"""Host-side logic of bench.py that needs no GPU: FLOP accounting, the activation-memory comparison,
the reference arm (oracle on a bounded sample), and the max-over-ranks reduction under a 2-process
gloo group (the N > 1 path of the benchmark has no data-path collective: ranks are independent
shards and only the timing is reduced)."""
import json
import os
import subprocess
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2607_17644_b200.inputs import CONFIGS, LagaShape  # noqa: E402


def test_flop_accounting_matches_the_closed_forms():
    fl = bench.flops(CONFIGS["c2"])
    pairs = 16384 * 16385 // 2
    assert fl["fwd"] == 2 * 16 * pairs * 320 + 2 * 16384 * 512 * 4096
    assert fl["bwd"] == 2 * 16 * pairs * 832 + 4 * 16384 * 512 * 4096
    assert abs((fl["fwd"] + fl["bwd"]) / 1e12 - 5.1543) < 1e-3          # the headline 5.154 TFLOP per step
    assert abs(bench.flops(CONFIGS["c1"])["fwd"] / 1e12 - 0.1031) < 1e-4
    tiny = bench.flops(LagaShape(S=1, h=1))
    assert tiny["fwd"] == 2 * 320 + 2 * 512 * 256


def test_activation_memory_comparison():
    sh = CONFIGS["c2"]
    m = bench.activation_memory(sh, ws_fwd=100, ws_bwd=200, allocated_in_step=0)
    tok_head = sh.S * sh.h
    assert m["explicit_form_bytes"] == tok_head * (128 * 2 + 4) + tok_head * 320 * 2 * 2 + tok_head * 4
    assert m["laga_bytes"] == tok_head * (128 * 2 + 4) + 200


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                          "--warmup", "0", "--ref-sample-tokens", "256"], capture_output=True, text=True, check=True)
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == bench.METRIC and d["unit"] == "TFLOP/s"
    assert d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle" and d["gpu_launches"] == 0
    assert d["e2e"]["h2d_bytes_per_step"] == 0


def _rank_main(rank, world, port, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist
    dist.init_process_group(backend="gloo", rank=rank, world_size=world)
    results[rank] = bench.max_over_ranks(10.0 + 5.0 * rank, world, device="cpu")   # the benchmark's own reduction
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_with_two_gloo_ranks():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    results = ctx.Manager().dict()
    from conftest import free_port
    port = free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, results)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(120)
        assert p.exitcode == 0
    assert results[0] == results[1] == 15.0
    # whole-job value under weak scaling: N shards' work over the slowest rank's time
    fl = bench.flops(CONFIGS["c2"])
    total = fl["fwd"] + fl["bwd"]
    assert abs(2 * total / (results[0] * 1e-3) / 1e12 - 2 * total / 15e-3 / 1e12) < 1e-9


def test_gpus_n_without_a_launcher_starts_n_ranks():
    """`python bench.py --gpus 2` with no WORLD_SIZE in the environment must itself start two ranks (one per
    GPU on the real run) and print ONE line whose n_gpus is 2 with the max over the ranks' times.  --dry-run
    swaps the GPU work for a made-up step time (10 ms on rank 0, 15 ms on rank 1) over gloo."""
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--dry-run"], env=env,
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip().startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["ms_per_step"] == 15.0 and d["scaling"] == "weak"


def test_error_metrics_and_sample():
    g = torch.tensor([1.0, 2.0, 4.0])
    r = torch.tensor([1.0, 2.0, 3.0], dtype=torch.float64)
    m = bench.error_metrics(g, r)
    assert m["max_abs"] == 1.0 and abs(m["rel_l2"] - 1.0 / 14 ** 0.5) < 1e-12
    assert abs(m["scaled_max_abs"] - 1.0 / (14 / 3) ** 0.5) < 1e-12
    sub, tensors = bench.oracle_sample(100, "c1")
    assert sub.S == 100 and sub.h == 1 and tuple(tensors[0].shape) == (100, 1, 192) and tuple(tensors[3].shape) == (512, 256)
