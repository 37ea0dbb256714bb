"""Host-side logic of bench.py: byte/flop accounting against parameter counts worked out by hand, and the
multi-rank plumbing (replicas, max over ranks) on two gloo ranks."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench
import ppd_inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_algorithmic_bytes_match_the_shapes():
    s7, s13 = ppd_inputs.LLAMA_7B, ppd_inputs.LLAMA_13B
    assert bench.layer_bytes(s7) == 2 * (202_383_360 - 2 * 4096)          # bf16 matrices of one layer
    assert abs(bench.greedy_step_bytes(s7, 0) - 13.215e9) < 2e6           # d W_L + W_H
    assert abs(bench.greedy_step_bytes(s13, 0) - 25.704e9) < 3e6
    assert bench.kv_layer_bytes(s7, 1) * s7.n_layers == 524_288           # KV bytes per position, all layers
    assert bench.kv_layer_bytes(s13, 1) * s13.n_layers == 819_200
    # PPD: + one head after a hit, + head + b layers after a miss
    g = bench.greedy_step_bytes(s7, 640)
    per_layer = bench.layer_bytes(s7) + bench.kv_layer_bytes(s7, 640)
    assert bench.ppd_step_bytes(s7, 640, 16, True) == g + bench.head_bytes(s7)
    assert bench.ppd_step_bytes(s7, 640, 16, False) == g + bench.head_bytes(s7) + 16 * per_layer
    assert bench.ppd_step_bytes(s7, 640, 8, False) == g + bench.head_bytes(s7) + 8 * per_layer
    assert bench.ppd_step_bytes(s7, 640, 24, False) == g + bench.head_bytes(s7) + 8 * per_layer
    # flops: 2 per weight per row; k branch rows for b layers
    extra = bench.ppd_step_flops(s7, 0, 3, 16, False) - bench.greedy_step_flops(s7, 0)
    assert extra == 3 * 16 * bench.layer_bytes(s7) + bench.head_bytes(s7)


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    got = bench.max_over_ranks([1.0 + rank, 10.0 - rank, 5.0], dist, "cpu")
    dist.barrier()
    if rank == 0:
        with open(out, "w") as f:
            json.dump(got, f)
    dist.destroy_process_group()


def test_max_over_two_gloo_ranks(tmp_path):
    out = str(tmp_path / "r.json")
    mp.spawn(_rank_main, args=(2, 29531 + os.getpid() % 500, out), nprocs=2, join=True)
    assert json.load(open(out)) == [2.0, 10.0, 5.0]
    assert bench.max_over_ranks([3.0, 4.0]) == [3.0, 4.0]      # no process group: identity


def test_reference_arm_only_rank0_prints(tmp_path):
    """The oracle arm under a multi-rank launch: rank 0 alone runs and prints, the others exit 0."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "2", "--warmup", "3", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny",
                        "--steps", "2", "--warmup", "3", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "ms/token" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["higher_is_better"] is False and line["steps"] == 2
