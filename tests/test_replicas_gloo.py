"""Host-side logic of the multi-GPU benchmark arm, on CPU with gloo and two ranks.

The path does not shard across GPUs (replicas only): N ranks run N independent replicas, the timed
region is bracketed by barriers, the step time is the MAX over ranks and the throughput is the sum of
what all ranks processed.  These tests run that reduction, and the reference arm's rule that only
rank 0 works and prints, as real two-process jobs."""
import json
import os
import subprocess
import sys

import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import torch
    ms = bench.reduce_max_ms(dist, 10.0 + 5.0 * rank, torch.device("cpu"))       # ranks measured 10 and 15 ms
    value = bench.aggregate_throughput(world, bytes_per_rank=3_000_000, ms_per_step=ms)
    dist.barrier()
    if rank == 0:
        with open(out, "w") as f:
            json.dump({"ms": ms, "value": value}, f)
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value(tmp_path):
    out = str(tmp_path / "r.json")
    mp.spawn(_worker, args=(2, 29611, out), nprocs=2, join=True)
    r = json.load(open(out))
    assert r["ms"] == 15.0                                        # the slowest rank sets the step time
    assert r["value"] == pytest.approx(2 * 3_000_000 / 15e-3 / 1e9)   # both replicas' bytes over that time


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""          # other ranks exit without work


def test_byte_accounting_matches_the_documented_figures():
    # 4096 x 4096 at M = 1, fp32 out: 4 231 172 bytes; a whole LLaMA-2-7B layer: 50 969 372 bytes
    assert bench.product_bytes(1, 4096, 4096) == 4_231_172
    import synth
    assert sum(bench.product_bytes(1, n, k) for _, n, k in synth.LLAMA2_7B) == 50_969_372
    assert bench.product_bytes(1, 4096, 4096, bits=4) == 4096 * 4096 // 2 + 4 * 4096 + 4100 + 4 * 4096
