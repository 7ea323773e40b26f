"""CPU, two gloo ranks: the multi-process conventions bench.py relies on for N > 1.

The path does not shard (replicas only), so there is no data-path collective to test; what N > 1
adds is (a) the max-over-ranks reduction of the per-rank times and the whole-job aggregate, and
(b) the reference arm, which only rank 0 runs and prints.
"""
import json
import os
import subprocess
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parents[1]
sys.path.insert(0, str(ROOT))
import bench  # noqa: E402


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    per_rank_ms = [10.0, 14.0][rank]
    total_ms, e2e_ms = bench.max_over_ranks(dist, torch.device("cpu"), per_rank_ms, per_rank_ms * 2)
    value = bench.aggregate_gbs(world, 58.6e9, total_ms, steps=2)
    out[rank] = (total_ms, e2e_ms, value)
    dist.destroy_process_group()


def test_times_are_max_over_ranks_and_value_is_whole_job():
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(2, 29631, out), nprocs=2, join=True)
        a, b = out[0], out[1]
    assert a == b
    assert a[0] == 14.0 and a[1] == 28.0                       # the slower rank sets the time
    assert abs(a[2] - 2 * 58.6e9 / (14.0 / 2 * 1e-3) / 1e9) < 1e-6   # two replicas' bytes over that time


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29632")
    outs = []
    for rank in (0, 1):
        env.update(RANK=str(rank), LOCAL_RANK=str(rank))
        res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                              "--warmup", "0", "--cpu-seconds", "1"], env=env, capture_output=True, text=True, timeout=600)
        assert res.returncode == 0, res.stderr
        outs.append(res.stdout.strip())
    assert outs[1] == ""
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["unit"] == "GB/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"] == {"value": line["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert line["gpu_launches"] == 0 and line["vs_baseline"] is None
