"""Host-side logic of bench.py that needs no GPU: multi-rank aggregation under gloo (world size 2), and the
CPU reference arm's JSON contract."""
import json
import os
import subprocess
import sys

import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    times = [1.0 + rank, 5.0 - rank, 2.5]                      # rank 0: 1, 5, 2.5 ; rank 1: 2, 4, 2.5
    got = bench.max_over_ranks(times, dist, "cpu")
    dist.barrier()
    if rank == 0:
        json.dump({"max": got, "value": bench.job_throughput(world, 1e9, got[0])}, open(out, "w"))
    dist.destroy_process_group()


def test_max_over_ranks_and_job_value_gloo(tmp_path):
    out = str(tmp_path / "r.json")
    mp.spawn(_worker, args=(2, 29000 + os.getpid() % 2000, out), nprocs=2, join=True)
    r = json.load(open(out))
    assert r["max"] == [2.0, 5.0, 2.5]                          # slowest rank per timer
    assert r["value"] == 2 * 1e9 / (2.0e-3) / 1e9               # all ranks' bytes over the slowest rank's time


def test_single_process_is_identity():
    import bench
    assert bench.max_over_ranks([3.0, 1.0]) == [3.0, 1.0]
    assert bench.job_throughput(1, 234881024, 0.04) == 234881024 / 0.04e-3 / 1e9


def test_reference_arm_prints_contract_line_and_other_ranks_stay_silent():
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "3"],
                       capture_output=True, text=True, env=env, timeout=600)
    assert p.returncode == 0, p.stderr
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "hif8_encode_decode_throughput" and line["unit"] == "GB/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["value"] == line["value"] > 0
    env1 = dict(os.environ, RANK="1", WORLD_SIZE="2")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1"],
                       capture_output=True, text=True, env=env1, timeout=600)
    assert p.returncode == 0 and p.stdout.strip() == ""
