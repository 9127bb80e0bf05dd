"""CPU test (gloo, world size 2) of the multi-replica path of bench.py: times are reduced with MAX over the
ranks and the reported throughput counts the images of all replicas against the slowest one."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms, e2e = bench.max_over_ranks([10.0 + 5.0 * rank, 2.0 - rank], world, "cpu")
    q.put((rank, ms, e2e, bench.aggregate_images_per_s(64 * 20, world, ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_are_timed_as_the_slowest_and_counted_together():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, e2e, val in res:
        assert ms == 15.0 and e2e == 2.0                       # max over ranks, element-wise
        assert val == pytest.approx(2 * 64 * 20 / 0.015)


def test_single_replica_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 4.0], 1, "cpu") == [3.0, 4.0]
    assert bench.aggregate_images_per_s(128, 1, 1000.0) == 128.0


def test_reference_arm_prints_one_json_line_with_the_required_keys():
    import json
    import subprocess
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c2", "--steps", "1",
                          "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    d = json.loads(out.stdout.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == dict(value=d["value"], unit=d["unit"], h2d_bytes_per_step=0, d2h_bytes_per_step=0)
    assert d["unit"] == "images/s" and d["higher_is_better"] is True and d["value"] > 0
