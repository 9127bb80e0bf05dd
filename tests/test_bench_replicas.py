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


def test_gpus_flag_starts_one_process_per_rank_when_no_launcher_did():
    """`python bench.py --gpus 2 ...` without torchrun: the script starts two ranks itself; with the reference arm rank 0
    alone prints the line (n_gpus 2) and the other rank exits 0 without work."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference", "--workload", "c2",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600, cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    assert json.loads(lines[0])["n_gpus"] == 2


def test_spawned_ranks_get_the_launcher_environment(tmp_path):
    """spawn_ranks hands every child RANK, LOCAL_RANK, WORLD_SIZE and a loop-back rendezvous address."""
    sys.path.insert(0, ROOT)
    import bench
    import subprocess
    script = tmp_path / "echo_env.py"
    script.write_text("import os, sys\n"
                      "open(sys.argv[1] + os.environ['RANK'], 'w').write(' '.join(os.environ[k] for k in "
                      "('RANK', 'LOCAL_RANK', 'WORLD_SIZE', 'MASTER_ADDR')) + ' ' + str(int(os.environ['MASTER_PORT']) > 0))\n")
    real = bench.__file__
    try:
        bench.__file__ = str(script)
        assert bench.spawn_ranks(3, [str(tmp_path / "r")]) == 0
    finally:
        bench.__file__ = real
    for r in range(3):
        assert (tmp_path / f"r{r}").read_text() == f"{r} {r} 3 127.0.0.1 True"


def _dp_worker(rank, world, port, q):
    """A stand-in layer whose phases only write rank-dependent numbers into the exchange buffers: what is checked is
    the schedule (which buffer is summed after which phase, the loss with the gradients, nothing after the update)."""
    sys.path.insert(0, ROOT)
    from paper_2402_14139_b200 import nf
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    bufs = [torch.zeros(4, dtype=torch.float64), torch.zeros(4, dtype=torch.float64), torch.zeros(6)]
    loss = torch.zeros(1)
    log = []

    def run_phase(k):
        log.append(("phase", k, [b.clone() for b in bufs]))
        if k < 3:
            bufs[k].fill_(float(10 * k + rank + 1))
        if k == 2:
            loss.fill_(0.25 * (rank + 1))

    nf.run_dp_phases(run_phase, lambda k: bufs[k], loss, lambda t: dist.all_reduce(t))
    q.put((rank, [b.tolist() for b in bufs], float(loss.item()), [(k, [b.tolist() for b in snap]) for _, k, snap in log]))
    dist.barrier()
    dist.destroy_process_group()


def test_data_parallel_exchange_schedule_over_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() * 3 + 1) % 2000
    procs = [ctx.Process(target=_dp_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, bufs, loss, log in res:
        assert bufs[0] == [3.0] * 4 and bufs[1] == [23.0] * 4 and bufs[2] == [43.0] * 6      # (10k+1) + (10k+2)
        assert loss == 0.75
        assert [k for k, _ in log] == [0, 1, 2, 3]
        assert log[1][1][0] == [3.0] * 4          # buffer 0 was already summed when phase 1 started
        assert log[2][1][1] == [23.0] * 4 and log[3][1][2] == [43.0] * 6
