"""GPU parity of the data-parallel local step: the batch is cut into `world` shards, each held by its own layer
object (one rank each), the phases run in lockstep and the exchange buffers are added across the ranks exactly as
an all-reduce would.  BatchNorm sees the whole batch, so every rank must reproduce the checker's step on the
WHOLE batch: its slice of the activation, the loss, every gradient, the updated parameters and running statistics;
and the ranks must stay bit-identical to one another.  (One process drives all ranks in turn: no kernel waits for
another rank.)"""
import numpy as np
import pytest

from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    nf.nf_set_stream(None)
    return nf, torch


CASES = [
    (0, 2, dict(N=6, Cin=3, Cout=8, H=10, W=12, F=6, classes=10, stride=1, pool=False)),
    (0, 3, dict(N=6, Cin=4, Cout=8, H=8, W=8, F=4, classes=5, stride=2, pool=False, loss="mse")),
    (1, 2, dict(N=8, Cin=3, Cout=64, H=16, W=16, F=16, classes=10, stride=1, pool=True)),
    (1, 2, dict(N=8, Cin=64, Cout=64, H=16, W=112, F=16, classes=10, stride=1, pool=False)),   # folded kernels, fused BN-backward sums
    (1, 4, dict(N=16, Cin=64, Cout=128, H=16, W=16, F=32, classes=20, stride=2, pool=False, aux_pool="max")),
    (1, 2, dict(N=512, Cin=64, Cout=64, H=4, W=4, F=64, classes=128, stride=1, pool=False)),  # tiled large-batch head
]


@pytest.mark.parametrize("ci", range(len(CASES)))
def test_sharded_step_equals_whole_batch_step(env, ci):
    nf, torch = env
    dtype, world, c = CASES[ci]
    bf16 = dtype == 1
    tol = pu.TOL[dtype]
    Nl = c["N"] // world
    P, x, y = pu.seeded_case(c, 0x4E46D000 + ci, bf16=bf16)
    O = pu.oracle_layer(c, P, store_bf16=bf16)
    cl = dict(c, N=Nl)
    ranks = [pu.gpu_layer(nf, cl, P, nf.NF_BF16 if bf16 else nf.NF_F32) for _ in range(world)]
    xs = [pu.to_device_nhwc(torch, x[r * Nl:(r + 1) * Nl], dtype) for r in range(world)]
    ys = [torch.from_numpy(y[r * Nl:(r + 1) * Nl].copy()).cuda() for r in range(world)]
    losses = [torch.zeros(1, device="cuda") for _ in range(world)]
    acts = [G.new_act() for G in ranks]
    lib = nf.lib()

    def all_reduce(tensors):
        total = torch.stack(tensors).sum(dim=0)
        for t in tensors:
            t.copy_(total)

    for step in range(2):
        loss_o, act_o, tr = O.step(x, y, 0.02, update=True, grads=True)
        for phase in range(4):
            for r, G in enumerate(ranks):
                rc = lib.nf_layer_step_dp(G.h, phase, nf._ptr(xs[r]), nf._ptr(ys[r]), 0.02, nf._ptr(losses[r]), nf._ptr(acts[r]), world)
                assert rc == 0, (phase, r, rc)
            if phase < 3:
                all_reduce([G.dp_buffer(phase) for G in ranks])
            if phase == 2:
                all_reduce(losses)
        torch.cuda.synchronize()
        assert all(G.status() == 0 for G in ranks)
        for r, G in enumerate(ranks):
            assert abs(float(losses[r].item()) - loss_o) <= tol["loss"] * abs(loss_o), (step, r)
            assert pu.max_err(pu.from_device_nhwc(acts[r]), act_o[r * Nl:(r + 1) * Nl]) <= tol["t"] * np.abs(act_o).max() / max(np.abs(act_o[r * Nl:(r + 1) * Nl]).max(), 1e-30)
            for k in pu.PNAMES:
                assert pu.max_err(G.get_param(k, nf.NF_K_GRAD), tr["g" + k]) <= tol["t"], (step, r, "grad " + k)
                assert pu.max_err(G.get_param(k), O.p[k]) <= tol["t"], (step, r, "param " + k)
                assert np.array_equal(G.get_param(k), ranks[0].get_param(k)), (step, r, "ranks diverged in " + k)
            assert pu.max_err(G.get_param("rmean"), O.rmean) <= tol["t"] and pu.max_err(G.get_param("rvar"), O.rvar) <= tol["t"]
            assert np.array_equal(G.get_param("rvar"), ranks[0].get_param("rvar"))
        if bf16:      # both sides continue from the checker's state (see parity_util.check_step)
            for k in pu.PNAMES:
                v32, m32 = O.p[k].astype(np.float32), O.v[k].astype(np.float32)
                O.set(**{k: v32, "v" + k: m32})
                for G in ranks:
                    G.set_param(k, v32)
                    G.set_param(k, m32, kind=nf.NF_K_MOMENTUM)
            for k in ("rmean", "rvar"):
                v32 = getattr(O, k).astype(np.float32)
                O.set(**{k: v32})
                for G in ranks:
                    G.set_param(k, v32)
    for G in ranks:
        G.close()


def test_dp_argument_errors(env):
    nf, torch = env
    c = dict(N=2, Cin=3, Cout=8, H=8, W=8, F=4, classes=3, stride=1, pool=False)
    P, x, y = pu.seeded_case(c, 5, bf16=False)
    G = pu.gpu_layer(nf, c, P, nf.NF_F32)
    xd, yd = pu.to_device_nhwc(torch, x, 0), torch.from_numpy(y).cuda()
    loss, act = torch.zeros(1, device="cuda"), G.new_act()
    lib = nf.lib()
    assert lib.nf_layer_step_dp(G.h, 4, nf._ptr(xd), nf._ptr(yd), 0.1, nf._ptr(loss), nf._ptr(act), 2) == nf.NF_EINVAL
    assert lib.nf_layer_step_dp(G.h, 0, nf._ptr(xd), nf._ptr(yd), 0.1, nf._ptr(loss), nf._ptr(act), 0) == nf.NF_EINVAL
    assert G.dp_buffer(0).numel() == 16 and G.dp_buffer(1).numel() == 16 and G.dp_buffer(2).dtype == torch.float32
    G.close()


def _rank_main(rank, world, port, q):
    """One rank of the two-process run: its own process and CUDA context on the shared GPU, sums exchanged through a
    gloo process group (staged through host memory)."""
    import os
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import torch
    import torch.distributed as dist
    from paper_2402_14139_b200 import nf
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    nf.lib()
    nf.nf_set_stream(None)
    c = dict(N=8, Cin=64, Cout=64, H=16, W=16, F=16, classes=10, stride=1, pool=False)
    Nl = c["N"] // world
    P, x, y = pu.seeded_case(c, 0x4E46D100, bf16=True)
    G = pu.gpu_layer(nf, dict(c, N=Nl), P, nf.NF_BF16)
    xd = pu.to_device_nhwc(torch, x[rank * Nl:(rank + 1) * Nl], 1)
    yd = torch.from_numpy(y[rank * Nl:(rank + 1) * Nl].copy()).cuda()
    loss, act = torch.zeros(1, device="cuda"), G.new_act()

    def all_reduce(t):
        h = t.cpu()
        dist.all_reduce(h)
        t.copy_(h)

    G.step_dp(xd, yd, 0.02, loss, act, world, all_reduce)
    torch.cuda.synchronize()
    q.put((rank, G.status(), float(loss.item()), {k: G.get_param(k) for k in pu.PNAMES},
           {k: G.get_param(k, nf.NF_K_GRAD) for k in pu.PNAMES}, pu.from_device_nhwc(act)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_processes_exchange_through_a_process_group():
    import os
    import torch.multiprocessing as mp
    c = dict(N=8, Cin=64, Cout=64, H=16, W=16, F=16, classes=10, stride=1, pool=False)
    P, x, y = pu.seeded_case(c, 0x4E46D100, bf16=True)
    O = pu.oracle_layer(c, P, store_bf16=True)
    loss_o, act_o, tr = O.step(x, y, 0.02, update=True, grads=True)
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() * 7) % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted([q.get(timeout=300) for _ in range(2)], key=lambda t: t[0])
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    tol = pu.TOL[1]
    for rank, status, loss, params, grads, act in res:
        assert status == 0 and abs(loss - loss_o) <= tol["loss"] * abs(loss_o)
        assert np.abs(act - act_o[rank * 4:(rank + 1) * 4]).max() <= tol["t"] * np.abs(act_o).max()
        for k in pu.PNAMES:
            assert pu.max_err(grads[k], tr["g" + k]) <= tol["t"], k
            assert pu.max_err(params[k], O.p[k]) <= tol["t"], k
            assert np.array_equal(params[k], res[0][3][k]), k


def test_dp_driver_single_process_runs_the_block():
    """The torchrun driver with one process: the phased step with an identity all-reduce trains the c2 block."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-m", "paper_2402_14139_b200.dp", "--workload", "c2", "--steps", "3", "--warmup", "1"],
                         capture_output=True, text=True, timeout=600, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    d = json.loads(out.stdout.strip().splitlines()[-1])
    assert d["n_gpus"] == 1 and d["status"] == [0, 0, 0, 0] and all(np.isfinite(d["losses"])) and d["images_per_s"] > 0
