"""Data-parallel block step: one process per GPU (torchrun), the batch of a block sharded over the ranks, BatchNorm
statistics and gradients summed with NCCL all-reduce between the phases of nf_layer_step_dp, so that every rank
performs exactly the update of the whole batch.

    python -m torch.distributed.run --nnodes=1 --nproc-per-node 4 --master-addr 127.0.0.1 --master-port 29511 \\
        -m paper_2402_14139_b200.dp --workload c4 --steps 20

With one process (no torchrun) the all-reduce is the identity and the step equals nf_block_step.
Per layer and step the exchange is 2 x 2*Cout doubles, the parameter gradients (fp32) and one float.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np

from . import synth, workloads


def dp_block_step(layers, x, labels, lr, losses, acts, world, all_reduce):
    """Chains Layer.step_dp over the layers of a block on this rank's shard; losses[i] and acts[i] belong to layer i."""
    cur = x
    for i, L in enumerate(layers):
        L.step_dp(cur, labels, lr, losses[i:i + 1], acts[i], world, all_reduce)
        cur = acts[i]


def main():
    import torch
    import torch.distributed as dist
    from . import nf
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c4", choices=sorted(workloads.ALL))
    ap.add_argument("--block", type=int, default=0)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    args = ap.parse_args()
    rank, world, local = int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1)), int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    nf.lib()
    stream = torch.cuda.current_stream()
    nf.nf_set_stream(stream)
    wl = workloads.ALL[args.workload]()
    N, ls = wl["blocks"][args.block]
    if N % world:
        raise SystemExit(f"batch {N} does not divide over {world} ranks")
    Nl = N // world
    dt = nf.NF_F32 if wl["dtype"] == "f32" else nf.NF_BF16
    tdt = torch.float32 if dt == nf.NF_F32 else torch.bfloat16
    seed = 0x4E46DD00
    layers = []
    for li, l in enumerate(ls):       # the same seeded weights on every rank
        L = nf.Layer(l["Cin"], l["Cout"], l["H"], l["W"], l["F"], wl["classes"], Nl, stride=l["stride"], maxpool=l["pool"], dtype=dt)
        L.set_param("W", synth.normal(seed, 100 * li + 1, L.shapes["W"], np.sqrt(2.0 / (9 * l["Cin"]))))
        L.set_param("Wa", synth.normal(seed, 100 * li + 2, L.shapes["Wa"], np.sqrt(2.0 / (9 * l["Cout"]))))
        L.set_param("Wf", synth.normal(seed, 100 * li + 3, L.shapes["Wf"], np.sqrt(2.0 / (4 * l["F"]))))
        layers.append(L)
    g = torch.Generator(device="cuda")
    g.manual_seed(seed + rank)
    l0 = ls[0]
    x = torch.randn((Nl, l0["H"], l0["W"], l0["Cin"]), generator=g, device="cuda", dtype=torch.float32).to(tdt)
    labels = torch.randint(0, wl["classes"], (Nl,), generator=g, device="cuda", dtype=torch.int32)
    losses = torch.zeros(len(ls), device="cuda")
    acts = [L.new_act() for L in layers]
    all_reduce = (lambda t: dist.all_reduce(t)) if world > 1 else (lambda t: None)

    def sync():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        dp_block_step(layers, x, labels, 0.01, losses, acts, world, all_reduce)
    sync()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        dp_block_step(layers, x, labels, 0.01, losses, acts, world, all_reduce)
    e1.record(stream)
    sync()
    t = torch.tensor([e0.elapsed_time(e1)], device="cuda", dtype=torch.float64)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms = float(t.item())
    status = [L.status() for L in layers]
    if rank == 0:
        print(json.dumps(dict(mode="data-parallel", workload=wl["name"], block=args.block, n_gpus=world, global_batch=N, steps=args.steps,
                              ms_per_step=round(ms / args.steps, 4), images_per_s=round(N * args.steps / ms * 1e3, 1), scaling="strong",
                              losses=[round(v, 4) for v in losses.cpu().tolist()], status=status)))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
