#!/usr/bin/env python
"""Benchmark of the local-layer training step (one JSON line on stdout).

  python bench.py --gpus N --steps K --warmup W [--workload c4|c2] [--impl reference]

A step = one pass of the whole hot path over one batch: every layer of the block runs its local
step in turn (conv+BN+ReLU forward, aux head forward/backward, weight gradients, SGD update).
The K timed steps are K replays of a CUDA graph recorded from nf_block_step (--no-graph launches the kernels one by
one instead); the per-op table and the roofline come from the same K steps launched one by one right after.
Multi-GPU: independent replicas, one process per GPU (the step has no exchange to shard over),
timed as the max over ranks; value = images of all ranks / that time.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "local-layer train-step images/s (bf16)"
FALLBACK_PEAKS = dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0)


# DRAM bytes per image (read + write) of the kernels behind each traced op on the c4 layers 64->64 at 224x224,
# from one ncu capture of the batch-24 case (profiles/ncu_full_c4s_conv_bn_kernels.md); every tensor is streamed
# once, so traffic grows in proportion to the batch.  Valid for the kernels as captured; None elsewhere.
NCU_TRAFFIC_C4_BYTES_PER_IMAGE = dict(conv_fwd=(154.31 + 107.70) * 1e6 / 24, wgrad=(324.60 + 3.75) * 1e6 / 24,
                                      # aux forward with the fused BatchNorm + ReLU: reads y, writes a, the sign mask and the
                                      # pooling partials (h is not stored)
                                      aux_fwd=(154.21 + 115.70) * 1e6 / 24,
                                      # second pass of the aux input gradient: reads dh and y, writes dy; the finalize kernel < 1 MB
                                      bn_bwd=(192.74 + 108.21) * 1e6 / 24,
                                      # dh from the mask + aux weight gradient; the two small partial-sum kernels move < 1 MB
                                      aux_wgrad=(2.45 + 0.01 + 201.43 + 3.72) * 1e6 / 24,
                                      # first pass of the input gradient (dh and y read, sums only)
                                      aux_dgrad=(192.74 + 5.13) * 1e6 / 24)


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"]))), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML every 100 ms."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.stop_flag, self.sm, self.reasons, self.max_mhz, self.power = index, False, [], set(), None, []
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap"}
        while not self.stop_flag:
            try:
                self.sm.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1e3)
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.1)

    def summary(self):
        return dict(sm_mhz=float(np.median(self.sm)) if self.sm else None, sm_max_mhz=self.max_mhz,
                    reasons=sorted(self.reasons), power_w=round(float(np.median(self.power)), 1) if self.power else None)


def max_over_ranks(values, world, device):
    """Element-wise maximum of a list of floats over all ranks (replicas are timed as the slowest one)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def aggregate_images_per_s(images_per_rank, world, ms_max):
    """Whole-job throughput of `world` independent replicas: all images / the slowest replica's time."""
    return images_per_rank * world / (ms_max / 1e3)


def build_block(nf, torch, wl, bi, seed, host_io):
    """Layers of block bi with Kaiming-normal conv/linear weights (seeded), as an nf.Block."""
    from paper_2402_14139_b200 import synth
    N, ls = wl["blocks"][bi]
    dt = nf.NF_F32 if wl["dtype"] == "f32" else nf.NF_BF16
    layers = []
    for li, l in enumerate(ls):
        L = nf.Layer(l["Cin"], l["Cout"], l["H"], l["W"], l["F"], wl["classes"], N, stride=l["stride"],
                     maxpool=l["pool"], dtype=dt, host_io=(2 if host_io and li == 0 else 0))
        t = 100 * (bi * 32 + li)
        L.set_param("W", synth.normal(seed, t + 1, L.shapes["W"], np.sqrt(2.0 / (9 * l["Cin"]))))
        L.set_param("Wa", synth.normal(seed, t + 2, L.shapes["Wa"], np.sqrt(2.0 / (9 * l["Cout"]))))
        L.set_param("Wf", synth.normal(seed, t + 3, L.shapes["Wf"], np.sqrt(2.0 / (4 * l["F"]))))
        layers.append(L)
    return nf.Block(layers), layers


def op_model(l, N, classes, es, fam):
    """Algorithmic work of each traced op of one layer step: kind -> ('tensor'|'alu', flops, bytes) for the
    contractions (the caller takes whichever of the two rooflines binds) or ('hbm', None, bytes)."""
    from paper_2402_14139_b200 import workloads as W
    fl = W.step_flops(l, N)
    Ho, Wo = (l["H"] - 1) // l["stride"] + 1, (l["W"] - 1) // l["stride"] + 1
    Ha, Wa = W.out_hw(l)
    nx = N * l["H"] * l["W"] * l["Cin"]
    ny, na, nh = N * Ho * Wo * l["Cout"], N * Ha * Wa * l["Cout"], N * Ha * Wa * l["F"]
    nparam = 9 * l["Cin"] * l["Cout"] + 2 * l["Cout"] + 9 * l["Cout"] * l["F"] + l["F"] + classes * (4 * l["F"] + 1)
    tc = lambda k: "tensor" if fam[k] == "tcgen05" else "alu"
    fused = len(fam) > 4 and fam[4] == "fused"   # BatchNorm + ReLU applied inside the aux forward kernel
    masked = len(fam) > 5 and fam[5] == "mask"   # h never stored: pooled in the aux forward's epilogue, sign bits kept
    two_pass = len(fam) > 6 and fam[6] == "two-pass"   # da never stored: the input gradient runs once for the sums, once for dy
    return dict(conv_fwd=(tc(0), fl["conv_fwd"], es * (nx + ny)),          # read x, write y
                wgrad=(tc(1), fl["wgrad"], es * (nx + ny)),                # read x and dy
                # read a, write h; fused: read y, write a and h
                aux_fwd=(tc(2), fl["aux_fwd"], es * ((ny if fused else 0) + na + (0 if masked else nh))),
                # h -> dh (from the sign mask: dh written only); a, dh -> gWa
                aux_wgrad=(tc(3), fl["aux_bwd"] / 2, es * ((2 if masked else 3) * nh + na)),
                # dh -> da (two-pass: dh and y read, sums only)
                aux_dgrad=(tc(3), fl["aux_bwd"] / 2, es * (nh + (ny if two_pass else na))),
                # read y, write a; fused: only the statistics are finished here (partial sums in, coefficients out)
                bn_fwd=("hbm", None, 4 * 2 * l["Cout"] * 1184 if fused else es * (ny + na)),
                # read y and da, write dy; two-pass: the second run of the input gradient reads dh and y and writes dy
                bn_bwd=("hbm", None, es * (nh + 2 * ny) if two_pass else es * (2 * ny + na)),
                head=("hbm", None, es * nh + 4 * N * (8 * l["F"] + 2 * classes)),
                sgd=("hbm", None, 18 * nparam))                            # theta, v read+write (fp32), g read, bf16 copy write


def kernel_table(trace, ls, N, classes, es, fam, peaks, tensor_peak_key):
    """Per traced (op, layer): time per launch, share of the step and the fraction of the roofline that binds it, largest
    share first.  Tensor-bound ops are held against peaks[tensor_peak_key] (burst or sustained measured bf16 rate)."""
    kernels = []
    tot_ms = sum(v[0] for v in trace.values())
    for (op, slot), (tms, cnt) in sorted(trace.items(), key=lambda kv: -kv[1][0]):
        kind, flops, nbytes = op_model(ls[slot], N, classes, es, fam[slot])[op]
        if op == "sgd":   # nf_block_step updates all layers of the block in one launch, traced at layer position 0
            nbytes = sum(op_model(l, N, classes, es, f)["sgd"][2] for l, f in zip(ls, fam))
        per = tms / cnt
        # a contraction with few filters moves more bytes per flop than the machine balance: its bound is HBM
        if kind != "hbm" and nbytes / (peaks["hbm_gbs"] * 1e9) > flops / (peaks[tensor_peak_key] * 1e12):
            kind = "hbm"
        if kind == "hbm":
            ach, peak, unit = nbytes / per / 1e6, peaks["hbm_gbs"], "GB/s"
        else:
            ach, peak, unit = flops / per / 1e9, peaks[tensor_peak_key], "TFLOP/s"
        kernels.append(dict(op=op, layer=slot, bound=kind, ms_per_launch=round(per, 4), share=round(tms / tot_ms, 4),
                            achieved=round(ach, 2), peak=peak, unit=unit, frac=round(ach / peak, 4)))
    return kernels


def run_ours(args, rank, world):
    import torch
    from paper_2402_14139_b200 import nf, workloads
    nf.lib()
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    wl = workloads.ALL[args.workload]()
    bi = args.block
    N, ls = wl["blocks"][bi]
    seed = 0x4E460000 + int(args.workload[1]) + 1000 * rank + (50 if args.workload.endswith("s") else 0)
    es = 4 if wl["dtype"] == "f32" else 2
    tdt = torch.float32 if es == 4 else torch.bfloat16
    stream = torch.cuda.current_stream()
    nf.nf_set_stream(stream)
    block, layers = build_block(nf, torch, wl, bi, seed, host_io=True)
    C, H, Wd = ls[0]["Cin"], ls[0]["H"], ls[0]["W"]
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    x_bytes = N * H * Wd * C * es
    # inputs smaller than L2 (126 MB) are rotated through a pool larger than L2
    n_pool = 1 if x_bytes > 256e6 else min(64, int(300e6 // max(x_bytes, 1)) + 2)
    xs = [torch.randn((N, H, Wd, C), generator=g, device="cuda", dtype=torch.float32).to(tdt) for _ in range(n_pool)]
    if bi > 0:  # later blocks read cached post-ReLU activations: non-negative, about half zeros
        xs = [t.clamp_(min=0) for t in xs]
    labels = torch.randint(0, wl["classes"], (N,), generator=g, device="cuda", dtype=torch.int32)
    loss = torch.zeros(len(ls), dtype=torch.float32, device="cuda")
    flush = torch.empty(int(256e6), dtype=torch.uint8, device="cuda") if n_pool == 1 and x_bytes <= 256e6 else None
    lr = 0.01

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()

    for i in range(args.warmup):
        block.step(xs[i % n_pool], labels, lr, loss)
    barrier()
    graphs = None
    if args.graph:
        try:
            graphs = [block.capture(x, labels, lr, loss) for x in xs]
        except RuntimeError as e:      # capture refused by this driver/runtime: time the eager launches instead
            print(f"bench: CUDA graph capture failed ({e}); timing eager launches", file=sys.stderr)
            args.graph = False
            nf.nf_set_stream(stream)
    step = (lambda i: graphs[i % n_pool].replay()) if args.graph else (lambda i: block.step(xs[i % n_pool], labels, lr, loss))
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = nf.nf_launch_count()
    nf.nf_trace_enable(not args.graph)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    launches = nf.nf_launch_count() - launches0
    if args.graph:  # a replayed graph has no per-op events and counts no launches: the same K steps are run once more,
        # launched one by one with the per-op events on, for the `kernels` table, the roofline and the launch count
        nf.nf_trace_enable(True)
        launches0 = nf.nf_launch_count()
        for i in range(args.steps):
            block.step(xs[i % n_pool], labels, lr, loss)
        barrier()
        launches = nf.nf_launch_count() - launches0
    trace = nf.nf_trace_read(len(ls))
    nf.nf_trace_enable(False)
    sampler.stop_flag = True
    sampler.join(timeout=2)
    status = [L.status() for L in layers]
    losses = loss.cpu().tolist()
    if any(status) or not all(np.isfinite(losses)):
        raise RuntimeError(f"device status {status}, losses {losses}")

    # end to end: host buffers through the C ABI, copies inside the timed region
    xh = xs[0].cpu().pin_memory()
    lh = labels.cpu().pin_memory()
    loss_h = torch.zeros(len(ls), dtype=torch.float32).pin_memory()
    e2e_steps = max(3, min(args.steps, 10))
    # every step copies its batch host -> device once; the copy of step k+1 runs while step k trains
    block.step_host_next(xh, lh, lr, loss_h, xh, lh)
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        block.step_host_next(xh, lh, lr, loss_h, xh, lh)
    barrier()
    e2e_s = time.perf_counter() - t0

    ms, e2e_s = max_over_ranks([ms, e2e_s], world, "cuda")

    peaks, peak_src = load_peaks()
    fam = [[L.kernel_family(k) for k in range(7)] for L in layers]
    clocks = sampler.summary()
    # Which measured bf16 peak the tensor kernels are held against: the timed region and the per-op pass last a fraction
    # of a second each, so unless the sampled SM clock has already dropped well below its maximum these are burst
    # conditions and the burst figure is the denominator; the `sustained` record below uses the sustained one.
    burst = ms < 1000.0 and (clocks["sm_mhz"] is None or clocks["sm_max_mhz"] is None or clocks["sm_mhz"] >= 0.95 * clocks["sm_max_mhz"])
    tkey = "bf16_tflops" if burst else "bf16_tflops_sustained"
    kernels = kernel_table(trace, ls, N, wl["classes"], es, fam, peaks, tkey)
    best = kernels[0]
    traffic = None
    if wl["name"] in ("c4", "c4s") and best["layer"] in (0, 1) and best["op"] in NCU_TRAFFIC_C4_BYTES_PER_IMAGE:
        traffic = round(NCU_TRAFFIC_C4_BYTES_PER_IMAGE[best["op"]] * N)
    roof = dict(bound=best["bound"], achieved=best["achieved"], peak=best["peak"], unit=best["unit"],
                frac=best["frac"], traffic=traffic, kernel=f'{best["op"]}[layer {best["layer"]}]',
                peak_source=f"{peak_src} ({'burst' if burst else 'sustained'} bf16 figure)" if best["bound"] != "hbm" else peak_src)
    step_flops = sum(sum(workloads.step_flops(l, N).values()) for l in ls)

    # The same step under seconds of continuous load: graph replays for at least --sustain seconds (the part settles at a
    # lower SM clock under its power cap), then the per-op pass once more while the device is still hot.
    sustained = None
    if args.sustain > 0 and args.graph:
        per = ms / args.steps
        k_s = max(args.steps, int(args.sustain * 1e3 / per) + 1)
        s2 = ClockSampler(local)
        s2.start()
        e0.record(stream)
        for i in range(k_s):
            step(i)
        e1.record(stream)
        torch.cuda.synchronize()
        ms_s = e0.elapsed_time(e1)
        nf.nf_trace_enable(True)
        for i in range(max(args.steps, int(1e3 / per))):
            block.step(xs[i % n_pool], labels, lr, loss)
        trace_s = nf.nf_trace_read(len(ls))
        nf.nf_trace_enable(False)
        s2.stop_flag = True
        s2.join(timeout=2)
        (ms_s,) = max_over_ranks([ms_s], world, "cuda")
        ks = kernel_table(trace_s, ls, N, wl["classes"], es, fam, peaks, "bf16_tflops_sustained")
        sustained = dict(seconds=round(ms_s / 1e3, 2), steps=k_s, ms_per_step=round(ms_s / k_s, 4),
                         value=round(aggregate_images_per_s(N * k_s, world, ms_s), 2), clocks=s2.summary(),
                         step_tflops=round(step_flops / (ms_s / k_s) / 1e9, 1),
                         step_frac_of_sustained_bf16=round(step_flops / (ms_s / k_s) / 1e9 / peaks["bf16_tflops_sustained"], 4),
                         peak_source=f"{peak_src} (sustained bf16 figure)",
                         tensor_kernels=[dict(op=k["op"], layer=k["layer"], ms_per_launch=k["ms_per_launch"], achieved=k["achieved"],
                                              frac=k["frac"]) for k in ks if k["bound"] == "tensor"])

    out = None
    if rank == 0:
        out = dict(metric=METRIC, value=round(aggregate_images_per_s(N * args.steps, world, ms), 2), unit="images/s", n_gpus=world, steps=args.steps,
                   warmup=args.warmup, ms_per_step=round(ms / args.steps, 4), higher_is_better=True, scaling="weak",
                   vs_baseline=None, dtype="bf16" if es == 2 else "f32", data="synthetic",
                   config=dict(workload=f"{wl['name']}: " + " ".join(workloads.ALL[args.workload].__doc__.split(".")[0].split()),
                               block=bi, batch=N, layers=len(ls), l2="inputs larger than L2" if n_pool == 1 else
                               f"{n_pool} input batches rotated (pool larger than L2)", replicas=world, cuda_graph=bool(args.graph),
                               per_op_timing="the same K steps launched one by one after the timed graph replays" if args.graph else "inside the timed region",
                               kernel_families=fam),
                   clocks=clocks, gpu_launches=int(launches),
                   step_tflops=round(step_flops / (ms / args.steps) / 1e9, 1), sustained=sustained,
                   e2e=dict(value=round(aggregate_images_per_s(N * e2e_steps, world, e2e_s * 1e3), 2), unit="images/s",
                            h2d_bytes_per_step=int(x_bytes + 4 * N), d2h_bytes_per_step=int(4 * len(ls))),
                   roofline=roof, kernels=kernels, final_losses=[round(v, 4) for v in losses])
    return out, wl, bi


def oracle_sample(wl, bi, n_sample, seed, steps=1):
    """Times the CPU checker, as it stands, on n_sample images through every layer of the block."""
    from oracle import nfo
    from paper_2402_14139_b200 import synth
    N, ls = wl["blocks"][bi]
    layers = []
    for li, l in enumerate(ls):
        L = nfo.Layer(l["Cin"], l["Cout"], l["H"], l["W"], l["F"], wl["classes"], n_sample, stride=l["stride"],
                      pool=l["pool"], store_bf16=(wl["dtype"] == "bf16"))
        L.set(W=synth.normal(seed, 100 * li + 1, L.shapes["W"], np.sqrt(2.0 / (9 * l["Cin"]))),
              Wa=synth.normal(seed, 100 * li + 2, L.shapes["Wa"], np.sqrt(2.0 / (9 * l["Cout"]))),
              Wf=synth.normal(seed, 100 * li + 3, L.shapes["Wf"], np.sqrt(2.0 / (4 * l["F"]))))
        layers.append(L)
    x0 = synth.normal(seed, 7, (n_sample, ls[0]["Cin"], ls[0]["H"], ls[0]["W"]))
    y = synth.labels(seed, 8, n_sample, wl["classes"])
    times = []
    for _ in range(steps):
        t0 = time.perf_counter()
        x = x0
        for L in layers:
            _, x, _ = L.step(x, y, 0.01)
        times.append(time.perf_counter() - t0)
    return times, nfo.threads()


def run_reference(args):
    """The reference arm: the CPU checker on the host cores, same metric and workload."""
    from paper_2402_14139_b200 import workloads
    wl = workloads.ALL[args.workload]()
    n_sample = 1 if args.workload.startswith("c4") else min(8, wl["blocks"][0][0])
    oracle_sample(wl, 0, n_sample, 1, steps=max(0, min(args.warmup, 1)))
    times, cores = oracle_sample(wl, 0, n_sample, 2, steps=args.steps)
    total = sum(times)
    v = round(n_sample * args.steps / total, 4)
    sample = f"{n_sample} image(s) per step through all {len(wl['blocks'][0][1])} layers of the block"
    return dict(impl="reference", metric=METRIC, value=v, unit="images/s", n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=round(1e3 * total / args.steps, 2), higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=f"{wl['name']}: " + " ".join(workloads.ALL[args.workload].__doc__.split(".")[0].split()),
                            sample=sample),
                cpu_baseline=dict(value=v, unit="images/s", cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=v, unit="images/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)


def spawn_ranks(n, argv, backend_env=None):
    """Starts this script once per rank (RANK / LOCAL_RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT in the environment, as
    torch.distributed.run would) and waits; rank 0's output is the job's.  Returns the largest exit code."""
    import socket
    import subprocess
    with socket.socket() as sk:          # a free port on the loop-back interface for the rendezvous
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), **(backend_env or {}))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + list(argv), env=env,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    return max(p.wait() for p in procs)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c4", choices=["c2", "c3", "c4", "c4s", "c5", "c6"])
    ap.add_argument("--block", type=int, default=0, help="which block of a multi-block workload (c3, c5) to step")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sustain", type=float, default=3.0,
                    help="seconds of back-to-back graph replays for the `sustained` record (0 skips it)")
    ap.add_argument("--no-graph", dest="graph", action="store_false",
                    help="launch the kernels of a step one by one; by default a step is one replay of a CUDA graph recorded from "
                         "nf_block_step (same kernels in the same order, no launch gaps: 6 %% on c4, 30 %% on c2)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started without a launcher: one process per GPU is started here, each a replica of this command
        sys.exit(spawn_ranks(args.gpus, sys.argv[1:]))
    rank, world = int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))
    if world != args.gpus:
        print(f"bench: --gpus {args.gpus} but WORLD_SIZE={world}; timing {world} replica(s)", file=sys.stderr)
    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args)), flush=True)
        return
    out, wl, bi = run_ours(args, rank, world)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            n_sample = 4 if args.workload.startswith("c4") else wl["blocks"][bi][0]
            times, cores = oracle_sample(wl, bi, n_sample, 3)
            out["cpu_baseline"] = dict(value=round(n_sample / times[0], 4), unit="images/s", cores=cores, kind="oracle",
                                       sample=f"one step of {n_sample} images through all layers of the block "
                                              f"({times[0]:.1f} s)")
        print(json.dumps(out), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
