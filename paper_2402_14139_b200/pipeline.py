"""Block-wise local learning over a dataset resident in HBM (Algorithm 2 with its outer loops, the
activation cache and the re-batching step), driven through the C-ABI binding.

For each block in order: for each epoch, a seeded permutation of the sample indices is cut into
batches of the block's own batch size (a last partial batch is dropped), every batch is assembled by
nf_cache_gather from the block's input set (the images for block 1, the cached activations of the
previous block otherwise) and stepped through all layers of the block with nf_block_step.  When a
block has finished, its output for every sample is written to the cache by nf_block_cache (forward
only, running statistics) and becomes the next block's input set.  Earlier blocks are never run again.

Storage tier (the paper keeps the activation cache outside the GPU when it does not fit): with cache="host" the
cache of every block lives in pinned host memory.  The cache fill copies each finished chunk to it asynchronously;
training assembles batch k+1 with nf_cache_gather straight from the pinned rows on a second stream while
batch k trains (two batch buffers, events between the streams), so the PCIe transfer hides behind the step.
The gather is a bit-exact row copy, so both tiers give identical results.  With cache="disk" the cache is a file in
`spill_dir` (for caches beyond host memory): the cache fill writes each finished chunk through a pinned staging buffer into
the memory-mapped file, and training has a reader thread collect the rows of batch k+1 from the file into pinned memory
while batch k trains; the rows travel as raw bytes, so this tier is bit-identical too.  With `offload` set, a finished
block's parameters, momentum and running statistics leave the device as well (one .npz file per block, or host arrays):
only the active block holds device memory, and load_block() brings a finished block back (for the selected exit model).

With a validation set, every trained layer is also evaluated as an exit point (nf_layer_predict on the
validation activations that the earlier layers produced, nf_count_equal against the labels); the
resulting (layer, accuracy, parameters) table goes through nf_select_exit.

    python -m paper_2402_14139_b200.pipeline --workload c5 --images 10000 --epochs 3
"""
from __future__ import annotations

import argparse
import json
import os
import threading
import time

import numpy as np

from . import synth, workloads


def build_layers(nf, wl, block_index, seed):
    """nf.Layer objects of one block with seeded Kaiming-normal weights, and the nf.Block over them."""
    N, ls = wl["blocks"][block_index]
    dt = nf.NF_F32 if wl["dtype"] == "f32" else nf.NF_BF16
    layers = []
    for li, l in enumerate(ls):
        L = nf.Layer(l["Cin"], l["Cout"], l["H"], l["W"], l["F"], wl["classes"], N, stride=l["stride"], maxpool=l["pool"], dtype=dt)
        t = 100 * (block_index * 32 + li)
        L.set_param("W", synth.normal(seed, t + 1, L.shapes["W"], np.sqrt(2.0 / (9 * l["Cin"]))))
        L.set_param("Wa", synth.normal(seed, t + 2, L.shapes["Wa"], np.sqrt(2.0 / (9 * l["Cout"]))))
        L.set_param("Wf", synth.normal(seed, t + 3, L.shapes["Wf"], np.sqrt(2.0 / (4 * l["F"]))))
        layers.append(L)
    return layers, nf.Block(layers)


def plan_blocks(nf, layers, classes, budget_bytes, batch_cap, rho=0.4, batches=(512, 1024, 2048, 4096), dtype="bf16"):
    """Profiler + Partitioner: the linear memory model of every layer (nf_profile_layer), its largest batch under the
    budget (nf_max_batch) and Algorithm 1 (nf_partition).  Returns [(first_layer, last_layer, batch_size)].
    The profiled batch sizes are large enough that the split-reduction scratch of small late layers has reached its
    final size (below that the memory need is not yet a straight line)."""
    dt = nf.NF_F32 if dtype == "f32" else nf.NF_BF16
    max_batch = []
    for l in layers:
        _, slope, icpt = nf.nf_profile_layer(l["Cin"], l["Cout"], l["H"], l["W"], l["F"], classes, list(batches), stride=l["stride"],
                                             maxpool=l["pool"], dtype=dt)
        t = nf.nf_max_batch(slope, icpt, budget_bytes)
        if t < 1:
            raise ValueError(f"layer {len(max_batch)} does not fit the budget even at batch size 1")
        max_batch.append(min(t, 2**31 - 1))
    return nf.nf_partition(max_batch, batch_cap, rho)


def measure_layer_memory(nf, torch, l, classes, batches, dtype="bf16"):
    """The Profiler as the paper describes it: the layer is actually trained for one step at each of the given batch
    sizes and the peak device memory of that step is read from the allocator's counters (everything the step touches:
    workspace, input batch, labels, loss and the output activation).  Returns the measured bytes per batch size."""
    dt = nf.NF_F32 if dtype == "f32" else nf.NF_BF16
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    out = []
    for N in batches:
        torch.cuda.synchronize()
        torch.cuda.empty_cache()
        base = torch.cuda.memory_allocated()
        torch.cuda.reset_peak_memory_stats()
        L = nf.Layer(l["Cin"], l["Cout"], l["H"], l["W"], l["F"], classes, int(N), stride=l["stride"], maxpool=l["pool"], dtype=dt)
        x = torch.zeros((int(N), l["H"], l["W"], l["Cin"]), dtype=tdt, device="cuda")
        y = torch.zeros(int(N), dtype=torch.int32, device="cuda")
        loss = torch.zeros(1, device="cuda")
        act = L.new_act()
        L.step(x, y, 0.0, loss, act)
        torch.cuda.synchronize()
        out.append(float(torch.cuda.max_memory_allocated() - base))
        L.close()
        del L, x, y, loss, act
    torch.cuda.empty_cache()
    return out


def plan_blocks_measured(nf, torch, layers, classes, budget_bytes, batch_cap, rho=0.4, batches=(8, 16, 32), dtype="bf16"):
    """plan_blocks with the MEASURED Profiler: memory per layer from measure_layer_memory at a few small batch sizes, the
    line through the measurements (nf_fit_line), the largest batch under the budget and Algorithm 1."""
    max_batch, model = [], []
    for l in layers:
        by = measure_layer_memory(nf, torch, l, classes, batches, dtype)
        slope, icpt = nf.nf_fit_line(list(batches), by)
        model.append((slope, icpt))
        max_batch.append(max(1, min(nf.nf_max_batch(slope, icpt, budget_bytes), 2**31 - 1)))
    return nf.nf_partition(max_batch, batch_cap, rho), model


def load_block(nf, wl, block_index, state):
    """Rebuilds the layers of a finished block on the device from what train_blockwise off-loaded: `state` is the list of
    per-layer dicts, or the path of the block's .npz file.  Returns (layers, nf.Block)."""
    N, ls = wl["blocks"][block_index]
    dt = nf.NF_F32 if wl["dtype"] == "f32" else nf.NF_BF16
    if isinstance(state, str):
        z = np.load(state)
        state = [{k.split(".", 1)[1]: z[k] for k in z.files if k.startswith(f"{li}.")} for li in range(len(ls))]
    layers = []
    for l, st in zip(ls, state):
        L = nf.Layer(l["Cin"], l["Cout"], l["H"], l["W"], l["F"], wl["classes"], N, stride=l["stride"], maxpool=l["pool"], dtype=dt)
        L.import_state(st)
        layers.append(L)
    return layers, nf.Block(layers)


class _DiskBatches:
    """Batches drawn by index from a memory-mapped cache file: a reader thread copies the rows of the next batch into one
    of two pinned buffers (reads hit the page cache or the drive) while the current batch trains."""

    def __init__(self, torch, mm, labels_host, N):
        self.mm, self.labels = mm, labels_host
        row = tuple(mm.shape[1:])
        self.pin = [torch.empty((N,) + row, dtype=torch.int16).pin_memory() for _ in range(2)]
        self.pin_l = [torch.empty(N, dtype=torch.int32).pin_memory() for _ in range(2)]
        self.thread = None

    def start(self, k, idx_host):
        def work():
            order = np.argsort(idx_host, kind="stable")          # ascending file offsets, rows put back in batch order
            self.pin[k % 2].numpy()[order] = self.mm[idx_host[order]]
            self.pin_l[k % 2].numpy()[:] = self.labels[idx_host]
        self.thread = threading.Thread(target=work)
        self.thread.start()

    def wait(self):
        self.thread.join()


def evaluate_exits(nf, torch, layers, N, val_cur, val_labels):
    """Run the validation activations through the layers of one trained block, each layer as an exit.
    Returns ([correct count per layer], the block's output for the validation set)."""
    V = val_cur.shape[0]
    counts = torch.zeros(len(layers), dtype=torch.int64, device=val_cur.device)
    pred = torch.empty(N, dtype=torch.int32, device=val_cur.device)
    acts = [L.new_act() for L in layers]
    last = layers[-1]
    out = torch.empty((V, last.Ha, last.Wa, last.Cout), dtype=val_cur.dtype, device=val_cur.device)
    for s in range(0, V, N):
        cnt = min(N, V - s)
        x = val_cur[s:s + cnt]
        for li, L in enumerate(layers):
            dst = out[s:s + cnt] if li == len(layers) - 1 else acts[li]
            L.predict(x, pred, act_out=dst, count=cnt)
            nf.nf_count_equal(pred[:cnt], val_labels[s:s + cnt], counts[li:li + 1])
            x = dst
    return counts.cpu().tolist(), out


def train_blockwise(nf, torch, wl, data, labels, epochs=1, lr=0.01, seed=1, log=None, val=None, cache="hbm", spill_dir=None,
                    offload=None):
    """data: device (or pinned host) tensor [K, H, W, C] of the first layer's dtype; labels: device int32 [K];
    cache: "hbm" keeps each block's output for all samples on the device, "host" in pinned host memory, "disk" in a
    memory-mapped file under spill_dir (bf16 workloads);
    offload: None keeps nothing of a finished block but its cache; "host" stores its layers' state (Layer.export_state) in
    the block's record under "state"; a directory path writes block<i>.npz there and records the path;
    val: optional (device tensor [V, H, W, C], device int32 [V]) validation set.
    Returns (per-block records, the last block's cached output) and, with val, also the exit report
    dict(table=[(layer, accuracy, parameters)], selected=layer index)."""
    K = data.shape[0]
    report = []
    cur = data
    labels_host = labels.cpu().numpy() if cache == "disk" else None
    val_cur, exits, main_params = (val[0] if val else None), [], 0
    for bi, (N, ls) in enumerate(wl["blocks"]):
        N = min(N, K)
        capped = dict(wl, blocks=[(N, l2) if i == bi else (n2, l2) for i, (n2, l2) in enumerate(wl["blocks"])])
        layers, block = build_layers(nf, capped, bi, seed)
        dev = labels.device
        tdt = torch.float32 if wl["dtype"] == "f32" else torch.bfloat16
        bufs = [(torch.empty((N,) + tuple(cur.shape[1:]), dtype=tdt, device=dev), torch.empty(N, dtype=torch.int32, device=dev))
                for _ in range(2)]
        loss = torch.zeros(len(ls), dtype=torch.float32, device=dev)
        main, side = torch.cuda.current_stream(), torch.cuda.Stream()
        ready = [torch.cuda.Event(), torch.cuda.Event()]      # batch buffer filled (side stream)
        free = [torch.cuda.Event(), torch.cuda.Event()]       # batch buffer consumed (main stream)
        perms = [torch.from_numpy(synth.permutation(seed + 7919 * bi, ep, K)).to(dev) for ep in range(epochs)]
        per_ep = K // N
        total = epochs * per_ep

        def assemble(k):      # batch k into buffer k % 2, on the side stream
            idx = perms[k // per_ep][(k % per_ep) * N:(k % per_ep + 1) * N].contiguous()
            if k >= 2:
                side.wait_event(free[k % 2])
            nf.nf_set_stream(side)
            nf.nf_cache_gather(cur, labels, idx, bufs[k % 2][0], bufs[k % 2][1])
            ready[k % 2].record(side)
            nf.nf_set_stream(main)
            return idx        # kept alive by the caller until the gather has run

        disk_in = isinstance(cur, np.memmap)
        if disk_in:      # the block's input set is a cache file: rows come through pinned buffers filled by a reader thread
            feeder = _DiskBatches(torch, cur, labels_host, N)
            perms_h = [synth.permutation(seed + 7919 * bi, ep, K) for ep in range(epochs)]
            batch_idx = lambda k: perms_h[k // per_ep][(k % per_ep) * N:(k % per_ep + 1) * N]
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        steps, keep = 0, []
        side.wait_stream(main)
        if total and disk_in:
            feeder.start(0, batch_idx(0))
        elif total:
            keep.append(assemble(0))
        for k in range(total):
            if disk_in:
                feeder.wait()                                   # rows of batch k are in pinned buffer k % 2
                if k >= 2:
                    side.wait_event(free[k % 2])
                with torch.cuda.stream(side):
                    bufs[k % 2][0].view(torch.int16).copy_(feeder.pin[k % 2], non_blocking=True)
                    bufs[k % 2][1].copy_(feeder.pin_l[k % 2], non_blocking=True)
                    ready[k % 2].record(side)
                if k + 1 < total:
                    if k >= 1:
                        ready[(k + 1) % 2].synchronize()        # its pinned buffer has been copied out
                    feeder.start(k + 1, batch_idx(k + 1))
            elif k + 1 < total:
                keep.append(assemble(k + 1))
            main.wait_event(ready[k % 2])
            block.step(bufs[k % 2][0], bufs[k % 2][1], lr, loss)
            free[k % 2].record(main)
            steps += 1
            keep = keep[-3:]
        torch.cuda.synchronize()
        t_train = time.perf_counter() - t0
        status = [L.status() for L in layers]
        if any(status):
            raise RuntimeError(f"block {bi}: device status {status}")
        # fill the cache: the block's output for every sample, in chunks of the block's batch size
        last = layers[-1]
        oshape = (K, last.Ha, last.Wa, last.Cout)
        host, disk = cache == "host", cache == "disk"
        if disk:
            if tdt != torch.bfloat16 or not spill_dir:
                raise ValueError('cache="disk" needs a bf16 workload and a spill_dir')
            out = np.lib.format.open_memmap(os.path.join(spill_dir, f"cache_block{bi}.npy"), mode="w+", dtype=np.int16, shape=oshape)
            pin_out = [torch.empty((N,) + oshape[1:], dtype=torch.int16).pin_memory() for _ in range(2)]
            done_out = [torch.cuda.Event(), torch.cuda.Event()]
        elif host:
            out = torch.empty(oshape, dtype=tdt, pin_memory=True)
        else:
            out = torch.empty(oshape, dtype=tdt, device=dev)
        in_dev = (not disk_in) and cur.is_cuda
        stage_in = None if in_dev else torch.empty((N,) + tuple(cur.shape[1:]), dtype=tdt, device=dev)
        stage_out = [torch.empty((N,) + oshape[1:], dtype=tdt, device=dev) for _ in range(2)] if (host or disk) else None
        t1 = time.perf_counter()
        pending = []      # disk: (chunk start, count, buffer) whose device -> pinned copy is in flight
        for ci, s in enumerate(range(0, K, N)):
            cnt = min(N, K - s)
            if disk_in:                   # the block's input set is a cache file: read the chunk, then bring it in
                stage_in[:cnt].view(torch.int16).copy_(torch.from_numpy(np.ascontiguousarray(cur[s:s + cnt])))
                src = stage_in[:cnt]
            elif stage_in is not None:    # ... or lives in host memory
                stage_in[:cnt].copy_(cur[s:s + cnt], non_blocking=True)
                src = stage_in[:cnt]
            else:
                src = cur[s:s + cnt]
            if disk:                      # forward into a device chunk, copy it to pinned memory, write the previous one out
                if len(pending) == 2:
                    s0, c0, b0 = pending.pop(0)
                    done_out[b0].synchronize()
                    out[s0:s0 + c0] = pin_out[b0][:c0].numpy()
                b = ci % 2
                block.cache(src, stage_out[b][:cnt], count=cnt)
                pin_out[b][:cnt].copy_(stage_out[b][:cnt].view(torch.int16), non_blocking=True)
                done_out[b].record(main)
                pending.append((s, cnt, b))
            elif host:                    # forward into a device chunk, then an asynchronous copy to the pinned cache
                so = stage_out[ci % 2]
                block.cache(src, so[:cnt], count=cnt)
                out[s:s + cnt].copy_(so[:cnt], non_blocking=True)
            else:
                block.cache(src, out[s:s + cnt], count=cnt)
        torch.cuda.synchronize()
        for s0, c0, b0 in pending:
            out[s0:s0 + c0] = pin_out[b0][:c0].numpy()
        if disk:
            out.flush()
        t_cache = time.perf_counter() - t1
        rec = dict(block=bi, layers=len(ls), batch=N, steps=steps, train_s=round(t_train, 4), cache_s=round(t_cache, 4),
                   train_images_per_s=round(steps * N / max(t_train, 1e-9), 1), losses=[round(v, 4) for v in loss.cpu().tolist()])
        report.append(rec)
        if val:
            correct, val_cur = evaluate_exits(nf, torch, layers, N, val_cur, val[1])
            for L, c in zip(layers, correct):       # exit at layer n: main paths of layers 1..n + the aux head of layer n
                main_params += L.param_count(0)
                exits.append((len(exits), c / val[0].shape[0], main_params + L.param_count(1)))
            rec["exit_val_accuracy"] = [round(e[1], 4) for e in exits[-len(layers):]]
        if offload:       # the finished block leaves the device: parameters, momentum and running statistics
            state = [L.export_state() for L in layers]
            if offload == "host":
                rec["state"] = state
            else:
                path = os.path.join(offload, f"block{bi}.npz")
                np.savez(path, **{f"{li}.{k}": v for li, st in enumerate(state) for k, v in st.items()})
                rec["state"] = path
        if log:
            log({k: v for k, v in rec.items() if k != "state" or isinstance(v, str)})
        block.close()
        for L in layers:
            L.close()
        cur = out
    if val:
        sel = nf.nf_select_exit([e[1] for e in exits], [e[2] for e in exits])
        return report, cur, dict(table=exits, selected=sel)
    return report, cur


def main():
    import torch
    from . import nf
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="c5", choices=sorted(workloads.ALL))
    ap.add_argument("--images", type=int, default=10000)
    ap.add_argument("--epochs", type=int, default=3)
    ap.add_argument("--lr", type=float, default=0.01)
    ap.add_argument("--val-images", type=int, default=0, help="evaluate every layer as an exit on this many held-out images")
    ap.add_argument("--budget-gb", type=float, default=0.0, help="re-plan the blocks with the Profiler and Algorithm 1 under this memory budget")
    ap.add_argument("--rho", type=float, default=0.4)
    ap.add_argument("--cache", default="hbm", choices=["hbm", "host", "disk"], help="where the activation cache of a finished block lives")
    ap.add_argument("--spill-dir", default=None, help='directory of the cache files (--cache disk) and of the off-loaded blocks')
    ap.add_argument("--offload", action="store_true", help="write each finished block's parameters to <spill-dir>/block<i>.npz")
    ap.add_argument("--measured-profiler", action="store_true", help="with --budget-gb: profile by running steps instead of sizing buffers")
    args = ap.parse_args()
    nf.lib()
    nf.nf_set_stream(torch.cuda.current_stream())
    wl = workloads.ALL[args.workload]()
    if args.budget_gb > 0 and "layers" in wl:
        if args.measured_profiler:
            plan, _ = plan_blocks_measured(nf, torch, wl["layers"], wl["classes"], args.budget_gb * 1e9, args.images, args.rho, dtype=wl["dtype"])
        else:
            plan = plan_blocks(nf, wl["layers"], wl["classes"], args.budget_gb * 1e9, args.images, args.rho, dtype=wl["dtype"])
        print(json.dumps(dict(planned_blocks=plan)), flush=True)
        wl = dict(wl, blocks=[(bs, wl["layers"][f:l + 1]) for f, l, bs in plan])
    C, H, W = wl["in_shape"]
    g = torch.Generator(device="cuda")
    g.manual_seed(0x4E460005)
    tdt = torch.float32 if wl["dtype"] == "f32" else torch.bfloat16
    data = torch.randn((args.images, H, W, C), generator=g, device="cuda", dtype=torch.float32).to(tdt)
    labels = torch.randint(0, wl["classes"], (args.images,), generator=g, device="cuda", dtype=torch.int32)
    val = None
    if args.val_images:
        val = (torch.randn((args.val_images, H, W, C), generator=g, device="cuda", dtype=torch.float32).to(tdt),
               torch.randint(0, wl["classes"], (args.val_images,), generator=g, device="cuda", dtype=torch.int32))
    t0 = time.perf_counter()
    res = train_blockwise(nf, torch, wl, data, labels, epochs=args.epochs, lr=args.lr, log=lambda r: print(json.dumps(r), flush=True),
                          val=val, cache=args.cache, spill_dir=args.spill_dir,
                          offload=(args.spill_dir if args.offload else None))
    wall = time.perf_counter() - t0
    if val:
        print(json.dumps(dict(exit_table=[(l, round(a, 4), p) for l, a, p in res[2]["table"]], selected_exit=res[2]["selected"])))
    n_layers = sum(len(ls) for _, ls in wl["blocks"])
    print(json.dumps(dict(workload=wl["name"], images=args.images, epochs=args.epochs, layers=n_layers, wall_s=round(wall, 3),
                          images_per_s_whole_pass=round(args.images * args.epochs / wall, 1))))


if __name__ == "__main__":
    main()
