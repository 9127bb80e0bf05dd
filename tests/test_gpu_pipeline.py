"""GPU test of the block-wise driver: two small blocks over a 24-image dataset; the cache handed to block 2
is what nf_block_cache produces, batches are re-assembled by permutation, nothing reruns block 1."""
import numpy as np
import pytest

from paper_2402_14139_b200 import pipeline, synth

pytestmark = pytest.mark.gpu


def _wl():
    l = lambda Cin, Cout, H, F, pool=False: dict(Cin=Cin, Cout=Cout, H=H, W=H, F=F, stride=1, pool=pool)
    return dict(name="mini", dtype="bf16", classes=4, in_shape=(3, 16, 16),
                blocks=[(6, [l(3, 64, 16, 8), l(64, 64, 16, 8, pool=True)]), (8, [l(64, 128, 8, 16)])])


def test_blockwise_pass_runs_and_learns_a_learnable_task():
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    nf.nf_set_stream(None)
    K = 24
    x = synth.normal(5, 1, (K, 16, 16, 3))
    lab = (np.arange(K) % 4).astype(np.int32)
    for k in range(K):                       # class = which quadrant carries a bright patch: learnable by conv + pooled head
        u, v = lab[k] // 2, lab[k] % 2
        x[k, u * 8:(u + 1) * 8, v * 8:(v + 1) * 8, :] += 2.0
    data = torch.from_numpy(synth.round_bf16(x)).cuda().to(torch.bfloat16)
    labels = torch.from_numpy(lab).cuda()
    recs = []
    report, out = pipeline.train_blockwise(nf, torch, _wl(), data, labels, epochs=25, lr=0.05, seed=3, log=recs.append)
    assert [r["block"] for r in report] == [0, 1] and report[0]["steps"] == 25 * 4 and report[1]["steps"] == 25 * 3
    assert out.shape == (K, 8, 8, 128) and torch.isfinite(out.float()).all()
    assert all(np.isfinite(r["losses"]).all() for r in report)
    assert report[0]["losses"][-1] < 0.7 * np.log(4)       # the local loss of block 1's last layer fell well below chance


def test_exit_evaluation_over_the_blockwise_pass():
    """Every trained layer is evaluated as an exit on held-out samples of the same learnable task: accuracies are
    counts over the validation set, parameter totals grow with depth, the selected exit follows the rule, and the
    deepest exits classify the task they were trained on."""
    import torch
    from oracle import nfo
    from paper_2402_14139_b200 import nf
    nf.lib()
    nf.nf_set_stream(None)

    def make(K, tid):
        x = synth.normal(5, tid, (K, 16, 16, 3))
        lab = (np.arange(K) % 4).astype(np.int32)
        for k in range(K):
            u, v = lab[k] // 2, lab[k] % 2
            x[k, u * 8:(u + 1) * 8, v * 8:(v + 1) * 8, :] += 2.0
        return torch.from_numpy(synth.round_bf16(x)).cuda().to(torch.bfloat16), torch.from_numpy(lab).cuda()

    data, labels = make(24, 1)
    val = make(20, 2)                         # 20 is not a multiple of either block's batch size: ragged last chunk
    report, out, ex = pipeline.train_blockwise(nf, torch, _wl(), data, labels, epochs=25, lr=0.05, seed=3, val=val)
    table = ex["table"]
    assert [t[0] for t in table] == [0, 1, 2]
    assert all(abs(t[1] * 20 - round(t[1] * 20)) < 1e-9 and 0.0 <= t[1] <= 1.0 for t in table)
    main = [9 * 3 * 64 + 128, 9 * 64 * 64 + 128, 9 * 64 * 128 + 256]
    aux = [9 * 64 * 8 + 8 + 4 * (32 + 1), 9 * 64 * 8 + 8 + 4 * (32 + 1), 9 * 128 * 16 + 16 + 4 * (64 + 1)]
    assert [t[2] for t in table] == [main[0] + aux[0], main[0] + main[1] + aux[1], sum(main) + aux[2]]
    assert ex["selected"] == nfo.select_exit([t[1] for t in table], [t[2] for t in table])
    assert max(t[1] for t in table) >= 0.9


def test_host_cache_tier_gives_identical_results():
    """The activation cache in pinned host memory (asynchronous fill, batches gathered from it on a second stream
    while the previous batch trains) is a storage choice only: final cache and losses are bit-identical to the
    run that keeps the cache on the device, also when the dataset itself sits in host memory."""
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    nf.nf_set_stream(None)
    K = 24
    x = synth.round_bf16(synth.normal(6, 1, (K, 16, 16, 3)))
    data = torch.from_numpy(x).cuda().to(torch.bfloat16)
    labels = torch.from_numpy(synth.labels(6, 2, K, 4)).cuda()
    r0, out0 = pipeline.train_blockwise(nf, torch, _wl(), data, labels, epochs=3, lr=0.05, seed=3)
    r1, out1 = pipeline.train_blockwise(nf, torch, _wl(), data, labels, epochs=3, lr=0.05, seed=3, cache="host")
    r2, out2 = pipeline.train_blockwise(nf, torch, _wl(), data.cpu().pin_memory(), labels, epochs=3, lr=0.05, seed=3, cache="host")
    assert out0.is_cuda and not out1.is_cuda and out1.is_pinned()
    for r, out in ((r1, out1), (r2, out2)):
        assert [b["losses"] for b in r] == [b["losses"] for b in r0]
        assert torch.equal(out.cuda().view(torch.int16), out0.view(torch.int16))
    nf.nf_set_stream(None)


def test_disk_cache_tier_and_offloaded_blocks_give_identical_results(tmp_path):
    """The storage tier beyond host memory: the activation cache as a memory-mapped file (rows read back by a reader
    thread while the previous batch trains) and finished blocks written out as .npz files.  Storage only: losses and the
    final cache are bit-identical to the run that keeps everything on the device, and a block reloaded from its file
    reproduces its cached output bit for bit."""
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    nf.nf_set_stream(None)
    K = 24
    x = synth.round_bf16(synth.normal(6, 1, (K, 16, 16, 3)))
    data = torch.from_numpy(x).cuda().to(torch.bfloat16)
    labels = torch.from_numpy(synth.labels(6, 2, K, 4)).cuda()
    r0, out0 = pipeline.train_blockwise(nf, torch, _wl(), data, labels, epochs=3, lr=0.05, seed=3, offload="host")
    r1, out1 = pipeline.train_blockwise(nf, torch, _wl(), data, labels, epochs=3, lr=0.05, seed=3, cache="disk", spill_dir=str(tmp_path),
                                        offload=str(tmp_path))
    assert isinstance(out1, np.memmap) and (tmp_path / "cache_block0.npy").exists() and (tmp_path / "cache_block1.npy").exists()
    assert [b["losses"] for b in r1] == [b["losses"] for b in r0]
    assert np.array_equal(np.asarray(out1), out0.view(torch.int16).cpu().numpy())
    # a finished block comes back from its file (and from the host copy) and reproduces the cache it left behind
    for state in (r1[0]["state"], r0[0]["state"]):
        layers, block = pipeline.load_block(nf, _wl(), 0, state)
        again = torch.empty((6, 8, 8, 64), dtype=torch.bfloat16, device="cuda")
        block.cache(data[:6].contiguous(), again)
        torch.cuda.synchronize()
        cache0 = np.load(tmp_path / "cache_block0.npy", mmap_mode="r")
        assert np.array_equal(again.view(torch.int16).cpu().numpy(), np.asarray(cache0[:6]))
        block.close()
        for L in layers:
            L.close()
    nf.nf_set_stream(None)


def test_measured_profiler_agrees_with_the_sized_one():
    """The Profiler that trains one step per batch size and reads the device's peak-memory counter against the one that adds
    up the library's own buffers: the measured bytes can only exceed the sized ones by the allocator's rounding, both give a
    straight line in the batch size.  The measured one also counts the step's output activation (which the sized model
    books on the consumer: the next layer's input or the cache), so its largest batch under a budget is up to about a
    quarter smaller and never noticeably larger; Algorithm 1 runs on either."""
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    nf.nf_set_stream(None)
    wl = _wl()
    ls = [l for _, b in wl["blocks"] for l in b]
    batches = (8, 16, 32)
    for l in ls:
        measured = pipeline.measure_layer_memory(nf, torch, l, wl["classes"], batches)
        sized, slope_s, icpt_s = nf.nf_profile_layer(l["Cin"], l["Cout"], l["H"], l["W"], l["F"], wl["classes"], list(batches),
                                                     stride=l["stride"], maxpool=l["pool"])
        slope_m, icpt_m = nf.nf_fit_line(list(batches), measured)
        for m, s in zip(measured, sized):
            assert s <= m <= s + 8 * 2 ** 20, (m, s)           # never less than the buffers; at most a few allocator blocks more
        assert abs(slope_m - slope_s) <= 0.05 * slope_s + 2 ** 20 / 8
    budget = 64e6
    plan_m, model = pipeline.plan_blocks_measured(nf, torch, ls, wl["classes"], budget, 512, batches=batches)
    max_m = [nf.nf_max_batch(sl, ic, budget) for sl, ic in model]
    for l, bm in zip(ls, max_m):
        _, sl, ic = nf.nf_profile_layer(l["Cin"], l["Cout"], l["H"], l["W"], l["F"], wl["classes"], list(batches), stride=l["stride"],
                                        maxpool=l["pool"])
        bs = nf.nf_max_batch(sl, ic, budget)
        assert 0.7 * bs <= bm <= 1.02 * bs + 1, (bm, bs)
    assert plan_m == nf.nf_partition([min(b, 2 ** 31 - 1) for b in max_m], 512, 0.4)
    assert plan_m[0][0] == 0 and plan_m[-1][1] == len(ls) - 1
    nf.nf_set_stream(None)
