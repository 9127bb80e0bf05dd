"""GPU parity on the shapes of the benchmark workloads c2, c3 and c5 (c1 and c4 have their own files).

Every compared step starts from seeded parameters and from inputs produced by the generators or by the
CHECKER (never by the GPU): layer l+1 of a chain is fed the checker's activation of layer l, which is
bf16-valued in the bf16 configurations and therefore identical on both sides."""
import numpy as np
import pytest

from paper_2402_14139_b200 import synth, workloads
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    nf.nf_set_stream(None)
    return nf, torch


_cfg = pu.layer_cfg


def _step_both(nf, torch, c, P, x, y, lr=0.01):
    return pu.step_both(nf, torch, c, P, x, y, lr)


def test_c2_vgg_block_full_batch_chain(env):
    nf, torch = env
    wl = workloads.c2()
    N, ls = wl["blocks"][0]
    x = synth.round_bf16(synth.normal(0x4E460002, 8, (N, 3, 32, 32))).astype(np.float64)
    y = synth.labels(0x4E460002, 9, N, wl["classes"])
    for li, l in enumerate(ls):
        c = _cfg(l, N, wl["classes"])
        P, _, _ = pu.seeded_case(dict(c, N=1), 0x4E460200 + li, bf16=True)
        errs, x, O, G = _step_both(nf, torch, c, P, x, y)
        fam = [G.kernel_family(k) for k in range(4)]
        assert fam == ["tcgen05"] * 4, fam        # the RGB first layer too: its input is padded to 64 channels
        G.close()


def test_c2_block_against_unrounded_fp64_checker(env):
    """What the bf16 storage costs on the VGG block at its full batch of 128: the same chain against the checker in
    pure fp64 (store_bf16 off), with the bounds parity_util.UNROUNDED_TOL derives from the arithmetic."""
    nf, torch = env
    wl = workloads.c2()
    N, ls = wl["blocks"][0]
    x = synth.round_bf16(synth.normal(0x4E460002, 8, (N, 3, 32, 32))).astype(np.float64)
    y = synth.labels(0x4E460002, 9, N, wl["classes"])
    for li, l in enumerate(ls):
        c = _cfg(l, N, wl["classes"])
        P, _, _ = pu.seeded_case(dict(c, N=1), 0x4E460200 + li, bf16=True)
        errs, act_o, O, G = pu.step_both(nf, torch, c, P, x, y, store_bf16=False, tol=pu.UNROUNDED_TOL)
        assert errs["act"] <= pu.UNROUNDED_TOL["act"], errs
        print(f"c2 layer {li} vs unrounded fp64:", {k: f"{v:.2e}" for k, v in errs.items()})
        G.close()
        x = synth.round_bf16(act_o).astype(np.float64)


def _c3_layers():
    wl = workloads.c3()
    return [(b, li, N, l) for b, (N, ls) in enumerate(wl["blocks"]) for li, l in enumerate(ls)]


def _one_layer(nf, torch, l, N, classes, seed):
    c = _cfg(l, N, classes)
    P, _, _ = pu.seeded_case(dict(c, N=1), seed, bf16=True)
    x = synth.normal(seed, 8, (N, l["Cin"], l["H"], l["W"]))
    if l["Cin"] != 3:
        x = np.maximum(x, 0.0)                              # deeper layers see post-ReLU activations
    x = synth.round_bf16(x).astype(np.float64)
    y = synth.labels(seed, 9, N, classes)
    errs, _, _, G = _step_both(nf, torch, c, P, x, y)
    G.close()
    return errs


@pytest.mark.parametrize("k", range(17))
def test_c3_every_layer_at_its_block_batch_size(env, k):
    """All 17 layers of the ResNet-18-shaped stack, each at the batch size of its block (64 / 128 / 256 / 512)."""
    nf, torch = env
    b, li, N, l = _c3_layers()[k]
    errs = _one_layer(nf, torch, l, N, workloads.c3()["classes"], 0x4E460300 + 16 * b + li)
    print(f"c3 block {b} layer {li} N={N}:", {k2: f"{v:.2e}" for k2, v in errs.items()})


# batch sizes for the 13 layer shapes of the VGG-16 workload: the block batch sizes (1260 ... 8602) are cut to what the
# checker steps in a few seconds, more samples where the maps are small so that several tensor-core tiles are covered
C5_BATCH = [8, 8, 12, 12, 24, 24, 24, 48, 48, 48, 160, 160, 160]


@pytest.mark.parametrize("k", range(13))
def test_c5_every_layer_shape(env, k):
    nf, torch = env
    wl = workloads.c5()
    errs = _one_layer(nf, torch, wl["layers"][k], C5_BATCH[k], wl["classes"], 0x4E460540 + k)
    print(f"c5 layer {k} N={C5_BATCH[k]}:", {k2: f"{v:.2e}" for k2, v in errs.items()})


def test_c5_partition_train_cache_rebatch_next_block(env):
    """The mechanism of the full pass on VGG-16 shapes, at a scale the checker finishes in seconds:
    Algorithm 1 on the analytic memory model -> train block 1 -> cache its output for the whole
    (small) dataset -> re-batch by a seeded permutation -> train block 2 on the cached activations."""
    nf, torch = env
    wl = workloads.c5()
    ls = wl["layers"]
    per_image = [workloads.layer_bytes_per_image(l, wl["classes"]) for l in ls]
    max_batch = [int(4e9 // b) for b in per_image]
    blocks = nf.nf_partition(max_batch, 10000, 0.4)
    from oracle import nfo
    assert blocks == nfo.partition(max_batch, 10000, 0.4)
    # five blocks under the 4 GB budget; with this library's buffers the early, memory-hungry layers stand alone
    assert [(f, l) for f, l, _ in blocks] == [(0, 0), (1, 1), (2, 3), (4, 5), (6, 12)]
    assert all(bs == min(max_batch[f:l + 1]) for f, l, bs in blocks)
    assert [bs for _, _, bs in blocks] == sorted(bs for _, _, bs in blocks)                    # later blocks: larger batches

    K, N1, N2, classes = 12, 4, 6, wl["classes"]      # dataset of 12 images; block 1 trains at 4, block 2 at 6
    data = synth.round_bf16(synth.normal(0x4E460005, 8, (K, 3, 64, 64))).astype(np.float64)
    labels = synth.labels(0x4E460005, 9, K, classes)
    b1 = ls[blocks[0][0]:blocks[1][1] + 1]      # the first two (single-layer) blocks trained as one chain here
    O1, G1 = [], []
    for li, l in enumerate(b1):
        c = _cfg(l, N1, classes)
        P, _, _ = pu.seeded_case(dict(c, N=1), 0x4E460500 + li, bf16=True)
        O1.append(pu.oracle_layer(c, P, store_bf16=True))
        G1.append(pu.gpu_layer(nf, c, P, nf.NF_BF16))
    blk1 = nf.Block(G1)
    loss = torch.zeros(2, device="cuda")
    for s in range(K // N1):                                # one epoch over the dataset at block 1's batch size
        xb, yb = data[s * N1:(s + 1) * N1], labels[s * N1:(s + 1) * N1]
        blk1.step(pu.to_device_nhwc(torch, xb, 1), torch.from_numpy(yb).cuda(), 0.01, loss)
        _, a, _ = O1[0].step(xb, yb, 0.01)
        l2, _, _ = O1[1].step(a, yb, 0.01)
        for g, o in zip(G1, O1):                            # both sides continue from the checker's state
            for k in pu.PNAMES:
                v32, m32 = o.p[k].astype(np.float32), o.v[k].astype(np.float32)
                o.set(**{k: v32, "v" + k: m32})
                g.set_param(k, v32)
                g.set_param(k, m32, kind=nf.NF_K_MOMENTUM)
            for k in ("rmean", "rvar"):
                v32 = getattr(o, k).astype(np.float32)
                o.set(**{k: v32})
                g.set_param(k, v32)
    torch.cuda.synchronize()
    assert abs(float(loss[1].item()) - l2) <= 3e-3 * abs(l2)
    # cache: block 1's output for all K samples (chunks of N1), against the checker's eval forward
    cache = torch.zeros((K, 32, 32, 64), dtype=torch.bfloat16, device="cuda")
    for s in range(K // N1):
        blk1.cache(pu.to_device_nhwc(torch, data[s * N1:(s + 1) * N1], 1), cache[s * N1:(s + 1) * N1])
    ref_cache = O1[1].eval_forward(O1[0].eval_forward(data))
    torch.cuda.synchronize()
    assert pu.max_err(pu.from_device_nhwc(cache), ref_cache) <= pu.TOL[1]["t"]
    # re-batch at block 2's size: indices and labels bit-exact, rows bit-exact
    perm = synth.permutation(0x4E460005, 77, K)
    idx = torch.from_numpy(perm[:N2].copy()).cuda()
    lab_d = torch.from_numpy(labels).cuda()
    xb2 = torch.zeros((N2, 32, 32, 64), dtype=torch.bfloat16, device="cuda")
    yb2 = torch.zeros(N2, dtype=torch.int32, device="cuda")
    nf.nf_cache_gather(cache, lab_d, idx, xb2, yb2)
    torch.cuda.synchronize()
    assert np.array_equal(yb2.cpu().numpy(), labels[perm[:N2]])
    assert torch.equal(xb2.view(torch.int16), cache[idx.long()].view(torch.int16))
    # block 2, first layer, on the re-batched cache; the checker gets ITS OWN cached rows
    l = ls[2]
    c = _cfg(l, N2, classes)
    P, _, _ = pu.seeded_case(dict(c, N=1), 0x4E460510, bf16=True)
    x2 = synth.round_bf16(ref_cache[perm[:N2]]).astype(np.float64)
    _, _, _, G2 = _step_both(nf, torch, c, P, x2, labels[perm[:N2]])
    G2.close()
