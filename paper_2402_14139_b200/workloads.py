"""Shapes of the five synthetic workloads (layer lists only; no arithmetic of the method).

Each workload is a list of blocks; a block is (batch_size, [layer dict]).  A layer dict has
Cin, Cout, H, W (input size), stride, pool (a 2x2 max-pool belongs to the layer), F (aux filters).
The datasets the paper trains on are replaced by seeded synthetic tensors of the same shapes:
CIFAR-10-shaped (c1, c2), CIFAR-100-shaped (c3), an ImageNet-shaped post-stem tensor (c4) and
Tiny-ImageNet-shaped 64x64 inputs (c5).
"""
from __future__ import annotations


def _layer(Cin, Cout, H, W, F, stride=1, pool=False):
    return dict(Cin=Cin, Cout=Cout, H=H, W=W, F=F, stride=stride, pool=pool)


def out_hw(l):
    Ho, Wo = (l["H"] - 1) // l["stride"] + 1, (l["W"] - 1) // l["stride"] + 1
    return (Ho // 2, Wo // 2) if l["pool"] else (Ho, Wo)


def c1():
    """Single fp32 local-learning layer: x[8,3,32,32], conv 3->16, aux F=4, 10 classes."""
    return dict(name="c1", dtype="f32", classes=10, in_shape=(3, 32, 32), blocks=[(8, [_layer(3, 16, 32, 32, 4)])])


def c2():
    """VGG-style 4-layer block, bf16, batch 128, 32x32x3, 10 classes, F = 32,32,16,16."""
    ls = [_layer(3, 64, 32, 32, 32), _layer(64, 64, 32, 32, 32), _layer(64, 128, 32, 32, 16),
          _layer(128, 128, 32, 32, 16)]
    return dict(name="c2", dtype="bf16", classes=10, in_shape=(3, 32, 32), blocks=[(128, ls)])


def c3():
    """ResNet-18-shaped stack (no skips): stem 3->64, 4 stages x 4 convs (64,128,256,512), the first conv of
    stages 2-4 has stride 2; blocks = stages (stem in block 1) at batch 64/128/256/512, F 64/32/16/8."""
    blocks, C, S = [], 64, 32
    for b, (width, N, F) in enumerate([(64, 64, 64), (128, 128, 32), (256, 256, 16), (512, 512, 8)]):
        ls = []
        if b == 0:
            ls.append(_layer(3, 64, 32, 32, F))
        for k in range(4):
            stride = 2 if (b > 0 and k == 0) else 1
            ls.append(_layer(C, width, S, S, F, stride=stride))
            C = width
            S = (S - 1) // stride + 1
        blocks.append((N, ls))
    return dict(name="c3", dtype="bf16", classes=100, in_shape=(3, 32, 32), blocks=blocks)


def c4():
    """ImageNet-shaped single block: x[64,64,224,224] bf16 post-stem; conv 64->64 x2, then 64->128 stride 2;
    F = 16; 1000 classes.  The conv roofline workload."""
    ls = [_layer(64, 64, 224, 224, 16), _layer(64, 64, 224, 224, 16), _layer(64, 128, 224, 224, 16, stride=2)]
    return dict(name="c4", dtype="bf16", classes=1000, in_shape=(64, 224, 224), blocks=[(64, ls)])


def c4s():
    """c4 with batch 24 (input 154 MB, still larger than L2): the case profiler captures run on."""
    d = c4()
    d["name"] = "c4s"
    d["blocks"] = [(24, d["blocks"][0][1])]
    return d


VGG16 = [64, 64, "P", 128, 128, "P", 256, 256, 256, "P", 512, 512, 512, "P", 512, 512, 512, "P"]


def vgg_layers(cfg, S, aux_per_stage, Cin=3):
    """Layer list of a VGG-shaped net; a max-pool is counted with the conv layer it follows."""
    ls, stage = [], 0
    for i, v in enumerate(cfg):
        if v == "P":
            stage += 1
            continue
        pool = i + 1 < len(cfg) and cfg[i + 1] == "P"
        ls.append(_layer(Cin, v, S, S, aux_per_stage[stage], pool=pool))
        Cin = v
        if pool:
            S //= 2
    return ls


def c5(block_batches=None):
    """VGG-16-shaped net on 64x64x3, 200 classes; aux filters 64,32,16,8,4 per stage.  The default blocks
    (block_batches = [(first, last, batch)]) are what Algorithm 1 returns for layer_bytes_per_image() under a
    4 GB budget with rho = 0.4 and the batch size capped at the 10 000-image dataset: five blocks."""
    ls = vgg_layers(VGG16, 64, [64, 32, 16, 8, 4])
    if block_batches is None:
        block_batches = [(0, 0, 1260), (1, 1, 1904), (2, 3, 3045), (4, 5, 5935), (6, 12, 8602)]
    blocks = [(bs, ls[f:l + 1]) for f, l, bs in block_batches]
    return dict(name="c5", dtype="bf16", classes=200, in_shape=(3, 64, 64), blocks=blocks, layers=ls)


def c6(block_batches=None):
    """VGG-16-shaped net on 32x32x3, 100 classes, with the auxiliary filter counts of the AAN-LL rule (32 for the two
    layers before the first down-sampling, 256 after).  The default blocks are what the Profiler calls of the library
    (nf_profile_layer at batch sizes 512..4096, nf_max_batch under a 2 GB budget) and Algorithm 1 (rho = 0.4, batch size
    capped at the 50 000-image dataset) return: six blocks (the RGB first layer, whose input batch is also held as a
    64-channel padded copy, stands alone)."""
    chans = [v for v in VGG16 if v != "P"]
    lo, hi = min(chans) // 2, max(chans) // 2
    ls, S, Cin, k = [], 32, 3, 0
    for i, v in enumerate(VGG16):
        if v == "P":
            continue
        pool = i + 1 < len(VGG16) and VGG16[i + 1] == "P"
        ls.append(_layer(Cin, v, S, S, lo if k < 2 else hi, pool=pool))
        Cin, k = v, k + 1
        if pool:
            S //= 2
    if block_batches is None:
        block_batches = [(0, 0, 2486), (1, 2, 3452), (3, 5, 6366), (6, 8, 13526), (9, 9, 25672), (10, 12, 50000)]
    blocks = [(bs, ls[f:l + 1]) for f, l, bs in block_batches]
    return dict(name="c6", dtype="bf16", classes=100, in_shape=(3, 32, 32), blocks=blocks, layers=ls)


def layer_bytes_per_image(l, classes, esize=2):
    """Device bytes one more image costs a layer of this library (stored activations and gradients):
    y, dy (conv output size), a, da (after pool), h, dh (aux conv output) plus the small head tensors."""
    Ho, Wo = (l["H"] - 1) // l["stride"] + 1, (l["W"] - 1) // l["stride"] + 1
    Ha, Wa = out_hw(l)
    return esize * (2 * Ho * Wo * l["Cout"] + 2 * Ha * Wa * l["Cout"] + 2 * Ha * Wa * l["F"]) \
        + 4 * (2 * 4 * l["F"] + 2 * classes + 1) + esize * l["H"] * l["W"] * l["Cin"]


def step_flops(l, N):
    """Algorithmic FLOPs of one local step of a layer: main conv forward and weight gradient, aux conv
    forward, weight gradient and input gradient (2 flops per multiply-add, true channel counts)."""
    Ho, Wo = (l["H"] - 1) // l["stride"] + 1, (l["W"] - 1) // l["stride"] + 1
    Ha, Wa = out_hw(l)
    main = 2.0 * N * Ho * Wo * l["Cin"] * l["Cout"] * 9
    aux = 2.0 * N * Ha * Wa * l["Cout"] * l["F"] * 9
    return dict(conv_fwd=main, wgrad=main, aux_fwd=aux, aux_bwd=2 * aux)


ALL = dict(c1=c1, c2=c2, c3=c3, c4=c4, c5=c5, c4s=c4s, c6=c6)
