"""GPU parity: the CUDA library (through its C ABI) against the fp64 CPU checker, element by element,
on the same seeded inputs.  Tolerances are those of parity_util.TOL."""
import numpy as np
import pytest

from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    return nf, torch


# config 1 of the benchmark suite: single fp32 layer, 8x3x32x32, 3->16, F=4, 10 classes
CFG1 = dict(N=8, Cin=3, Cout=16, H=32, W=32, F=4, classes=10, stride=1, pool=False)

SMALL = [
    dict(N=4, Cin=3, Cout=5, H=6, W=6, F=3, classes=7, stride=1, pool=False),      # ragged channel counts
    dict(N=3, Cin=2, Cout=4, H=8, W=8, F=2, classes=5, stride=2, pool=False),      # stride 2
    dict(N=3, Cin=3, Cout=4, H=8, W=8, F=3, classes=4, stride=1, pool=True),       # max-pool layer
    dict(N=2, Cin=2, Cout=3, H=5, W=7, F=2, classes=3, stride=1, pool=False),      # odd sizes, overlapping bins
    dict(N=2, Cin=35, Cout=18, H=19, W=21, F=5, classes=11, stride=2, pool=False), # several tiles + ragged tails
    dict(N=2, Cin=1, Cout=1, H=1, W=1, F=1, classes=2, stride=1, pool=False),      # degenerate 1x1 image
    dict(N=2, Cin=4, Cout=8, H=2, W=2, F=2, classes=3, stride=1, pool=True),       # pool down to 1x1
    dict(N=70, Cin=3, Cout=4, H=4, W=4, F=6, classes=300, stride=1, pool=False),   # class-sliced head: 43 slices, 2 sample chunks
]
WIDE_HEAD = dict(N=2, Cin=2, Cout=3, H=4, W=4, F=520, classes=3, stride=1, pool=False)  # 2080 head inputs: one block per sample


def test_config1_fp32_single_step(env):
    nf, torch = env
    w = pu.check_step(nf, torch, CFG1, seed=0x4E460001, dtype=nf.NF_F32, lr=0.01, steps=1)
    print("config1 fp32 worst relative errors:", w)


def test_config1_fp32_three_steps(env):
    nf, torch = env
    pu.check_step(nf, torch, CFG1, seed=0x4E460001, dtype=nf.NF_F32, lr=0.01, steps=3)


@pytest.mark.parametrize("ci", range(len(SMALL)))
def test_small_shapes_fp32(env, ci):
    nf, torch = env
    pu.check_step(nf, torch, SMALL[ci], seed=100 + ci, dtype=nf.NF_F32, lr=0.05, steps=2)


def test_head_wider_than_the_sliced_kernels_fp32(env):
    nf, torch = env
    pu.check_step(nf, torch, WIDE_HEAD, seed=150, dtype=nf.NF_F32, lr=1e-3, steps=2)


@pytest.mark.parametrize("ci", range(len(SMALL) - 3))
def test_small_shapes_bf16(env, ci):
    nf, torch = env
    pu.check_step(nf, torch, SMALL[ci], seed=200 + ci, dtype=nf.NF_BF16, lr=0.05, steps=1)


def test_uniform_head_loss_is_log_classes(env):
    nf, torch = env
    c = CFG1
    P, x, y = pu.seeded_case(c, 5, bf16=False)
    P["Wf"][:] = 0
    P["bf"][:] = 0
    G = pu.gpu_layer(nf, c, P, nf.NF_F32)
    loss = torch.zeros(1, device="cuda")
    act = G.new_act()
    G.step(pu.to_device_nhwc(torch, x, 0), torch.from_numpy(y).cuda(), 0.0, loss, act)
    assert abs(float(loss.item()) - np.log(10)) <= 1e-5 * np.log(10)
    g = G.get_param("bf", nf.NF_K_GRAD)
    assert abs(g.sum()) < 1e-6          # softmax-CE gradients sum to zero across classes


def test_bad_label_is_flagged_and_clamped(env):
    nf, torch = env
    c = CFG1
    P, x, y = pu.seeded_case(c, 6, bf16=False)
    G = pu.gpu_layer(nf, c, P, nf.NF_F32)
    y = y.copy()
    y[3] = 10
    loss = torch.zeros(1, device="cuda")
    G.step(pu.to_device_nhwc(torch, x, 0), torch.from_numpy(y).cuda(), 0.0, loss, G.new_act())
    assert G.status() & nf.NF_ELABEL
    assert G.status() == 0
    assert np.isfinite(float(loss.item()))


def test_argument_errors(env):
    nf, torch = env
    c = CFG1
    P, x, y = pu.seeded_case(c, 7, bf16=False)
    G = pu.gpu_layer(nf, c, P, nf.NF_F32)
    xd = pu.to_device_nhwc(torch, x, 0)
    yd = torch.from_numpy(y).cuda()
    loss = torch.zeros(1, device="cuda")
    act = G.new_act()
    with pytest.raises(nf.NfError):
        G.step(xd, yd, 0.1, loss, None)                      # act_out is required
    with pytest.raises(nf.NfError):
        G.step(xd.view(-1)[1:], yd, 0.1, loss, act)          # 4-byte offset: not 16-byte aligned
    with pytest.raises(nf.NfError):
        G.set_param("W", np.zeros((16, 3, 3, 3), np.float32), kind=nf.NF_K_GRAD)


def test_step_host_matches_device_step(env):
    nf, torch = env
    c = CFG1
    P, x, y = pu.seeded_case(c, 8, bf16=False)
    A = pu.gpu_layer(nf, c, P, nf.NF_F32)
    B = pu.gpu_layer(nf, c, P, nf.NF_F32, host_io=True)
    xh = torch.from_numpy(np.ascontiguousarray(np.transpose(x, (0, 2, 3, 1)))).pin_memory()
    yh = torch.from_numpy(y).pin_memory()
    loss_a = torch.zeros(1, device="cuda")
    act_a = A.new_act()
    A.step(xh.cuda(), yh.cuda(), 0.01, loss_a, act_a)
    loss_h = torch.zeros(1).pin_memory()
    act_h = torch.empty(act_a.shape, dtype=act_a.dtype).pin_memory()
    B.step_host(xh, yh, 0.01, loss_h, act_h)
    assert float(loss_h.item()) == float(loss_a.item())
    assert torch.equal(act_h, act_a.cpu())
    assert np.array_equal(A.get_param("W"), B.get_param("W"))


# shapes the tcgen05 kernels cover (bf16, channel counts multiples of 64, tileable image sizes)
TC = [
    dict(N=4, Cin=64, Cout=64, H=32, W=32, F=16, classes=10, stride=1, pool=False),
    dict(N=6, Cin=128, Cout=128, H=16, W=16, F=16, classes=10, stride=1, pool=True),
    dict(N=3, Cin=64, Cout=128, H=16, W=32, F=8, classes=20, stride=1, pool=False),
    dict(N=4, Cin=64, Cout=64, H=16, W=16, F=4, classes=10, stride=1, pool=False),    # aux tile padded 4 -> 16
    dict(N=4, Cin=64, Cout=64, H=16, W=16, F=32, classes=10, stride=1, pool=False),
    dict(N=12, Cin=64, Cout=64, H=16, W=16, F=64, classes=10, stride=1, pool=True),
    dict(N=4, Cin=64, Cout=64, H=16, W=16, F=12, classes=10, stride=1, pool=False),   # F not a multiple of 8
    dict(N=6, Cin=64, Cout=128, H=32, W=32, F=16, classes=10, stride=2, pool=False),  # stride-2 tensor-core kernels
    dict(N=3, Cin=64, Cout=64, H=16, W=112, F=16, classes=10, stride=1, pool=False),  # folded-tap forward (W % 14 == 0)
    dict(N=3, Cin=64, Cout=128, H=16, W=112, F=8, classes=10, stride=1, pool=False),  # folded aux forward, two K chunks, F < 16
    dict(N=3, Cin=64, Cout=64, H=16, W=112, F=40, classes=10, stride=1, pool=False),  # folded aux forward, group width 64
    dict(N=3, Cin=64, Cout=64, H=16, W=112, F=32, classes=10, stride=1, pool=False),  # folded aux input gradient, 32-channel K
    dict(N=9, Cin=128, Cout=128, H=8, W=8, F=16, classes=10, stride=1, pool=True),    # 8x8 maps: 2 images per tile (ragged), aux at 4x4
    dict(N=16, Cin=64, Cout=64, H=4, W=4, F=8, classes=10, stride=1, pool=False),     # 4x4 maps: 8 images per tile
    dict(N=12, Cin=64, Cout=128, H=16, W=16, F=32, classes=10, stride=2, pool=False), # stride 2 down to 8x8, multi-image tiles
    dict(N=8, Cin=64, Cout=64, H=16, W=16, F=128, classes=10, stride=1, pool=False),    # more than 64 aux filters: main-conv kernels
    dict(N=16, Cin=128, Cout=128, H=16, W=16, F=256, classes=100, stride=1, pool=True), # the classic setting of 256 aux filters
    dict(N=200, Cin=64, Cout=64, H=2, W=2, F=32, classes=10, stride=1, pool=True),       # aux conv on 1x1 maps: 128 images per tile
    dict(N=520, Cin=64, Cout=128, H=2, W=2, F=128, classes=10, stride=1, pool=True),     # the same with more than 64 aux filters
    dict(N=300, Cin=64, Cout=64, H=1, W=1, F=16, classes=10, stride=1, pool=False),      # everything on 1x1 maps
    dict(N=32, Cin=128, Cout=256, H=8, W=8, F=16, classes=10, stride=1, pool=False),     # per-tap weight gradient, 256-wide instructions
    dict(N=16, Cin=64, Cout=256, H=16, W=16, F=32, classes=10, stride=2, pool=False),    # the same with stride 2
    dict(N=6, Cin=128, Cout=256, H=16, W=32, F=16, classes=10, stride=1, pool=True),     # 256-wide forward on a map that tiles
    dict(N=3, Cin=64, Cout=64, H=16, W=56, F=16, classes=10, stride=1, pool=False),   # width not a multiple of 16: input gradient with folded taps
    dict(N=2, Cin=64, Cout=128, H=8, W=112, F=24, classes=10, stride=1, pool=False),  # unfolded input gradient: two channel tiles, 32-channel K, F < 32
    dict(N=5, Cin=64, Cout=64, H=16, W=16, F=16, classes=700, stride=1, pool=False),  # few samples, many classes: 47 class slices in the head
    dict(N=3, Cin=64, Cout=64, H=24, W=112, F=16, classes=10, stride=1, pool=False),   # fused normalisation, but a tile row straddles the pooling quadrants: h stored
    dict(N=2, Cin=64, Cout=64, H=32, W=56, F=40, classes=10, stride=1, pool=False),   # pooled epilogue with three 16-channel groups (F = 40), 2 x 2 tiles per quadrant
    dict(N=3, Cin=64, Cout=64, H=16, W=48, F=24, classes=10, stride=1, pool=False),   # folded kernels on a width that is no multiple of 14: ragged last tile column
    dict(N=2, Cin=128, Cout=64, H=8, W=64, F=8, classes=10, stride=1, pool=False),    # the same with two input-channel chunks in the aux forward's sibling, 64 columns
]


@pytest.mark.parametrize("ci", range(len(TC)))
def test_tensor_core_shapes_bf16(env, ci):
    nf, torch = env
    c = TC[ci]
    P, x, y = pu.seeded_case(c, 1, bf16=True)
    G = pu.gpu_layer(nf, c, P, nf.NF_BF16)
    assert G.kernel_family(0) == "tcgen05" and G.kernel_family(1) == "tcgen05"
    if c["F"] > 64 or c["H"] <= 2:
        assert G.kernel_family(2) == "tcgen05" and G.kernel_family(3) == "tcgen05"
    G.close()
    w = pu.check_step(nf, torch, c, seed=400 + ci, dtype=nf.NF_BF16, lr=0.02, steps=2)
    print(w)


SWEEP_SEEDS = [7001, 7002, 7003, 7004, 7005]


@pytest.mark.parametrize("seed", SWEEP_SEEDS)
@pytest.mark.parametrize("ci", range(len(TC)))
def test_tensor_core_shapes_bf16_seed_sweep(env, ci, seed):
    """Every shape above over a fixed set of seeds that was written down before the first run, two steps each, the second
    on a batch of its own (as training draws one): no seed, batch or size is chosen among passing ones.  A case that
    exceeds the tolerance while the two sides provably took different ReLU decisions is reported as XFAIL with the counts
    (parity_util.Verdict); one that exceeds it with identical decisions fails."""
    nf, torch = env
    pu.check_step(nf, torch, TC[ci], seed=seed + 100 * ci, dtype=nf.NF_BF16, lr=0.02, steps=2, fresh_batch=True)


def test_fused_normalisation_is_selected(env):
    """Where the folded aux forward applies (width a multiple of 14, no pool) it also applies BatchNorm + ReLU and writes
    act_out, so the parity cases of those shapes above check the fused kernel; other shapes keep the separate pass."""
    nf, torch = env
    for c, want in ((TC[8], "fused"), (TC[9], "fused"), (TC[3], "separate"), (TC[1], "separate")):
        P, x, y = pu.seeded_case(c, 1, bf16=True)
        G = pu.gpu_layer(nf, c, P, nf.NF_BF16)
        assert G.kernel_family(4) == want, (c, G.kernel_family(4))
        # 16 x 112 maps: a 14 x 8 tile never straddles a pooling quadrant (8 x 56), so the same kernel also pools h in its
        # epilogue and keeps only its sign bits
        assert G.kernel_family(5) == ("mask" if want == "fused" else "stored")
        G.close()
    P, x, y = pu.seeded_case(TC[0], 1, bf16=True)      # 32 columns: three 14-column tiles, the last one ragged; no whole-tile quadrants
    G = pu.gpu_layer(nf, TC[0], P, nf.NF_BF16)
    assert G.kernel_family(4) == "fused" and G.kernel_family(5) == "stored"
    G.close()
    c = dict(TC[8], H=24)       # 24 rows: the quadrant boundary (row 12) cuts through a tile row, h is stored
    P, x, y = pu.seeded_case(c, 1, bf16=True)
    G = pu.gpu_layer(nf, c, P, nf.NF_BF16)
    assert G.kernel_family(4) == "fused" and G.kernel_family(5) == "stored"
    G.close()


LARGE_HEAD = [
    (0, dict(N=600, Cin=8, Cout=16, H=4, W=4, F=32, classes=256, stride=1, pool=False)),      # fp32, 600*128*256 products
    (1, dict(N=512, Cin=64, Cout=64, H=4, W=4, F=64, classes=128, stride=1, pool=False)),     # bf16 tensor-core layer
    (1, dict(N=700, Cin=64, Cout=64, H=2, W=2, F=128, classes=100, stride=1, pool=True)),     # ragged tiles, 512 head inputs
]


@pytest.mark.parametrize("ci", range(len(LARGE_HEAD)))
@pytest.mark.parametrize("loss", ["ce", "mse"])
def test_large_batch_head(env, ci, loss):
    """Batches large enough for the tiled head kernels (logits, dp and gWf as matrix products, the batch
    reduction of gWf in ranges): whole steps against the checker, then the early-exit forward."""
    nf, torch = env
    dtype, c = LARGE_HEAD[ci]
    c = dict(c, loss=loss)
    pu.check_step(nf, torch, c, seed=900 + ci, dtype=dtype, lr=0.02, steps=2)
    bf16 = dtype == 1
    P, x, _ = pu.seeded_case(c, 950 + ci, bf16=bf16)
    if c["Cin"] == 64:
        x = np.maximum(x, 0.0)
    O = pu.oracle_layer(c, P, store_bf16=bf16)
    G = pu.gpu_layer(nf, c, P, nf.NF_BF16 if bf16 else nf.NF_F32)
    _, logits_o, pred_o = O.predict(x)
    logits_d = torch.zeros((c["N"], c["classes"]), device="cuda")
    pred_d = torch.zeros(c["N"], dtype=torch.int32, device="cuda")
    G.predict(pu.to_device_nhwc(torch, x, dtype), pred_d, logits_out=logits_d)
    torch.cuda.synchronize()
    tol = pu.TOL[dtype]["t"] * np.abs(logits_o).max()
    lg = logits_d.cpu().numpy()
    assert np.abs(lg - logits_o).max() <= tol
    assert np.array_equal(pred_d.cpu().numpy(), np.argmax(lg, axis=1))
    top2 = np.sort(logits_o, axis=1)[:, -2:]
    decided = (top2[:, 1] - top2[:, 0]) > 2 * tol
    assert decided.sum() > c["N"] // 8 and np.array_equal(pred_d.cpu().numpy()[decided], pred_o[decided])
    G.close()


@pytest.mark.parametrize("ci", [0, 8, 5])
def test_stored_intermediates_match_checker(env, ci):
    """The tensors a step leaves in the workspace (nf_layer_stored_tensor), element by element against the checker's trace: the
    conv output y, the pooled aux output p, the logits, dp, dh (rebuilt from the sign mask where h is never stored) and the
    gradient dy at the conv output; da too where the layer stores it (two-pass layers never form it in memory).  On the layers
    that keep a sign mask instead of h the mask itself is compared bit for bit with the checker's h > 0."""
    nf, torch = env
    c = TC[ci]
    P, x, y = pu.seeded_case(c, 1300 + ci, bf16=True)
    O = pu.oracle_layer(c, P, store_bf16=True)
    G = pu.gpu_layer(nf, c, P, nf.NF_BF16)
    loss = torch.zeros(1, device="cuda")
    G.step(pu.to_device_nhwc(torch, x, 1), torch.from_numpy(y).cuda(), 0.02, loss, G.new_act())
    torch.cuda.synchronize()
    _, _, tr = O.step(x, y, 0.02, update=False, trace=True)
    t = pu.TOL[1]["t"]
    F = c["F"]
    assert pu.max_err(pu.from_device_nhwc(G.stored("y")), tr["y"]) <= t
    pg = G.stored("p").cpu().numpy().reshape(c["N"], -1, 4)[:, :F].reshape(c["N"], -1)
    assert pu.max_err(pg, tr["p"]) <= t
    assert pu.max_err(G.stored("logits").cpu().numpy(), tr["logits"]) <= t
    dpg = G.stored("dp").cpu().numpy().reshape(c["N"], -1, 4)[:, :F].reshape(c["N"], -1)
    assert pu.max_err(dpg, tr["dp"]) <= t
    if G.kernel_family(5) == "mask":
        m = np.unpackbits(G.stored("hmask").cpu().numpy(), axis=3, bitorder="little")[..., :F].transpose(0, 3, 1, 2).astype(bool)
        flips = int((m != (tr["h"] > 0)).sum())
        assert flips <= 2, flips                      # a sign may differ where h is within rounding of zero
    else:
        flips = int(((pu.from_device_nhwc(G.stored("h"))[:, :F] > 0) != (tr["h"] > 0)).sum())
    if flips == 0:      # with identical ReLU decisions the backward tensors agree element by element
        assert pu.max_err(pu.from_device_nhwc(G.stored("dh"))[:, :F], tr["dh"]) <= t
        if G.kernel_family(6) == "stored":
            assert pu.max_err(pu.from_device_nhwc(G.stored("da")), tr["da"]) <= t
        assert pu.max_err(pu.from_device_nhwc(G.stored("dy")), tr["dy"]) <= t
    G.close()
