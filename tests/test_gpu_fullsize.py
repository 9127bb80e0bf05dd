"""Full-size checks in the launch configuration the benchmark times (c4: 64 x 224 x 224 x 64, bf16).

The checker cannot run a whole 64-image step in seconds, so: (a) the two dense contractions are run
stand-alone at full size and compared on sampled outputs the checker computes one by one, and (b) the
whole block step is run at full size and checked through properties that hold at any size."""
import numpy as np
import pytest

from oracle import nfo
from paper_2402_14139_b200 import synth, workloads
from tests import parity_util as pu

pytestmark = pytest.mark.gpu

N, C, H, W = 64, 64, 224, 224


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    nf.nf_set_stream(None)
    return nf, torch


@pytest.fixture(scope="module")
def big(env):
    nf, torch = env
    x = np.empty((N, H, W, C), dtype=np.float32)          # channels-last, bf16 values
    g = np.empty((N, H, W, C), dtype=np.float32)
    for n in range(N):                                    # per-image chunks keep the host footprint low
        x[n] = synth.round_bf16(synth.normal(0x4E460004, 100 + n, (H, W, C)))
        g[n] = synth.round_bf16(synth.normal(0x4E460004, 300 + n, (H, W, C)))
    w = synth.round_bf16(synth.normal(0x4E460004, 1, (C, C, 3, 3), np.sqrt(2.0 / (9 * C))))
    return x, g, w


def test_full_size_forward_on_sampled_outputs(env, big):
    nf, torch = env
    x, g, w = big
    xd = torch.from_numpy(x).cuda().to(torch.bfloat16)
    wk = np.ascontiguousarray(np.transpose(w.reshape(C, C, 9), (2, 0, 1)))
    wd = torch.from_numpy(wk).cuda().to(torch.bfloat16)
    yd = torch.empty((N, H, W, C), device="cuda", dtype=torch.bfloat16)
    nf.nf_conv3x3_forward(nf.NF_BF16, xd, wd, 1, yd)
    torch.cuda.synchronize()
    assert nf.nf_op_status() == 0
    rng = np.random.default_rng(7)
    S = 3000
    ns, is_, js = rng.integers(0, N, S), rng.integers(0, H, S), rng.integers(0, W, S)
    is_[:200] = rng.choice([0, H - 1], 200)               # image borders and tile seams included
    js[100:300] = rng.choice([0, W - 1, 15, 16], 200)
    patches = np.zeros((S, C, 3, 3))
    xp = np.pad(x, ((0, 0), (1, 1), (1, 1), (0, 0)))
    for k in range(S):
        patches[k] = np.transpose(xp[ns[k], is_[k]:is_[k] + 3, js[k]:js[k] + 3, :], (2, 0, 1))
    ref = nfo.conv3x3(patches, w.astype(np.float64))[:, :, 1, 1]          # the checker, one output pixel each
    got = yd[torch.from_numpy(ns).cuda(), torch.from_numpy(is_).cuda(), torch.from_numpy(js).cuda()].float().cpu().numpy()
    assert np.abs(got - ref).max() <= pu.TOL[1]["t"] * np.abs(ref).max()


def test_full_size_weight_gradient_on_sampled_outputs(env, big):
    nf, torch = env
    x, g, w = big
    xd = torch.from_numpy(x).cuda().to(torch.bfloat16)
    gd = torch.from_numpy(g).cuda().to(torch.bfloat16)
    scratch = torch.empty(nf.nf_conv3x3_wgrad_scratch_bytes(N, H, W, C, C, 1), dtype=torch.uint8, device="cuda")
    dw = torch.empty((9, C, C), device="cuda", dtype=torch.float32)
    nf.nf_conv3x3_wgrad(nf.NF_BF16, xd, gd, 1, scratch, dw)
    torch.cuda.synchronize()
    assert nf.nf_op_status() == 0
    got = dw.cpu().numpy()
    rng = np.random.default_rng(8)
    scale = np.abs(got).max()
    for co, ci in zip(rng.integers(0, C, 6), rng.integers(0, C, 6)):
        xs = np.ascontiguousarray(x[:, :, :, ci])[:, None].astype(np.float64)      # [N,1,H,W]
        gs = np.ascontiguousarray(g[:, :, :, co])[:, None].astype(np.float64)
        ref = nfo.conv3x3_wgrad(xs, gs)[0, 0].reshape(9)                            # all nine taps of (co, ci)
        assert np.abs(got[:, co, ci] - ref).max() <= pu.TOL[1]["t"] * scale


def test_full_size_block_step_properties(env):
    """c4 block (three layers, N=64) as bench.py builds it: reproducible bit for bit, status clean,
    uniform head gives ln(classes), softmax-CE gradients sum to zero, momentum after the first step
    equals the gradient."""
    import bench
    nf, torch = env
    wl = workloads.c4()
    losses, params = [], []
    g = torch.Generator(device="cuda")
    g.manual_seed(11)
    x = torch.randn((N, H, W, C), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    labels = torch.randint(0, 1000, (N,), generator=g, device="cuda", dtype=torch.int32)
    for rep in range(2):
        block, layers = bench.build_block(nf, torch, wl, 0, 0x4E460004, host_io=False)
        for L in layers:
            L.set_param("Wf", np.zeros(L.shapes["Wf"], np.float32))
        loss = torch.zeros(3, device="cuda")
        block.step(x, labels, 0.01, loss)
        torch.cuda.synchronize()
        assert [L.status() for L in layers] == [0, 0, 0]
        assert [L.kernel_family(k) for L in layers for k in range(4)] == ["tcgen05"] * 12
        losses.append(loss.cpu().numpy().copy())
        params.append([layers[0].get_param("W"), layers[2].get_param("Wa"), layers[1].get_param("gamma")])
        if rep == 0:
            for L in layers:
                assert abs(L.get_param("bf", nf.NF_K_GRAD).sum()) < 1e-5
                np.testing.assert_array_equal(L.get_param("W", nf.NF_K_MOMENTUM), L.get_param("W", nf.NF_K_GRAD))
        block.close()
        for L in layers:
            L.close()
        del block, layers
        torch.cuda.empty_cache()
    np.testing.assert_allclose(losses[0], np.log(1000.0), rtol=1e-5)
    assert np.array_equal(losses[0], losses[1])
    for a, b in zip(params[0], params[1]):
        assert np.array_equal(a, b)
