"""GPU parity of layers with an identity shortcut (residual networks): the shortcut tensor is added to the BatchNorm
output before the ReLU and carries no gradient.  Whole steps, the eval forward used by the cache and by early-exit
evaluation, and a two-layer residual block chained through nf_block_step, against the checker."""
import numpy as np
import pytest

from paper_2402_14139_b200 import synth
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
    (0, dict(N=4, Cin=8, Cout=8, H=10, W=12, F=6, classes=10, stride=1, pool=False)),
    (0, dict(N=4, Cin=4, Cout=8, H=8, W=8, F=4, classes=5, stride=1, pool=True)),
    (1, dict(N=8, Cin=64, Cout=64, H=16, W=112, F=16, classes=10, stride=1, pool=False)),   # folded tensor-core kernels
    (1, dict(N=8, Cin=64, Cout=128, H=16, W=16, F=32, classes=10, stride=2, pool=False)),
    (1, dict(N=12, Cin=64, Cout=64, H=16, W=16, F=64, classes=10, stride=1, pool=True)),
]


def _skip_for(c, seed, bf16):
    Ho, Wo = (c["H"] - 1) // c["stride"] + 1, (c["W"] - 1) // c["stride"] + 1
    s = np.maximum(synth.normal(seed, 31, (c["N"], c["Cout"], Ho, Wo)), 0.0)
    return synth.round_bf16(s).astype(np.float64) if bf16 else s.astype(np.float32).astype(np.float64)


@pytest.mark.parametrize("ci", range(len(CASES)))
def test_step_predict_and_cache_with_shortcut(env, ci):
    nf, torch = env
    dtype, c = CASES[ci]
    bf16 = dtype == 1
    tol = pu.TOL[dtype]
    seed = 0x4E46A000 + ci
    P, x, y = pu.seeded_case(c, seed, bf16=bf16)
    skip = _skip_for(c, seed, bf16)
    O = pu.oracle_layer(c, P, store_bf16=bf16)
    G = pu.gpu_layer(nf, c, P, nf.NF_BF16 if bf16 else nf.NF_F32)
    xd, yd = pu.to_device_nhwc(torch, x, dtype), torch.from_numpy(y).cuda()
    sd = pu.to_device_nhwc(torch, skip, dtype)
    G.set_skip(sd)
    loss_d, act_d = torch.zeros(1, device="cuda"), G.new_act()
    loss_o, act_o, tr = O.step(x, y, 0.02, update=True, grads=True, skip=skip)
    loss_plain = pu.oracle_layer(c, P, store_bf16=bf16).step(x, y, 0.02, update=False)[0]
    G.step(xd, yd, 0.02, loss_d, act_d)
    torch.cuda.synchronize()
    assert G.status() == 0
    assert abs(float(loss_d.item()) - loss_o) <= tol["loss"] * abs(loss_o) < abs(loss_plain - loss_o)
    assert pu.max_err(pu.from_device_nhwc(act_d), act_o) <= tol["t"]
    for k in pu.PNAMES:
        assert pu.max_err(G.get_param(k, nf.NF_K_GRAD), tr["g" + k]) <= tol["t"], "grad " + k
        assert pu.max_err(G.get_param(k), O.p[k]) <= tol["t"], "param " + k
    # eval forward: early-exit prediction and the cache of a one-layer block, both with the shortcut
    for k in pu.PNAMES + ("rmean", "rvar"):
        v32 = (O.p[k] if k in O.p else getattr(O, k)).astype(np.float32)
        O.set(**{k: v32})
        G.set_param(k, v32)
    act_e, logits_o, _ = O.predict(x, skip=skip)
    pred_d, logits_d = torch.zeros(c["N"], dtype=torch.int32, device="cuda"), torch.zeros((c["N"], c["classes"]), device="cuda")
    G.predict(xd, pred_d, act_out=act_d, logits_out=logits_d)
    blk = nf.Block([G])
    cache = G.new_act()
    blk.cache(xd, cache)
    torch.cuda.synchronize()
    assert pu.max_err(pu.from_device_nhwc(act_d), act_e) <= tol["t"]
    assert np.abs(logits_d.cpu().numpy() - logits_o).max() <= tol["t"] * np.abs(logits_o).max()
    assert torch.equal(cache.view(torch.int16 if bf16 else torch.int32), act_d.view(torch.int16 if bf16 else torch.int32))
    # removing the shortcut restores the plain layer
    G.set_skip(None)
    G.predict(xd, pred_d, act_out=act_d)
    torch.cuda.synchronize()
    assert pu.max_err(pu.from_device_nhwc(act_d), O.eval_forward(x)) <= tol["t"]
    blk.close()
    G.close()


def test_two_layer_residual_block_through_block_step(env):
    """conv-BN-ReLU, then conv-BN-(+block input)-ReLU: the second layer's shortcut is the block's input buffer."""
    nf, torch = env
    c = dict(N=8, Cin=64, Cout=64, H=16, W=16, F=16, classes=10, stride=1, pool=False)
    P1, x, y = pu.seeded_case(c, 0x4E46A100, bf16=True)
    P2, _, _ = pu.seeded_case(c, 0x4E46A101, bf16=True)
    x = np.maximum(x, 0.0)
    O1, O2 = pu.oracle_layer(c, P1, store_bf16=True), pu.oracle_layer(c, P2, store_bf16=True)
    G1, G2 = pu.gpu_layer(nf, c, P1, nf.NF_BF16), pu.gpu_layer(nf, c, P2, nf.NF_BF16)
    xd, yd = pu.to_device_nhwc(torch, x, 1), torch.from_numpy(y).cuda()
    G2.set_skip(xd)
    blk = nf.Block([G1, G2])
    loss_d, act_d = torch.zeros(2, device="cuda"), G2.new_act()
    l1, a1, _ = O1.step(x, y, 0.02, update=True)
    l2, a2, tr2 = O2.step(a1, y, 0.02, update=True, grads=True, skip=x)
    blk.step(xd, yd, 0.02, loss_d, act_d)
    torch.cuda.synchronize()
    tol = pu.TOL[1]
    got = loss_d.cpu().numpy()
    assert abs(got[0] - l1) <= tol["loss"] * abs(l1) and abs(got[1] - l2) <= 3 * tol["loss"] * abs(l2)
    assert pu.max_err(pu.from_device_nhwc(act_d), a2) <= tol["t"]
    for k in pu.PNAMES:
        assert pu.max_err(G2.get_param(k, nf.NF_K_GRAD), tr2["g" + k]) <= tol["t"], k
    assert nf.lib().nf_layer_set_skip(G2.h, xd.data_ptr() + 2) == nf.NF_EALIGN
    blk.close()
    G1.close()
    G2.close()


PROJ_CASES = [  # (dtype, layer config, channels of the block input) -- the block input has twice the layer's map size
    (0, dict(N=4, Cin=6, Cout=10, H=6, W=6, F=3, classes=5, stride=1, pool=False), 5),
    (1, dict(N=8, Cin=128, Cout=128, H=16, W=16, F=32, classes=100, stride=1, pool=False), 64),   # ResNet-18 stage 2, second conv
    (1, dict(N=6, Cin=64, Cout=64, H=8, W=8, F=16, classes=10, stride=1, pool=True), 32),          # with a pool after the sum
]


@pytest.mark.parametrize("ci", range(len(PROJ_CASES)))
def test_projection_shortcut_step_matches_checker(env, ci):
    """A layer joined by a projection shortcut (1x1 convolution with stride 2 on the block input + BatchNorm), two steps:
    the shortcut s, the layer's loss, activation and gradients, the gradient dz at the sum, the projection's own gradients,
    updated parameters, momentum and running statistics, and the eval-mode shortcut, all against the checker."""
    nf, torch = env
    from oracle import nfo
    dtype, c, Cs = PROJ_CASES[ci]
    bf = dtype == 1
    tol = pu.TOL[dtype]
    rnd = synth.round_bf16 if bf else (lambda a: np.asarray(a, dtype=np.float32))
    P, x, y = pu.seeded_case(c, 600 + ci, bf16=bf)
    xb = rnd(np.maximum(synth.normal(600 + ci, 20, (c["N"], Cs, 2 * c["H"], 2 * c["W"])), 0.0))
    Wp = rnd(synth.normal(600 + ci, 21, (c["Cout"], Cs), np.sqrt(2.0 / Cs)))
    gp = (1.0 + 0.2 * synth.normal(600 + ci, 22, (c["Cout"],))).astype(np.float32)
    bp = (0.1 * synth.normal(600 + ci, 23, (c["Cout"],))).astype(np.float32)
    O = pu.oracle_layer(c, P, store_bf16=bf)
    OP = nfo.Projection(Cs, c["Cout"], store_bf16=bf)
    OP.p["W"][...], OP.p["gamma"][...], OP.p["beta"][...] = Wp, gp, bp
    G = pu.gpu_layer(nf, c, P, dtype)
    GP = nf.Projection(Cs, c["Cout"], 2 * c["H"], 2 * c["W"], c["N"], dtype=dtype)
    for k, v in (("W", Wp), ("gamma", gp), ("beta", bp)):
        GP.set_param(k, v)
    xd, xbd = pu.to_device_nhwc(torch, x, dtype), pu.to_device_nhwc(torch, xb, dtype)
    yd = torch.from_numpy(y).cuda()
    s_d, dz_d, act_d = GP.new_out(), GP.new_out(), G.new_act()
    loss_d = torch.zeros(1, device="cuda")
    G.set_skip(s_d)
    G.set_skip_grad(dz_d)
    assert G.kernel_family(6) == "stored"
    for it in range(2):
        s_o = OP.forward(xb)
        loss_o, act_o, tr = O.step(x, y, 0.02, update=True, trace=True, skip=s_o)
        pg = OP.backward(tr["dz"], 0.02)
        GP.forward(xbd, s_d)
        G.step(xd, yd, 0.02, loss_d, act_d)
        GP.backward(xbd, dz_d, 0.02)
        torch.cuda.synchronize()
        assert G.status() == 0
        assert abs(float(loss_d.item()) - loss_o) <= tol["loss"] * abs(loss_o)
        assert pu.max_err(pu.from_device_nhwc(s_d), s_o) <= tol["t"]
        assert pu.max_err(pu.from_device_nhwc(act_d), act_o) <= tol["t"]
        assert pu.max_err(pu.from_device_nhwc(dz_d), tr["dz"]) <= tol["t"]
        for k in pu.PNAMES:
            assert pu.max_err(G.get_param(k, nf.NF_K_GRAD), tr["g" + k]) <= tol["t"], (it, k)
        for k, g in (("W", "gW"), ("gamma", "ggamma"), ("beta", "gbeta")):
            assert pu.max_err(GP.get_param(k, nf.NF_K_GRAD), pg[g]) <= tol["t"], (it, "proj grad", k)
            assert pu.max_err(GP.get_param(k), OP.p[k]) <= tol["t"], (it, "proj param", k)
            assert pu.max_err(GP.get_param(k, nf.NF_K_MOMENTUM), OP.v[k]) <= tol["t"], (it, "proj momentum", k)
        assert pu.max_err(GP.get_param("rmean"), OP.rmean) <= tol["t"] and pu.max_err(GP.get_param("rvar"), OP.rvar) <= tol["t"]
        if bf:      # both sides continue from the checker's state (bf16 trajectories drift otherwise)
            for k in pu.PNAMES:
                v32, m32 = O.p[k].astype(np.float32), O.v[k].astype(np.float32)
                O.set(**{k: v32, "v" + k: m32})
                G.set_param(k, v32)
                G.set_param(k, m32, kind=nf.NF_K_MOMENTUM)
            for k in ("rmean", "rvar"):
                v32 = getattr(O, k).astype(np.float32)
                O.set(**{k: v32})
                G.set_param(k, v32)
            for k in ("W", "gamma", "beta"):
                v32, m32 = OP.p[k].astype(np.float32), OP.v[k].astype(np.float32)
                OP.p[k][...], OP.v[k][...] = v32, m32
                GP.set_param(k, v32)
                GP.set_param(k, m32, kind=nf.NF_K_MOMENTUM)
            OP.rmean[...], OP.rvar[...] = OP.rmean.astype(np.float32), OP.rvar.astype(np.float32)
            GP.set_param("rmean", OP.rmean)
            GP.set_param("rvar", OP.rvar)
    GP.forward_eval(xbd[:3].contiguous(), s_d, count=3)
    torch.cuda.synchronize()
    assert pu.max_err(pu.from_device_nhwc(s_d[:3]), OP.eval_forward(xb[:3])) <= tol["t"]
    G.close()
    GP.close()
