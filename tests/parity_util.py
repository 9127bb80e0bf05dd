"""Shared helpers of the GPU parity tests: build the same layer on both sides from seeded inputs,
run one local step on each, and compare every output tensor within the stated tolerances.

Tolerances (written here once, used by every parity test):
  fp32 path : max-abs error <= 1e-4 * max|tensor| for outputs and gradients, loss relative error <= 1e-5
  bf16 path : max-abs error <= 3e-2 * max|tensor|,                           loss relative error <= 1e-3
In the bf16 path the checker keeps its two stored tensors (conv output, activation) in bfloat16 as
the kernels do, so ReLU masks and pool argmax are decided in the same precision on both sides;
all of its arithmetic stays fp64.
"""
import numpy as np

from oracle import nfo
from paper_2402_14139_b200 import synth

TOL = {0: dict(t=1e-4, loss=1e-5), 1: dict(t=3e-2, loss=1e-3)}
PNAMES = ("W", "gamma", "beta", "Wa", "ba", "Wf", "bf")


def seeded_case(c, seed, bf16):
    """Parameters and one batch for config dict c (keys N,Cin,Cout,H,W,F,classes,stride,pool)."""
    r = synth.round_bf16 if bf16 else (lambda a: np.asarray(a, dtype=np.float32))
    f32 = lambda a: np.asarray(a, dtype=np.float32)
    P = dict(
        W=r(synth.normal(seed, 1, (c["Cout"], c["Cin"], 3, 3), np.sqrt(2.0 / (c["Cin"] * 9)))),
        gamma=f32(1.0 + 0.2 * synth.normal(seed, 2, (c["Cout"],))),
        beta=f32(0.1 * synth.normal(seed, 3, (c["Cout"],))),
        Wa=r(synth.normal(seed, 4, (c["F"], c["Cout"], 3, 3), np.sqrt(2.0 / (c["Cout"] * 9)))),
        ba=f32(0.05 * synth.normal(seed, 5, (c["F"],))),
        Wf=f32(synth.normal(seed, 6, (c["classes"], 4 * c["F"]), np.sqrt(2.0 / (4 * c["F"])))),
        bf=f32(0.05 * synth.normal(seed, 7, (c["classes"],))))
    x = r(synth.normal(seed, 8, (c["N"], c["Cin"], c["H"], c["W"])))   # NCHW
    y = synth.labels(seed, 9, c["N"], c["classes"])
    return P, x, y


def oracle_layer(c, P, momentum=0.9, store_bf16=False):
    L = nfo.Layer(c["Cin"], c["Cout"], c["H"], c["W"], c["F"], c["classes"], c["N"], stride=c.get("stride", 1),
                  pool=c.get("pool", False), momentum=momentum, store_bf16=store_bf16, loss=c.get("loss", "ce"),
                  aux_pool=c.get("aux_pool", "avg"))
    L.set(**{k: np.asarray(v, dtype=np.float64) for k, v in P.items()})
    return L


def gpu_layer(nf, c, P, dtype, momentum=0.9, host_io=False):
    L = nf.Layer(c["Cin"], c["Cout"], c["H"], c["W"], c["F"], c["classes"], c["N"], stride=c.get("stride", 1),
                 maxpool=c.get("pool", False), dtype=dtype, momentum=momentum, host_io=host_io, loss=c.get("loss", "ce"),
                 aux_pool=c.get("aux_pool", "avg"))
    for k, v in P.items():
        L.set_param(k, v)
    return L


def to_device_nhwc(torch, x_nchw, dtype):
    t = torch.from_numpy(np.ascontiguousarray(np.transpose(x_nchw, (0, 2, 3, 1)), dtype=np.float32))
    return t.to(device="cuda", dtype=torch.float32 if dtype == 0 else torch.bfloat16).contiguous()


def from_device_nhwc(t):
    return np.transpose(t.float().cpu().numpy(), (0, 3, 1, 2)).astype(np.float64)


def max_err(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    scale = max(np.abs(ref).max(), 1e-30)
    return float(np.abs(np.asarray(got, dtype=np.float64) - ref).max() / scale)


def check_step(nf, torch, c, seed, dtype, lr=0.01, steps=1, report=None):
    """Run `steps` consecutive local steps on both sides on the same batch and compare after each:
    act_out, loss, every gradient, every updated parameter, momentum and running statistics.

    fp32 runs free.  In bf16, rounding of slightly different masters to different bfloat16 neighbours
    makes free-running trajectories drift apart, so after each compared step both sides are reset to
    the CHECKER's state rounded to fp32 (never the other way round)."""
    P, x, y = seeded_case(c, seed, bf16=(dtype == 1))
    O = oracle_layer(c, P, store_bf16=(dtype == 1))
    G = gpu_layer(nf, c, P, dtype)
    xd = to_device_nhwc(torch, x, dtype)
    yd = torch.from_numpy(y).cuda()
    loss_d = torch.zeros(1, dtype=torch.float32, device="cuda")
    act_d = G.new_act()
    tol = TOL[dtype]
    worst = {}
    for it in range(steps):
        loss_o, act_o, tr = O.step(x, y, lr, update=True, grads=True)
        G.step(xd, yd, lr, loss_d, act_d)
        torch.cuda.synchronize()
        assert G.status() == 0
        loss_g = float(loss_d.item())
        e = abs(loss_g - loss_o) / abs(loss_o)
        worst["loss"] = max(worst.get("loss", 0), e)
        assert e <= tol["loss"], (it, "loss", loss_g, loss_o)
        e = max_err(from_device_nhwc(act_d), act_o)
        worst["act"] = max(worst.get("act", 0), e)
        assert e <= tol["t"], (it, "act_out", e)
        for k in PNAMES:
            e = max_err(G.get_param(k, nf.NF_K_GRAD), tr["g" + k])
            worst["g" + k] = max(worst.get("g" + k, 0), e)
            assert e <= tol["t"], (it, "grad " + k, e)
            e = max_err(G.get_param(k), O.p[k])
            assert e <= tol["t"], (it, "param " + k, e)
            e = max_err(G.get_param(k, nf.NF_K_MOMENTUM), O.v[k])
            assert e <= tol["t"], (it, "momentum " + k, e)
        assert max_err(G.get_param("rmean"), O.rmean) <= tol["t"]
        assert max_err(G.get_param("rvar"), O.rvar) <= tol["t"]
        if dtype == 1 and it + 1 < steps:
            for k in PNAMES:
                v32, m32 = O.p[k].astype(np.float32), O.v[k].astype(np.float32)
                O.set(**{k: v32, "v" + k: m32})
                G.set_param(k, v32)
                G.set_param(k, m32, kind=nf.NF_K_MOMENTUM)
            for k in ("rmean", "rvar"):
                v32 = getattr(O, k).astype(np.float32)
                O.set(**{k: v32})
                G.set_param(k, v32)
    if report is not None:
        report.update(worst)
    G.close()
    return worst
