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

# Bounds for comparing the bf16 path with the checker in PURE fp64 (nothing rounded after the inputs and weights), fixed
# from the arithmetic: bfloat16 keeps 8 significant bits, so one rounding is off by at most 2^-8 of the value (half a
# unit in the last place, worst just above a power of two); act_out carries two of them (y, then a), the first on
# scale*y = a - shift whose size exceeds a's by the channel's shift (allowed here up to a fifth of the largest
# activation) -> 2^-7 * 1.1 of the largest element; the loss averages such noise over the head inputs and the batch ->
# well under 1e-2; rounding y moves about 0.2 % of the ReLU decisions (those with |z|
# below half an ulp of y times the scale), and a gradient that is a sum of noise-like terms moves by about
# sqrt(0.002) = 4.5 % of its own size when that share of its terms is switched -> gated at 1e-1 of the largest element.
UNROUNDED_TOL = dict(t=1e-1, loss=1e-2, act=2.0 ** -7 * 1.1)


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


def rms_err(got, ref):
    ref = np.asarray(ref, dtype=np.float64)
    d = np.asarray(got, dtype=np.float64) - ref
    return float(np.sqrt(np.mean(d * d)) / max(np.sqrt(np.mean(ref * ref)), 1e-30))


class Verdict:
    """Collects the per-tensor errors of one or more compared steps and judges them.

    The stated tolerance is on the LARGEST element error relative to the largest element, and it must hold whenever both
    sides take the same ReLU decisions.  In the bf16 path they occasionally do not, through no arithmetic fault: where the
    fp32 and fp64 accumulations of a conv output straddle a bfloat16 rounding boundary, y (and the activation a computed
    from it) differs by one unit in the last place between the two sides, and an auxiliary-conv output h (or a z) that lies
    that close to zero then gets opposite ReLU decisions.  One flipped h switches dp/|bin| on or off for that element, and
    through the input-gradient convolution it reaches every channel; on a small problem (a few thousand h elements) that
    one element is several per cent of the whole gradient.  Rule, applied per compared step:
      - the loss always has to meet its tolerance;
      - if every tensor meets the largest-element tolerance: fine;
      - otherwise the decisions of both sides are compared element by element (sign of the activation a, sign of the aux
        output h, and the winner of every max-pool window where the layer has a pool).  No
        differing decision: the test FAILS.  k differing decisions among n/2 active elements can move the energy of the
        gradients by about k/(n/2), so every root-mean-square error must stay below tol + 3*sqrt(k/(n/2)), else it FAILS;
        within that bound the test ends as XFAIL with the numbers -- never as passed."""

    def __init__(self, tol, what, soft_ok=True):
        self.tol, self.what, self.soft, self.worst, self.soft_ok = tol, what, [], {}, soft_ok
        self.pending, self.notes = [], []

    def add(self, name, got, ref, step=0):
        e = max_err(got, ref)
        self.worst[name] = max(self.worst.get(name, 0.0), e)
        if e > self.tol["t"]:
            assert self.soft_ok, (self.what, step, name, "max", e)
            self.pending.append((step, name, round(e, 4), round(rms_err(got, ref), 5)))
        return e

    def add_loss(self, got, ref, step=0):
        e = abs(got - ref) / abs(ref)
        self.worst["loss"] = max(self.worst.get("loss", 0.0), e)
        assert e <= self.tol["loss"], (self.what, step, "loss", got, ref)
        return e

    def judge_step(self, count_decisions):
        """count_decisions() -> [(differing decisions, elements)] for a, h and the pool winners of the step just compared."""
        if not self.pending:
            return
        counts = count_decisions()
        k = sum(c[0] for c in counts)
        assert k > 0, (self.what, "tolerance exceeded with identical decisions", self.pending)
        allowed = self.tol["t"] + 3.0 * float(np.sqrt(sum(c[0] / max(c[1] / 2.0, 1.0) for c in counts)))
        for step, name, e, r in self.pending:
            assert r <= allowed, (self.what, step, name, "rms", r, "allowed", allowed, "decisions", counts)
        self.notes.append(f"{self.pending} with {counts} (differing, elements) decisions for a, h, pool winners")
        self.soft += self.pending
        self.pending = []

    def finish(self):
        assert not self.pending, "judge_step was not called"
        if self.soft:
            import pytest
            pytest.xfail(f"{self.what}: largest-element tolerance {self.tol['t']} exceeded on (step, tensor, max, rms) "
                         + "; ".join(self.notes))
        return self.worst


def relu_decisions(nf, G, c, state, x, y, lr, act_g, store_bf16=True):
    """[(differing, elements)] for the activation a and the aux output h between the library (act_g and its stored h) and a
    fresh checker layer stepped from `state` (parameters, momentum, running statistics before the step) without update."""
    O = oracle_layer(c, {k: state[k] for k in PNAMES}, store_bf16=store_bf16)
    O.set(**{"v" + k: state["v" + k] for k in PNAMES}, rmean=state["rmean"], rvar=state["rvar"])
    _, act_o, tr = O.step(x, y, lr, update=False, trace=True)
    if G.kernel_family(5) == "mask":      # h itself was never stored: the library kept one sign bit per element
        m = G.stored("hmask").cpu().numpy()                                        # [N, Ha, Wa, Fp/8]
        pos_g = np.unpackbits(m, axis=3, bitorder="little")[..., :c["F"]].transpose(0, 3, 1, 2).astype(bool)
    else:
        pos_g = from_device_nhwc(G.stored("h"))[:, :c["F"]] > 0
    counts = [(int(((act_g > 0) != (act_o > 0)).sum()), act_o.size), (int((pos_g != (tr["h"] > 0)).sum()), tr["h"].size)]
    if c.get("pool"):
        # which element of each 2 x 2 window wins the max-pool (it alone receives the gradient): the library's stored y put
        # through the checker's BatchNorm coefficients, rounded as stored, first maximum in scan order
        y_g = from_device_nhwc(G.stored("y"))
        ch = (1, -1, 1, 1)
        z = state["gamma"].reshape(ch) * (y_g - tr["mu"].reshape(ch)) / np.sqrt(tr["var"].reshape(ch) + 1e-5) + state["beta"].reshape(ch)
        r = synth.round_bf16(np.maximum(z, 0.0)) if store_bf16 else np.maximum(z, 0.0)
        n_, c_, h_, w_ = r.shape
        win = r.reshape(n_, c_, h_ // 2, 2, w_ // 2, 2).transpose(0, 1, 2, 4, 3, 5).reshape(n_, c_, h_ // 2, w_ // 2, 4)
        arg_g = np.argmax(win, axis=4)
        counts.append((int(((arg_g != tr["argmax"]) & (act_o > 0)).sum()), act_o.size))
    return counts


def oracle_state(O):
    st = {k: O.p[k].copy() for k in PNAMES}
    st.update({"v" + k: O.v[k].copy() for k in PNAMES})
    st.update(rmean=O.rmean.copy(), rvar=O.rvar.copy())
    return st


def layer_cfg(l, N, classes):
    """Config dict of a workload layer (paper_2402_14139_b200.workloads) at batch size N."""
    return dict(N=N, Cin=l["Cin"], Cout=l["Cout"], H=l["H"], W=l["W"], F=l["F"], classes=classes, stride=l["stride"],
                pool=l["pool"])


def step_both(nf, torch, c, P, x, y, lr=0.01, store_bf16=True, tol=None, gate=True):
    """One bf16 step on both sides from the same state and inputs (x NCHW float64 holding bf16 values).

    Returns (errors per tensor, the checker's act_out, checker layer, library layer).  With store_bf16=False the checker
    keeps every tensor in fp64 (only the inputs and the weights are bf16-valued), which measures what the
    reduced-precision storage of the library costs; the caller then passes its own bounds in `tol`."""
    tol = tol or TOL[1]
    O = oracle_layer(c, P, store_bf16=store_bf16)
    G = gpu_layer(nf, c, P, nf.NF_BF16)
    xd = to_device_nhwc(torch, x, 1)
    loss_d = torch.zeros(1, device="cuda")
    act_d = G.new_act()
    state = oracle_state(O)
    loss_o, act_o, tr = O.step(x, y, lr, update=True, grads=True)
    G.step(xd, torch.from_numpy(np.ascontiguousarray(y, dtype=np.int32)).cuda(), lr, loss_d, act_d)
    torch.cuda.synchronize()
    assert G.status() == 0
    V = Verdict(tol, f"layer {c}")
    V.add_loss(float(loss_d.item()), loss_o)
    act_g = from_device_nhwc(act_d)
    V.add("act", act_g, act_o)
    for k in PNAMES:
        V.add("g" + k, G.get_param(k, nf.NF_K_GRAD), tr["g" + k])
        V.add("p" + k, G.get_param(k), O.p[k])
    V.add("rmean", G.get_param("rmean"), O.rmean)
    V.add("rvar", G.get_param("rvar"), O.rvar)
    errs = dict(V.worst)
    if gate:
        V.judge_step(lambda: relu_decisions(nf, G, c, state, x, y, lr, act_g, store_bf16))
        V.finish()
    else:
        V.pending = []
    return errs, act_o, O, G


def check_step(nf, torch, c, seed, dtype, lr=0.01, steps=1, report=None, fresh_batch=False):
    """Run `steps` consecutive local steps on both sides and compare after each:
    act_out, loss, every gradient, every updated parameter, momentum and running statistics.
    fresh_batch: every step draws its own seeded batch (as training does); otherwise all steps reuse the first one.

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
    V = Verdict(TOL[dtype], f"{c} seed {seed}", soft_ok=(dtype == 1))     # fp32 has no rounded storage: no exception
    for it in range(steps):
        if fresh_batch and it > 0:
            r = synth.round_bf16 if dtype == 1 else (lambda a: np.asarray(a, dtype=np.float32))
            x = r(synth.normal(seed, 8 + 16 * it, (c["N"], c["Cin"], c["H"], c["W"])))
            y = synth.labels(seed, 9 + 16 * it, c["N"], c["classes"])
            xd = to_device_nhwc(torch, x, dtype)
            yd = torch.from_numpy(y).cuda()
        state = oracle_state(O)
        loss_o, act_o, tr = O.step(x, y, lr, update=True, grads=True)
        G.step(xd, yd, lr, loss_d, act_d)
        torch.cuda.synchronize()
        assert G.status() == 0
        V.add_loss(float(loss_d.item()), loss_o, it)
        act_g = from_device_nhwc(act_d)
        V.add("act", act_g, act_o, it)
        for k in PNAMES:
            V.add("g" + k, G.get_param(k, nf.NF_K_GRAD), tr["g" + k], it)
            V.add("p" + k, G.get_param(k), O.p[k], it)
            V.add("v" + k, G.get_param(k, nf.NF_K_MOMENTUM), O.v[k], it)
        V.add("rmean", G.get_param("rmean"), O.rmean, it)
        V.add("rvar", G.get_param("rvar"), O.rvar, it)
        V.judge_step(lambda: relu_decisions(nf, G, c, state, x, y, lr, act_g))
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
        report.update(V.worst)
    G.close()
    return V.finish()
