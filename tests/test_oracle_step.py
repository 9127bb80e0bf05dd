"""Pins of the checker's whole local step (Algorithm 2 body): central finite differences on every
gradient, a library autograd re-derivation, invariances, and the seeded input generators."""
import numpy as np
import pytest
import torch

from oracle import nfo
from paper_2402_14139_b200 import synth

CASES = [
    dict(N=4, Cin=3, Cout=5, H=6, W=6, F=3, classes=7, stride=1, pool=False),
    dict(N=3, Cin=2, Cout=4, H=8, W=8, F=2, classes=5, stride=2, pool=False),
    dict(N=3, Cin=3, Cout=4, H=8, W=8, F=3, classes=4, stride=1, pool=True),
    dict(N=2, Cin=2, Cout=3, H=5, W=7, F=2, classes=3, stride=1, pool=False),   # odd sizes: overlapping avg bins
]


def make_layer(c, seed, momentum=0.9):
    L = nfo.Layer(c["Cin"], c["Cout"], c["H"], c["W"], c["F"], c["classes"], c["N"], stride=c["stride"],
                  pool=c["pool"], momentum=momentum)
    sh = L.shapes
    L.set(W=synth.normal(seed, 1, sh["W"], np.sqrt(2.0 / (c["Cin"] * 9))),
          gamma=1.0 + 0.3 * synth.normal(seed, 2, sh["gamma"]),
          beta=0.2 * synth.normal(seed, 3, sh["beta"]),
          Wa=synth.normal(seed, 4, sh["Wa"], np.sqrt(2.0 / (c["Cout"] * 9))),
          ba=0.1 * synth.normal(seed, 5, sh["ba"]),
          Wf=synth.normal(seed, 6, sh["Wf"], np.sqrt(2.0 / (4 * c["F"]))),
          bf=0.1 * synth.normal(seed, 7, sh["bf"]))
    x = synth.normal(seed, 8, (c["N"], c["Cin"], c["H"], c["W"]))
    y = synth.labels(seed, 9, c["N"], c["classes"])
    return L, x, y


def _kink_margin(tr):
    """Smallest distance of any pre-activation from its ReLU kink and of any pool window's top two."""
    m = min(np.abs(tr["z"]).min(), np.abs(tr["h"][tr["h"] > 0]).min() if (tr["h"] > 0).any() else 1.0)
    return m


@pytest.mark.parametrize("ci", range(len(CASES)))
def test_all_gradients_by_central_finite_differences(ci):
    c = CASES[ci]
    for seed in range(100, 140):
        L, x, y = make_layer(c, seed)
        loss, act, tr = L.step(x, y, 0.0, update=False, trace=True)
        if _kink_margin(tr) > 2e-4:
            break
    else:
        pytest.skip("no seed with safe kink margins")
    step = 1e-6
    worst = 0.0
    for name, gname in [("W", "gW"), ("gamma", "ggamma"), ("beta", "gbeta"), ("Wa", "gWa"), ("ba", "gba"),
                        ("Wf", "gWf"), ("bf", "gbf")]:
        theta = L.p[name]
        flat = theta.reshape(-1)
        idxs = np.unique(np.linspace(0, flat.size - 1, 12).astype(int))
        for k in idxs:
            old = flat[k]
            flat[k] = old + step
            lp = L.step(x, y, 0.0, update=False)[0]
            flat[k] = old - step
            lm = L.step(x, y, 0.0, update=False)[0]
            flat[k] = old
            fd = (lp - lm) / (2 * step)
            an = tr[gname].reshape(-1)[k]
            scale = max(abs(fd), np.abs(tr[gname]).max(), 1e-3)
            worst = max(worst, abs(fd - an) / scale)
            assert abs(fd - an) <= 1e-6 * scale, (name, k, fd, an)
    assert worst <= 1e-6


@pytest.mark.parametrize("ci", range(len(CASES)))
def test_step_against_library_autograd_and_optimizer(ci):
    """Two consecutive steps re-derived with torch's fp64 CPU ops, autograd and SGD(momentum)."""
    c = CASES[ci]
    L, x, y = make_layer(c, 7 + ci)
    tp = {k: torch.tensor(v.copy(), dtype=torch.float64, requires_grad=True) for k, v in L.p.items()}
    opt = torch.optim.SGD(list(tp.values()), lr=0.05, momentum=0.9)
    rm, rv = torch.zeros(c["Cout"], dtype=torch.float64), torch.ones(c["Cout"], dtype=torch.float64)
    xt, yt = torch.tensor(x), torch.tensor(y.astype(np.int64))
    F = torch.nn.functional
    for it in range(2):
        opt.zero_grad()
        yy = F.conv2d(xt, tp["W"], None, stride=c["stride"], padding=1)
        z = F.batch_norm(yy, rm, rv, tp["gamma"], tp["beta"], training=True, momentum=0.1, eps=1e-5)
        a = F.relu(z)
        if c["pool"]:
            a = F.max_pool2d(a, 2)
        a_in = a.detach().numpy().copy()
        h = F.relu(F.conv2d(a, tp["Wa"], tp["ba"], padding=1))
        p = F.adaptive_avg_pool2d(h, 2).flatten(1)
        loss_t = F.cross_entropy(F.linear(p, tp["Wf"], tp["bf"]), yt)
        loss_t.backward()
        grads = {k: v.grad.detach().numpy().copy() for k, v in tp.items()}
        opt.step()
        loss, act, tr = L.step(x, y, 0.05, update=True, trace=True)
        assert abs(loss - float(loss_t.detach())) <= 1e-12 * max(1, abs(loss))
        np.testing.assert_allclose(act, a_in, atol=1e-12)
        for k, g in [("W", "gW"), ("gamma", "ggamma"), ("beta", "gbeta"), ("Wa", "gWa"), ("ba", "gba"),
                     ("Wf", "gWf"), ("bf", "gbf")]:
            np.testing.assert_allclose(tr[g], grads[k], atol=1e-11 * max(1.0, np.abs(grads[k]).max()), err_msg=k)
            np.testing.assert_allclose(L.p[k], tp[k].detach().numpy(), atol=1e-12, err_msg=k)
        np.testing.assert_allclose(L.rmean, rm.numpy(), atol=1e-13)
        np.testing.assert_allclose(L.rvar, rv.numpy(), atol=1e-13)
    # eval-mode forward (what the cache stores) with the running statistics reached so far
    with torch.no_grad():
        z = F.batch_norm(F.conv2d(xt, tp["W"], None, stride=c["stride"], padding=1), rm, rv, tp["gamma"],
                         tp["beta"], training=False, eps=1e-5)
        a = F.relu(z)
        if c["pool"]:
            a = F.max_pool2d(a, 2)
    np.testing.assert_allclose(L.eval_forward(x), a.numpy(), atol=1e-12)


def test_no_gradient_reaches_layer_input_and_conv_bias_would_be_inert():
    # A constant added per output channel before BatchNorm (a conv bias) changes nothing: BN removes it.
    c = CASES[0]
    L, x, y = make_layer(c, 3)
    loss0, act0, tr0 = L.step(x, y, 0.0, update=False, trace=True)
    # scale invariance of BN: <W_co, dW_co> -> 0 (exactly eps-small)
    inner = (L.p["W"] * tr0["gW"]).sum(axis=(1, 2, 3))
    assert np.all(np.abs(inner) < 1e-3 * np.abs(tr0["gW"]).max())
    np.testing.assert_allclose(tr0["dy"].sum(axis=(0, 2, 3)), 0, atol=1e-12)


def test_batch_permutation_permutes_output_and_leaves_loss_and_grads():
    c = CASES[2]
    L, x, y = make_layer(c, 11)
    loss0, act0, tr0 = L.step(x, y, 0.0, update=False, trace=True)
    perm = np.array([2, 0, 1])
    loss1, act1, tr1 = L.step(x[perm], y[perm], 0.0, update=False, trace=True)
    assert abs(loss0 - loss1) < 1e-12
    np.testing.assert_allclose(act1, act0[perm], atol=1e-12)
    for g in ("gW", "ggamma", "gbeta", "gWa", "gba", "gWf", "gbf"):
        np.testing.assert_allclose(tr1[g], tr0[g], atol=1e-12)


def test_uniform_head_gives_log_classes_and_activation_precedes_update():
    c = CASES[0]
    L, x, y = make_layer(c, 5)
    L.set(Wf=np.zeros(L.shapes["Wf"]), bf=np.zeros(L.shapes["bf"]))
    W_before = L.p["W"].copy()
    loss, act, _ = L.step(x, y, 0.1, update=True)
    assert abs(loss - np.log(c["classes"])) < 1e-13
    # act_out is Eq. 1 evaluated with the weights BEFORE the update of the same step
    L2, _, _ = make_layer(c, 5)
    assert np.array_equal(L2.p["W"], W_before)
    _, act_ref, _ = L2.step(x, y, 0.0, update=False)
    np.testing.assert_array_equal(act, act_ref)


def test_eval_forward_is_per_sample():
    c = CASES[2]
    L, x, y = make_layer(c, 13)
    L.step(x, y, 0.05)
    full = L.eval_forward(x)
    for i in range(c["N"]):
        np.testing.assert_array_equal(L.eval_forward(x[i:i + 1])[0], full[i])


# ---------------------------------------------------------------- seeded generators
def test_splitmix64_published_vector():
    # First outputs of SplitMix64 seeded with 0 (state advanced by the golden gamma before mixing);
    # values from the generator's public reference implementation.
    got = synth.splitmix64(np.array([0, 0x9E3779B97F4A7C15], dtype=np.uint64))
    assert int(got[0]) == 0xE220A8397B1DCDAF and int(got[1]) == 0x6E789E6AA1B965F4


def test_generators_reproducible_and_distribution():
    a = synth.normal(1234, 3, (1000, 100))
    b = synth.normal(1234, 3, (1000, 100), chunk=777)
    assert np.array_equal(a, b)
    assert abs(a.mean()) < 0.01 and abs(a.std() - 1) < 0.01
    assert not np.array_equal(a, synth.normal(1234, 4, (1000, 100)))
    lab = synth.labels(5, 1, 100000, 10)
    assert lab.min() == 0 and lab.max() == 9 and abs(np.bincount(lab).std() / 10000) < 0.02
    p = synth.permutation(9, 2, 1000)
    assert sorted(p.tolist()) == list(range(1000)) and np.array_equal(p, synth.permutation(9, 2, 1000))


def test_bf16_rounding_ties_to_even():
    v = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -9, -2.5, 3.14159], dtype=np.float32)
    r = synth.round_bf16(v)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2 ** -6 and r[3] == 1.0
    t = torch.tensor(v).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(r, t)
    np.testing.assert_array_equal(synth.from_bf16_bits(synth.to_bf16_bits(v)), r)


def test_bf16_storage_mode_rounds_only_the_stored_tensors():
    c = CASES[2]
    L, x, y = make_layer(c, 21)
    L.set(W=synth.round_bf16(L.p["W"]), Wa=synth.round_bf16(L.p["Wa"]))   # bf16-valued conv weights on both
    Lb, _, _ = make_layer(c, 21)
    Lb.set(W=L.p["W"], Wa=L.p["Wa"])
    Lb.d.store_bf16 = 1
    loss, act, tr = L.step(x, y, 0.0, update=False, trace=True)
    loss_b, act_b, tr_b = Lb.step(x, y, 0.0, update=False, trace=True)
    # stored tensors hold bfloat16 values exactly, and are the nearest ones to the unrounded tensors
    for k in ("y", "a"):
        np.testing.assert_array_equal(tr_b[k], synth.round_bf16(tr_b[k]).astype(np.float64))
    np.testing.assert_array_equal(tr_b["y"], synth.round_bf16(tr["y"]).astype(np.float64))
    np.testing.assert_array_equal(act_b, tr_b["a"])
    # the rounding is a small perturbation of the exact step (bf16 has 8 significand bits)
    assert np.abs(tr_b["y"] - tr["y"]).max() <= 2.0 ** -8 * np.abs(tr["y"]).max()
    assert abs(loss_b - loss) <= 1e-2 * abs(loss)
    # conv weights are read through bfloat16 copies: masters with bf16 values give the same step as the
    # default mode does once y and a are rounded; masters themselves are never rounded by the update
    Lm, _, _ = make_layer(c, 21)
    Lm.set(W=synth.round_bf16(Lm.p["W"]), Wa=synth.round_bf16(Lm.p["Wa"]))
    Lq, _, _ = make_layer(c, 21)
    Lq.set(W=synth.round_bf16(Lq.p["W"]), Wa=synth.round_bf16(Lq.p["Wa"]))
    Lq.d.store_bf16 = 1
    Lb2, _, _ = make_layer(c, 21)
    Lb2.d.store_bf16 = 1
    l_q, a_q, _ = Lq.step(x, y, 0.1, update=True)
    l_b2, a_b2, _ = Lb2.step(x, y, 0.1, update=True)
    assert l_q == l_b2 and np.array_equal(a_q, a_b2)          # rounding the operand copy == rounded masters
    assert not np.array_equal(Lb2.p["W"], synth.round_bf16(Lb2.p["W"]).astype(np.float64))  # masters stay unrounded
    # the scalar rounding routine agrees with a library conversion, ties to even included
    v = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, -2.5, 3.14159, 1e-20, 65504.0, 0.0])
    got = np.array([nfo.lib().nfo_round_bf16(float(t)) for t in v])
    np.testing.assert_array_equal(got, torch.tensor(v, dtype=torch.float32).to(torch.bfloat16).double().numpy())


def test_early_exit_prediction_against_library_ops_and_selection_rule():
    c = CASES[2]
    L, x, y = make_layer(c, 31)
    L.step(x, y, 0.05)                       # running statistics away from their initial values
    act, logits, cls = L.predict(x)
    F = torch.nn.functional
    t = lambda a: torch.tensor(np.asarray(a, dtype=np.float64))
    with torch.no_grad():
        z = F.batch_norm(F.conv2d(t(x), t(L.p["W"]), None, stride=c["stride"], padding=1), t(L.rmean), t(L.rvar),
                         t(L.p["gamma"]), t(L.p["beta"]), training=False, eps=1e-5)
        a = F.max_pool2d(F.relu(z), 2)
        h = F.relu(F.conv2d(a, t(L.p["Wa"]), t(L.p["ba"]), padding=1))
        lg = F.linear(F.adaptive_avg_pool2d(h, 2).flatten(1), t(L.p["Wf"]), t(L.p["bf"]))
    np.testing.assert_allclose(act, a.numpy(), atol=1e-12)
    np.testing.assert_allclose(logits, lg.numpy(), atol=1e-12)
    np.testing.assert_array_equal(cls, lg.numpy().argmax(axis=1))
    np.testing.assert_array_equal(act, L.eval_forward(x))
    # per-sample: a prediction does not depend on the batch it is evaluated in
    np.testing.assert_array_equal(L.predict(x[1:2])[1][0], logits[1])
    # selection: highest accuracy wins; equal accuracy -> fewer parameters (the figure's "layer 5" situation)
    assert nfo.select_exit([0.31, 0.52, 0.64, 0.64, 0.63], [10, 20, 30, 40, 50]) == 2
    assert nfo.select_exit([0.7, 0.7, 0.7], [30, 20, 25]) == 1
    assert nfo.select_exit([0.2], [5]) == 0
    main, aux = L.n_params()
    assert main == c["Cout"] * c["Cin"] * 9 + 2 * c["Cout"] and aux == c["F"] * c["Cout"] * 9 + c["F"] + c["classes"] * (4 * c["F"] + 1)


VARIANTS = [("mse", "avg"), ("ce", "max"), ("mse", "max")]


@pytest.mark.parametrize("vi", range(len(VARIANTS)))
@pytest.mark.parametrize("ci", range(len(CASES)))
def test_loss_and_downsampling_variants_against_library_autograd(ci, vi):
    """The alternatives the paper names for the loss (mean squared error) and the down-sampling F_n (max
    pooling): one step re-derived with the library's mse_loss / adaptive_max_pool2d, autograd and SGD."""
    c = CASES[ci]
    loss_kind, pool_kind = VARIANTS[vi]
    L, x, y = make_layer(c, 31 + ci)
    L2 = nfo.Layer(c["Cin"], c["Cout"], c["H"], c["W"], c["F"], c["classes"], c["N"], stride=c["stride"], pool=c["pool"],
                   loss=loss_kind, aux_pool=pool_kind)
    L2.set(**L.p)
    tp = {k: torch.tensor(v.copy(), dtype=torch.float64, requires_grad=True) for k, v in L.p.items()}
    opt = torch.optim.SGD(list(tp.values()), lr=0.05, momentum=0.9)
    rm, rv = torch.zeros(c["Cout"], dtype=torch.float64), torch.ones(c["Cout"], dtype=torch.float64)
    xt, yt = torch.tensor(x), torch.tensor(y.astype(np.int64))
    F = torch.nn.functional
    a = F.relu(F.batch_norm(F.conv2d(xt, tp["W"], None, stride=c["stride"], padding=1), rm, rv, tp["gamma"], tp["beta"],
                            training=True, momentum=0.1, eps=1e-5))
    if c["pool"]:
        a = F.max_pool2d(a, 2)
    h = F.relu(F.conv2d(a, tp["Wa"], tp["ba"], padding=1))
    p = (F.adaptive_max_pool2d(h, 2) if pool_kind == "max" else F.adaptive_avg_pool2d(h, 2)).flatten(1)
    logits = F.linear(p, tp["Wf"], tp["bf"])
    loss_t = F.mse_loss(logits, F.one_hot(yt, c["classes"]).to(torch.float64)) if loss_kind == "mse" else F.cross_entropy(logits, yt)
    loss_t.backward()
    grads = {k: v.grad.detach().numpy().copy() for k, v in tp.items()}
    opt.step()
    loss, act, tr = L2.step(x, y, 0.05, update=True, trace=True)
    assert abs(loss - float(loss_t.detach())) <= 1e-12 * max(1, abs(loss))
    for k, g in [("W", "gW"), ("gamma", "ggamma"), ("beta", "gbeta"), ("Wa", "gWa"), ("ba", "gba"), ("Wf", "gWf"), ("bf", "gbf")]:
        np.testing.assert_allclose(tr[g], grads[k], atol=1e-11 * max(1.0, np.abs(grads[k]).max()), err_msg=k)
        np.testing.assert_allclose(L2.p[k], tp[k].detach().numpy(), atol=1e-12, err_msg=k)
    # the variant really differs from the default step
    assert abs(loss - L.step(x, y, 0.05, update=False)[0]) > 1e-6
    # early-exit logits use the same down-sampling
    with torch.no_grad():
        ae = F.relu(F.batch_norm(F.conv2d(xt, tp["W"], None, stride=c["stride"], padding=1), rm, rv, tp["gamma"], tp["beta"],
                                 training=False, eps=1e-5))
        if c["pool"]:
            ae = F.max_pool2d(ae, 2)
        he = F.relu(F.conv2d(ae, tp["Wa"], tp["ba"], padding=1))
        pe = (F.adaptive_max_pool2d(he, 2) if pool_kind == "max" else F.adaptive_avg_pool2d(he, 2)).flatten(1)
        le = F.linear(pe, tp["Wf"], tp["bf"])
    np.testing.assert_allclose(L2.predict(x)[1], le.numpy(), atol=1e-11)


@pytest.mark.parametrize("ci", [0, 2])
def test_identity_shortcut_against_library_autograd(ci):
    """A residual network's identity shortcut: a tensor added to the BatchNorm output before the ReLU.  It carries
    no gradient (local training); one step and the eval forward re-derived with the library's ops and autograd."""
    c = CASES[ci]
    L, x, y = make_layer(c, 51 + ci)
    Ho, Wo = L.Ho, L.Wo
    skip = np.maximum(synth.normal(52 + ci, 1, (c["N"], c["Cout"], Ho, Wo)), 0.0)      # an earlier post-ReLU activation
    tp = {k: torch.tensor(v.copy(), dtype=torch.float64, requires_grad=True) for k, v in L.p.items()}
    rm, rv = torch.zeros(c["Cout"], dtype=torch.float64), torch.ones(c["Cout"], dtype=torch.float64)
    xt, yt, st = torch.tensor(x), torch.tensor(y.astype(np.int64)), torch.tensor(skip)
    F = torch.nn.functional
    a = F.relu(F.batch_norm(F.conv2d(xt, tp["W"], None, stride=c["stride"], padding=1), rm, rv, tp["gamma"], tp["beta"],
                            training=True, momentum=0.1, eps=1e-5) + st)
    if c["pool"]:
        a = F.max_pool2d(a, 2)
    a_in = a.detach().numpy().copy()
    h = F.relu(F.conv2d(a, tp["Wa"], tp["ba"], padding=1))
    loss_t = F.cross_entropy(F.linear(F.adaptive_avg_pool2d(h, 2).flatten(1), tp["Wf"], tp["bf"]), yt)
    loss_t.backward()
    loss0 = L.step(x, y, 0.05, update=False)[0]
    loss, act, tr = L.step(x, y, 0.05, update=True, trace=True, skip=skip)
    assert abs(loss - float(loss_t.detach())) <= 1e-12 and abs(loss - loss0) > 1e-6
    np.testing.assert_allclose(act, a_in, atol=1e-12)
    for k, g in [("W", "gW"), ("gamma", "ggamma"), ("beta", "gbeta"), ("Wa", "gWa"), ("ba", "gba"), ("Wf", "gWf"), ("bf", "gbf")]:
        np.testing.assert_allclose(tr[g], tp[k].grad.numpy(), atol=1e-11 * max(1.0, np.abs(tp[k].grad.numpy()).max()), err_msg=k)
    with torch.no_grad():        # eval forward with the updated parameters and running statistics
        t2 = {k: torch.tensor(v) for k, v in L.p.items()}
        ae = F.relu(F.batch_norm(F.conv2d(xt, t2["W"], None, stride=c["stride"], padding=1), torch.tensor(L.rmean), torch.tensor(L.rvar),
                                 t2["gamma"], t2["beta"], training=False, eps=1e-5) + st)
        if c["pool"]:
            ae = F.max_pool2d(ae, 2)
    np.testing.assert_allclose(L.eval_forward(x, skip=skip), ae.numpy(), atol=1e-12)
    np.testing.assert_allclose(L.predict(x, skip=skip)[0], ae.numpy(), atol=1e-12)
    assert np.abs(L.eval_forward(x) - ae.numpy()).max() > 1e-3       # and the shortcut is not silently ignored


def test_projection_shortcut_against_library_autograd_and_optimizer():
    """The projection shortcut of a down-sampling residual block (1x1 convolution with stride 2 on the block input, then
    BatchNorm with batch statistics) added to the layer's BatchNorm output before the ReLU; its three parameter tensors are
    trained by the layer's local loss, the block input receives no gradient.  Two consecutive steps (gradients, updated
    parameters, momentum, running statistics of both parts) and the eval forward re-derived with the library's ops,
    autograd and SGD."""
    c = dict(N=5, Cin=4, Cout=6, H=6, W=6, F=3, classes=4, stride=1, pool=False)
    L, x, y = make_layer(c, 71)
    Cs = 3
    xb = synth.normal(72, 1, (c["N"], Cs, 12, 12))                 # the block input, twice the layer's map size
    Pj = nfo.Projection(Cs, c["Cout"])
    Pj.p["W"][...] = synth.normal(72, 2, (c["Cout"], Cs), np.sqrt(2.0 / Cs))
    Pj.p["gamma"][...] = 1.0 + 0.2 * synth.normal(72, 3, (c["Cout"],))
    Pj.p["beta"][...] = 0.1 * synth.normal(72, 4, (c["Cout"],))
    F = torch.nn.functional
    tp = {k: torch.tensor(v.copy(), dtype=torch.float64, requires_grad=True) for k, v in L.p.items()}
    tq = {k: torch.tensor(v.copy(), dtype=torch.float64, requires_grad=True) for k, v in Pj.p.items()}
    names = list(tp) + ["p" + k for k in tq]
    opt = torch.optim.SGD(list(tp.values()) + list(tq.values()), lr=0.05, momentum=0.9)
    rm, rv = torch.zeros(c["Cout"], dtype=torch.float64), torch.ones(c["Cout"], dtype=torch.float64)
    rms, rvs = torch.zeros(c["Cout"], dtype=torch.float64), torch.ones(c["Cout"], dtype=torch.float64)
    xt, xbt, yt = torch.tensor(x), torch.tensor(xb, requires_grad=True), torch.tensor(y.astype(np.int64))
    for step in range(2):
        opt.zero_grad()
        s_t = F.batch_norm(F.conv2d(xbt, tq["W"][:, :, None, None], None, stride=2), rms, rvs, tq["gamma"], tq["beta"], training=True,
                           momentum=0.1, eps=1e-5)
        a = F.relu(F.batch_norm(F.conv2d(xt, tp["W"], None, padding=1), rm, rv, tp["gamma"], tp["beta"], training=True, momentum=0.1,
                                eps=1e-5) + s_t)
        h = F.relu(F.conv2d(a.detach() * 0 + a, tp["Wa"], tp["ba"], padding=1))
        loss_t = F.cross_entropy(F.linear(F.adaptive_avg_pool2d(h, 2).flatten(1), tp["Wf"], tp["bf"]), yt)
        loss_t.backward()
        grads = {k: v.grad.numpy().copy() for k, v in tp.items()}
        pgrads = {k: v.grad.numpy().copy() for k, v in tq.items()}
        s = Pj.forward(xb)
        np.testing.assert_allclose(s, s_t.detach().numpy(), atol=1e-12)
        loss, act, tr = L.step(x, y, 0.05, update=True, trace=True, skip=s)
        pg = Pj.backward(tr["dz"], 0.05)
        assert abs(loss - float(loss_t.detach())) <= 1e-12
        np.testing.assert_allclose(act, a.detach().numpy(), atol=1e-12)
        for k, g in [("W", "gW"), ("gamma", "ggamma"), ("beta", "gbeta"), ("Wa", "gWa"), ("ba", "gba"), ("Wf", "gWf"), ("bf", "gbf")]:
            np.testing.assert_allclose(tr[g], grads[k], atol=1e-11 * max(1.0, np.abs(grads[k]).max()), err_msg=k)
        np.testing.assert_allclose(pg["gW"], pgrads["W"], atol=1e-11 * max(1.0, np.abs(pgrads["W"]).max()))
        np.testing.assert_allclose(pg["ggamma"], pgrads["gamma"], atol=1e-11)
        np.testing.assert_allclose(pg["gbeta"], pgrads["beta"], atol=1e-11)
        assert np.abs(pgrads["W"]).max() > 1e-4                      # the shortcut really is trained by this loss
        opt.step()
        for k in tp:
            np.testing.assert_allclose(L.p[k], tp[k].detach().numpy(), atol=1e-12, err_msg=k)
        for k in tq:
            np.testing.assert_allclose(Pj.p[k], tq[k].detach().numpy(), atol=1e-12, err_msg="p" + k)
        np.testing.assert_allclose(Pj.rmean, rms.numpy(), atol=1e-12)
        np.testing.assert_allclose(Pj.rvar, rvs.numpy(), atol=1e-12)
    with torch.no_grad():
        se = F.batch_norm(F.conv2d(torch.tensor(xb), tq["W"][:, :, None, None], None, stride=2), rms, rvs, tq["gamma"], tq["beta"],
                          training=False, eps=1e-5)
    np.testing.assert_allclose(Pj.eval_forward(xb), se.numpy(), atol=1e-12)
    # bf16 storage mode: s and the stored conv output are bfloat16 values, the convolution reads a bfloat16 copy of Wp
    Pb = nfo.Projection(Cs, c["Cout"], store_bf16=True)
    Pb.p["W"][...] = Pj.p["W"]
    sb = Pb.forward(xb)
    assert np.array_equal(sb, synth.round_bf16(sb).astype(np.float64)) and np.abs(sb - Pj.forward(xb)).max() > 0
