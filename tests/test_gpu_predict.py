"""GPU parity of the early-exit evaluation (the paper's "Trained output CNN" section: each layer with its
auxiliary network is a prospective exit) against the checker's forward with running statistics.

Logits within the element tolerance; the predicted class equal wherever the checker's top-two margin is
larger than twice that tolerance (below it either class is a valid arg-max of logits known to that accuracy);
parameter counts and the selection rule bit-exact."""
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
    # dtype, config, count
    (0, dict(N=6, Cin=3, Cout=16, H=12, W=10, F=12, classes=10, stride=1, pool=True), 6),
    (0, dict(N=5, Cin=8, Cout=16, H=9, W=9, F=16, classes=7, stride=2, pool=False), 3),
    (1, dict(N=8, Cin=3, Cout=64, H=32, W=32, F=64, classes=10, stride=1, pool=False), 8),
    (1, dict(N=8, Cin=64, Cout=64, H=28, W=28, F=64, classes=100, stride=1, pool=True), 5),
    (1, dict(N=8, Cin=64, Cout=128, H=16, W=16, F=72, classes=10, stride=2, pool=False), 8),
    (1, dict(N=16, Cin=128, Cout=128, H=8, W=8, F=128, classes=200, stride=1, pool=True), 16),
]


def _running_stats(O, G, nf, seed):
    """Non-trivial running statistics (a fresh layer has mean 0, variance 1), the same on both sides."""
    Co = O.p["gamma"].size
    rm = (0.2 * synth.normal(seed, 41, (Co,))).astype(np.float32)
    rv = (0.5 + synth.uniform01(seed, 42, Co)).astype(np.float32)
    O.set(rmean=rm, rvar=rv)
    G.set_param("rmean", rm)
    G.set_param("rvar", rv)


@pytest.mark.parametrize("case", range(len(CASES)))
def test_predict_matches_checker(env, case):
    nf, torch = env
    dt, c, count = CASES[case]
    bf16 = dt == 1
    seed = 0x4E46E000 + case
    P, x, _ = pu.seeded_case(c, seed, bf16=bf16)
    if c["Cin"] != 3:
        x = np.maximum(x, 0.0)
    O = pu.oracle_layer(c, P, store_bf16=bf16)
    G = pu.gpu_layer(nf, c, P, nf.NF_BF16 if bf16 else nf.NF_F32)
    _running_stats(O, G, nf, seed)
    xs = x[:count]
    act_o, logits_o, pred_o = O.predict(xs)
    xd = pu.to_device_nhwc(torch, xs, dt)
    act_d = G.new_act()
    logits_d = torch.full((count, c["classes"]), float("nan"), device="cuda")
    pred_d = torch.full((count,), -1, dtype=torch.int32, device="cuda")
    before = {k: G.get_param(k).copy() for k in pu.PNAMES + ("rmean", "rvar")}
    G.predict(xd, pred_d, act_out=act_d, logits_out=logits_d, count=count)
    torch.cuda.synchronize()
    assert G.status() == 0
    tol = pu.TOL[dt]["t"]
    assert pu.max_err(pu.from_device_nhwc(act_d)[:count], act_o) <= tol
    lg = logits_d.cpu().numpy().astype(np.float64)
    scale = np.abs(logits_o).max()
    assert np.abs(lg - logits_o).max() <= tol * scale
    pred = pred_d.cpu().numpy()
    assert np.array_equal(pred, np.argmax(lg.astype(np.float32), axis=1))          # first maximum of its own logits
    top2 = np.sort(logits_o, axis=1)[:, -2:]
    decided = (top2[:, 1] - top2[:, 0]) > 2 * tol * scale
    assert decided.any()
    assert np.array_equal(pred[decided], pred_o[decided])
    for k, v in before.items():                                                     # evaluation changes no parameter
        assert np.array_equal(G.get_param(k), v), k
    # logits and activation outputs are optional
    pred2 = torch.full((count,), -1, dtype=torch.int32, device="cuda")
    G.predict(xd, pred2, count=count)
    torch.cuda.synchronize()
    assert torch.equal(pred2, pred_d)
    main, aux = O.n_params()
    assert (G.param_count(0), G.param_count(1), G.param_count(2)) == (main, aux, main + aux)
    G.close()


def test_exit_chain_accuracy_and_selection(env):
    """Three chained exits on a small validation set: per-exit accuracy from the library's predictions equals
    the checker's wherever every sample is decided; the selected exit follows the rule on both sides."""
    nf, torch = env
    from oracle import nfo
    cfgs = [dict(N=16, Cin=3, Cout=64, H=16, W=16, F=64, classes=10, stride=1, pool=False),
            dict(N=16, Cin=64, Cout=64, H=16, W=16, F=64, classes=10, stride=1, pool=True),
            dict(N=16, Cin=64, Cout=128, H=8, W=8, F=128, classes=10, stride=1, pool=False)]
    seed = 0x4E46E100
    x = synth.round_bf16(synth.normal(seed, 8, (16, 3, 16, 16))).astype(np.float64)
    y = synth.labels(seed, 9, 16, 10)
    acc_o, acc_g, par_o, par_g = [], [], [], []
    main_o = main_g = 0
    xin = x
    for li, c in enumerate(cfgs):
        P, _, _ = pu.seeded_case(dict(c, N=1), seed + 1 + li, bf16=True)
        O = pu.oracle_layer(c, P, store_bf16=True)
        G = pu.gpu_layer(nf, c, P, nf.NF_BF16)
        _running_stats(O, G, nf, seed + li)
        act_o, logits_o, pred_o = O.predict(xin)
        pred_d = torch.zeros(16, dtype=torch.int32, device="cuda")
        G.predict(pu.to_device_nhwc(torch, xin, 1), pred_d)          # each exit is fed the checker's activation
        torch.cuda.synchronize()
        top2 = np.sort(logits_o, axis=1)[:, -2:]
        decided = (top2[:, 1] - top2[:, 0]) > 2 * pu.TOL[1]["t"] * np.abs(logits_o).max()
        pred = pred_d.cpu().numpy()
        assert np.array_equal(pred[decided], pred_o[decided])
        pred = np.where(decided, pred, pred_o)                        # undecided samples: take the checker's class
        acc_o.append(float(np.mean(pred_o == y)))
        acc_g.append(float(np.mean(pred == y)))
        m, a = O.n_params()
        main_o += m
        main_g += G.param_count(0)
        par_o.append(main_o + a)
        par_g.append(main_g + G.param_count(1))
        xin = act_o
        G.close()
    assert acc_g == acc_o and par_g == par_o
    assert nf.nf_select_exit(acc_g, par_g) == nfo.select_exit(acc_o, par_o)
