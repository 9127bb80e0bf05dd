"""Pins of the fp64 CPU checker against mathematics, library routines and the paper's printed values.

None of these tests touches the CUDA library.  Each is chosen so that a plausible mistake in the
checker (dropped term, wrong sign or index, transposed operand) fails at least one of them.
"""
import os

import numpy as np
import pytest
import scipy.signal
import scipy.special

from oracle import nfo
from paper_2402_14139_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(20240214)


# ---------------------------------------------------------------- convolution (Eq. 1, Eq. 2)
def _corr_lib(x, w, bias, stride):
    """Same conv through scipy's correlate2d on a zero-padded image (a library routine)."""
    N, Ci, H, W = x.shape
    Co = w.shape[0]
    y = np.zeros((N, Co, H, W))
    for n in range(N):
        for co in range(Co):
            for ci in range(Ci):
                y[n, co] += scipy.signal.correlate2d(np.pad(x[n, ci], 1), w[co, ci], mode="valid")
            if bias is not None:
                y[n, co] += bias[co]
    return y[:, :, ::stride, ::stride]


@pytest.mark.parametrize("shape,stride", [((2, 3, 5, 7), 1), ((1, 2, 6, 6), 2), ((2, 1, 7, 5), 2), ((1, 4, 1, 1), 1)])
def test_conv_matches_library_correlation(shape, stride):
    x = rng.standard_normal(shape)
    w = rng.standard_normal((3, shape[1], 3, 3))
    b = rng.standard_normal(3)
    np.testing.assert_allclose(nfo.conv3x3(x, w, b, stride), _corr_lib(x, w, b, stride), rtol=0, atol=1e-12)
    np.testing.assert_allclose(nfo.conv3x3(x, w, None, stride), _corr_lib(x, w, None, stride), rtol=0, atol=1e-12)


def test_conv_centre_tap_is_identity_and_ones_count_neighbours():
    x = rng.standard_normal((2, 3, 6, 5))
    w = np.zeros((3, 3, 3, 3))
    for c in range(3):
        w[c, c, 1, 1] = 1.0
    np.testing.assert_array_equal(nfo.conv3x3(x, w), x)
    y = nfo.conv3x3(np.ones((1, 2, 5, 5)), np.ones((1, 2, 3, 3)))[0, 0]
    assert y[2, 2] == 18 and y[0, 2] == 12 and y[0, 0] == 8 and y[4, 4] == 8 and y[2, 0] == 12


def test_conv_single_off_centre_tap_shifts_the_right_way():
    # w[kh=0,kw=2] = 1 reads x[i-1, j+1]: catches a flipped (true-convolution) or transposed kernel.
    x = np.arange(20.0).reshape(1, 1, 4, 5)
    w = np.zeros((1, 1, 3, 3))
    w[0, 0, 0, 2] = 1.0
    y = nfo.conv3x3(x, w)[0, 0]
    assert y[1, 0] == x[0, 0, 0, 1] and y[0, 0] == 0.0 and y[3, 4] == 0.0 and y[3, 3] == x[0, 0, 2, 4]


@pytest.mark.parametrize("stride", [1, 2])
def test_conv_adjoint_identities(stride):
    # <conv(x,W), g> = <W, wgrad(x,g)> = <x, dgrad(W,g)>
    x = rng.standard_normal((2, 3, 6, 7))
    w = rng.standard_normal((4, 3, 3, 3))
    y = nfo.conv3x3(x, w, None, stride)
    g = rng.standard_normal(y.shape)
    lhs = float((y * g).sum())
    assert abs(lhs - float((w * nfo.conv3x3_wgrad(x, g, stride)).sum())) < 1e-11 * max(1, abs(lhs))
    assert abs(lhs - float((x * nfo.conv3x3_dgrad(w, g, 6, 7, stride)).sum())) < 1e-11 * max(1, abs(lhs))


# ---------------------------------------------------------------- BatchNorm
def test_bn_forward_against_numpy_and_invariants():
    y = rng.standard_normal((4, 3, 5, 6)) * 3 + 1.5
    gamma, beta = rng.standard_normal(3), rng.standard_normal(3)
    mu, var, xhat, z = nfo.bn_train(y, gamma, beta, 1e-5)
    np.testing.assert_allclose(mu, y.mean(axis=(0, 2, 3)), atol=1e-13)
    np.testing.assert_allclose(var, y.var(axis=(0, 2, 3)), atol=1e-12)  # biased
    np.testing.assert_allclose(z.mean(axis=(0, 2, 3)), beta, atol=1e-12)
    np.testing.assert_allclose(z.var(axis=(0, 2, 3)), gamma ** 2 * var / (var + 1e-5), rtol=1e-10)


def test_bn_backward_orthogonality_and_finite_difference():
    y = rng.standard_normal((3, 2, 4, 4))
    gamma, beta = np.array([1.3, -0.7]), np.array([0.2, 0.1])
    mu, var, xhat, z = nfo.bn_train(y, gamma, beta, 1e-5)
    dz = rng.standard_normal(y.shape)
    dg, db, dy = nfo.bn_bwd(dz, xhat, gamma, var, 1e-5)
    np.testing.assert_allclose(dy.sum(axis=(0, 2, 3)), 0, atol=1e-12)
    # sum(xhat^2) = M v/(v+eps), hence sum(dy*xhat) = gamma/sqrt(v+eps) * dgamma * eps/(v+eps): zero as eps -> 0
    np.testing.assert_allclose((dy * xhat).sum(axis=(0, 2, 3)), gamma / np.sqrt(var + 1e-5) * dg * 1e-5 / (var + 1e-5),
                               atol=1e-12)
    np.testing.assert_allclose(dg, (dz * xhat).sum(axis=(0, 2, 3)), atol=1e-12)
    np.testing.assert_allclose(db, dz.sum(axis=(0, 2, 3)), atol=1e-12)
    f = lambda yy: float((nfo.bn_train(yy, gamma, beta, 1e-5)[3] * dz).sum())
    for idx in [(0, 0, 0, 0), (2, 1, 3, 2), (1, 0, 2, 1)]:
        e = np.zeros_like(y)
        e[idx] = 1e-6
        fd = (f(y + e) - f(y - e)) / 2e-6
        assert abs(fd - dy[idx]) <= 1e-6 * max(1.0, abs(fd))


# ---------------------------------------------------------------- pooling
def test_maxpool_and_argmax_first_maximum():
    r = rng.standard_normal((2, 3, 4, 6))
    a, arg = nfo.maxpool2(r)
    ref = r.reshape(2, 3, 2, 2, 3, 2).max(axis=(3, 5))
    np.testing.assert_array_equal(a, ref)
    win = r.reshape(2, 3, 2, 2, 3, 2).transpose(0, 1, 2, 4, 3, 5).reshape(2, 3, 2, 3, 4)
    np.testing.assert_array_equal(arg, win.argmax(axis=-1))
    t = np.zeros((1, 1, 2, 2))
    t[0, 0, 0, 1] = t[0, 0, 1, 0] = 5.0
    assert nfo.maxpool2(t)[1][0, 0, 0, 0] == 1  # first of two equal maxima in scan order


def test_adaptive_avgpool_even_odd_and_single_pixel():
    h = rng.standard_normal((2, 3, 4, 6))
    np.testing.assert_allclose(nfo.avgpool_2x2(h), h.reshape(2, 3, 2, 2, 2, 3).mean(axis=(3, 5)), atol=1e-14)
    h3 = np.arange(9.0).reshape(1, 1, 3, 3)  # odd: bins [0,2) and [1,3) overlap on the middle row/column
    np.testing.assert_allclose(nfo.avgpool_2x2(h3)[0, 0], [[2.0, 3.0], [5.0, 6.0]], atol=1e-14)
    h1 = np.full((1, 2, 1, 1), 7.0)
    np.testing.assert_array_equal(nfo.avgpool_2x2(h1), np.full((1, 2, 2, 2), 7.0))
    # backward is the adjoint of forward
    for (H, W) in [(4, 6), (3, 3), (1, 1), (5, 2)]:
        hh = rng.standard_normal((2, 2, H, W))
        dp = rng.standard_normal((2, 2, 2, 2))
        assert abs((nfo.avgpool_2x2(hh) * dp).sum() - (hh * nfo.avgpool_2x2_bwd(dp, H, W)).sum()) < 1e-12


# ---------------------------------------------------------------- loss (Eq. 3)
def test_softmax_ce_uniform_logits_rows_sum_to_zero_and_library_logsumexp():
    for K in (10, 100, 1000):
        labels = rng.integers(0, K, 7)
        loss, dl = nfo.softmax_ce(np.full((7, K), 3.25), labels)
        assert abs(loss - np.log(K)) < 1e-13
    logits = rng.standard_normal((5, 10)) * 4
    labels = rng.integers(0, 10, 5)
    loss, dl = nfo.softmax_ce(logits, labels)
    ref = np.mean(scipy.special.logsumexp(logits, axis=1) - logits[np.arange(5), labels])
    assert abs(loss - ref) < 1e-13
    np.testing.assert_allclose(dl.sum(axis=1), 0, atol=1e-15)
    assert np.all(np.abs(dl) <= 1.0 / 5 + 1e-15)
    sm = scipy.special.softmax(logits, axis=1)
    sm[np.arange(5), labels] -= 1
    np.testing.assert_allclose(dl, sm / 5, atol=1e-14)
    big = logits + 1e4  # shift invariance / no overflow
    assert abs(nfo.softmax_ce(big, labels)[0] - ref) < 1e-9


# ---------------------------------------------------------------- update (Algorithm 2, last step)
def test_sgd_first_step_and_constant_gradient_closed_form():
    th0 = rng.standard_normal(11)
    g = rng.standard_normal(11)
    th, v = th0.copy(), np.zeros(11)
    nfo.sgd(th, v, g, 0.01, 0.9)
    np.testing.assert_allclose(th, th0 - 0.01 * g, atol=1e-16)
    for _ in range(6):
        nfo.sgd(th, v, g, 0.01, 0.9)
    T, mu = 7, 0.9
    coef = sum((1 - mu ** t) / (1 - mu) for t in range(1, T + 1))
    np.testing.assert_allclose(th, th0 - 0.01 * g * coef, atol=1e-14)
    th, v = th0.copy(), np.zeros(11)
    nfo.sgd(th, v, g, 0.1, 0.0)  # the paper's plain SGD (Appendix B) is the mu = 0 case
    nfo.sgd(th, v, g, 0.1, 0.0)
    np.testing.assert_allclose(th, th0 - 0.2 * g, atol=1e-15)


# ---------------------------------------------------------------- Algorithm 1
def _read_cols(name):
    with open(os.path.join(GOLD, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def test_partition_on_paper_batch_sizes():
    mb = [int(v) for v in _read_cols("vgg19_max_batch_630mb.txt")[0]]
    assert len(mb) == 16
    # derived by hand from Algorithm 1 with rho = 0.4 (consecutive-layer comparison), B = 512
    blocks = nfo.partition(mb, 512, 0.4)
    assert blocks == [(0, 2, 30), (3, 3, 60), (4, 7, 90), (8, 11, 195), (12, 15, 512)]
    assert nfo.partition(mb, 10 ** 9, 0.4)[-1] == (12, 15, 810)
    # every layer lands in exactly one block and a block never exceeds any member's feasible size
    for B in (64, 200, 512):
        bl = nfo.partition(mb, B, 0.4)
        assert [f for f, _, _ in bl] == [0] + [l + 1 for _, l, _ in bl[:-1]] and bl[-1][1] == 15
        for f, l, bs in bl:
            assert bs == min(min(mb[f:l + 1]), B)
    assert nfo.partition([10, 14, 15], 100, 0.4) == [(0, 2, 10)]   # inclusive threshold: |14-10| = 0.4*10
    assert nfo.partition([10, 15], 100, 0.4) == [(0, 0, 10), (1, 1, 15)]


def test_linear_memory_model_on_paper_points():
    rows = np.array(_read_cols("vgg11_layer_memory.txt"), dtype=float)
    b, l1 = rows[:, 0], rows[:, 1]
    slope, icpt = np.polyfit(b, l1, 1)
    assert abs(slope - 17.19) < 0.02
    t = nfo.max_batch_from_line(slope, icpt, 630.0)
    assert icpt + slope * t <= 630.0 < icpt + slope * (t + 1)
    assert t == 36


def test_mse_loss_against_library_closed_form_and_finite_differences():
    """Eq. 3 with the mean-squared-error loss: library mse_loss on one-hot targets (and its autograd
    gradient), the closed form for constant logits, and a central finite difference of one entry."""
    import torch
    N, K = 5, 7
    logits = synth.normal(61, 1, (N, K))
    labels = synth.labels(61, 2, N, K)
    loss, dl = nfo.mse_onehot(logits, labels)
    zt = torch.tensor(logits, dtype=torch.float64, requires_grad=True)
    tt = torch.nn.functional.one_hot(torch.tensor(labels.astype(np.int64)), K).to(torch.float64)
    ref = torch.nn.functional.mse_loss(zt, tt)
    ref.backward()
    assert abs(loss - float(ref.detach())) < 1e-14
    np.testing.assert_allclose(dl, zt.grad.numpy(), atol=1e-15)
    # constant logits c: L = ((K-1) c^2 + (c-1)^2) / K whatever the labels
    c = 0.3
    assert abs(nfo.mse_onehot(np.full((4, K), c), synth.labels(61, 3, 4, K))[0] - ((K - 1) * c * c + (c - 1) ** 2) / K) < 1e-15
    e = 1e-6
    lp, lm = logits.copy(), logits.copy()
    lp[2, 3] += e
    lm[2, 3] -= e
    assert abs((nfo.mse_onehot(lp, labels)[0] - nfo.mse_onehot(lm, labels)[0]) / (2 * e) - dl[2, 3]) < 1e-9


def test_adaptive_maxpool_even_odd_ties_and_adjoint_routing():
    """F_n as max pooling: even sizes against a reshape-max, odd sizes against hand-computed overlapping bins,
    the first maximum on ties, and the backward routes each bin's gradient to exactly that position."""
    h = synth.normal(62, 1, (2, 3, 4, 6))
    p, arg = nfo.maxpool_2x2_adaptive(h)
    np.testing.assert_array_equal(p, h.reshape(2, 3, 2, 2, 2, 3).max(axis=(3, 5)))
    for n in range(2):
        for f in range(3):
            for b in range(4):
                i, j = divmod(int(arg[n, f, b // 2, b % 2]), 6)
                assert h[n, f, i, j] == p[n, f, b // 2, b % 2] and i // 2 == b // 2 and j // 3 == b % 2
    h3 = np.arange(9.0).reshape(1, 1, 3, 3)            # bins overlap in the middle row and column
    p3, a3 = nfo.maxpool_2x2_adaptive(h3)
    np.testing.assert_array_equal(p3[0, 0], [[4.0, 5.0], [7.0, 8.0]])
    np.testing.assert_array_equal(a3[0, 0], [[4, 5], [7, 8]])
    ties = np.zeros((1, 1, 4, 4))
    ties[0, 0, 1, 0] = ties[0, 0, 0, 1] = 2.0         # two equal maxima in bin (0,0): row-major scan meets (0,1) first
    assert nfo.maxpool_2x2_adaptive(ties)[1][0, 0, 0, 0] == 1
    dp = synth.normal(62, 2, (2, 3, 2, 2))
    dh = nfo.maxpool_2x2_adaptive_bwd(dp, arg, 4, 6)
    assert np.count_nonzero(dh) == dp.size and abs(dh.sum() - dp.sum()) < 1e-13
    assert abs((p * dp).sum() - (h * dh).sum()) < 1e-12          # <pool(h), dp> = <h, pool^T dp> at the chosen positions
    c = np.zeros((1, 1, 3, 3))
    c[0, 0, 1, 1] = 5.0                                # the centre of an odd map is the maximum of all four bins
    pc, ac = nfo.maxpool_2x2_adaptive(c)
    assert nfo.maxpool_2x2_adaptive_bwd(np.ones((1, 1, 2, 2)), ac, 3, 3)[0, 0, 1, 1] == 4.0
