"""ctypes front end of the fp64 CPU checker in ``nfo.c``.

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the tests, the smoke check and the
CPU-baseline leg of the benchmark may import this.  It shares nothing with the
CUDA library.  Arrays are numpy float64 in NCHW order.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libnfo.so")
_SRC = os.path.join(_HERE, "nfo.c")


def build(force: bool = False) -> str:
    """Compile nfo.c into libnfo.so beside it (gcc -O2 -fopenmp)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _SO, _SRC, "-lm"])
    return _SO


_lib = None
_dp = C.POINTER(C.c_double)
_ip = C.POINTER(C.c_int32)


class Dims(C.Structure):
    _fields_ = [(k, C.c_int) for k in ("N", "Cin", "Cout", "H", "W", "stride", "pool", "F", "classes")] + \
               [(k, C.c_double) for k in ("eps", "momentum", "bn_momentum")] + \
               [(k, C.c_int) for k in ("store_bf16", "loss", "aux_pool")] + [("skip", C.c_void_p)]


_PNAMES = ("W", "gamma", "beta", "Wa", "ba", "Wf", "bf")
_PFIELDS = _PNAMES + tuple("v" + k for k in _PNAMES) + ("rmean", "rvar")
_TFIELDS = ("y", "mu", "var", "xhat", "z", "a", "h", "p", "logits", "dlogits", "dp", "dh", "da", "dz", "dy",
            "gW", "ggamma", "gbeta", "gWa", "gba", "gWf", "gbf")


class _Params(C.Structure):
    _fields_ = [(k, _dp) for k in _PFIELDS]


class _Trace(C.Structure):
    _fields_ = [(k, _dp) for k in _TFIELDS] + [("argmax", _ip)]


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.nfo_layer_step.restype = C.c_double
        _lib.nfo_softmax_ce.restype = C.c_double
        _lib.nfo_mse_onehot.restype = C.c_double
        _lib.nfo_threads.restype = C.c_int
        _lib.nfo_round_bf16.restype = C.c_double
        _lib.nfo_round_bf16.argtypes = [C.c_double]
    return _lib


def threads() -> int:
    return int(lib().nfo_threads())


def _d(a):
    return a.ctypes.data_as(_dp)


def _c64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def out_size(H: int, stride: int) -> int:
    return (H - 1) // stride + 1


def conv3x3(x, w, bias=None, stride=1):
    x, w = _c64(x), _c64(w)
    N, Ci, H, W = x.shape
    Co = w.shape[0]
    y = np.empty((N, Co, out_size(H, stride), out_size(W, stride)))
    b = _c64(bias) if bias is not None else None
    lib().nfo_conv3x3(_d(x), N, Ci, H, W, _d(w), Co, _d(b) if b is not None else None, stride, _d(y))
    return y


def conv3x3_wgrad(x, g, stride=1):
    x, g = _c64(x), _c64(g)
    N, Ci, H, W = x.shape
    Co = g.shape[1]
    dw = np.empty((Co, Ci, 3, 3))
    lib().nfo_conv3x3_wgrad(_d(x), N, Ci, H, W, _d(g), Co, stride, _d(dw))
    return dw


def conv3x3_dgrad(w, g, H, W, stride=1):
    w, g = _c64(w), _c64(g)
    Co, Ci = w.shape[:2]
    N = g.shape[0]
    dx = np.empty((N, Ci, H, W))
    lib().nfo_conv3x3_dgrad(_d(w), Ci, Co, _d(g), N, H, W, stride, _d(dx))
    return dx


def conv1x1(x, w, stride=2):
    x, w = _c64(x), _c64(w)
    N, Ci, H, W = x.shape
    Co = w.shape[0]
    y = np.empty((N, Co, out_size(H, stride), out_size(W, stride)))
    lib().nfo_conv1x1(_d(x), N, Ci, H, W, _d(w), Co, stride, _d(y))
    return y


def conv1x1_wgrad(x, g, stride=2):
    x, g = _c64(x), _c64(g)
    N, Ci, H, W = x.shape
    Co = g.shape[1]
    dw = np.empty((Co, Ci))
    lib().nfo_conv1x1_wgrad(_d(x), N, Ci, H, W, _d(g), Co, stride, _d(dw))
    return dw


def bn_train(y, gamma, beta, eps=1e-5):
    y = _c64(y)
    N, Cc, H, W = y.shape
    mu, var = np.empty(Cc), np.empty(Cc)
    xhat, z = np.empty_like(y), np.empty_like(y)
    lib().nfo_bn_train(_d(y), N, Cc, H * W, _d(_c64(gamma)), _d(_c64(beta)), C.c_double(eps),
                       _d(mu), _d(var), _d(xhat), _d(z))
    return mu, var, xhat, z


def bn_bwd(dz, xhat, gamma, var, eps=1e-5):
    dz, xhat = _c64(dz), _c64(xhat)
    N, Cc, H, W = dz.shape
    dg, db, dy = np.empty(Cc), np.empty(Cc), np.empty_like(dz)
    lib().nfo_bn_bwd(_d(dz), _d(xhat), N, Cc, H * W, _d(_c64(gamma)), _d(_c64(var)), C.c_double(eps),
                     _d(dg), _d(db), _d(dy))
    return dg, db, dy


def maxpool2(r):
    r = _c64(r)
    N, Cc, H, W = r.shape
    a = np.empty((N, Cc, H // 2, W // 2))
    arg = np.empty(a.shape, dtype=np.int32)
    lib().nfo_maxpool2(_d(r), N, Cc, H, W, _d(a), arg.ctypes.data_as(_ip))
    return a, arg


def avgpool_2x2(h):
    h = _c64(h)
    N, F, H, W = h.shape
    p = np.empty((N, F, 2, 2))
    lib().nfo_avgpool_2x2(_d(h), N, F, H, W, _d(p))
    return p


def avgpool_2x2_bwd(dp, H, W):
    dp = _c64(dp)
    N, F = dp.shape[:2]
    dh = np.empty((N, F, H, W))
    lib().nfo_avgpool_2x2_bwd(_d(dp), N, F, H, W, _d(dh))
    return dh


def maxpool_2x2_adaptive(h):
    """Adaptive max pool to 2x2 and the position i*W+j of the first maximum of every bin."""
    h = _c64(h)
    N, F, H, W = h.shape
    p = np.empty((N, F, 2, 2))
    arg = np.empty((N, F, 2, 2), dtype=np.int32)
    lib().nfo_maxpool_2x2_adaptive(_d(h), N, F, H, W, _d(p), arg.ctypes.data_as(_ip))
    return p, arg


def maxpool_2x2_adaptive_bwd(dp, arg, H, W):
    dp = _c64(dp)
    arg = np.ascontiguousarray(arg, dtype=np.int32)
    N, F = dp.shape[:2]
    dh = np.empty((N, F, H, W))
    lib().nfo_maxpool_2x2_adaptive_bwd(_d(dp), arg.ctypes.data_as(_ip), N, F, H, W, _d(dh))
    return dh


def mse_onehot(logits, labels):
    logits = _c64(logits)
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    N, K = logits.shape
    dl = np.empty_like(logits)
    loss = lib().nfo_mse_onehot(_d(logits), labels.ctypes.data_as(_ip), N, K, _d(dl))
    return float(loss), dl


def fc(p, Wf, bf):
    p, Wf, bf = _c64(p), _c64(Wf), _c64(bf)
    N, D = p.shape
    K = Wf.shape[0]
    out = np.empty((N, K))
    lib().nfo_fc(_d(p), N, D, _d(Wf), _d(bf), K, _d(out))
    return out


def softmax_ce(logits, labels):
    logits = _c64(logits)
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    N, K = logits.shape
    dl = np.empty_like(logits)
    loss = lib().nfo_softmax_ce(_d(logits), labels.ctypes.data_as(_ip), N, K, _d(dl))
    return float(loss), dl


def sgd(theta, v, g, lr, mu):
    """In-place momentum update of float64 arrays theta and v."""
    assert theta.dtype == np.float64 and v.dtype == np.float64 and theta.flags.c_contiguous and v.flags.c_contiguous
    lib().nfo_sgd(_d(theta), _d(v), _d(_c64(g)), C.c_size_t(theta.size), C.c_double(lr), C.c_double(mu))


class Layer:
    """Parameters, momentum and running statistics of one layer plus its auxiliary head (fp64)."""

    def __init__(self, Cin, Cout, H, W, F, classes, N, stride=1, pool=False, eps=1e-5, momentum=0.9,
                 bn_momentum=0.1, store_bf16=False, loss="ce", aux_pool="avg"):
        self.d = Dims(N, Cin, Cout, H, W, stride, int(pool), F, classes, eps, momentum, bn_momentum, int(store_bf16),
                      {"ce": 0, "mse": 1}[loss], {"avg": 0, "max": 1}[aux_pool], None)
        self.Ho, self.Wo = out_size(H, stride), out_size(W, stride)
        self.Ha, self.Wa = (self.Ho // 2, self.Wo // 2) if pool else (self.Ho, self.Wo)
        sh = dict(W=(Cout, Cin, 3, 3), gamma=(Cout,), beta=(Cout,), Wa=(F, Cout, 3, 3), ba=(F,),
                  Wf=(classes, 4 * F), bf=(classes,))
        self.shapes = sh
        self.p = {k: np.zeros(s) for k, s in sh.items()}
        self.p["gamma"][:] = 1.0
        self.v = {k: np.zeros(s) for k, s in sh.items()}
        self.rmean = np.zeros(Cout)
        self.rvar = np.ones(Cout)

    def set(self, **kw):
        for k, a in kw.items():
            if k in self.p:
                self.p[k][...] = np.asarray(a, dtype=np.float64).reshape(self.shapes[k])
            elif k in ("rmean", "rvar"):
                getattr(self, k)[...] = a
            elif k.startswith("v") and k[1:] in self.v:
                self.v[k[1:]][...] = np.asarray(a, dtype=np.float64).reshape(self.shapes[k[1:]])
            else:
                raise KeyError(k)

    def _params(self):
        P = _Params()
        for k in _PNAMES:
            setattr(P, k, _d(self.p[k]))
            setattr(P, "v" + k, _d(self.v[k]))
        P.rmean, P.rvar = _d(self.rmean), _d(self.rvar)
        return P

    def _trace_arrays(self):
        d = self.d
        ysh = (d.N, d.Cout, self.Ho, self.Wo)
        ash = (d.N, d.Cout, self.Ha, self.Wa)
        hsh = (d.N, d.F, self.Ha, self.Wa)
        sh = dict(y=ysh, mu=(d.Cout,), var=(d.Cout,), xhat=ysh, z=ysh, a=ash, h=hsh, p=(d.N, 4 * d.F),
                  logits=(d.N, d.classes), dlogits=(d.N, d.classes), dp=(d.N, 4 * d.F), dh=hsh, da=ash,
                  dz=ysh, dy=ysh, gW=self.shapes["W"], ggamma=(d.Cout,), gbeta=(d.Cout,),
                  gWa=self.shapes["Wa"], gba=(d.F,), gWf=self.shapes["Wf"], gbf=(d.classes,))
        arrs = {k: np.zeros(s) for k, s in sh.items()}
        arrs["argmax"] = np.zeros(ash, dtype=np.int32)
        return arrs

    def _with_skip(self, d, skip, n):
        """A copy of the dims with the shortcut tensor attached (kept alive by the returned array)."""
        if skip is None:
            return d, None
        s = _c64(skip)
        assert s.shape == (n, d.Cout, self.Ho, self.Wo), s.shape
        d = Dims.from_buffer_copy(d)
        d.skip = s.ctypes.data
        return d, s

    def step(self, x, labels, lr, update=True, trace=False, grads=False, skip=None):
        """One local training step.  Returns (loss, act_out, trace dict or None).

        ``trace=True`` keeps every intermediate; ``grads=True`` keeps only the parameter gradients
        and the batch statistics (cheap enough for large shapes)."""
        x = _c64(x)
        labels = np.ascontiguousarray(labels, dtype=np.int32)
        d, _keep = self._with_skip(self.d, skip, self.d.N)
        assert x.shape == (d.N, d.Cin, d.H, d.W), x.shape
        act = np.empty((d.N, d.Cout, self.Ha, self.Wa))
        P = self._params()
        T, arrs = None, None
        if trace:
            arrs = self._trace_arrays()
        elif grads:
            arrs = {k: np.zeros(s) for k, s in dict(
                mu=(d.Cout,), var=(d.Cout,), gW=self.shapes["W"], ggamma=(d.Cout,), gbeta=(d.Cout,),
                gWa=self.shapes["Wa"], gba=(d.F,), gWf=self.shapes["Wf"], gbf=(d.classes,),
                logits=(d.N, d.classes), p=(d.N, 4 * d.F)).items()}
        if arrs is not None:
            T = _Trace()
            for k, a in arrs.items():
                setattr(T, k, a.ctypes.data_as(_ip) if k == "argmax" else _d(a))
        loss = lib().nfo_layer_step(C.byref(d), _d(x), labels.ctypes.data_as(_ip), C.c_double(lr),
                                    C.byref(P), _d(act), C.byref(T) if T is not None else None, int(update))
        return float(loss), act, arrs

    def predict(self, x, skip=None):
        """Early-exit prediction for any batch size: (act_out, logits, classes); class = first arg-max."""
        x = _c64(x)
        d = Dims.from_buffer_copy(self.d)
        d.N = x.shape[0]
        d, _keep = self._with_skip(d, skip, d.N)
        act = np.empty((d.N, d.Cout, self.Ha, self.Wa))
        logits = np.empty((d.N, d.classes))
        P = self._params()
        lib().nfo_layer_predict(C.byref(d), _d(x), C.byref(P), _d(act), _d(logits))
        return act, logits, np.argmax(logits, axis=1).astype(np.int32)

    def n_params(self):
        """(main-path parameters W, gamma, beta; aux-head parameters Wa, ba, Wf, bf)."""
        main = sum(self.p[k].size for k in ("W", "gamma", "beta"))
        aux = sum(self.p[k].size for k in ("Wa", "ba", "Wf", "bf"))
        return main, aux

    def eval_forward(self, x, skip=None):
        """Eval-mode forward (running statistics) for any batch size."""
        x = _c64(x)
        d = Dims.from_buffer_copy(self.d)
        d.N = x.shape[0]
        d, _keep = self._with_skip(d, skip, d.N)
        out = np.empty((d.N, d.Cout, self.Ha, self.Wa))
        P = self._params()
        lib().nfo_layer_eval(C.byref(d), _d(x), C.byref(P), _d(out))
        return out


class Projection:
    """Projection shortcut of a down-sampling residual block: s = BN(Wp (*) x_b), a 1x1 convolution with stride 2 on the
    block input x_b followed by BatchNorm with batch statistics.  The paper trains ResNet-18 without saying how such a
    shortcut enters a layer-local step; the reading here: it is part of the layer whose BatchNorm output it is added to
    (x_{n+1} = P(ReLU(BN(theta_n x_n) + s))), so its parameters (Wp, gamma_p, beta_p) are trained by that layer's local
    loss: the gradient at the sum, dz, is also the gradient at s; no gradient reaches x_b.  Same optimiser and running-
    statistics conventions as the layer.  In the bf16 configuration the stored conv output and s are rounded to bfloat16
    and the convolution reads a bfloat16 copy of Wp, as the layer does for y, a and W."""

    def __init__(self, Cin, Cout, stride=2, eps=1e-5, momentum=0.9, bn_momentum=0.1, store_bf16=False):
        self.Cin, self.Cout, self.stride, self.eps, self.momentum, self.bn_momentum = Cin, Cout, stride, eps, momentum, bn_momentum
        self.store_bf16 = store_bf16
        self.p = dict(W=np.zeros((Cout, Cin)), gamma=np.ones(Cout), beta=np.zeros(Cout))
        self.v = {k: np.zeros_like(a) for k, a in self.p.items()}
        self.rmean, self.rvar = np.zeros(Cout), np.ones(Cout)

    def _round(self, a):
        if not self.store_bf16:
            return a
        return np.asarray(np.float64(_bf16_array(a)))

    def forward(self, xb):
        """s for a batch, with batch statistics; keeps what backward needs."""
        wq = self._round(self.p["W"])
        ys = self._round(conv1x1(xb, wq, self.stride))
        mu, var, shat, s = bn_train(ys, self.p["gamma"], self.p["beta"], self.eps)
        self._saved = (_c64(xb), ys.shape, mu, var, shat)
        return self._round(s)

    def backward(self, dz, lr, update=True):
        """Gradients from the gradient dz at the sum, then the momentum update.  Returns dict(gW, ggamma, gbeta)."""
        xb, shape, mu, var, shat = self._saved
        gg, gb, dys = bn_bwd(_c64(dz).reshape(shape), shat, self.p["gamma"], var, self.eps)
        g = dict(W=conv1x1_wgrad(xb, dys, self.stride), gamma=gg, beta=gb)
        if update:
            M = shat.size // self.Cout
            for k in ("W", "gamma", "beta"):
                sgd(self.p[k], self.v[k], g[k], lr, self.momentum)
            self.rmean[...] = (1 - self.bn_momentum) * self.rmean + self.bn_momentum * mu
            self.rvar[...] = (1 - self.bn_momentum) * self.rvar + self.bn_momentum * var * M / (M - 1)
        return dict(gW=g["W"], ggamma=gg, gbeta=gb)

    def eval_forward(self, xb):
        """s with the running statistics (cache fill, early-exit evaluation)."""
        ys = self._round(conv1x1(xb, self._round(self.p["W"]), self.stride))
        ch = (1, -1, 1, 1)
        s = self.p["gamma"].reshape(ch) * (ys - self.rmean.reshape(ch)) / np.sqrt(self.rvar.reshape(ch) + self.eps) + self.p["beta"].reshape(ch)
        return self._round(s)


def _bf16_array(a):
    """float64 array rounded to bfloat16 through the C routine's rule (round to nearest even via float32)."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    r = ((u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)) << np.uint64(16)
    return (r & np.uint64(0xFFFFFFFF)).astype(np.uint32).view(np.float32).reshape(f.shape)


def select_exit(val_accuracy, params):
    """Exit-point rule of the paper's "Trained output CNN" section: the layer whose early-exit model has the
    highest validation accuracy; among equals, the one with the fewest parameters.  Returns its index."""
    best = 0
    for i in range(1, len(val_accuracy)):
        if val_accuracy[i] > val_accuracy[best] or (val_accuracy[i] == val_accuracy[best] and params[i] < params[best]):
            best = i
    return best


def partition(max_batch, B, rho):
    """Algorithm 1 after its first loop: cap each layer's largest feasible batch size at B, then
    greedily group consecutive layers while |b[i+1]-b[i]| <= rho*b[i]; a block trains at the
    smallest batch size of its members.  Returns [(first_layer, last_layer, batch_size)], 0-based."""
    b = [min(int(t), int(B)) for t in max_batch]
    blocks, i, L = [], 0, len(b)
    while i < L:
        first, bs = i, b[i]
        while i + 1 < L and abs(b[i + 1] - b[i]) <= rho * b[i]:
            bs = min(bs, b[i + 1])
            i += 1
        blocks.append((first, i, bs))
        i += 1
    return blocks


def aan_filters(channels, first_downsample):
    """AAN-LL rule (Section "Opportunity 1"): layers before the first down-sampling operation get half the smallest
    filter count of the CNN, the later ones half the largest."""
    lo, hi = min(channels), max(channels)
    return [max(1, (lo if i < first_downsample else hi) // 2) for i in range(len(channels))]


def fit_line(batches, bytes_):
    """Least-squares line through (batch, bytes): the Profiler's layer-wise linear model.  Returns (slope, intercept)."""
    x = np.asarray(batches, dtype=np.float64)
    y = np.asarray(bytes_, dtype=np.float64)
    xm, ym = x.mean(), y.mean()
    slope = float(((x - xm) * (y - ym)).sum() / ((x - xm) ** 2).sum())
    return slope, float(ym - slope * xm)


def max_batch_from_line(slope, intercept, M):
    """Algorithm 1, first loop: largest integer batch t with intercept + slope*t <= M."""
    return int(np.floor((M - intercept) / slope + 1e-12))
