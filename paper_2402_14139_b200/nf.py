"""Thin ctypes binding of libnf.so: argument marshalling only, same names as include/nf.h.

Every step of the path runs inside the library's CUDA kernels.  There is no CPU fallback: if
libnf.so is missing or a call fails, an exception is raised.  torch is used for device memory
and streams only.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libnf.so")

NF_OK, NF_EINVAL, NF_EALIGN, NF_ENOWS, NF_EUNSUPPORTED, NF_ECUDA = 0, -1, -2, -3, -4, -5
NF_ELABEL, NF_ENONFINITE, NF_ETIMEOUT, NF_EINDEX = 1, 2, 4, 8
NF_F32, NF_BF16 = 0, 1
NF_LOSS_CE, NF_LOSS_MSE = 0, 1
NF_POOL_AVG, NF_POOL_MAX = 0, 1
NF_P_W, NF_P_GAMMA, NF_P_BETA, NF_P_WA, NF_P_BA, NF_P_WF, NF_P_BF, NF_P_RMEAN, NF_P_RVAR = range(9)
NF_K_VALUE, NF_K_MOMENTUM, NF_K_GRAD = 0, 0x100, 0x200
PARAM_IDS = dict(W=NF_P_W, gamma=NF_P_GAMMA, beta=NF_P_BETA, Wa=NF_P_WA, ba=NF_P_BA, Wf=NF_P_WF, bf=NF_P_BF,
                 rmean=NF_P_RMEAN, rvar=NF_P_RVAR)

EXPORTS = ["nf_layer_create", "nf_layer_destroy", "nf_layer_configure", "nf_layer_workspace_bytes",
           "nf_layer_bind_workspace", "nf_layer_set_param", "nf_layer_get_param", "nf_layer_step",
           "nf_layer_step_host", "nf_layer_status", "nf_block_create", "nf_block_destroy", "nf_block_cache",
           "nf_block_cache_n", "nf_layer_predict", "nf_layer_param_count", "nf_select_exit", "nf_count_equal", "nf_aan_filters", "nf_profile_layer", "nf_fit_line", "nf_max_batch", "nf_layer_step_dp", "nf_layer_dp_buffer", "nf_layer_set_skip", "nf_layer_set_skip_grad", "nf_proj_create", "nf_proj_destroy", "nf_proj_configure",
           "nf_proj_workspace_bytes", "nf_proj_bind_workspace", "nf_proj_set_param", "nf_proj_get_param", "nf_proj_forward",
           "nf_proj_forward_eval", "nf_proj_backward", "nf_layer_stored_tensor", "nf_block_step", "nf_block_step_host", "nf_block_step_host_next", "nf_trace_enable", "nf_trace_read",
           "nf_cache_gather", "nf_selftest_bounded_wait", "nf_conv3x3_forward", "nf_conv3x3_wgrad_scratch_bytes", "nf_conv3x3_wgrad", "nf_conv3x3_wgrad_static", "nf_op_status", "nf_partition", "nf_set_stream", "nf_launch_count",
           "nf_layer_kernel_family", "nf_strerror", "nf_last_cuda_error"]


class NfError(RuntimeError):
    pass


class nf_layer_opts(C.Structure):
    _fields_ = [("N", C.c_int), ("stride", C.c_int), ("maxpool", C.c_int), ("dtype", C.c_int),
                ("momentum", C.c_float), ("bn_eps", C.c_float), ("bn_momentum", C.c_float), ("host_io", C.c_int),
                ("loss", C.c_int), ("aux_pool", C.c_int)]


_lib = None


def lib():
    """The loaded C-ABI library.  Raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_SO):
            raise NfError(f"{_SO} not found: build it with `python -m paper_2402_14139_b200.build`")
        L = C.CDLL(_SO)
        vp, ip, fp = C.c_void_p, C.c_void_p, C.c_void_p
        L.nf_layer_create.restype = vp
        L.nf_layer_create.argtypes = [C.c_int] * 6
        L.nf_layer_destroy.restype = None
        L.nf_layer_destroy.argtypes = [vp]
        L.nf_layer_configure.argtypes = [vp, C.POINTER(nf_layer_opts)]
        L.nf_layer_workspace_bytes.restype = C.c_size_t
        L.nf_layer_workspace_bytes.argtypes = [vp]
        L.nf_layer_bind_workspace.argtypes = [vp, vp, C.c_size_t]
        L.nf_layer_set_param.argtypes = [vp, C.c_int, fp, C.c_size_t]
        L.nf_layer_get_param.argtypes = [vp, C.c_int, fp, C.c_size_t]
        L.nf_layer_step.argtypes = [vp, vp, ip, C.c_float, fp, vp]
        L.nf_layer_step_host.argtypes = [vp, vp, ip, C.c_float, fp, vp]
        L.nf_layer_status.argtypes = [vp]
        L.nf_block_create.restype = vp
        L.nf_block_create.argtypes = [C.POINTER(vp), C.c_int]
        L.nf_block_destroy.restype = None
        L.nf_block_destroy.argtypes = [vp]
        L.nf_block_cache.argtypes = [vp, vp, vp]
        L.nf_block_cache_n.argtypes = [vp, vp, vp, C.c_int]
        L.nf_layer_predict.argtypes = [vp, vp, C.c_int, vp, fp, ip]
        L.nf_layer_param_count.restype = C.c_longlong
        L.nf_layer_param_count.argtypes = [vp, C.c_int]
        L.nf_count_equal.argtypes = [ip, ip, C.c_longlong, vp]
        L.nf_layer_set_skip.argtypes = [vp, vp]
        L.nf_layer_set_skip_grad.argtypes = [vp, vp]
        L.nf_proj_create.restype = vp
        L.nf_proj_create.argtypes = [C.c_int] * 4
        L.nf_proj_destroy.restype = None
        L.nf_proj_destroy.argtypes = [vp]
        L.nf_proj_configure.argtypes = [vp, C.c_int, C.c_int, C.c_float, C.c_float, C.c_float]
        L.nf_proj_workspace_bytes.restype = C.c_size_t
        L.nf_proj_workspace_bytes.argtypes = [vp]
        L.nf_proj_bind_workspace.argtypes = [vp, vp, C.c_size_t]
        L.nf_proj_set_param.argtypes = [vp, C.c_int, fp, C.c_size_t]
        L.nf_proj_get_param.argtypes = [vp, C.c_int, fp, C.c_size_t]
        L.nf_proj_forward.argtypes = [vp, vp, vp]
        L.nf_proj_forward_eval.argtypes = [vp, vp, C.c_int, vp]
        L.nf_proj_backward.argtypes = [vp, vp, vp, C.c_float]
        L.nf_layer_stored_tensor.argtypes = [vp, C.c_int, C.POINTER(C.c_void_p), C.POINTER(C.c_size_t)]
        L.nf_layer_step_dp.argtypes = [vp, C.c_int, vp, ip, C.c_float, fp, vp, C.c_int]
        L.nf_layer_dp_buffer.argtypes = [vp, C.c_int, C.POINTER(C.c_void_p), C.POINTER(C.c_size_t)]
        L.nf_aan_filters.argtypes = [C.POINTER(C.c_int), C.c_int, C.c_int, C.POINTER(C.c_int)]
        L.nf_profile_layer.argtypes = [C.c_int] * 6 + [C.POINTER(nf_layer_opts), C.POINTER(C.c_int), C.c_int, C.POINTER(C.c_double),
                                       C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.nf_fit_line.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_double), C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.nf_max_batch.restype = C.c_longlong
        L.nf_max_batch.argtypes = [C.c_double, C.c_double, C.c_double]
        L.nf_select_exit.argtypes = [C.POINTER(C.c_double), C.POINTER(C.c_longlong), C.c_int]
        L.nf_block_step.argtypes = [vp, vp, ip, C.c_float, fp, vp]
        L.nf_block_step_host.argtypes = [vp, vp, ip, C.c_float, fp, vp]
        L.nf_block_step_host_next.argtypes = [vp, vp, ip, C.c_float, fp, vp, vp, ip]
        L.nf_trace_enable.argtypes = [C.c_int]
        L.nf_trace_read.argtypes = [C.c_int, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_longlong)]
        L.nf_cache_gather.argtypes = [vp, ip, C.c_int, ip, C.c_int, C.c_size_t, vp, ip]
        L.nf_conv3x3_forward.argtypes = [C.c_int, vp, vp] + [C.c_int] * 6 + [vp]
        L.nf_conv3x3_wgrad_scratch_bytes.restype = C.c_size_t
        L.nf_conv3x3_wgrad_scratch_bytes.argtypes = [C.c_int] * 6
        L.nf_conv3x3_wgrad.argtypes = [C.c_int, vp, vp] + [C.c_int] * 6 + [vp, C.c_size_t, vp]
        L.nf_conv3x3_wgrad_static.argtypes = [C.c_int, vp, vp] + [C.c_int] * 6 + [vp]
        L.nf_selftest_bounded_wait.argtypes = [C.c_ulonglong, vp]
        L.nf_partition.argtypes = [C.POINTER(C.c_int), C.c_int, C.c_int, C.c_double, C.POINTER(C.c_int),
                                   C.POINTER(C.c_int)]
        L.nf_set_stream.argtypes = [vp]
        L.nf_launch_count.restype = C.c_longlong
        L.nf_layer_kernel_family.restype = C.c_char_p
        L.nf_layer_kernel_family.argtypes = [vp, C.c_int]
        L.nf_strerror.restype = C.c_char_p
        L.nf_strerror.argtypes = [C.c_int]
        L.nf_last_cuda_error.restype = C.c_char_p
        _lib = L
    return _lib


def _check(rc: int, what: str):
    if rc != NF_OK:
        msg = lib().nf_strerror(rc).decode()
        if rc == NF_ECUDA:
            msg += ": " + lib().nf_last_cuda_error().decode()
        raise NfError(f"{what}: {msg} ({rc})")


def nf_strerror(rc: int) -> str:
    return lib().nf_strerror(rc).decode()


def nf_launch_count() -> int:
    return int(lib().nf_launch_count())


def nf_set_stream(stream=None):
    """stream: a torch.cuda.Stream, a raw cudaStream_t integer, or None for the default stream."""
    h = 0 if stream is None else int(getattr(stream, "cuda_stream", stream))
    _check(lib().nf_set_stream(C.c_void_p(h)), "nf_set_stream")


def nf_partition(max_batch, B: int, rho: float):
    """Algorithm 1: returns [(first_layer, last_layer, batch_size)] (0-based, inclusive)."""
    n = len(max_batch)
    mb = (C.c_int * n)(*[int(v) for v in max_batch])
    first, bs = (C.c_int * n)(), (C.c_int * n)()
    nb = lib().nf_partition(mb, n, int(B), float(rho), first, bs)
    if nb < 0:
        _check(nb, "nf_partition")
    out = []
    for i in range(nb):
        last = (first[i + 1] - 1) if i + 1 < nb else n - 1
        out.append((first[i], last, bs[i]))
    return out


TRACE_OPS = ("conv_fwd", "bn_fwd", "aux_fwd", "head", "aux_wgrad", "bn_bwd", "wgrad", "sgd", "aux_dgrad")


def nf_trace_enable(on: bool):
    _check(lib().nf_trace_enable(int(on)), "nf_trace_enable")


def nf_trace_read(slots: int = 1):
    """{(op name, layer slot): (total ms, timed groups)} since nf_trace_enable(True); synchronises."""
    out = {}
    for i, name in enumerate(TRACE_OPS):
        for s in range(slots):
            ms, n = C.c_double(), C.c_longlong()
            _check(lib().nf_trace_read(i, s, C.byref(ms), C.byref(n)), "nf_trace_read")
            if n.value:
                out[(name, s)] = (ms.value, n.value)
    return out


def run_dp_phases(run_phase, buffer_of, loss_out, all_reduce):
    """The exchange schedule of the data-parallel step: phase k, then the sum over ranks of exchange buffer k
    (k = 0, 1, 2); the loss share is summed with the gradients; phase 3 (the update) needs no exchange."""
    for k in range(4):
        run_phase(k)
        if k < 3:
            all_reduce(buffer_of(k))
        if k == 2:
            all_reduce(loss_out)


def nf_aan_filters(channels, first_downsample: int):
    """AAN-LL rule: aux filter count per layer (half the smallest channel count before the first down-sampling, half the largest after)."""
    n = len(channels)
    ch = (C.c_int * n)(*[int(v) for v in channels])
    out = (C.c_int * n)()
    _check(lib().nf_aan_filters(ch, n, int(first_downsample), out), "nf_aan_filters")
    return list(out)


def nf_profile_layer(Cin, Cout, H, W, F, classes, batches, stride=1, maxpool=False, dtype=NF_BF16, loss="ce", aux_pool="avg"):
    """Memory model of one layer: (bytes at each batch size, slope, intercept) of bytes = intercept + slope * batch."""
    k = len(batches)
    o = nf_layer_opts(1, stride, int(maxpool), dtype, 0.9, 1e-5, 0.1, 0, {"ce": 0, "mse": 1}[loss], {"avg": 0, "max": 1}[aux_pool])
    b = (C.c_int * k)(*[int(v) for v in batches])
    by = (C.c_double * k)()
    sl, ic = C.c_double(), C.c_double()
    _check(lib().nf_profile_layer(Cin, Cout, H, W, F, classes, C.byref(o), b, k, by, C.byref(sl), C.byref(ic)), "nf_profile_layer")
    return list(by), sl.value, ic.value


def nf_fit_line(batches, bytes_):
    """Least-squares line bytes = intercept + slope * batch through measured pairs: (slope, intercept)."""
    k = len(batches)
    x = (C.c_double * k)(*[float(v) for v in batches])
    y = (C.c_double * k)(*[float(v) for v in bytes_])
    sl, ic = C.c_double(), C.c_double()
    _check(lib().nf_fit_line(x, y, k, C.byref(sl), C.byref(ic)), "nf_fit_line")
    return sl.value, ic.value


def nf_max_batch(slope, intercept, budget_bytes) -> int:
    return int(lib().nf_max_batch(float(slope), float(intercept), float(budget_bytes)))


def nf_count_equal(a, b, count_out):
    """count_out (device int64[1]) += number of equal entries of the device int32 tensors a and b."""
    _check(lib().nf_count_equal(_ptr(a), _ptr(b), int(a.numel()), _ptr(count_out)), "nf_count_equal")


def nf_select_exit(val_accuracy, params) -> int:
    """Index of the exit with the highest validation accuracy, fewest parameters among equals."""
    n = len(val_accuracy)
    acc = (C.c_double * n)(*[float(v) for v in val_accuracy])
    par = (C.c_longlong * n)(*[int(v) for v in params])
    rc = lib().nf_select_exit(acc, par, n)
    if rc < 0:
        _check(rc, "nf_select_exit")
    return rc


def _ptr(t):
    return C.c_void_p(t.data_ptr()) if t is not None else None


class Layer:
    """One layer with its auxiliary head on the current CUDA device (wraps nf_layer_* calls)."""

    def __init__(self, Cin, Cout, H, W, F, classes, N, stride=1, maxpool=False, dtype=NF_BF16, momentum=0.9,
                 bn_eps=1e-5, bn_momentum=0.1, host_io=False, device="cuda", loss="ce", aux_pool="avg"):
        import torch
        self._torch = torch
        self.Cin, self.Cout, self.H, self.W, self.F, self.classes, self.N = Cin, Cout, H, W, F, classes, N
        self.stride, self.maxpool, self.dtype = stride, bool(maxpool), dtype
        self.Ho, self.Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
        self.Ha, self.Wa = (self.Ho // 2, self.Wo // 2) if maxpool else (self.Ho, self.Wo)
        self.h = lib().nf_layer_create(Cin, Cout, H, W, F, classes)
        if not self.h:
            raise NfError("nf_layer_create failed")
        o = nf_layer_opts(N, stride, int(maxpool), dtype, momentum, bn_eps, bn_momentum, int(host_io),
                          {"ce": NF_LOSS_CE, "mse": NF_LOSS_MSE}[loss], {"avg": NF_POOL_AVG, "max": NF_POOL_MAX}[aux_pool])
        _check(lib().nf_layer_configure(self.h, C.byref(o)), "nf_layer_configure")
        self.ws_bytes = int(lib().nf_layer_workspace_bytes(self.h))
        self.ws = torch.empty(self.ws_bytes + 256, dtype=torch.uint8, device=device)
        base = (self.ws.data_ptr() + 255) // 256 * 256
        _check(lib().nf_layer_bind_workspace(self.h, C.c_void_p(base), self.ws_bytes), "nf_layer_bind_workspace")
        self.shapes = dict(W=(Cout, Cin, 3, 3), gamma=(Cout,), beta=(Cout,), Wa=(F, Cout, 3, 3), ba=(F,),
                           Wf=(classes, 4 * F), bf=(classes,), rmean=(Cout,), rvar=(Cout,))
        self.tdtype = torch.float32 if dtype == NF_F32 else torch.bfloat16
        self.device = device

    def close(self):
        if getattr(self, "h", None):
            lib().nf_layer_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_param(self, name, array, kind=NF_K_VALUE):
        a = np.ascontiguousarray(array, dtype=np.float32).reshape(self.shapes[name])
        _check(lib().nf_layer_set_param(self.h, PARAM_IDS[name] | kind, a.ctypes.data_as(C.c_void_p), a.size),
               f"nf_layer_set_param({name})")

    def get_param(self, name, kind=NF_K_VALUE):
        a = np.empty(self.shapes[name], dtype=np.float32)
        _check(lib().nf_layer_get_param(self.h, PARAM_IDS[name] | kind, a.ctypes.data_as(C.c_void_p), a.size),
               f"nf_layer_get_param({name})")
        return a

    STATE = ("W", "gamma", "beta", "Wa", "ba", "Wf", "bf")

    def export_state(self):
        """Everything that defines the trained layer, as host arrays: the seven parameter tensors, their momentum buffers
        (keys "v" + name) and the running statistics.  With it a finished layer can leave the device (the paper keeps only
        the active block in GPU memory) and be rebuilt later by import_state."""
        st = {k: self.get_param(k) for k in self.STATE}
        st.update({"v" + k: self.get_param(k, NF_K_MOMENTUM) for k in self.STATE})
        st.update(rmean=self.get_param("rmean"), rvar=self.get_param("rvar"))
        return st

    def import_state(self, st):
        for k in self.STATE:
            self.set_param(k, st[k])
            self.set_param(k, st["v" + k], kind=NF_K_MOMENTUM)
        self.set_param("rmean", st["rmean"])
        self.set_param("rvar", st["rvar"])

    def new_act(self):
        return self._torch.empty((self.N, self.Ha, self.Wa, self.Cout), dtype=self.tdtype, device=self.device)

    def step(self, x, labels, lr, loss_out, act_out):
        """nf_layer_step on device tensors: x [N,H,W,Cin], labels int32 [N], loss_out float32 [1],
        act_out [N,Ha,Wa,Cout]; asynchronous."""
        _check(lib().nf_layer_step(self.h, _ptr(x), _ptr(labels), float(lr), _ptr(loss_out), _ptr(act_out)),
               "nf_layer_step")

    def step_host(self, x_host, labels_host, lr, loss_host, act_host=None):
        """nf_layer_step_host on host tensors (pinned for speed); synchronous."""
        _check(lib().nf_layer_step_host(self.h, _ptr(x_host), _ptr(labels_host), float(lr), _ptr(loss_host),
                                        _ptr(act_host)), "nf_layer_step_host")

    def predict(self, x, pred_out, act_out=None, logits_out=None, count=None):
        """nf_layer_predict: early-exit forward for `count` (default N) samples; device tensors."""
        _check(lib().nf_layer_predict(self.h, _ptr(x), int(self.N if count is None else count), _ptr(act_out), _ptr(logits_out),
                                      _ptr(pred_out)), "nf_layer_predict")

    def set_skip(self, skip):
        """nf_layer_set_skip: identity shortcut [N, Ho, Wo, Cout] added before the ReLU in later calls (None removes it)."""
        self._skip = skip       # keeps the tensor alive
        _check(lib().nf_layer_set_skip(self.h, _ptr(skip)), "nf_layer_set_skip")

    STORED = dict(y=0, dy=1, h=2, dh=3, da=4, p=5, dp=6, logits=7, hmask=8)

    def stored(self, name):
        """nf_layer_stored_tensor as a tensor view of the workspace: y, dy [N,Ho,Wo,Cout]; h, dh [N,Ha,Wa,Fp]; da [N,Ha,Wa,Cout]
        (layer dtype; Fp = F rounded up to a multiple of 8); p, dp [N,4*Fp]; logits [N,classes] (float32)."""
        ptr, nbytes = C.c_void_p(), C.c_size_t()
        _check(lib().nf_layer_stored_tensor(self.h, self.STORED[name], C.byref(ptr), C.byref(nbytes)), "nf_layer_stored_tensor")
        off = ptr.value - self.ws.data_ptr()
        raw = self.ws[off:off + nbytes.value]
        Fp = (self.F + 7) // 8 * 8
        if name in ("p", "dp", "logits"):
            return raw.view(self._torch.float32).view(self.N, -1)
        if name == "hmask":     # uint8 [N, Ha, Wa, Fp/8]: bit f%8 of byte f/8 is set where h > 0
            return raw.view(self.N, self.Ha, self.Wa, Fp // 8)
        shape = dict(y=(self.N, self.Ho, self.Wo, self.Cout), dy=(self.N, self.Ho, self.Wo, self.Cout), h=(self.N, self.Ha, self.Wa, Fp),
                     dh=(self.N, self.Ha, self.Wa, Fp), da=(self.N, self.Ha, self.Wa, self.Cout))[name]
        return raw.view(self.tdtype).view(shape)

    def set_skip_grad(self, dz_out):
        """nf_layer_set_skip_grad: every later step also writes the gradient at the shortcut sum to dz_out [N, Ho, Wo, Cout]."""
        self._skip_grad = dz_out
        _check(lib().nf_layer_set_skip_grad(self.h, _ptr(dz_out)), "nf_layer_set_skip_grad")

    def dp_buffer(self, which):
        """The exchange buffer `which` of the data-parallel step as a tensor view of the workspace (float64 for 0 and 1, float32 for 2)."""
        ptr, nbytes = C.c_void_p(), C.c_size_t()
        _check(lib().nf_layer_dp_buffer(self.h, which, C.byref(ptr), C.byref(nbytes)), "nf_layer_dp_buffer")
        off = ptr.value - self.ws.data_ptr()
        return self.ws[off:off + nbytes.value].view(self._torch.float64 if which < 2 else self._torch.float32)

    def step_dp(self, x, labels, lr, loss_out, act_out, world, all_reduce):
        """nf_layer_step_dp through its four phases; all_reduce(tensor) must add the tensor over all ranks in place."""
        def phase(k):
            _check(lib().nf_layer_step_dp(self.h, k, _ptr(x), _ptr(labels), float(lr), _ptr(loss_out), _ptr(act_out), int(world)),
                   "nf_layer_step_dp")
        run_dp_phases(phase, self.dp_buffer, loss_out, all_reduce)

    def param_count(self, part=2) -> int:
        return int(lib().nf_layer_param_count(self.h, part))

    def status(self) -> int:
        rc = lib().nf_layer_status(self.h)
        if rc < 0:
            _check(rc, "nf_layer_status")
        return rc

    def kernel_family(self, op: int) -> str:
        """op 0-3: "tcgen05" or "cuda-core" for main forward, main weight gradient, aux forward, aux backward;
        op 4: "fused" when BatchNorm + ReLU run inside the aux forward kernel, else "separate";
        op 5: "mask" when that kernel pools h in its epilogue and keeps only its sign bits, else "stored";
        op 6: "two-pass" when the aux input gradient runs once for the BatchNorm-backward sums and once more to write dy, so
        that da is never stored, else "stored"."""
        return lib().nf_layer_kernel_family(self.h, op).decode()


class Projection:
    """Projection shortcut of a down-sampling residual block (wraps nf_proj_*): s = BN(Wp (*) x_b), 1x1 convolution with
    stride 2 on the block input x_b [N, H, W, Cin], trained by the local loss of the layer it joins."""

    def __init__(self, Cin, Cout, H, W, N, dtype=NF_BF16, momentum=0.9, bn_eps=1e-5, bn_momentum=0.1, device="cuda"):
        import torch
        self._torch = torch
        self.Cin, self.Cout, self.H, self.W, self.N, self.dtype = Cin, Cout, H, W, N, dtype
        self.Ho, self.Wo = (H - 1) // 2 + 1, (W - 1) // 2 + 1
        self.h = lib().nf_proj_create(Cin, Cout, H, W)
        if not self.h:
            raise NfError("nf_proj_create failed")
        _check(lib().nf_proj_configure(self.h, N, dtype, momentum, bn_eps, bn_momentum), "nf_proj_configure")
        nbytes = int(lib().nf_proj_workspace_bytes(self.h))
        self.ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=device)
        base = (self.ws.data_ptr() + 255) // 256 * 256
        _check(lib().nf_proj_bind_workspace(self.h, C.c_void_p(base), nbytes), "nf_proj_bind_workspace")
        self.shapes = dict(W=(Cout, Cin), gamma=(Cout,), beta=(Cout,), rmean=(Cout,), rvar=(Cout,))
        self.tdtype = torch.float32 if dtype == NF_F32 else torch.bfloat16
        self.device = device

    def close(self):
        if getattr(self, "h", None):
            lib().nf_proj_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_param(self, name, array, kind=NF_K_VALUE):
        a = np.ascontiguousarray(array, dtype=np.float32).reshape(self.shapes[name])
        _check(lib().nf_proj_set_param(self.h, PARAM_IDS[name] | kind, a.ctypes.data_as(C.c_void_p), a.size), f"nf_proj_set_param({name})")

    def get_param(self, name, kind=NF_K_VALUE):
        a = np.empty(self.shapes[name], dtype=np.float32)
        _check(lib().nf_proj_get_param(self.h, PARAM_IDS[name] | kind, a.ctypes.data_as(C.c_void_p), a.size), f"nf_proj_get_param({name})")
        return a

    def new_out(self):
        return self._torch.empty((self.N, self.Ho, self.Wo, self.Cout), dtype=self.tdtype, device=self.device)

    def forward(self, xb, s_out):
        _check(lib().nf_proj_forward(self.h, _ptr(xb), _ptr(s_out)), "nf_proj_forward")

    def forward_eval(self, xb, s_out, count=None):
        _check(lib().nf_proj_forward_eval(self.h, _ptr(xb), int(self.N if count is None else count), _ptr(s_out)), "nf_proj_forward_eval")

    def backward(self, xb, dz, lr):
        _check(lib().nf_proj_backward(self.h, _ptr(xb), _ptr(dz), float(lr)), "nf_proj_backward")


class Block:
    """Consecutive layers trained at one batch size (wraps nf_block_*)."""

    def __init__(self, layers):
        self.layers = list(layers)
        arr = (C.c_void_p * len(layers))(*[l.h for l in layers])
        self.h = lib().nf_block_create(arr, len(layers))
        if not self.h:
            raise NfError("nf_block_create failed: layers do not chain or have no workspace")

    def cache(self, x, out, count=None):
        if count is None:
            _check(lib().nf_block_cache(self.h, _ptr(x), _ptr(out)), "nf_block_cache")
        else:
            _check(lib().nf_block_cache_n(self.h, _ptr(x), _ptr(out), int(count)), "nf_block_cache_n")

    def step(self, x, labels, lr, loss_out, act_out=None):
        """nf_block_step: loss_out is a float32 device tensor with one entry per layer."""
        _check(lib().nf_block_step(self.h, _ptr(x), _ptr(labels), float(lr), _ptr(loss_out), _ptr(act_out)),
               "nf_block_step")

    def capture(self, x, labels, lr, loss_out, act_out=None):
        """Records one nf_block_step on these (fixed) device buffers into a CUDA graph and returns it; graph.replay()
        then runs the whole step as one launch, which pays off when the kernels are short (small batches or maps).
        Run one eager step first: the first use of a kernel sets its attributes, which is not part of a step."""
        torch = self.layers[0]._torch
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            nf_set_stream(torch.cuda.current_stream())
            self.step(x, labels, lr, loss_out, act_out)
        nf_set_stream(torch.cuda.current_stream())
        return g

    def step_host_next(self, x_host, labels_host, lr, loss_host, next_x_host=None, next_labels_host=None, act_host=None):
        """nf_block_step_host_next: trains on (x_host, labels_host) while the next batch is copied to the device."""
        _check(lib().nf_block_step_host_next(self.h, _ptr(x_host), _ptr(labels_host), float(lr), _ptr(loss_host), _ptr(act_host),
                                             _ptr(next_x_host), _ptr(next_labels_host)), "nf_block_step_host_next")

    def step_host(self, x_host, labels_host, lr, loss_host, act_host=None):
        _check(lib().nf_block_step_host(self.h, _ptr(x_host), _ptr(labels_host), float(lr), _ptr(loss_host),
                                        _ptr(act_host)), "nf_block_step_host")

    def close(self):
        if getattr(self, "h", None):
            lib().nf_block_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def nf_cache_gather(cache, cache_labels, idx, out, out_labels):
    """out[i] = cache[idx[i]] (rows) and labels likewise; device tensors, idx int32.  An index outside the cache's rows
    yields a zero row, label -1 and NF_EINDEX in nf_op_status()."""
    row_bytes = cache[0].numel() * cache.element_size()
    _check(lib().nf_cache_gather(_ptr(cache), _ptr(cache_labels), int(cache.shape[0]), _ptr(idx), int(idx.numel()), row_bytes,
                                 _ptr(out), _ptr(out_labels)), "nf_cache_gather")


def nf_conv3x3_forward(dtype, x, w, stride, y):
    """y = conv3x3(x, w): x [N,H,W,Cin], w [9,Cout,Cin] (both of dtype), y [N,Ho,Wo,Cout]; device tensors."""
    N, H, W, Cin = x.shape
    _check(lib().nf_conv3x3_forward(dtype, _ptr(x), _ptr(w), N, H, W, Cin, w.shape[1], stride, _ptr(y)),
           "nf_conv3x3_forward")


def nf_conv3x3_wgrad_scratch_bytes(N, H, W, Cin, Cout, stride) -> int:
    return int(lib().nf_conv3x3_wgrad_scratch_bytes(N, H, W, Cin, Cout, stride))


def nf_conv3x3_wgrad(dtype, x, g, stride, scratch, dw):
    """dw [9,Cout,Cin] float32 = weight gradient of conv3x3 for input x and output gradient g; scratch is a
    uint8 device tensor of at least nf_conv3x3_wgrad_scratch_bytes()."""
    N, H, W, Cin = x.shape
    _check(lib().nf_conv3x3_wgrad(dtype, _ptr(x), _ptr(g), N, H, W, Cin, g.shape[3], stride, _ptr(scratch),
                                  scratch.numel(), _ptr(dw)), "nf_conv3x3_wgrad")


NF_STATIC_SCRATCH_BYTES = 16 << 20


def nf_conv3x3_wgrad_static(dtype, x, g, stride, dw):
    """nf_conv3x3_wgrad for callers with no scratch to give: the partial sums go to a 16 MiB array built
    into the library, so nothing is allocated.  Problems that need more are refused (NfError).  Calls
    share that array, so do not let two of them overlap on the GPU."""
    N, H, W, Cin = x.shape
    _check(lib().nf_conv3x3_wgrad_static(dtype, _ptr(x), _ptr(g), N, H, W, Cin, g.shape[3], stride, _ptr(dw)),
           "nf_conv3x3_wgrad_static")


def nf_selftest_bounded_wait(limit_ns: int, waited_ns_out):
    """One small CTA waits limit_ns on a barrier nobody arrives at and gives up; waited_ns_out: device int64[1]."""
    _check(lib().nf_selftest_bounded_wait(int(limit_ns), _ptr(waited_ns_out)), "nf_selftest_bounded_wait")


def nf_op_status() -> int:
    rc = lib().nf_op_status()
    if rc < 0:
        _check(rc, "nf_op_status")
    return rc
