"""GPU parity of the alternatives the method names for the loss of Eq. 3 (mean squared error) and for the
down-sampling F_n of Eq. 2 (max pooling): whole local steps and the early-exit forward against the checker,
same tolerances as the default configuration."""
import numpy as np
import pytest

from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    nf.nf_set_stream(None)
    return nf, torch


SHAPES = [
    (0, dict(N=4, Cin=3, Cout=8, H=10, W=12, F=6, classes=10, stride=1, pool=False)),
    (0, dict(N=3, Cin=4, Cout=8, H=9, W=7, F=4, classes=5, stride=1, pool=False)),       # odd sizes: overlapping bins
    (0, dict(N=4, Cin=8, Cout=16, H=12, W=12, F=8, classes=7, stride=2, pool=False)),
    (1, dict(N=8, Cin=3, Cout=64, H=16, W=16, F=16, classes=10, stride=1, pool=False)),
    (1, dict(N=8, Cin=64, Cout=64, H=28, W=28, F=16, classes=100, stride=1, pool=True)),  # tensor-core kernels
    (1, dict(N=16, Cin=64, Cout=128, H=16, W=16, F=32, classes=10, stride=2, pool=False)),
]
VARIANTS = [("mse", "avg"), ("ce", "max"), ("mse", "max")]


@pytest.mark.parametrize("vi", range(len(VARIANTS)))
@pytest.mark.parametrize("si", range(len(SHAPES)))
def test_variant_step_parity(env, si, vi):
    nf, torch = env
    dtype, c = SHAPES[si]
    loss, aux_pool = VARIANTS[vi]
    c = dict(c, loss=loss, aux_pool=aux_pool)
    pu.check_step(nf, torch, c, 0x4E46F000 + 16 * si + vi, dtype, steps=2)


@pytest.mark.parametrize("si", [1, 4])
def test_variant_predict_uses_the_same_downsampling(env, si):
    nf, torch = env
    dtype, c = SHAPES[si]
    c = dict(c, loss="mse", aux_pool="max")
    bf16 = dtype == 1
    P, x, _ = pu.seeded_case(c, 0x4E46F100 + si, bf16=bf16)
    if c["Cin"] != 3:
        x = np.maximum(x, 0.0)
    O = pu.oracle_layer(c, P, store_bf16=bf16)
    G = pu.gpu_layer(nf, c, P, nf.NF_BF16 if bf16 else nf.NF_F32)
    _, logits_o, _ = O.predict(x)
    logits_d = torch.zeros((c["N"], c["classes"]), device="cuda")
    pred_d = torch.zeros(c["N"], dtype=torch.int32, device="cuda")
    G.predict(pu.to_device_nhwc(torch, x, dtype), pred_d, logits_out=logits_d)
    torch.cuda.synchronize()
    assert np.abs(logits_d.cpu().numpy() - logits_o).max() <= pu.TOL[dtype]["t"] * np.abs(logits_o).max()
    G.close()


def test_unknown_variant_is_rejected(env):
    nf, torch = env
    import ctypes as C
    h = nf.lib().nf_layer_create(8, 8, 8, 8, 8, 4)
    o = nf.nf_layer_opts(2, 1, 0, nf.NF_F32, 0.9, 1e-5, 0.1, 0, 7, 0)
    assert nf.lib().nf_layer_configure(h, C.byref(o)) == nf.NF_EINVAL
    o = nf.nf_layer_opts(2, 1, 0, nf.NF_F32, 0.9, 1e-5, 0.1, 0, 0, 3)
    assert nf.lib().nf_layer_configure(h, C.byref(o)) == nf.NF_EINVAL
    nf.lib().nf_layer_destroy(h)
