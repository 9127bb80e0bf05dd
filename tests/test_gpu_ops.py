"""GPU parity of the stand-alone contractions (conv forward, weight gradient) against the CPU checker."""
import numpy as np
import pytest

from oracle import nfo
from paper_2402_14139_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu

SHAPES = [  # N, Cin, Cout, H, W, stride
    (2, 3, 5, 9, 7, 1),
    (3, 20, 33, 12, 10, 2),
    (2, 64, 64, 32, 32, 1),
    (2, 64, 128, 16, 16, 2),
    (1, 128, 64, 8, 24, 1),
    (2, 128, 128, 32, 32, 1),   # tensor-core forward: two channel chunks, 128-wide channel tile
    (1, 64, 64, 64, 48, 1),     # tensor-core forward: 16x8 pixel tiles, several tiles per CTA row
    (3, 64, 192, 8, 32, 1),     # tensor-core forward: 32x4 pixel tiles, three 64-wide channel tiles
    (1, 64, 64, 16, 8, 1),      # tensor-core forward: 8x16 pixel tiles, a single tile
    (2, 64, 128, 32, 32, 2),    # tensor-core stride 2: 16x16 output, strided TMA boxes
    (1, 128, 64, 64, 32, 2),    # tensor-core stride 2: two channel chunks, 32x16 output
    (2, 64, 64, 16, 28, 1),     # 64->64 forward with the column taps folded into N: 14-pixel-wide tiles
    (1, 64, 64, 8, 14, 1),      # the same kernel on a single tile
    (3, 64, 64, 24, 56, 1),     # several tiles per CTA row and per image
    (4, 64, 64, 8, 8, 1),       # small feature map: tiles of two whole 8x8 images, one TMA box per tap
    (5, 64, 128, 8, 8, 1),      # the same with a ragged last tile (5 images, 2 per tile)
    (16, 128, 128, 4, 4, 1),    # eight 4x4 images per tile, two channel chunks
    (6, 128, 128, 16, 16, 2),   # stride 2 down to 8x8: strided boxes over two images
    (3, 256, 64, 4, 4, 1),
    (2, 64, 64, 31, 33, 2),     # stride 2 with odd input sizes: 16x17 output is not tileable -> CUDA-core path
]


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    return nf, torch


def _case(shape, seed, bf16):
    N, Ci, Co, H, W, s = shape
    r = (lambda a: synth.round_bf16(a).astype(np.float64)) if bf16 else (lambda a: a.astype(np.float32).astype(np.float64))
    x = r(synth.normal(seed, 1, (N, Ci, H, W)))
    w = r(synth.normal(seed, 2, (Co, Ci, 3, 3), np.sqrt(2.0 / (9 * Ci))))
    Ho, Wo = nfo.out_size(H, s), nfo.out_size(W, s)
    g = r(synth.normal(seed, 3, (N, Co, Ho, Wo)))
    return x, w, g


@pytest.mark.parametrize("si", range(len(SHAPES)))
@pytest.mark.parametrize("dtype", [0, 1])
def test_conv_forward_and_wgrad(env, si, dtype):
    nf, torch = env
    shape = SHAPES[si]
    N, Ci, Co, H, W, s = shape
    x, w, g = _case(shape, 300 + si, dtype == 1)
    tol = pu.TOL[dtype]["t"]
    td = torch.float32 if dtype == 0 else torch.bfloat16
    xd = pu.to_device_nhwc(torch, x, dtype)
    gd = pu.to_device_nhwc(torch, g, dtype)
    wk = np.ascontiguousarray(np.transpose(w.reshape(Co, Ci, 9), (2, 0, 1)))          # [tap][Cout][Cin]
    wd = torch.from_numpy(wk.astype(np.float32)).to(device="cuda", dtype=td)
    yd = torch.empty((N, gd.shape[1], gd.shape[2], Co), device="cuda", dtype=td)
    nf.nf_conv3x3_forward(dtype, xd, wd, s, yd)
    assert pu.max_err(pu.from_device_nhwc(yd), nfo.conv3x3(x, w, None, s)) <= tol
    assert nf.nf_op_status() == 0
    scratch = torch.empty(nf.nf_conv3x3_wgrad_scratch_bytes(N, H, W, Ci, Co, s), dtype=torch.uint8, device="cuda")
    dw = torch.empty((9, Co, Ci), device="cuda", dtype=torch.float32)
    nf.nf_conv3x3_wgrad(dtype, xd, gd, s, scratch, dw)
    ref = np.transpose(nfo.conv3x3_wgrad(x, g, s).reshape(Co, Ci, 9), (2, 0, 1))
    assert pu.max_err(dw.cpu().numpy(), ref) <= tol
    with pytest.raises(nf.NfError):
        nf.nf_conv3x3_wgrad(dtype, xd, gd, s, scratch[:16], dw)     # scratch too small


def test_bounded_wait_runs_out_and_reports_a_timeout(env):
    """The wait routine of the tensor-core kernels, in isolation: one small CTA waits on a barrier that nobody arrives at,
    with a 1 ms limit.  It must give up by itself (the call returns, the context stays usable), report about the limit as
    the time waited, and raise NF_ETIMEOUT in the status word; a kernel launched afterwards runs normally."""
    nf, torch = env
    assert nf.nf_op_status() == 0
    waited = torch.zeros(1, dtype=torch.int64, device="cuda")
    nf.nf_selftest_bounded_wait(1_000_000, waited)
    torch.cuda.synchronize()
    assert nf.nf_op_status() == nf.NF_ETIMEOUT
    assert nf.nf_op_status() == 0
    assert 1_000_000 <= int(waited.item()) < 100_000_000
    x = torch.ones(1024, device="cuda")
    assert float((x * 2).sum().item()) == 2048.0              # the device still answers
    with pytest.raises(nf.NfError):
        nf.nf_selftest_bounded_wait(0, waited)
    with pytest.raises(nf.NfError):
        nf.nf_selftest_bounded_wait(2_000_000_000, waited)    # limits above one second are refused
