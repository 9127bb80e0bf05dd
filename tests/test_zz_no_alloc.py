"""The allocation-free weight gradient (nf_conv3x3_wgrad_static) against the ordinary entry point.

A trainer that runs on a fixed device-memory budget may have nothing left to allocate when it needs
a weight gradient, so the library offers a variant whose partial sums live in a 16 MiB array built
into the library.  This file checks, through the C ABI, that the variant returns what
nf_conv3x3_wgrad returns (within the tolerance of the other parity tests) and what the CPU checker
computes, on calls in a row with different problems -- each later call finds the array full of the
previous call's partials -- and that it refuses problems larger than its array.  The shapes cover the
CUDA-core kernel (fp32; bf16 with 32 input channels) and the tensor-core kernel (bf16, 64 -> 64 channels,
12 pixel splits of 147 KB).  It is collected last on purpose.
"""
import numpy as np
import pytest

from oracle import nfo
from paper_2402_14139_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def _run_both(nf, torch, dtype, N, Ci, Co, H, W, s, seed):
    rnd = synth.round_bf16 if dtype == 1 else (lambda a: np.asarray(a, dtype=np.float32))
    Ho, Wo = (H - 1) // s + 1, (W - 1) // s + 1
    x, g = rnd(synth.normal(seed, 1, (N, Ci, H, W))), rnd(synth.normal(seed, 2, (N, Co, Ho, Wo)))
    xd, gd = pu.to_device_nhwc(torch, x, dtype), pu.to_device_nhwc(torch, g, dtype)
    scratch = torch.empty(nf.nf_conv3x3_wgrad_scratch_bytes(N, H, W, Ci, Co, s), dtype=torch.uint8, device="cuda")
    want = torch.empty((9, Co, Ci), device="cuda", dtype=torch.float32)
    nf.nf_conv3x3_wgrad(dtype, xd, gd, s, scratch, want)
    got = torch.full((9, Co, Ci), float("nan"), device="cuda", dtype=torch.float32)
    nf.nf_conv3x3_wgrad_static(dtype, xd, gd, s, got)
    torch.cuda.synchronize()
    ref = nfo.conv3x3_wgrad(x, g, stride=s)                                   # [Co][Ci][3][3]
    ref = np.transpose(ref.reshape(Co, Ci, 9), (2, 0, 1))                    # the library's [tap][Co][Ci]
    return got.cpu().numpy(), want.cpu().numpy(), ref


def test_static_scratch_wgrad_matches_on_two_calls_in_a_row():
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    nf.nf_set_stream(None)
    # bf16 on the CUDA-core kernel, several split partials; fp32, another shape, stale partials in the array; bf16 on the
    # tensor-core kernel (64 -> 64 channels, three 16 x 32 maps: 12 pixel splits); the first shape once more
    cases = [(nf.NF_BF16, (4, 32, 48, 16, 16, 1), 901), (nf.NF_F32, (3, 20, 33, 12, 10, 2), 902),
             (nf.NF_BF16, (3, 64, 64, 16, 32, 1), 903), (nf.NF_BF16, (4, 32, 48, 16, 16, 1), 904)]
    for dtype, shape, seed in cases:
        assert nf.nf_conv3x3_wgrad_scratch_bytes(*[shape[k] for k in (0, 3, 4, 1, 2, 5)]) <= nf.NF_STATIC_SCRATCH_BYTES
        got, want, ref = _run_both(nf, torch, dtype, *shape, seed)
        assert np.isfinite(got).all()
        assert pu.max_err(got, want) <= pu.TOL[dtype]["t"]
        assert pu.max_err(got, ref) <= pu.TOL[dtype]["t"]
    assert nf.nf_op_status() == 0


def test_static_scratch_wgrad_refuses_what_does_not_fit():
    import torch
    from paper_2402_14139_b200 import nf
    N, Ci, Co, H, W = 2, 512, 512, 4, 4
    assert nf.nf_conv3x3_wgrad_scratch_bytes(N, H, W, Ci, Co, 1) > nf.NF_STATIC_SCRATCH_BYTES
    x = torch.zeros((N, H, W, Ci), device="cuda", dtype=torch.bfloat16)
    g = torch.zeros((N, H, W, Co), device="cuda", dtype=torch.bfloat16)
    dw = torch.zeros((9, Co, Ci), device="cuda", dtype=torch.float32)
    before = nf.nf_launch_count()
    with pytest.raises(nf.NfError, match="workspace"):
        nf.nf_conv3x3_wgrad_static(nf.NF_BF16, x, g, 1, dw)
    assert nf.nf_launch_count() == before
