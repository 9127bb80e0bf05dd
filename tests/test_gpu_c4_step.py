"""Whole local steps of the ImageNet-shaped block (workload c4) at its own map size, 224 x 224, against the CPU checker.

The three layers (64->64, 64->64, 64->128 with stride 2; 16 auxiliary filters; 1000 classes) are stepped one after the
other as Algorithm 2 does, each on the CHECKER's activation of the layer before, so both sides always see the same
bf16-valued input.  Every tensor of the step is compared element by element: loss, act_out, the seven gradients, the
updated parameters and the running statistics.  Only the batch is smaller than the benchmark's 64 images (the checker
needs about a second per image); the tile geometry per image (16 x 28 tiles of 14 x 8 pixels, 14 x 28 of 16 x 8 for the
input gradient, 7 x 14 on the stride-2 layer) and the kernels selected are those of the benchmark run.  The batch sizes
4 and 8 leave every CTA a different, uneven number of tiles (12.1 and 24.2 on 148 SMs).
"""
import numpy as np
import pytest

from paper_2402_14139_b200 import synth, workloads
from tests import parity_util as pu

pytestmark = pytest.mark.gpu

SEED = 0x4E460004


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    nf.nf_set_stream(None)
    return nf, torch


def _chain(nf, torch, N, store_bf16, tol, seed=SEED, gate=True):
    wl = workloads.c4()
    _, ls = wl["blocks"][0]
    x = synth.round_bf16(synth.normal(seed, 8, (N, ls[0]["Cin"], ls[0]["H"], ls[0]["W"]))).astype(np.float64)
    y = synth.labels(seed, 9, N, wl["classes"])
    out = []
    for li, l in enumerate(ls):
        c = pu.layer_cfg(l, N, wl["classes"])
        P, _, _ = pu.seeded_case(dict(c, N=1), seed + 0x400 + li, bf16=True)
        errs, act_o, O, G = pu.step_both(nf, torch, c, P, x, y, lr=0.01, store_bf16=store_bf16, tol=tol, gate=gate)
        assert [G.kernel_family(k) for k in range(4)] == ["tcgen05"] * 4
        assert G.kernel_family(4) == "fused"     # 224 and 112 are multiples of 14: BatchNorm + ReLU run inside the aux forward
        G.close()
        out.append(errs)
        # the next layer reads the bf16 activation both sides agree on: the checker's, rounded as the cache stores it
        x = synth.round_bf16(act_o).astype(np.float64)
    return out


@pytest.mark.parametrize("N", [4, 8])
def test_c4_block_steps_match_checker_at_224(env, N):
    nf, torch = env
    for li, errs in enumerate(_chain(nf, torch, N, True, pu.TOL[1])):
        print(f"c4 N={N} layer {li}:", {k: f"{v:.2e}" for k, v in errs.items()})


def test_c4_block_steps_against_unrounded_fp64_checker(env):
    """What the bf16 storage of the library costs: the same chain against the checker WITHOUT its bf16 storage mode."""
    nf, torch = env
    for li, errs in enumerate(_chain(nf, torch, 4, False, pu.UNROUNDED_TOL)):
        assert errs["act"] <= pu.UNROUNDED_TOL["act"], errs
        print(f"c4 N=4 layer {li} vs unrounded fp64:", {k: f"{v:.2e}" for k, v in errs.items()})
