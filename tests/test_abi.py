"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every symbol the header
declares, and its host-only entry points behave (no kernel is launched here)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import nfo

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def nf():
    from paper_2402_14139_b200 import build
    build.build()
    from paper_2402_14139_b200 import nf as mod
    return mod


def test_every_declared_symbol_is_exported(nf):
    hdr = open(os.path.join(ROOT, "include", "nf.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = sorted(set(re.findall(r"\b(nf_[a-z_0-9]+)\s*\(", hdr)))
    assert len(declared) >= 20
    L = nf.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert sorted(nf.EXPORTS) == declared


def test_create_configure_and_workspace_size_are_host_only(nf):
    L = nf.lib()
    assert not L.nf_layer_create(0, 16, 32, 32, 4, 10)
    h = L.nf_layer_create(3, 16, 32, 32, 4, 10)
    assert h
    o = nf.nf_layer_opts(8, 1, 0, nf.NF_F32, 0.9, 1e-5, 0.1, 0)
    assert L.nf_layer_configure(h, C.byref(o)) == nf.NF_OK
    small = L.nf_layer_workspace_bytes(h)
    o.N = 64
    assert L.nf_layer_configure(h, C.byref(o)) == nf.NF_OK
    assert L.nf_layer_workspace_bytes(h) > small > 0
    for bad in (dict(N=0), dict(stride=3), dict(dtype=7), dict(momentum=1.5)):
        ob = nf.nf_layer_opts(8, 1, 0, nf.NF_F32, 0.9, 1e-5, 0.1, 0)
        for k, v in bad.items():
            setattr(ob, k, v)
        assert L.nf_layer_configure(h, C.byref(ob)) == nf.NF_EINVAL
    h2 = L.nf_layer_create(3, 16, 31, 31, 4, 10)   # 31x31 output cannot be max-pooled 2x2
    op = nf.nf_layer_opts(8, 1, 1, nf.NF_F32, 0.9, 1e-5, 0.1, 0)
    assert L.nf_layer_configure(h2, C.byref(op)) == nf.NF_EINVAL
    # calls that need a workspace refuse without one
    assert L.nf_layer_step(h, None, None, 0.1, None, None) == nf.NF_EINVAL
    buf = np.zeros(16, dtype=np.float32)
    assert L.nf_layer_get_param(h, nf.NF_P_GAMMA, buf.ctypes.data_as(C.c_void_p), 16) == nf.NF_ENOWS
    L.nf_layer_destroy(h)
    L.nf_layer_destroy(h2)
    assert nf.nf_strerror(nf.NF_ENOWS) and nf.nf_strerror(nf.NF_OK) == "ok"


def test_partition_matches_checker_and_paper_example(nf):
    gold = os.path.join(ROOT, "tests", "golden", "vgg19_max_batch_630mb.txt")
    mb = [int(v) for v in [ln for ln in open(gold) if not ln.startswith("#")][0].split()]
    assert nf.nf_partition(mb, 512, 0.4) == [(0, 2, 30), (3, 3, 60), (4, 7, 90), (8, 11, 195), (12, 15, 512)]
    rng = np.random.default_rng(1)
    for _ in range(200):
        n = int(rng.integers(1, 20))
        v = rng.integers(1, 2000, n).tolist()
        B = int(rng.integers(1, 1500))
        rho = float(rng.choice([0.0, 0.1, 0.4, 0.7]))
        assert nf.nf_partition(v, B, rho) == nfo.partition(v, B, rho)
    with pytest.raises(nf.NfError):
        nf.nf_partition([10, 0], 100, 0.4)


def test_select_exit_rule_matches_checker_on_the_host():
    """Highest validation accuracy wins; equal accuracies go to the smaller model; the first of full ties."""
    from oracle import nfo
    from paper_2402_14139_b200 import nf, synth
    assert nf.nf_select_exit([0.5, 0.7, 0.7, 0.6], [10, 30, 20, 40]) == 2
    assert nf.nf_select_exit([0.7, 0.7], [20, 20]) == 0
    assert nf.nf_select_exit([0.1], [5]) == 0
    for t in range(50):
        n = 1 + t % 9
        acc = [round(float(v) * 4) / 4 for v in synth.uniform01(0x4E46E200, t, n)]     # many ties
        par = [int(v * 5) for v in synth.uniform01(0x4E46E201, t, n)]
        assert nf.nf_select_exit(acc, par) == nfo.select_exit(acc, par)


def test_profiler_rule_line_fit_and_max_batch_on_the_host():
    """The Profiler's three host steps against the checker and against what the paper states: the AAN-LL rule
    (VGG: 32 filters before the first down-sampling, 256 after), the layer-wise linear memory model (the library's
    own memory need is linear in the batch size up to alignment; its slope is the stored bytes per image) and the
    largest batch under a budget."""
    import numpy as np
    from oracle import nfo
    from paper_2402_14139_b200 import nf, workloads
    vgg19 = [64, 64, 128, 128, 256, 256, 256, 256, 512, 512, 512, 512, 512, 512, 512, 512]
    want = [32, 32] + [256] * 14                      # the paper's worked example for VGG
    assert nf.nf_aan_filters(vgg19, 2) == want == nfo.aan_filters(vgg19, 2)
    resnet = [64] * 5 + [128] * 4 + [256] * 4 + [512] * 4
    assert nf.nf_aan_filters(resnet, 1) == nfo.aan_filters(resnet, 1) == [32] + [256] * 16
    # checker's line fit against the library routine numpy offers, then the library against the checker
    xs, ys = [8, 16, 32, 64, 96], [1.0e6, 1.9e6, 4.2e6, 8.1e6, 12.3e6]
    sl, ic = nfo.fit_line(xs, ys)
    ref = np.polyfit(xs, ys, 1)
    assert abs(sl - ref[0]) <= 1e-9 * abs(ref[0]) and abs(ic - ref[1]) <= 1e-6 * abs(ref[1])
    sl2, ic2 = nf.nf_fit_line(xs, ys)                 # the stand-alone fit the measured Profiler uses
    assert abs(sl2 - sl) <= 1e-9 * abs(sl) and abs(ic2 - ic) <= 1e-6 * abs(ic)
    with pytest.raises(nf.NfError):
        nf.nf_fit_line([8, 8], [1.0, 2.0])            # all batch sizes equal: no line
    l = dict(Cin=64, Cout=64, H=32, W=32, F=32, stride=1, pool=True)
    batches = [16, 32, 64, 128, 256]
    by, slope, icpt = nf.nf_profile_layer(l["Cin"], l["Cout"], l["H"], l["W"], l["F"], 10, batches, maxpool=True)
    s2, i2 = nfo.fit_line(batches, by)
    assert abs(slope - s2) <= 1e-9 * s2 and abs(icpt - i2) <= 1e-6 * max(abs(i2), 1.0)
    assert all(abs(b - (icpt + slope * n)) <= 0.01 * b for n, b in zip(batches, by))          # "linearly correlates with the batch size"
    per_image = workloads.layer_bytes_per_image(l, 10)
    assert abs(slope - per_image) <= 0.02 * per_image                                          # slope = stored bytes per image
    for budget in (64e6, 630e6, 4e9):
        t = nf.nf_max_batch(slope, icpt, budget)
        assert t == nfo.max_batch_from_line(slope, icpt, budget)
        assert icpt + slope * t <= budget < icpt + slope * (t + 1)
    assert nf.nf_max_batch(slope, icpt, 0.0) == 0


def test_planned_blocks_of_the_aan_workload_match_its_stored_default():
    """The block list stored in the c6 workload is what the Profiler and Algorithm 1 of the library return."""
    from paper_2402_14139_b200 import nf, pipeline, workloads
    wl = workloads.c6()
    assert [l["F"] for l in wl["layers"]] == nf.nf_aan_filters([l["Cout"] for l in wl["layers"]], 2)
    plan = pipeline.plan_blocks(nf, wl["layers"], wl["classes"], 2e9, 50000, 0.4)
    assert [(bs, len(ls)) for bs, ls in wl["blocks"]] == [(bs, l - f + 1) for f, l, bs in plan]


def test_projection_description_is_host_only(nf):
    """nf_proj_create / configure / workspace_bytes do no device work: they size the workspace a caller must provide."""
    L = nf.lib()
    assert not L.nf_proj_create(0, 8, 8, 8)
    h = L.nf_proj_create(64, 128, 32, 32)
    assert h
    assert L.nf_proj_configure(h, 8, nf.NF_BF16, 0.9, 1e-5, 0.1) == nf.NF_OK
    small = L.nf_proj_workspace_bytes(h)
    assert L.nf_proj_configure(h, 64, nf.NF_BF16, 0.9, 1e-5, 0.1) == nf.NF_OK
    big = L.nf_proj_workspace_bytes(h)
    # two stored tensors of N x 16 x 16 x 128 bf16 (conv output and its gradient) dominate the growth
    assert big > small > 0 and abs((big - small) - 2 * 56 * 16 * 16 * 128 * 2) <= 0.1 * (big - small)
    for bad in (dict(N=0), dict(dtype=5), dict(momentum=1.0), dict(eps=0.0)):
        a = dict(N=8, dtype=nf.NF_BF16, momentum=0.9, eps=1e-5)
        a.update(bad)
        assert L.nf_proj_configure(h, a["N"], a["dtype"], a["momentum"], a["eps"], 0.1) == nf.NF_EINVAL
    buf = np.zeros(128, dtype=np.float32)
    assert L.nf_proj_get_param(h, nf.NF_P_GAMMA, buf.ctypes.data_as(C.c_void_p), 128) == nf.NF_ENOWS    # no workspace bound
    assert L.nf_proj_forward(h, None, None) == nf.NF_EINVAL
    L.nf_proj_destroy(h)
