"""GPU tests of the block-level calls: nf_block_step chains layer steps, nf_block_cache is the eval-mode
forward the checker computes (and is per-sample), nf_cache_gather re-batches bit-exactly."""
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


def _two_layer(nf, torch, dtype, N, seed, pool_first=True, C=64, F=16):
    c1 = dict(N=N, Cin=C, Cout=C, H=16, W=16, F=F, classes=10, stride=1, pool=pool_first)
    hw = 8 if pool_first else 16
    c2 = dict(N=N, Cin=C, Cout=2 * C, H=hw, W=hw, F=8, classes=10, stride=1, pool=False)
    cases = []
    for k, c in enumerate((c1, c2)):
        P, x, y = pu.seeded_case(c, seed + k, bf16=(dtype == 1))
        cases.append((c, P, x, y))
    return cases


@pytest.mark.parametrize("dtype", [0, 1])
def test_block_step_equals_chained_layer_steps(env, dtype):
    nf, torch = env
    cases = _two_layer(nf, torch, dtype, 6, 700)
    A = [pu.gpu_layer(nf, c, P, dtype) for c, P, _, _ in cases]
    B = [pu.gpu_layer(nf, c, P, dtype) for c, P, _, _ in cases]
    blk = nf.Block(B)
    x = pu.to_device_nhwc(torch, cases[0][2], dtype)
    lab = torch.from_numpy(cases[0][3]).cuda()
    la = torch.zeros(2, device="cuda")
    a1, a2 = A[0].new_act(), A[1].new_act()
    A[0].step(x, lab, 0.01, la[0:1], a1)
    A[1].step(a1, lab, 0.01, la[1:2], a2)
    lb = torch.zeros(2, device="cuda")
    b2 = B[1].new_act()
    blk.step(x, lab, 0.01, lb, b2)
    torch.cuda.synchronize()
    assert torch.equal(la, lb) and torch.equal(a2, b2)
    for k in range(2):
        for name in pu.PNAMES:
            assert np.array_equal(A[k].get_param(name), B[k].get_param(name))


@pytest.mark.parametrize("dtype", [0, 1])
def test_block_cache_matches_checker_eval_forward_and_is_per_sample(env, dtype):
    nf, torch = env
    N = 6
    cases = _two_layer(nf, torch, dtype, N, 710)
    G = [pu.gpu_layer(nf, c, P, dtype) for c, P, _, _ in cases]
    O = [pu.oracle_layer(c, P, store_bf16=(dtype == 1)) for c, P, _, _ in cases]
    blk = nf.Block(G)
    x = cases[0][2]
    lab = cases[0][3]
    # one training step on both sides so that running statistics are not the initial 0/1
    xd = pu.to_device_nhwc(torch, x, dtype)
    loss = torch.zeros(2, device="cuda")
    blk.step(xd, torch.from_numpy(lab).cuda(), 0.01, loss)
    _, a_o, _ = O[0].step(x, lab, 0.01)
    O[1].step(a_o, lab, 0.01)
    if dtype == 1:   # take the checker's state on both sides (see parity_util.check_step)
        for g, o in zip(G, O):
            for k in pu.PNAMES:
                v32 = o.p[k].astype(np.float32)
                o.set(**{k: v32})
                g.set_param(k, v32)
            for k in ("rmean", "rvar"):
                v32 = getattr(o, k).astype(np.float32)
                o.set(**{k: v32})
                g.set_param(k, v32)
    out = G[1].new_act()
    blk.cache(xd, out)
    torch.cuda.synchronize()
    ref = O[1].eval_forward(O[0].eval_forward(x))
    assert pu.max_err(pu.from_device_nhwc(out), ref) <= pu.TOL[dtype]["t"]
    # a sample's cached row does not depend on its batch-mates: sample 3 alone, and a count of 2 < N
    one = torch.zeros_like(out)
    blk.cache(xd[3:4].contiguous(), one, count=1)
    two = torch.zeros_like(out)
    blk.cache(xd[4:6].contiguous(), two, count=2)
    torch.cuda.synchronize()
    assert torch.equal(one[0], out[3]) and torch.equal(two[:2], out[4:6])
    with pytest.raises(nf.NfError):
        blk.cache(xd, out, count=N + 1)
    assert all(l.status() == 0 for l in G)


def test_cache_gather_is_bit_exact(env):
    nf, torch = env
    K, row = 300, (4, 4, 24)
    cache = torch.from_numpy(synth.to_bf16_bits(synth.normal(3, 1, (K,) + row)).view(np.int16)).cuda().view(torch.bfloat16)
    labels = torch.from_numpy(synth.labels(3, 2, K, 100)).cuda()
    for it, n in enumerate((1, 77, 300)):
        idx = torch.from_numpy(synth.permutation(5 + it, 1, K)[:n].copy()).cuda()
        out = torch.zeros((n,) + row, dtype=torch.bfloat16, device="cuda")
        out_l = torch.full((n,), -1, dtype=torch.int32, device="cuda")
        nf.nf_cache_gather(cache, labels, idx, out, out_l)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), cache[idx.long()].view(torch.int16))
        assert torch.equal(out_l, labels[idx.long()])
    with pytest.raises(nf.NfError):
        nf.nf_cache_gather(cache, labels, idx, out, None)      # labels in without labels out


def test_cache_gather_skips_indices_outside_the_cache(env):
    """A stale or corrupt permutation entry (negative, or beyond the cache's rows) must not become an out-of-bounds read:
    the kernel checks every index, zero-fills that output row, sets its label to -1 and raises NF_EINDEX; the rows with
    valid indices are still copied bit for bit."""
    nf, torch = env
    K, row = 40, (2, 2, 16)
    cache = torch.from_numpy(synth.to_bf16_bits(synth.normal(4, 1, (K,) + row)).view(np.int16)).cuda().view(torch.bfloat16)
    labels = torch.from_numpy(synth.labels(4, 2, K, 10)).cuda()
    idx_h = np.array([3, -1, 39, 40, 7, 2 ** 31 - 1, -2 ** 31, 0], dtype=np.int32)
    idx = torch.from_numpy(idx_h).cuda()
    out = torch.full((len(idx_h),) + row, 7.0, dtype=torch.bfloat16, device="cuda")
    out_l = torch.full((len(idx_h),), 123, dtype=torch.int32, device="cuda")
    assert nf.nf_op_status() == 0
    nf.nf_cache_gather(cache, labels, idx, out, out_l)
    torch.cuda.synchronize()
    good = (idx_h >= 0) & (idx_h < K)
    gi = torch.from_numpy(np.nonzero(good)[0]).cuda()
    bi = torch.from_numpy(np.nonzero(~good)[0]).cuda()
    assert torch.equal(out[gi].view(torch.int16), cache[idx[gi].long()].view(torch.int16))
    assert torch.equal(out_l[gi], labels[idx[gi].long()])
    assert int(out[bi].view(torch.int16).abs().max()) == 0 and bool((out_l[bi] == -1).all())
    assert nf.nf_op_status() == nf.NF_EINDEX
    assert nf.nf_op_status() == 0                                 # reading clears the word


def test_prefetching_host_step_equals_plain_host_step():
    """A stream of different batches through nf_block_step_host_next (the next batch copied while this one trains)
    gives bit-identical losses and parameters to the plain host step; a call whose batch was not announced falls
    back to copying it itself."""
    import torch
    from paper_2402_14139_b200 import nf, synth
    from tests import parity_util as pu
    nf.lib()
    nf.nf_set_stream(None)
    c1 = dict(N=6, Cin=64, Cout=64, H=16, W=16, F=16, classes=10, stride=1, pool=False)
    c2 = dict(N=6, Cin=64, Cout=64, H=16, W=16, F=8, classes=10, stride=1, pool=True)
    P1, _, _ = pu.seeded_case(c1, 71, bf16=True)
    P2, _, _ = pu.seeded_case(c2, 72, bf16=True)

    def make(host_io):
        layers = [pu.gpu_layer(nf, c1, P1, nf.NF_BF16, host_io=host_io), pu.gpu_layer(nf, c2, P2, nf.NF_BF16)]
        return layers, nf.Block(layers)

    la, A = make(1)
    lb, B = make(2)
    xs = [torch.from_numpy(synth.round_bf16(synth.normal(73, k, (6, 16, 16, 64)))).to(torch.bfloat16).pin_memory() for k in range(4)]
    ys = [torch.from_numpy(synth.labels(74, k, 6, 10)).pin_memory() for k in range(4)]
    la_h, lb_h = torch.zeros(2).pin_memory(), torch.zeros(2).pin_memory()
    order = [0, 1, 2, 3, 1]
    for i, k in enumerate(order):
        A.step_host(xs[k], ys[k], 0.05, la_h)
        nxt = order[i + 1] if i + 1 < len(order) and i != 2 else None      # step 3's batch is NOT announced
        B.step_host_next(xs[k], ys[k], 0.05, lb_h, None if nxt is None else xs[nxt], None if nxt is None else ys[nxt])
        assert torch.equal(la_h, lb_h), (i, la_h, lb_h)
    for ga, gb in zip(la, lb):
        for name in pu.PNAMES:
            assert np.array_equal(ga.get_param(name), gb.get_param(name)), name
    # the plain layer (host_io = 1) has no second buffer: the call is refused
    assert nf.lib().nf_block_step_host_next(A.h, nf._ptr(xs[0]), nf._ptr(ys[0]), 0.05, nf._ptr(la_h), None, None, None) == nf.NF_EINVAL


def test_captured_block_step_replays_identically():
    """nf.Block.capture: the whole block step recorded into a CUDA graph; replays give bit-identical losses and
    parameters to the same number of eager steps."""
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    nf.nf_set_stream(None)
    c1 = dict(N=8, Cin=3, Cout=64, H=16, W=16, F=16, classes=10, stride=1, pool=False)
    c2 = dict(N=8, Cin=64, Cout=64, H=16, W=16, F=8, classes=10, stride=1, pool=True)
    P1, x, y = pu.seeded_case(c1, 81, bf16=True)
    P2, _, _ = pu.seeded_case(c2, 82, bf16=True)
    xd, yd = pu.to_device_nhwc(torch, x, 1), torch.from_numpy(y).cuda()

    def run(graph):
        layers = [pu.gpu_layer(nf, c1, P1, nf.NF_BF16), pu.gpu_layer(nf, c2, P2, nf.NF_BF16)]
        blk = nf.Block(layers)
        loss = torch.zeros(2, device="cuda")
        blk.step(xd, yd, 0.05, loss)                     # the eager step that must precede a capture
        if graph:
            g = blk.capture(xd, yd, 0.05, loss)
            for _ in range(3):
                g.replay()
        else:
            for _ in range(3):
                blk.step(xd, yd, 0.05, loss)
        torch.cuda.synchronize()
        out = loss.cpu().numpy().copy(), [L.get_param("W") for L in layers], [L.status() for L in layers]
        nf.nf_set_stream(None)
        return out

    (la, wa, sa), (lb, wb, sb) = run(False), run(True)
    assert sa == sb == [0, 0] and np.array_equal(la, lb)
    for a, b in zip(wa, wb):
        assert np.array_equal(a, b)
