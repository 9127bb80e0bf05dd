"""GPU test of the block-wise driver: two small blocks over a 24-image dataset; the cache handed to block 2
is what nf_block_cache produces, batches are re-assembled by permutation, nothing reruns block 1."""
import numpy as np
import pytest

from paper_2402_14139_b200 import pipeline, synth

pytestmark = pytest.mark.gpu


def _wl():
    l = lambda Cin, Cout, H, F, pool=False: dict(Cin=Cin, Cout=Cout, H=H, W=H, F=F, stride=1, pool=pool)
    return dict(name="mini", dtype="bf16", classes=4, in_shape=(3, 16, 16),
                blocks=[(6, [l(3, 64, 16, 8), l(64, 64, 16, 8, pool=True)]), (8, [l(64, 128, 8, 16)])])


def test_blockwise_pass_runs_and_learns_a_learnable_task():
    import torch
    from paper_2402_14139_b200 import nf
    nf.lib()
    nf.nf_set_stream(None)
    K = 24
    x = synth.normal(5, 1, (K, 16, 16, 3))
    lab = (np.arange(K) % 4).astype(np.int32)
    for k in range(K):                       # class = which quadrant carries a bright patch: learnable by conv + pooled head
        u, v = lab[k] // 2, lab[k] % 2
        x[k, u * 8:(u + 1) * 8, v * 8:(v + 1) * 8, :] += 2.0
    data = torch.from_numpy(synth.round_bf16(x)).cuda().to(torch.bfloat16)
    labels = torch.from_numpy(lab).cuda()
    recs = []
    report, out = pipeline.train_blockwise(nf, torch, _wl(), data, labels, epochs=25, lr=0.05, seed=3, log=recs.append)
    assert [r["block"] for r in report] == [0, 1] and report[0]["steps"] == 25 * 4 and report[1]["steps"] == 25 * 3
    assert out.shape == (K, 8, 8, 128) and torch.isfinite(out.float()).all()
    assert all(np.isfinite(r["losses"]).all() for r in report)
    assert report[0]["losses"][-1] < 0.7 * np.log(4)       # the local loss of block 1's last layer fell well below chance
