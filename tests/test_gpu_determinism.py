"""Results do not depend on how the local steps are issued: one call with K steps, K calls with one
step each, and the same work on a side stream while the default stream is busy all leave
bit-identical weights and losses (every reduction in the library has a fixed order)."""
import numpy as np
import pytest

from paper_1910_02120_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _run(w, W, b, X, y, split, stream=None):
    import torch
    from paper_1910_02120_b200 import api
    ctx = api.Ist(w.layer_dims, w.S, api.IST_BF16, w.B, device="cuda:0", stream=stream)
    Wd = [torch.tensor(x, device="cuda:0") for x in W]
    bd = [torch.tensor(x, device="cuda:0") for x in b]
    torch.cuda.synchronize()
    if stream is not None:                                # keep the default stream occupied meanwhile
        busy = torch.randn(4096, 4096, device="cuda:0")
        for _ in range(20):
            busy = busy @ busy * 1e-4
    ctx.bind_weights(Wd, bd)
    ctx.partition(9)
    if split:
        losses = torch.cat([ctx.local_steps(X[k * w.B:], y[k * w.B:], w.lr, 1, w.B, stride_subnet=w.K * w.B,
                                            stride_step=w.B) for k in range(w.K)], dim=1)
    else:
        losses = ctx.local_steps(X, y, w.lr, w.K, w.B)
    ctx.reassemble()
    ctx.sync_status()
    return [x.cpu().numpy() for x in Wd] + [x.cpu().numpy() for x in bd], losses.cpu().numpy()


def test_issue_pattern_and_stream_do_not_change_the_result():
    import torch
    w = synth.Workload("d", (256, 1024, 1024, 35), S=4, B=128, K=4, rounds=1, precision="bf16", x_dist="normal",
                       lr=0.02, seed=5)
    W, b, data = H.make_problem(w)
    X, y = H.gpu_inputs(w, data)
    ref, ref_loss = _run(w, W, b, X, y, split=False)
    got, got_loss = _run(w, W, b, X, y, split=True)
    assert np.array_equal(got_loss, ref_loss) and all(np.array_equal(g, r) for g, r in zip(got, ref))
    side = torch.cuda.Stream()
    got, got_loss = _run(w, W, b, X, y, split=False, stream=side)
    assert np.array_equal(got_loss, ref_loss) and all(np.array_equal(g, r) for g, r in zip(got, ref))
