"""Several IST rounds in a row (Sec. 2.1: re-partition after every K local steps): the CUDA
library follows the oracle's trajectory round by round, and on a learnable synthetic task the
reassembled full network improves from round to round."""
import numpy as np
import pytest

from paper_1910_02120_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("norm_eps", [None, 1e-5])
def test_four_rounds_follow_the_oracle(norm_eps):
    import torch
    from oracle import ist_oracle as O
    from paper_1910_02120_b200 import api
    dims, S, K, B, R, lr = (16, 48, 40, 5), 3, 3, 16, 4, 0.05
    n = 512
    X_all, y_all = synth.make_teacher_task(n, dims[0], dims[-1], 3)
    W, b = synth.make_weights(dims, 3, bias_scale=0.1)
    o = O.IstOracle(dims, S, norm_eps=norm_eps)
    o.bind_weights(W, b)
    dev = "cuda:0"
    ctx = api.Ist(dims, S, api.IST_FP32, 128, device=dev)
    Wd = [torch.tensor(x, device=dev) for x in W]
    bd = [torch.tensor(x, device=dev) for x in b]
    ctx.bind_weights(Wd, bd)
    if norm_eps is not None:
        ctx.enable_normalization(norm_eps)
    for r in range(R):
        rows = synth.draw_round_rows(n, S, K, B, 3, r)
        Xr, yr = X_all[rows], y_all[rows]                 # [S][K][B][N0], [S][K][B]
        ol = o.round(100 + r, Xr.astype(np.float64), yr, lr, K)
        gl = ctx.round(100 + r, torch.tensor(Xr.reshape(-1, dims[0]), device=dev),
                       torch.tensor(yr.reshape(-1), device=dev), lr, K, B)
        ctx.sync_status()
        np.testing.assert_allclose(gl.cpu().numpy(), ol, rtol=5e-4)
    for l in range(len(W)):
        H.assert_close(Wd[l].cpu().numpy(), o.W[l], 5e-4, f"W_{l + 1} after {R} rounds")
        H.assert_close(bd[l].cpu().numpy(), o.b[l], 5e-4, f"b_{l + 1} after {R} rounds")
    # the deployed network: statistics over a subset, then held-out loss
    Xe, ye = X_all[:128], y_all[:128]
    if norm_eps is not None:
        o.calibrate(Xe.astype(np.float64))
        ctx.calibrate(torch.tensor(Xe, device=dev), 128)
    ol, oc = o.eval(Xe.astype(np.float64), ye)
    gl, gc = ctx.eval(torch.tensor(Xe, device=dev), torch.tensor(ye, device=dev), 128)
    assert abs(gl.item() - ol) <= 1e-3 * abs(ol)
    assert abs(gc.item() - oc) <= 2


def test_ist_learns_a_synthetic_task_over_rounds():
    from paper_1910_02120_b200 import teacher_student as T
    recs = T.train((64, 512, 512, 10), S=4, K=10, B=64, rounds=30, lr=0.05, norm_eps=1e-5,
                   precision="bf16", seed=1, eval_every=5)
    first, last = recs[0], recs[-1]
    assert last["test_loss"] < 0.8 * first["test_loss"], recs
    assert last["test_acc"] > first["test_acc"] + 0.1 and last["test_acc"] > 0.35, recs
    assert last["subnet_loss"] < first["subnet_loss"], recs
