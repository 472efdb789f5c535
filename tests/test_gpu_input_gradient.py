"""The input gradient of a local step (Sec. 2.2, "IST for other architectures": what a trunk in front
of the partitioned fully connected layers is trained from), through ist_local_steps_dx, against the
oracle's delta_1 W_1^T row by row; the round itself must come out as without the extra output."""
import numpy as np
import pytest

from paper_1910_02120_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _wl(dims, S, B, K, precision, lr=0.05, seed=23):
    return synth.Workload("dx", tuple(dims), S=S, B=B, K=K, rounds=1, precision=precision,
                          x_dist="normal", lr=lr, seed=seed)


@pytest.mark.parametrize("precision,dims,S,B,K", [
    ("fp32", [20, 37, 5], 3, 7, 3),                  # nothing divides anything
    ("fp32", [12, 6], 1, 5, 2),                      # no hidden layer: delta_1 is the softmax gradient
    ("fp32", [64, 256, 128, 10], 2, 96, 2),
    ("bf16", [256, 1024, 1024, 35], 4, 256, 2),
    ("bf16", [264, 6144, 24], 3, 384, 1),            # CTA-pair tiles with ragged edges
    ("bf16", [40, 72, 136, 12], 2, 40, 2),           # small and ragged
])
def test_input_gradient_matches_oracle(precision, dims, S, B, K):
    import torch
    from oracle import ist_oracle as O
    w = _wl(dims, S, B, K, precision)
    W, b, data = H.make_problem(w)
    seed = 77
    o = O.IstOracle(w.layer_dims, w.S)
    o.bind_weights(W, b)
    o.partition(seed)
    olosses, odx = o.local_steps_dx(data.X, data.y, w.lr, w.K)
    o.reassemble()

    ctx, Wd, bd = H.gpu_context(w, W, b)
    X, y = H.gpu_inputs(w, data)
    ctx.partition(seed)
    dx = torch.full((X.shape[0], dims[0]), float("nan"), dtype=torch.float32, device="cuda:0")
    glosses = ctx.local_steps(X, y, w.lr, w.K, w.B, dx_out=dx)
    ctx.reassemble()
    ctx.sync_status()

    gdx = dx.cpu().numpy().astype(np.float64).reshape(odx.shape)
    assert np.isfinite(gdx).all()                    # every row of X was read by some step
    fro = np.linalg.norm(gdx - odx) / np.linalg.norm(odx)
    if precision == "fp32":
        H.assert_close(gdx, odx, 1e-4, "dX")
        assert np.max(np.abs(glosses.cpu().numpy() - olosses)) <= 1e-4 * np.abs(olosses).max()
    else:
        # like the weight updates, dX carries the ReLU-mask flips of the bf16 path
        assert fro <= 1e-1, f"dX: {fro:.3e}"
        assert abs(glosses.cpu().numpy().mean() - olosses.mean()) <= 1e-3
    rtol = 1e-4 if precision == "fp32" else 2e-2
    for l in range(len(W)):
        H.assert_close(Wd[l].cpu().numpy(), o.W[l], rtol, f"W_{l + 1}")
        H.assert_close(bd[l].cpu().numpy(), o.b[l], rtol, f"b_{l + 1}")


def test_input_gradient_refuses_sparse_inputs():
    import torch
    from paper_1910_02120_b200 import api
    w = synth.Workload("dxc", (3000, 130, 50), S=2, B=16, K=1, rounds=1, precision="fp32", x_dist="csr", seed=8)
    W, b, data = H.make_problem(w)
    ctx, Wd, bd = H.gpu_context(w, W, b)
    X, y = H.gpu_inputs(w, data)
    ctx.partition(1)
    dx = torch.zeros((2 * 16, 3000), dtype=torch.float32, device="cuda:0")
    with pytest.raises(api.IstError) as e:
        ctx.local_steps(X, y, w.lr, w.K, w.B, dx_out=dx)
    assert e.value.status == api.IST_ERR_UNSUPPORTED
    ctx.local_steps(X, y, w.lr, w.K, w.B)          # the context is still usable
    ctx.reassemble()
    ctx.sync_status()


@pytest.mark.parametrize("precision", ["fp32", "bf16"])
def test_trunk_in_front_of_the_partitioned_head_learns(precision):
    # Sec. 2.2, last paragraph, end to end: a small convolutional trunk (torch, one copy per
    # subnet, averaged at the end of a round) trained only from the library's input gradients,
    # the head by IST.  The loss of the subnets' local steps must fall clearly.
    from paper_1910_02120_b200 import trunk_head
    recs = trunk_head.train(rounds=30, S=4, K=10, B=64, lr=0.3, precision=precision, seed=3)
    first, last = recs[0]["subnet_loss"], recs[-1]["subnet_loss"]
    assert np.isfinite(last) and last < 0.9 * first, (first, last)     # measured 2.29 -> 1.91
