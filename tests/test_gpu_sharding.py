"""Subnets split over several contexts (Sec. 2.1 / 2.3) on one GPU: two contexts that each gather
and train half of the subnets and then swap their packed slices end with the oracle's full
network (within the path's tolerance) and with exactly the full network of one context training
all of them.  (The exchange between GPUs is an all-gather of the same slabs; its host side is
covered on CPU with gloo ranks.)"""
import numpy as np
import pytest

from paper_1910_02120_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("precision,dims,S,B,K", [
    ("fp32", (20, 64, 48, 7), 4, 12, 3),
    ("bf16", (64, 256, 128, 10), 4, 32, 3),
    ("bf16", (256, 4096, 4096, 16), 8, 512, 2),      # tensor-core pair tiles in both arrangements
])
def test_two_half_contexts_equal_one_full_context(precision, dims, S, B, K):
    import torch
    from paper_1910_02120_b200 import api
    w = synth.Workload("sh", dims, S=S, B=B, K=K, rounds=1, precision=precision, x_dist="normal", lr=0.02, seed=31)
    W, b, data = H.make_problem(w, bias_scale=0.1)
    X, y = H.gpu_inputs(w, data)
    seed = 77
    ref, Wr, br = H.gpu_context(w, W, b)
    ref_loss = ref.round(seed, X, y, w.lr, K, B)
    ref.sync_status()
    half = S // 2
    rows = half * K * B
    parts = []
    for r in range(2):
        ctx, Wd, bd = H.gpu_context(w, W, b)
        ctx.set_subnet_range(r * half, half)
        ctx.partition(seed)
        loss = ctx.local_steps(X[r * rows:(r + 1) * rows], y[r * rows:(r + 1) * rows], w.lr, K, B)
        assert torch.equal(loss, ref_loss[r * half:(r + 1) * half])
        parts.append((ctx, Wd, bd))
    for l in range(1, len(dims)):                      # the exchange: every context gets the other's slabs
        (m0, b0), (m1, b1) = parts[0][0].packed_layer(l), parts[1][0].packed_layer(l)
        m0[half:] = m1[half:]
        b0[half:] = b1[half:]
        m1[:half] = m0[:half]
        b1[:half] = b0[:half]
    o, _, oloss = H.oracle_round(w, W, b, data, seed)
    rtol = 2e-2 if precision == "bf16" else 1e-4
    for ctx, Wd, bd in parts:
        ctx.reassemble()
        ctx.sync_status()
        for l in range(len(dims) - 1):
            H.assert_close(Wd[l].cpu().numpy(), o.W[l], rtol, f"W_{l + 1} against the oracle")
            H.assert_close(bd[l].cpu().numpy(), o.b[l], rtol, f"b_{l + 1} against the oracle")
            assert torch.equal(Wd[l], Wr[l]), f"W_{l + 1}"
            assert torch.equal(bd[l], br[l]), f"b_{l + 1}"
    loss_tol = 1e-3 if precision == "bf16" else 1e-4 * abs(oloss.mean())
    assert abs(float(ref_loss.mean()) - oloss.mean()) <= loss_tol


def test_a_narrowed_context_gathers_only_its_own_subnets():
    """With a subnet range set, ist_partition leaves the other subnets' packed slabs alone
    (Sec. 2.3: a site receives its own slices only)."""
    import torch
    w = synth.Workload("sh", (64, 256, 128, 10), S=4, B=8, K=1, rounds=1, precision="bf16", x_dist="normal", seed=3)
    W, b, data = H.make_problem(w, bias_scale=0.1)
    ctx, Wd, bd = H.gpu_context(w, W, b)
    ctx.set_subnet_range(1, 2)
    for l in range(1, 4):
        m, bb = ctx.packed_layer(l)
        m.fill_(-7.0)
        bb.fill_(-7.0)
    ctx.partition(5)
    ctx.sync_status()
    from oracle import ist_oracle as O
    parts = O.partition(5, w.layer_dims, w.S)
    for l in range(1, 4):
        m, bb = ctx.packed_layer(l)
        for s in (0, 3):
            assert bool((m[s] == -7.0).all()) and bool((bb[s] == -7.0).all()), (l, s)
        for s in (1, 2):
            Ws, bs = O.slice_subnet(W, b, parts, s)
            gw, gb = ctx.get_subnet_params(l, s)
            assert np.array_equal(gw.cpu().numpy(), Ws[l - 1]) and np.array_equal(gb.cpu().numpy(), bs[l - 1])
    ctx.reassemble()


def test_subnet_range_is_checked():
    from paper_1910_02120_b200 import api
    w = synth.Workload("sh", (8, 16, 4), S=4, B=4, K=1, rounds=1, precision="fp32", x_dist="normal", seed=1)
    W, b, data = H.make_problem(w)
    ctx, Wd, bd = H.gpu_context(w, W, b)
    for first, count in [(-1, 2), (0, 0), (3, 2), (4, 1)]:
        with pytest.raises(api.IstError):
            ctx.set_subnet_range(first, count)
    ctx.set_subnet_range(1, 2)
    ctx.partition(3)
    with pytest.raises(api.IstError):
        ctx.set_subnet_range(0, 4)                     # not while a partition is in place
    ctx.reassemble()
