"""Independent uniform assignment of neurons to subnets (Sec. 2.1 / App. A, the other reading of
"uniform assignment"): unequal, seed-dependent group sizes through the whole round.  Index maps
bit-exact against the oracle, one round within the usual tolerances, slices exact."""
import numpy as np
import pytest

from paper_1910_02120_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _wl(dims, S, B, K, precision, lr=0.05, seed=41):
    return synth.Workload("iid", tuple(dims), S=S, B=B, K=K, rounds=1, precision=precision,
                          x_dist="normal", lr=lr, seed=seed)


@pytest.mark.parametrize("dims,S", [([8, 50, 6], 3), ([16, 1000, 777, 8], 7), ([4, 5000, 3], 64), ([4, 12, 9, 3], 9)])
def test_iid_partition_matches_oracle_bit_exact(dims, S):
    from oracle import ist_oracle as O
    w = _wl(dims, S, 4, 1, "fp32")
    W, b, _ = H.make_problem(w)
    ctx, Wd, bd = H.gpu_context(w, W, b, rule="iid")
    for seed in (0, 1, 2 ** 63 + 5):
        ctx.partition(seed)
        want = O.partition(seed, dims, S, rule="iid")
        sizes = []
        for l in range(1, len(dims) - 1):
            idx, off = (t.cpu().numpy() for t in ctx.get_partition(l))
            assert np.array_equal(idx, want[l - 1][0]) and np.array_equal(off, want[l - 1][1])
            sizes.append(np.diff(off))
        ctx.reassemble()
        ctx.sync_status()
    assert any(len(set(s.tolist())) > 1 for s in sizes)


@pytest.mark.parametrize("precision,dims,S,B,K", [
    ("fp32", [20, 37, 5], 3, 7, 3),
    ("fp32", [33, 129, 65, 130, 11], 4, 33, 2),
    ("bf16", [256, 1024, 1024, 35], 4, 256, 3),
    ("fp32", [16, 10, 9, 4], 8, 8, 2),             # nearly as many subnets as neurons: some groups are empty
    ("bf16", [16, 10, 9, 4], 8, 8, 2),
    ("bf16", [48, 515, 300, 10], 5, 24, 2),
    ("bf16", [256, 8192, 1000], 8, 512, 2),
])
def test_iid_round_matches_oracle(precision, dims, S, B, K):
    from oracle import ist_oracle as O
    w = _wl(dims, S, B, K, precision, lr=0.05 if precision == "fp32" else 0.01)
    W, b, data = H.make_problem(w, bias_scale=0.1)
    seed = 4242
    o, oparts, oloss = H.oracle_round(w, W, b, data, seed, rule="iid")
    ctx, gW, gb, gparts, gloss = H.gpu_round(w, W, b, data, seed, rule="iid")
    for (gi, go), (oi, oo) in zip(gparts, oparts):
        assert np.array_equal(gi, oi) and np.array_equal(go, oo)
    if precision == "fp32":
        np.testing.assert_allclose(gloss, oloss, rtol=1e-4)
        rtol_w, rtol_dw = 1e-4, 1e-3
    else:
        assert abs(gloss.mean() - oloss.mean()) <= 1e-3
        rtol_w, rtol_dw = 2e-2, 1e-1
    for l in range(len(W)):
        H.assert_close(gW[l], o.W[l], rtol_w, f"W_{l + 1}")
        H.assert_close(gb[l], o.b[l], rtol_w, f"b_{l + 1}")
        dg, do = gW[l].astype(np.float64) - W[l], o.W[l] - W[l]
        fro = np.linalg.norm(dg - do) / max(np.linalg.norm(do), 1e-300)
        assert fro <= rtol_dw, f"update of W_{l + 1}: {fro:.3e}"


def test_iid_slices_and_untouched_round_are_exact():
    import torch
    from oracle import ist_oracle as O
    dims, S = [24, 100, 72, 10], 4
    w = _wl(dims, S, 8, 1, "bf16")
    W, b, _ = H.make_problem(w, bias_scale=0.2)
    ctx, Wd, bd = H.gpu_context(w, W, b, rule="iid")
    ctx.partition(11)
    parts = O.partition(11, dims, S, rule="iid")
    W64 = [x.astype(np.float64) for x in W]
    b64 = [x.astype(np.float64) for x in b]
    for s in range(S):
        Ws, bs = O.slice_subnet(W64, b64, parts, s)
        for l in range(1, len(dims)):
            gWs, gbs = ctx.get_subnet_params(l, s)
            assert np.array_equal(gWs.cpu().numpy().astype(np.float64), Ws[l - 1])
            assert np.array_equal(gbs.cpu().numpy().astype(np.float64), bs[l - 1])
    ctx.reassemble()
    ctx.sync_status()
    for l in range(len(W)):
        assert np.array_equal(Wd[l].cpu().numpy(), W[l]) and np.array_equal(bd[l].cpu().numpy(), b[l])


@pytest.mark.parametrize("precision,dims,S,B", [("bf16", [64, 700, 520, 12], 3, 96), ("bf16", [256, 4096, 4096, 16], 8, 512)])
def test_iid_two_rounds_with_changing_group_sizes(precision, dims, S, B):
    """Unequal subnets work on their true shapes: tiles beyond a group's extent are skipped, so the
    buffers behind them keep values from the round before, when the group may have been larger.
    Two rounds with different draws must still follow the oracle."""
    w = _wl(dims, S, B, 2, precision, lr=0.01)
    W, b, data = H.make_problem(w, bias_scale=0.1)
    from oracle import ist_oracle as O
    o = O.IstOracle(w.layer_dims, w.S, partition_rule="iid")
    o.bind_weights(W, b)
    ctx, Wd, bd = H.gpu_context(w, W, b, rule="iid")
    X, y = H.gpu_inputs(w, data)
    sizes = []
    for seed in (11, 12):
        oloss = o.round(seed, data.X, data.y, w.lr, w.K)
        gloss = ctx.round(seed, X, y, w.lr, w.K, w.B).cpu().numpy()
        ctx.sync_status()
        sizes.append([np.diff(p[1]).tolist() for p in o.parts])
        assert abs(gloss.mean() - oloss.mean()) <= 1e-3
        for l in range(len(W)):
            H.assert_close(Wd[l].cpu().numpy(), o.W[l], 2e-2, f"W_{l + 1} after seed {seed}")
            H.assert_close(bd[l].cpu().numpy(), o.b[l], 2e-2, f"b_{l + 1} after seed {seed}")
    assert sizes[0] != sizes[1]
