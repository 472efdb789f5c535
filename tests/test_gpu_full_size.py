"""Parity at the full benchmark sizes, in the launch configuration bench.py times.

The CPU oracle cannot run a whole round of the wide configurations in test time, but it can run
one subnet: the test draws the partition with the oracle, slices that subnet out of the full
network, trains it for K local steps in fp64, and compares with what the library holds for the
same subnet after the same K steps (read back with ist_get_subnet_params before reassembly).
After reassembly, properties that hold at any size are checked on the device: entries outside
every subnet are bit-identical to the input, entries inside have moved."""
import numpy as np
import pytest

from paper_1910_02120_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def _sampled_subnet_round(w, s_check, rtol_w, rtol_dw, loss_tol, norm_eps=None, rule="balanced"):
    import torch
    from oracle import ist_oracle as O
    from paper_1910_02120_b200 import api
    dev = "cuda:0"
    W, b = synth.make_weights(w.layer_dims, w.seed)
    data = synth.make_round_inputs(w)
    seed = 31337
    parts = O.partition(seed, w.layer_dims, w.S, rule)
    Ws, bs = O.slice_subnet(W, b, parts, s_check)
    Ws0 = [x.copy() for x in Ws]
    Ws = [x.astype(np.float64) for x in Ws]
    bs = [x.astype(np.float64) for x in bs]
    oracle = O.IstOracle(w.layer_dims, w.S)
    X = (data.row_ptr, data.col, data.val) if data.is_csr else data.X
    olosses = []
    for k in range(w.K):
        xb, yb = oracle._batch(X, data.y, s_check, k)
        olosses.append(O.sgd_step(Ws, bs, xb, yb, w.lr, norm_eps=norm_eps))

    prec = api.IST_BF16 if w.precision == "bf16" else api.IST_FP32
    ctx = api.Ist(w.layer_dims, w.S, prec, w.B, input_is_csr=data.is_csr, device=dev,
                  partition_rule=api.IST_PART_IID if rule == "iid" else api.IST_PART_BALANCED)
    Wd = [torch.from_numpy(x).to(dev) for x in W]
    bd = [torch.from_numpy(x).to(dev) for x in b]
    ctx.bind_weights(Wd, bd)
    if norm_eps is not None:
        ctx.enable_normalization(norm_eps)
    Xd, yd = H.gpu_inputs(w, data)
    ctx.partition(seed)
    for l in range(1, ctx.t):
        gi, go = ctx.get_partition(l)
        assert np.array_equal(gi.cpu().numpy(), parts[l - 1][0]) and np.array_equal(go.cpu().numpy(), parts[l - 1][1])
    gloss = ctx.local_steps(Xd, yd, w.lr, w.K, w.B).cpu().numpy()
    for l in range(1, ctx.t + 1):
        gw, gb = ctx.get_subnet_params(l, s_check)
        gw, gb = gw.cpu().numpy(), gb.cpu().numpy()
        H.assert_close(gw, Ws[l - 1], rtol_w, f"W_{l} of subnet {s_check}")
        # biases start at zero here, so their value is their update: the update tolerance
        # (relative Frobenius error, as for the weight updates) applies
        if norm_eps is not None and l < ctx.t:
            # standardisation removes the batch mean: a hidden bias has no gradient and stays (near) zero
            assert np.max(np.abs(gb)) <= 1e-3 and np.max(np.abs(bs[l - 1])) <= 1e-9
        else:
            fro_b = np.linalg.norm(gb.astype(np.float64) - bs[l - 1]) / max(np.linalg.norm(bs[l - 1]), 1e-300)
            assert fro_b <= rtol_dw, f"b_{l} of subnet {s_check}: {fro_b:.3e}"
        do = Ws[l - 1] - Ws0[l - 1]
        fro = np.linalg.norm((gw.astype(np.float64) - Ws0[l - 1]) - do) / max(np.linalg.norm(do), 1e-300)
        assert fro <= rtol_dw, f"update of W_{l}: {fro:.3e}"
    assert np.max(np.abs(gloss[s_check] - np.array(olosses))) <= loss_tol, (gloss[s_check], olosses)
    ctx.reassemble()
    ctx.sync_status()
    # any-size properties, checked on the device
    for l in range(2, ctx.t):          # middle layers: cross-group blocks untouched, bit for bit
        g_prev = torch.empty(w.layer_dims[l - 1], dtype=torch.int64, device=dev)
        g_cur = torch.empty(w.layer_dims[l], dtype=torch.int64, device=dev)
        for s in range(w.S):
            g_prev[torch.from_numpy(O.group(parts, l - 1, s).astype(np.int64)).to(dev)] = s
            g_cur[torch.from_numpy(O.group(parts, l, s).astype(np.int64)).to(dev)] = s
        W0 = torch.from_numpy(W[l - 1]).to(dev)
        same = g_prev[:, None] == g_cur[None, :]
        assert torch.equal(Wd[l - 1][~same], W0[~same])
        assert (Wd[l - 1][same] != W0[same]).float().mean().item() > 0.5
    return ctx


def test_wide_pixel_config_full_size_one_subnet():
    # 3072 -> 16384 -> 16384 -> 10, S = 8, batch 512: the benchmark's shapes and tile choices
    w = synth.C3.scaled(K=2)
    _sampled_subnet_round(w, 5, 2e-2, 1e-1, 5e-3)


def test_speech_like_config_full_size_one_subnet():
    # 1024 -> 4096 -> 4096 -> 35, S = 4, batch 256, all K = 50 local steps
    _sampled_subnet_round(synth.C2, 2, 2e-2, 1e-1, 5e-3)


def test_extreme_classification_config_full_size_one_subnet():
    # CSR 135,909 -> 1024 -> 670,091, S = 8, batch 256: sparse first layer, k-split delta GEMM,
    # wide softmax at their real sizes
    w = synth.C4.scaled(K=1)
    _sampled_subnet_round(w, 1, 2e-2, 1e-1, 5e-3)


def test_wide_pixel_config_with_standardisation_one_subnet():
    # the same shapes with Sec. 2.2's batch standardisation: fp32 pre-activation epilogue on CTA pairs,
    # column kernels at batch 512
    w = synth.C3.scaled(K=1)
    _sampled_subnet_round(w, 3, 2e-2, 1e-1, 5e-3, norm_eps=1e-5)


def test_wide_pixel_config_independent_assignment_one_subnet():
    # unequal groups (capacity-padded slices) at the benchmark's width
    w = synth.C3.scaled(K=1)
    _sampled_subnet_round(w, 6, 2e-2, 1e-1, 5e-3, rule="iid")


def test_largest_sweep_width_indexes_beyond_two_to_the_31():
    """1024 -> 65536 -> 65536 -> 100 with two subnets: the middle layer has 2^32 entries, every
    subnet owns 2^30 of them.  No CPU run can follow that, so the round is checked through what holds
    at any size: with lr = 0 it returns the network bit for bit; with lr > 0 no entry outside a
    subnet's own block moves and nearly all inside do."""
    import torch
    from paper_1910_02120_b200 import api
    dev = "cuda:0"
    free, _ = torch.cuda.mem_get_info()
    if free < 70 * 2**30:
        pytest.skip("needs about 70 GB of device memory")
    Hw, S, B = 65536, 2, 512
    dims = (1024, Hw, Hw, 100)
    g = torch.Generator(device=dev)
    g.manual_seed(3)
    Wd = [torch.empty(dims[i], dims[i + 1], device=dev).uniform_(-0.01, 0.01, generator=g) for i in range(3)]
    bd = [torch.zeros(dims[i + 1], device=dev) for i in range(3)]
    ref = [w.clone() for w in Wd]
    X = torch.randn(S * B, dims[0], device=dev, generator=g).to(torch.bfloat16)
    y = torch.randint(0, 100, (S * B,), device=dev, dtype=torch.int32, generator=g)
    ctx = api.Ist(dims, S, api.IST_BF16, B, device=dev)
    ctx.bind_weights(Wd, bd)
    ctx.partition(11)
    (idx1, off1), (idx2, off2) = ctx.get_partition(1), ctx.get_partition(2)
    losses = ctx.local_steps(X, y, 0.0, 1, B)
    ctx.reassemble()
    ctx.sync_status()
    assert all(torch.equal(a, r) for a, r in zip(Wd, ref))
    assert torch.isfinite(losses).all() and (losses > 4.0).all() and (losses < 5.2).all()   # ln 100 = 4.6

    ctx.partition(11)
    ctx.local_steps(X, y, 0.5, 1, B)
    ctx.reassemble()
    ctx.sync_status()
    grp1 = torch.empty(Hw, dtype=torch.int64, device=dev)
    grp2 = torch.empty(Hw, dtype=torch.int64, device=dev)
    for s in range(S):
        grp1[idx1[off1[s]:off1[s + 1]].long()] = s
        grp2[idx2[off2[s]:off2[s + 1]].long()] = s
    moved_outside = moved_inside = inside = 0
    for r0 in range(0, Hw, 4096):
        moved = Wd[1][r0:r0 + 4096] != ref[1][r0:r0 + 4096]
        own = grp1[r0:r0 + 4096, None] == grp2[None, :]
        moved_outside += int((moved & ~own).sum())
        moved_inside += int((moved & own).sum())
        inside += int(own.sum())
    assert inside == Hw * Hw // S
    assert moved_outside == 0
    assert moved_inside > 0.99 * inside
    assert int((Wd[1][-1] != ref[1][-1]).sum()) > 0.99 * Hw // S                    # the last row is reached
    assert int((Wd[0] != ref[0]).sum()) > 0.99 * Wd[0].numel()
    del ctx, Wd, ref
    torch.cuda.empty_cache()
