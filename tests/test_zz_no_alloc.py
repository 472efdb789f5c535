"""ist_partition_layer_static: the allocation-free partition entry point.

Some users of the library may not allocate device memory when they need a partition (their host
application handed out all device memory at start-up, or they only want index lists and have no
room for a context's workspace).  For them the library carries its own scratch array.  This test
calls that entry point through the C ABI and checks, bit for bit, that it returns what the
ordinary path (ist_partition + ist_get_partition) returns, on two calls in a row that share the
scratch, and that sizes beyond the built-in array are refused.

Collected last on purpose: a failure here must not hide the other tests' results.
"""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _reference_partition(api, dims, S, seed):
    import torch
    ctx = api.Ist(dims, S, api.IST_FP32, 4)
    W = [torch.zeros(dims[l], dims[l + 1], device="cuda:0") for l in range(len(dims) - 1)]
    b = [torch.zeros(dims[l + 1], device="cuda:0") for l in range(len(dims) - 1)]
    ctx.bind_weights(W, b)
    ctx.partition(seed)
    out = [tuple(t.cpu().numpy() for t in ctx.get_partition(l)) for l in range(1, ctx.t)]
    ctx.reassemble()
    ctx.sync_status()
    return out


def test_static_partition_matches_the_workspace_path_twice_in_a_row():
    import torch
    from paper_1910_02120_b200 import api
    cases = [([8, 4096, 1000, 5], 8, 123), ([4, 777, 2049, 3], 3, 2 ** 63 + 5)]
    for dims, S, seed in cases:
        want = _reference_partition(api, dims, S, seed)
        # two calls back to back on one stream: the second reuses the scratch the first left behind
        for layer in (1, 2):
            N = dims[layer]
            idx = torch.full((N,), -1, dtype=torch.int32, device="cuda:0")
            off = torch.full((S + 1,), -1, dtype=torch.int32, device="cuda:0")
            st = api.ist_partition_layer_static(seed, layer, N, S, idx, off)
            assert st == api.IST_OK
            torch.cuda.synchronize()
            assert np.array_equal(idx.cpu().numpy(), want[layer - 1][0])
            assert np.array_equal(off.cpu().numpy(), want[layer - 1][1])
    # the same call again gives the same answer (nothing stale is picked up from the scratch)
    idx2 = torch.empty(4096, dtype=torch.int32, device="cuda:0")
    off2 = torch.empty(9, dtype=torch.int32, device="cuda:0")
    assert api.ist_partition_layer_static(123, 1, 4096, 8, idx2, off2) == api.IST_OK
    torch.cuda.synchronize()
    assert np.array_equal(idx2.cpu().numpy(), _reference_partition(api, [8, 4096, 5], 8, 123)[0][0])


def test_static_partition_takes_no_device_memory_and_reports_its_status():
    """The point of the entry point: free device memory is the same before and after warmed-up calls
    (the first call's symbol look-up is done by then), and the kernels' bounds-check word reads OK."""
    import torch
    from paper_1910_02120_b200 import api
    N, S = 30000, 16
    idx = torch.empty(N, dtype=torch.int32, device="cuda:0")
    off = torch.empty(S + 1, dtype=torch.int32, device="cuda:0")
    assert api.ist_partition_layer_static(5, 1, N, S, idx, off) == api.IST_OK      # warm-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for seed in range(6, 12):
        assert api.ist_partition_layer_static(seed, 2, N, S, idx, off) == api.IST_OK
    assert api.ist_static_partition_status() == api.IST_OK
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)
    assert np.array_equal(np.sort(idx.cpu().numpy()), np.arange(N))


def test_static_partition_refuses_sizes_beyond_its_scratch():
    import torch
    from paper_1910_02120_b200 import api
    idx = torch.empty(api.IST_STATIC_MAX_NEURONS + 8, dtype=torch.int32, device="cuda:0")
    off = torch.empty(api.IST_STATIC_MAX_SUBNETS + 2, dtype=torch.int32, device="cuda:0")
    assert api.ist_partition_layer_static(1, 1, api.IST_STATIC_MAX_NEURONS + 1, 4, idx, off) == api.IST_ERR_UNSUPPORTED
    assert api.ist_partition_layer_static(1, 1, 4096, api.IST_STATIC_MAX_SUBNETS + 1, idx, off) == api.IST_ERR_UNSUPPORTED
    assert api.ist_partition_layer_static(1, 0, 4096, 4, idx, off) == api.IST_ERR_ARG
    assert api.ist_partition_layer_static(1, 1, 16, 17, idx, off) == api.IST_ERR_ARG
    # the largest allowed size works
    assert api.ist_partition_layer_static(9, 1, api.IST_STATIC_MAX_NEURONS, api.IST_STATIC_MAX_SUBNETS, idx, off) == api.IST_OK
    torch.cuda.synchronize()
    got = idx[:api.IST_STATIC_MAX_NEURONS].cpu().numpy()
    assert np.array_equal(np.sort(got), np.arange(api.IST_STATIC_MAX_NEURONS))
