"""Argument and call-order checks of the optional modes: every misuse is an error code, never a fault."""
import pytest

from paper_1910_02120_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def test_normalisation_misuse_is_reported():
    import torch
    from paper_1910_02120_b200 import api
    w = synth.Workload("e", (8, 16, 12, 4), S=2, B=8, K=1, rounds=1, precision="fp32", x_dist="normal", seed=2)
    W, b, data = H.make_problem(w)
    ctx, Wd, bd = H.gpu_context(w, W, b)
    X, y = H.gpu_inputs(w, data)
    with pytest.raises(api.IstError):
        ctx.calibrate(X, 4)                               # mode not enabled
    nbytes = int(api.lib.ist_norm_workspace_bytes(ctx.handle))
    buf = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda:0")
    import ctypes
    assert api.lib.ist_enable_normalization(ctx.handle, ctypes.c_float(0.0), buf.data_ptr(), nbytes) == api.IST_ERR_ARG
    assert api.lib.ist_enable_normalization(ctx.handle, ctypes.c_float(1e-5), buf.data_ptr() + 8, nbytes) == api.IST_ERR_WORKSPACE
    assert api.lib.ist_enable_normalization(ctx.handle, ctypes.c_float(1e-5), buf.data_ptr(), nbytes - 256) == api.IST_ERR_WORKSPACE
    ctx.partition(1)
    assert api.lib.ist_enable_normalization(ctx.handle, ctypes.c_float(1e-5), buf.data_ptr(), nbytes) == api.IST_ERR_STATE
    ctx.reassemble()
    ctx.enable_normalization(1e-5)
    with pytest.raises(api.IstError):
        ctx.enable_normalization(1e-5)                    # already on
    with pytest.raises(api.IstError):
        ctx.calibrate(X, 9)                               # more rows than max_batch
    with pytest.raises(api.IstError):
        ctx.calibrate(X, 0)
    ctx.partition(2)
    with pytest.raises(api.IstError):
        ctx.calibrate(X, 4)                               # not while a partition is in place
    ctx.reassemble()
    ctx.calibrate(X, 8)
    ctx.eval(X, y, 8)
    ctx.sync_status()


def test_packed_layer_views_cover_all_subnets():
    from paper_1910_02120_b200 import api
    w = synth.Workload("e", (8, 24, 16, 4), S=4, B=8, K=1, rounds=1, precision="bf16", x_dist="normal", seed=2)
    W, b, data = H.make_problem(w)
    ctx, Wd, bd = H.gpu_context(w, W, b)
    with pytest.raises(api.IstError):
        ctx.packed_layer(0)
    with pytest.raises(api.IstError):
        ctx.packed_layer(4)
    m, bb = ctx.packed_layer(2)
    assert m.shape == (4, 6 * 8) and bb.shape == (4, 8)   # 6 rows per subnet; 4 columns in rows of 8
    ctx.partition(3)
    got = ctx.get_subnet_params(2, 1)[0]
    assert (m[1].view(6, 8)[:, :4] == got).all()
    ctx.reassemble()
