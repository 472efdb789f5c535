"""Shared test plumbing: runs the same seeded round through the CPU oracle and through the
CUDA library's C ABI, and compares tensors with the tolerance rule used throughout."""
import numpy as np

from paper_1910_02120_b200 import synth


def tensor_close(g, o, rtol):
    """max_i |g_i - o_i| <= rtol * max(|o_i|, RMS(o))  and  ||g - o||_F <= rtol * ||o||_F."""
    g = np.asarray(g, dtype=np.float64)
    o = np.asarray(o, dtype=np.float64)
    assert g.shape == o.shape, (g.shape, o.shape)
    if o.size == 0:
        return True, 0.0, 0.0
    rms = np.sqrt(np.mean(o * o))
    scale = np.maximum(np.abs(o), rms)
    scale = np.where(scale == 0, 1.0, scale)
    worst = float(np.max(np.abs(g - o) / scale))
    nrm = np.linalg.norm(o)
    fro = float(np.linalg.norm(g - o) / (nrm if nrm > 0 else 1.0))
    return (worst <= rtol and fro <= rtol), worst, fro


def assert_close(g, o, rtol, what=""):
    ok, worst, fro = tensor_close(g, o, rtol)
    assert ok, f"{what}: worst element ratio {worst:.3e}, Frobenius {fro:.3e}, rtol {rtol:.1e}"


def make_problem(w: synth.Workload, bias_scale=0.1, round_index=0):
    W, b = synth.make_weights(w.layer_dims, w.seed, bias_scale=bias_scale)
    data = synth.make_round_inputs(w, round_index)
    return W, b, data


def oracle_round(w: synth.Workload, W, b, data, seed, dtype=np.float64, norm_eps=None, rule="balanced"):
    from oracle import ist_oracle as O
    o = O.IstOracle(w.layer_dims, w.S, dtype=dtype, norm_eps=norm_eps, partition_rule=rule)
    o.bind_weights(W, b)
    X = (data.row_ptr, data.col, data.val) if data.is_csr else data.X
    parts = o.partition(seed)
    losses = o.local_steps(X, data.y, w.lr, w.K)
    o.reassemble()
    return o, parts, losses


def gpu_context(w: synth.Workload, W, b, device="cuda:0", rule="balanced"):
    import torch
    from paper_1910_02120_b200 import api
    prec = api.IST_BF16 if w.precision == "bf16" else api.IST_FP32
    ctx = api.Ist(w.layer_dims, w.S, prec, w.B, input_is_csr=(w.x_dist == "csr"), device=device,
                  partition_rule=api.IST_PART_IID if rule == "iid" else api.IST_PART_BALANCED)
    Wd = [torch.tensor(x, device=device) for x in W]
    bd = [torch.tensor(x, device=device) for x in b]
    ctx.bind_weights(Wd, bd)
    return ctx, Wd, bd


def gpu_inputs(w: synth.Workload, data, device="cuda:0", as_bf16=None):
    import torch
    y = torch.tensor(data.y.reshape(-1), dtype=torch.int32, device=device)
    if data.is_csr:
        X = (torch.tensor(data.row_ptr, dtype=torch.int32, device=device),
             torch.tensor(data.col, dtype=torch.int32, device=device),
             torch.tensor(data.val, dtype=torch.float32, device=device))
        return X, y
    X = torch.tensor(data.X.reshape(-1, w.layer_dims[0]), device=device)
    if as_bf16 is None:
        as_bf16 = w.precision == "bf16" and w.layer_dims[0] % 8 == 0
    if as_bf16:
        X = X.to(torch.bfloat16)
    return X, y


def gpu_round(w: synth.Workload, W, b, data, seed, device="cuda:0", as_bf16=None, norm_eps=None, rule="balanced"):
    ctx, Wd, bd = gpu_context(w, W, b, device, rule)
    if norm_eps is not None:
        ctx.enable_normalization(norm_eps)
    X, y = gpu_inputs(w, data, device, as_bf16)
    ctx.partition(seed)
    parts = [tuple(t.cpu().numpy() for t in ctx.get_partition(l)) for l in range(1, ctx.t)]
    losses = ctx.local_steps(X, y, w.lr, w.K, w.B)
    ctx.reassemble()
    ctx.sync_status()
    return ctx, [x.cpu().numpy() for x in Wd], [x.cpu().numpy() for x in bd], parts, losses.cpu().numpy()
