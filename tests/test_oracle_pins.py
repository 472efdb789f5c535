"""Pins for the CPU oracle: each test ties one part of oracle/ist_oracle.py to
something other than itself (a published vector, an invariant the paper states,
a closed form, brute force, or a library routine used only as a check)."""
import os

import numpy as np
import pytest
import torch

from oracle import ist_oracle as O
from paper_1910_02120_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _tiny(layer_dims, S, B, K, seed=11, bias_scale=0.3, n_classes=None):
    W, b = synth.make_weights(layer_dims, seed, bias_scale=bias_scale)
    X = synth.make_dense_inputs(S, K, B, layer_dims[0], "normal", seed)
    y = synth.make_labels((S, K, B), layer_dims[-1], seed)
    return W, b, X, y


# --- key mixer: published SplitMix64 vector -------------------------------------------

def test_splitmix64_published_vector():
    want = [int(l) for l in open(os.path.join(GOLDEN, "splitmix64_seed1234567.txt"))
            if l.strip() and not l.startswith("#")]
    assert O.splitmix64_stream(1234567, len(want)) == want


def test_keys_are_two_level_splitmix_streams():
    # layer seed = l-th output of the round stream; keys = outputs of the layer stream
    seed = 1234567
    want = [int(l) for l in open(os.path.join(GOLDEN, "splitmix64_seed1234567.txt"))
            if l.strip() and not l.startswith("#")]
    for layer in (1, 2, 3):
        keys = O.neuron_keys(seed, layer, 4)
        assert keys == O.splitmix64_stream(want[layer - 1], 4)
    # and a stream seeded with 1234567 itself reproduces the vector through neuron_keys'
    # inner generator: layer seed w such that stream(w) is checked above by composition.


# --- Sec. 2.1 / App. A: exactly one subnet per hidden neuron ---------------------------

@pytest.mark.parametrize("N,S", [(10, 3), (1024, 2), (1000, 7), (16, 16), (33, 1), (4096, 8)])
def test_partition_invariants(N, S):
    idx, off = O.partition_layer(99, 1, N, S)
    assert idx.dtype == np.int32 and off.dtype == np.int32
    assert sorted(idx.tolist()) == list(range(N))          # cover, each exactly once
    assert off[0] == 0 and off[-1] == N
    sizes = np.diff(off)
    for g in range(S):
        assert sizes[g] == N // S + (1 if g < N % S else 0)
        members = idx[off[g]:off[g + 1]]
        assert np.all(np.diff(members) > 0)                # ascending inside a group
    # membership indicators m^(s)_{l,i}: sum over s is 1 for every neuron
    m = np.zeros((S, N), dtype=np.int64)
    for g in range(S):
        m[g, idx[off[g]:off[g + 1]]] = 1
    assert np.all(m.sum(axis=0) == 1)


def test_partition_brute_force_small():
    # independent restatement on a tiny case: rank every neuron by (key, index)
    N, S, seed, layer = 11, 4, 5, 2
    keys = O.neuron_keys(seed, layer, N)
    rank = [sum((keys[j], j) < (keys[i], i) for j in range(N)) for i in range(N)]
    bounds = np.cumsum([0] + [N // S + (1 if g < N % S else 0) for g in range(S)])
    grp = [int(np.searchsorted(bounds, r, side="right") - 1) for r in rank]
    idx, off = O.partition_layer(seed, layer, N, S)
    for g in range(S):
        assert idx[off[g]:off[g + 1]].tolist() == [i for i in range(N) if grp[i] == g]


def test_partition_layers_and_seeds_differ_and_repeat():
    a = O.partition(3, [8, 256, 256, 4], 4)
    b = O.partition(3, [8, 256, 256, 4], 4)
    c = O.partition(4, [8, 256, 256, 4], 4)
    assert all(np.array_equal(x[0], y[0]) for x, y in zip(a, b))     # deterministic
    assert not np.array_equal(a[0][0], a[1][0])                      # layers independent
    assert not np.array_equal(a[0][0], c[0][0])                      # seeds differ


def test_partition_marginal_is_uniform():
    # P[m^(s)_{l,i} = 1] = 1/S (App. A): chi-square on the group of neuron 0 over seeds
    N, S, trials = 12, 4, 2000
    counts = np.zeros(S)
    for seed in range(trials):
        idx, off = O.partition_layer(seed, 1, N, S)
        pos = int(np.where(idx == 0)[0][0])
        counts[np.searchsorted(off, pos, side="right") - 1] += 1
    chi2 = ((counts - trials / S) ** 2 / (trials / S)).sum()
    assert chi2 < 16.27          # 99.9% quantile, 3 degrees of freedom
    # pairwise independence across layers: P[same group in layer 1 and 2] ~ 1/S^2 per group
    both = 0
    for seed in range(trials):
        p = O.partition(seed, [4, N, N, 3], S)
        g1 = np.searchsorted(p[0][1], int(np.where(p[0][0] == 0)[0][0]), side="right") - 1
        g2 = np.searchsorted(p[1][1], int(np.where(p[1][0] == 0)[0][0]), side="right") - 1
        both += int(g1 == 0 and g2 == 0)
    assert abs(both / trials - 1 / S ** 2) < 4 * np.sqrt((1 / S ** 2) * (1 - 1 / S ** 2) / trials)


def test_no_hidden_layer_requires_S1():
    with pytest.raises(ValueError):
        O.partition(1, [8, 4], 2)
    assert O.partition(1, [8, 4], 1) == []


# --- Sec. 2.1: copy-back; untouched round is the identity, bit for bit -------------------

@pytest.mark.parametrize("dtype", [np.float32, np.float64])
@pytest.mark.parametrize("dims,S", [([12, 40, 6], 3), ([9, 30, 26, 5], 4), ([7, 16, 24, 8, 3], 2)])
def test_untouched_round_is_identity(dims, S, dtype):
    W, b, _, _ = _tiny(dims, S, 4, 1)
    o = O.IstOracle(dims, S, dtype=dtype)
    o.bind_weights(W, b)
    o.partition(17)
    o.reassemble()
    for l in range(len(W)):
        assert np.array_equal(o.W[l], W[l].astype(dtype))
        assert np.array_equal(o.b[l], b[l].astype(dtype))


def test_cross_group_blocks_untouched_and_owned_blocks_change():
    dims, S, B, K = [10, 24, 20, 4], 4, 6, 3
    W, b, X, y = _tiny(dims, S, B, K)
    o = O.IstOracle(dims, S)
    o.bind_weights(W, b)
    parts = o.partition(5)
    o.local_steps(X, y, 0.1, K)
    o.reassemble()
    g1 = np.empty(dims[1], dtype=int)
    g2 = np.empty(dims[2], dtype=int)
    for s in range(S):
        g1[O.group(parts, 1, s)] = s
        g2[O.group(parts, 2, s)] = s
    same = g1[:, None] == g2[None, :]
    before = W[1].astype(np.float64)
    assert np.array_equal(o.W[1][~same], before[~same])       # footnote of Sec. 2.1
    assert np.all(o.W[1][same] != before[same]) or (o.W[1][same] != before[same]).mean() > 0.5
    # fraction of a middle layer that is owned: sum_s |G1^s||G2^s| = N1 N2 / S here
    assert same.sum() == dims[1] * dims[2] // S


def test_one_hidden_layer_every_weight_is_owned_once():
    dims, S = [6, 21, 5], 4
    parts = O.partition(2, dims, S)
    own1 = np.zeros((dims[0], dims[1]), dtype=int)
    own2 = np.zeros((dims[1], dims[2]), dtype=int)
    for s in range(S):
        g = O.group(parts, 1, s)
        own1[:, g] += 1
        own2[g, :] += 1
    assert np.all(own1 == 1) and np.all(own2 == 1)


# --- Sec. 2.3: per-site parameter counts (1/n of first/last, 1/n^2 of middle layers) ---

def test_slice_sizes_match_closed_forms():
    dims, S = [16, 64, 32, 48, 8], 4
    W, b, _, _ = _tiny(dims, S, 2, 1)
    parts = O.partition(1, dims, S)
    tot = [0] * (len(dims) - 1)
    for s in range(S):
        Ws, bs = O.slice_subnet(W, b, parts, s)
        assert Ws[0].shape == (16, 16) and Ws[1].shape == (16, 8)
        assert Ws[2].shape == (8, 12) and Ws[3].shape == (12, 8)
        assert Ws[1].size * S * S == W[1].size and Ws[0].size * S == W[0].size
        for l in range(4):
            tot[l] += Ws[l].size
    # summed over sites: N0 N1 + N_{t-1} N_t + sum_middle N_{i-1} N_i / n
    assert tot == [16 * 64, 64 * 32 // S, 32 * 48 // S, 48 * 8]


def test_slice_picks_the_indexed_entries():
    dims, S = [5, 12, 9, 3], 3
    W, b, _, _ = _tiny(dims, S, 2, 1)
    parts = O.partition(8, dims, S)
    for s in range(S):
        Ws, bs = O.slice_subnet(W, b, parts, s)
        G1, G2 = O.group(parts, 1, s), O.group(parts, 2, s)
        for i, r in enumerate(G1):
            for j, c in enumerate(G2):
                assert Ws[1][i, j] == W[1][r, c]
        for j, c in enumerate(G1):
            assert np.array_equal(Ws[0][:, j], W[0][:, c]) and bs[0][j] == b[0][c]
        for i, r in enumerate(G2):
            assert np.array_equal(Ws[2][i, :], W[2][r, :])
        assert np.array_equal(bs[2], b[2])


# --- training maths: autograd, finite differences, S = 1 ---------------------------------

def _torch_loss(Ws, bs, X, y):
    a = X
    for l in range(len(Ws)):
        a = a @ Ws[l] + bs[l]
        if l < len(Ws) - 1:
            a = torch.relu(a)
    return torch.nn.functional.cross_entropy(a, y, reduction="mean")


@pytest.mark.parametrize("dims", [[7, 5], [6, 9, 4], [5, 8, 7, 3]])
def test_gradients_match_torch_autograd(dims):
    W, b, X, y = _tiny(dims, 1, 10, 1)
    Ws = [w.astype(np.float64) for w in W]
    bs = [v.astype(np.float64) for v in b]
    loss, dW, db = O.gradients(Ws, bs, X[0, 0].astype(np.float64), y[0, 0])
    tW = [torch.tensor(w, requires_grad=True) for w in Ws]
    tb = [torch.tensor(v, requires_grad=True) for v in bs]
    tl = _torch_loss(tW, tb, torch.tensor(X[0, 0], dtype=torch.float64),
                     torch.tensor(y[0, 0], dtype=torch.long))
    tl.backward()
    assert abs(loss - tl.item()) < 1e-12
    for l in range(len(Ws)):
        np.testing.assert_allclose(dW[l], tW[l].grad.numpy(), rtol=1e-10, atol=1e-13)
        np.testing.assert_allclose(db[l], tb[l].grad.numpy(), rtol=1e-10, atol=1e-13)


def test_finite_difference_gradients():
    dims = [4, 6, 5, 3]
    W, b, X, y = _tiny(dims, 1, 5, 1, seed=3)
    Ws = [w.astype(np.float64) for w in W]
    bs = [v.astype(np.float64) for v in b]
    x, yy = X[0, 0].astype(np.float64), y[0, 0]
    loss, dW, db = O.gradients(Ws, bs, x, yy)
    h = 1e-6

    def f():
        z, _ = O.forward(Ws, bs, x)
        return O.softmax_xent(z[-1], yy.astype(np.int64))[0]

    z0, _ = O.forward(Ws, bs, x)
    assert min(np.abs(zz).min() for zz in z0[:-1]) > 1e-4      # away from ReLU kinks
    for params, grads in ((Ws, dW), (bs, db)):
        for l in range(len(params)):
            flat, g = params[l].reshape(-1), grads[l].reshape(-1)
            for i in range(flat.size):
                old = flat[i]
                flat[i] = old + h
                fp = f()
                flat[i] = old - h
                fm = f()
                flat[i] = old
                fd = (fp - fm) / (2 * h)
                assert abs(fd - g[i]) <= 1e-6 * max(1.0, abs(g[i])) + 1e-9


@pytest.mark.parametrize("dims", [[7, 5], [6, 9, 4], [5, 8, 7, 3]])
def test_input_gradient_matches_torch_autograd_and_central_differences(dims):
    # Sec. 2.2 "IST for other architectures": what a trunk in front of the partitioned layers is
    # trained from.  Pinned twice: against autograd of the same network in torch, and against
    # central differences of the oracle's own loss in every input entry.
    W, b, X, y = _tiny(dims, 1, 6, 1, seed=11)
    Ws = [w.astype(np.float64) for w in W]
    bs = [v.astype(np.float64) for v in b]
    x, yy = X[0, 0].astype(np.float64), y[0, 0]
    dx = O.input_gradient(Ws, bs, x, yy)
    assert dx.shape == x.shape
    tx = torch.tensor(x, requires_grad=True)
    tl = _torch_loss([torch.tensor(w) for w in Ws], [torch.tensor(v) for v in bs], tx,
                     torch.tensor(yy, dtype=torch.long))
    tl.backward()
    np.testing.assert_allclose(dx, tx.grad.numpy(), rtol=1e-10, atol=1e-13)

    def f(xx):
        z, _ = O.forward(Ws, bs, xx)
        return O.softmax_xent(z[-1], yy.astype(np.int64))[0]

    z0, _ = O.forward(Ws, bs, x)
    if len(Ws) > 1:
        assert min(np.abs(zz).min() for zz in z0[:-1]) > 1e-4      # away from ReLU kinks
    h = 1e-6
    for i in range(x.shape[0]):
        for j in range(x.shape[1]):
            xp, xm = x.copy(), x.copy()
            xp[i, j] += h
            xm[i, j] -= h
            fd = (f(xp) - f(xm)) / (2 * h)
            assert abs(fd - dx[i, j]) <= 1e-6 * max(1.0, abs(dx[i, j])) + 1e-9


def test_local_steps_dx_is_taken_before_each_update():
    # dX of step k is the input gradient at the parameters step k starts from; the losses and the
    # trained slices are those of local_steps
    dims, S, B, K, lr = [6, 12, 8, 4], 2, 5, 3, 0.05
    W, b, X, y = _tiny(dims, S, B, K, seed=4)
    o = O.IstOracle(dims, S)
    o.bind_weights(W, b)
    o.partition(9)
    ref = O.IstOracle(dims, S)
    ref.bind_weights(W, b)
    ref.partition(9)
    losses, dX = o.local_steps_dx(X, y, lr, K)
    assert dX.shape == X.shape
    for s in range(S):
        Ws, bs = ref.subnets[s]
        for k in range(K):
            xb, yb = ref._batch(X, y, s, k)
            np.testing.assert_array_equal(dX[s, k], O.input_gradient(Ws, bs, xb, yb))
            O.sgd_step(Ws, bs, xb, yb, lr)
    np.testing.assert_array_equal(losses, O.IstOracle.local_steps(_fresh(dims, S, W, b, 9), X, y, lr, K))
    for s in range(S):
        for l in range(len(W)):
            np.testing.assert_array_equal(o.subnets[s][0][l], ref.subnets[s][0][l])


def _fresh(dims, S, W, b, seed):
    o = O.IstOracle(dims, S)
    o.bind_weights(W, b)
    o.partition(seed)
    return o


def test_S1_round_is_plain_sgd():
    # xi = 1 in the paper's compression operator: the mask is the identity and IST is SGD.
    dims, B, K, lr = [6, 10, 8, 4], 7, 5, 0.05
    W, b, X, y = _tiny(dims, 1, B, K)
    o = O.IstOracle(dims, 1)
    o.bind_weights(W, b)
    parts = o.partition(123)
    for idx, off in parts:
        assert np.array_equal(idx, np.arange(idx.size))          # identity after in-group sort
    losses = o.local_steps(X, y, lr, K)
    o.reassemble()
    tW = [torch.tensor(w, dtype=torch.float64, requires_grad=True) for w in W]
    tb = [torch.tensor(v, dtype=torch.float64, requires_grad=True) for v in b]
    opt = torch.optim.SGD(tW + tb, lr=lr)
    for k in range(K):
        opt.zero_grad()
        l = _torch_loss(tW, tb, torch.tensor(X[0, k], dtype=torch.float64),
                        torch.tensor(y[0, k], dtype=torch.long))
        l.backward()
        opt.step()
        assert abs(l.item() - losses[0, k]) < 1e-12
    for l in range(len(W)):
        np.testing.assert_allclose(o.W[l], tW[l].detach().numpy(), rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(o.b[l], tb[l].detach().numpy(), rtol=1e-12, atol=1e-14)


def test_each_subnet_trains_as_its_own_small_mlp():
    # S > 1: subnet s after K steps equals torch SGD on the sliced parameters with its own data
    dims, S, B, K, lr = [6, 12, 9, 4], 3, 5, 4, 0.1
    W, b, X, y = _tiny(dims, S, B, K)
    o = O.IstOracle(dims, S)
    o.bind_weights(W, b)
    parts = o.partition(77)
    o.local_steps(X, y, lr, K)
    trained = [([w.copy() for w in Ws], [v.copy() for v in bs]) for Ws, bs in o.subnets]
    o.reassemble()
    bt = np.zeros(dims[-1])
    for s in range(S):
        G1, G2 = O.group(parts, 1, s), O.group(parts, 2, s)
        sl = [W[0][:, G1], W[1][np.ix_(G1, G2)], W[2][G2, :]]
        sb = [b[0][G1], b[1][G2], b[2]]
        tW = [torch.tensor(w, dtype=torch.float64, requires_grad=True) for w in sl]
        tb = [torch.tensor(v, dtype=torch.float64, requires_grad=True) for v in sb]
        opt = torch.optim.SGD(tW + tb, lr=lr)
        for k in range(K):
            opt.zero_grad()
            _torch_loss(tW, tb, torch.tensor(X[s, k], dtype=torch.float64),
                        torch.tensor(y[s, k], dtype=torch.long)).backward()
            opt.step()
        for l in range(3):
            np.testing.assert_allclose(trained[s][0][l], tW[l].detach().numpy(), rtol=1e-11, atol=1e-13)
        # copy-back landed at the indexed positions
        np.testing.assert_allclose(o.W[0][:, G1], tW[0].detach().numpy(), rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(o.W[1][np.ix_(G1, G2)], tW[1].detach().numpy(), rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(o.W[2][G2, :], tW[2].detach().numpy(), rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(o.b[0][G1], tb[0].detach().numpy(), rtol=1e-11, atol=1e-13)
        bt += tb[2].detach().numpy()
    np.testing.assert_allclose(o.b[2], bt / S, rtol=1e-12, atol=1e-14)   # averaged output bias


def test_one_hidden_layer_separability():
    # f_l = sum_s f_l^(s) (App. A): with one hidden layer the subnet logits add up to the
    # full network's logits once the S copies of the output bias are counted once.
    dims, S = [9, 30, 6], 5
    W, b, X, _ = _tiny(dims, S, 8, 1)
    W64 = [w.astype(np.float64) for w in W]
    b64 = [v.astype(np.float64) for v in b]
    parts = O.partition(4, dims, S)
    x = X[0, 0].astype(np.float64)
    full = O.forward(W64, b64, x)[0][-1]
    tot = np.zeros_like(full)
    for s in range(S):
        Ws, bs = O.slice_subnet(W64, b64, parts, s)
        tot += O.forward(Ws, bs, x)[0][-1]
    np.testing.assert_allclose(tot - (S - 1) * b64[1], full, rtol=1e-12, atol=1e-13)


def test_softmax_xent_special_cases():
    # equal logits: loss = log C; huge logits do not overflow
    z = np.zeros((3, 7))
    loss, d = O.softmax_xent(z, np.array([0, 3, 6]))
    assert abs(loss - np.log(7)) < 1e-15
    assert np.allclose(d.sum(axis=1), 0)
    z = np.array([[1000.0, 0.0], [0.0, -1000.0]])
    loss, d = O.softmax_xent(z, np.array([0, 0]))
    assert np.isfinite(loss) and abs(loss) < 1e-12


def test_eval_counts_and_ties():
    W = [np.zeros((2, 3))]
    b = [np.array([0.5, 0.5, 0.1])]
    loss, ok = O.evaluate(W, b, np.ones((4, 2)), np.array([0, 1, 2, 0]))
    assert ok == 2          # ties go to class 0


# --- sparse first layer equals the dense definition -----------------------------------

def test_csr_round_equals_dense_round():
    dims, S, B, K, lr = [40, 12, 9], 3, 6, 3, 0.1
    W, b = synth.make_weights(dims, 5, bias_scale=0.2)
    rp, col, val = synth.make_csr_inputs(S * K * B, dims[0], 5.0, 9)
    y = synth.make_labels((S, K, B), dims[-1], 9)
    dense = np.zeros((S * K * B, dims[0]), dtype=np.float32)
    for r in range(S * K * B):
        dense[r, col[rp[r]:rp[r + 1]]] = val[rp[r]:rp[r + 1]]
    o1 = O.IstOracle(dims, S)
    o1.bind_weights(W, b)
    l1 = o1.round(3, (rp, col, val), y, lr, K)
    o2 = O.IstOracle(dims, S)
    o2.bind_weights(W, b)
    l2 = o2.round(3, dense.reshape(S, K, B, dims[0]), y, lr, K)
    np.testing.assert_allclose(l1, l2, rtol=1e-12)
    for l in range(2):
        np.testing.assert_allclose(o1.W[l], o2.W[l], rtol=1e-11, atol=1e-14)
        np.testing.assert_allclose(o1.b[l], o2.b[l], rtol=1e-11, atol=1e-14)
    e1 = o1.eval((rp[:B + 1], col[:rp[B]], val[:rp[B]]), y[0, 0])
    e2 = o2.eval(dense[:B], y[0, 0])
    assert e1[1] == e2[1] and abs(e1[0] - e2[0]) < 1e-12


# --- documents the reading "scale = 1": the n^2 factor of Eq. (2) over-corrects -------

def test_masked_linear_unbiased_scale_is_S_not_S_squared():
    # Monte Carlo over partitions of sum_s m_l^(s) * (W (m_{l-1}^(s) * f)): its mean is
    # (1/S) W f on a middle layer, so the unbiasing factor is S; S^2 would overshoot.
    rng = np.random.default_rng(0)
    N, S, trials = 12, 3, 3000
    Wm = rng.standard_normal((N, N))
    f = rng.standard_normal(N)
    acc = np.zeros(N)
    for seed in range(trials):
        p = O.partition(seed, [2, N, N, 2], S)
        for s in range(S):
            Gin, Gout = O.group(p, 1, s), O.group(p, 2, s)
            acc[Gout] += f[Gin] @ Wm[np.ix_(Gin, Gout)]
    est = acc / trials
    full = f @ Wm
    err_S = np.linalg.norm(S * est - full) / np.linalg.norm(full)
    err_S2 = np.linalg.norm(S * S * est - full) / np.linalg.norm(full)
    assert err_S < 0.15 and err_S2 > 1.0


# --- Sec. 2.2: per-neuron batch standardisation -------------------------------------------------

def _torch_loss_norm(Ws, bs, X, y, eps):
    a = X
    for l in range(len(Ws)):
        a = a @ Ws[l] + bs[l]
        if l < len(Ws) - 1:
            a = torch.nn.functional.batch_norm(a, None, None, training=True, eps=eps)   # no affine, batch stats
            a = torch.relu(a)
    return torch.nn.functional.cross_entropy(a, y, reduction="mean")


@pytest.mark.parametrize("dims", [[6, 9, 4], [5, 8, 7, 3]])
def test_norm_gradients_match_torch_batch_norm(dims):
    eps = 1e-5
    W, b, X, y = _tiny(dims, 1, 12, 1)
    Ws = [w.astype(np.float64) for w in W]
    bs = [v.astype(np.float64) for v in b]
    loss, dW, db = O.gradients_norm(Ws, bs, X[0, 0].astype(np.float64), y[0, 0], eps)
    tW = [torch.tensor(w, requires_grad=True) for w in Ws]
    tb = [torch.tensor(v, requires_grad=True) for v in bs]
    tl = _torch_loss_norm(tW, tb, torch.tensor(X[0, 0], dtype=torch.float64), torch.tensor(y[0, 0], dtype=torch.long), eps)
    tl.backward()
    assert abs(loss - tl.item()) < 1e-12
    for l in range(len(Ws)):
        np.testing.assert_allclose(dW[l], tW[l].grad.numpy(), rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(db[l], tb[l].grad.numpy(), rtol=1e-9, atol=1e-12)
    # a hidden bias cancels in the standardisation: its gradient vanishes
    for l in range(len(Ws) - 1):
        assert np.max(np.abs(db[l])) < 1e-12


def test_norm_forward_has_zero_mean_unit_variance():
    dims = [7, 20, 15, 4]
    W, b, X, _ = _tiny(dims, 1, 64, 1)
    _, _, zh, _ = O.forward_norm([w.astype(np.float64) for w in W], [v.astype(np.float64) for v in b],
                                 X[0, 0].astype(np.float64), 0.0)
    for h in zh:
        assert np.max(np.abs(h.mean(axis=0))) < 1e-12
        np.testing.assert_allclose(h.var(axis=0), 1.0, rtol=1e-10)


def test_norm_round_and_deployment_statistics():
    # S = 1 round with standardisation equals torch SGD on the batch-normalised network, and
    # evaluation with calibrated statistics equals the training-mode forward on the same rows
    dims, B, K, lr, eps = [6, 10, 8, 4], 16, 3, 0.05, 1e-5
    W, b, X, y = _tiny(dims, 1, B, K)
    o = O.IstOracle(dims, 1, norm_eps=eps)
    o.bind_weights(W, b)
    losses = o.round(5, X, y, lr, K)
    tW = [torch.tensor(w, dtype=torch.float64, requires_grad=True) for w in W]
    tb = [torch.tensor(v, dtype=torch.float64, requires_grad=True) for v in b]
    opt = torch.optim.SGD(tW + tb, lr=lr)
    for k in range(K):
        opt.zero_grad()
        l = _torch_loss_norm(tW, tb, torch.tensor(X[0, k], dtype=torch.float64), torch.tensor(y[0, k], dtype=torch.long), eps)
        l.backward()
        opt.step()
        assert abs(l.item() - losses[0, k]) < 1e-11
    for l in range(3):
        np.testing.assert_allclose(o.W[l], tW[l].detach().numpy(), rtol=1e-10, atol=1e-13)
    o.calibrate(X[0, 0])
    ev_loss, _ = o.eval(X[0, 0], y[0, 0])
    with torch.no_grad():
        ref = _torch_loss_norm([w.detach() for w in tW], [v.detach() for v in tb],
                               torch.tensor(X[0, 0], dtype=torch.float64), torch.tensor(y[0, 0], dtype=torch.long), eps)
    assert abs(ev_loss - ref.item()) < 1e-11


# ---------------------------------------------------------------------------------------------
# independent uniform assignment (the other reading of "uniform assignment", Sec. 2.1 / App. A)
# ---------------------------------------------------------------------------------------------

def test_iid_partition_is_the_multiply_high_of_the_keys():
    # brute force with Python integers on the keys (which the published SplitMix64 vector pins)
    seed, layer, N, S = 99, 2, 257, 5
    keys = [int(k) for k in O.neuron_keys(seed, layer, N)]
    idx, off = O.partition_layer_iid(seed, layer, N, S)
    assert off[0] == 0 and off[-1] == N
    for g in range(S):
        want = [i for i in range(N) if (keys[i] * S) // 2 ** 64 == g]
        assert list(idx[off[g]:off[g + 1]]) == want
    assert sorted(idx.tolist()) == list(range(N))           # every neuron in exactly one group


def test_iid_group_sizes_are_binomial_not_fixed():
    N, S, trials = 240, 4, 400
    sizes = np.array([np.diff(O.partition_layer_iid(1000 + s, 1, N, S)[1]) for s in range(trials)])
    assert sizes.sum(axis=1).tolist() == [N] * trials
    # mean N/S, variance N (1/S)(1 - 1/S) = 45 per group; the balanced rule would give variance 0
    assert np.all(np.abs(sizes.mean(axis=0) - N / S) < 4 * np.sqrt(45 / trials))
    assert np.all(np.abs(sizes.var(axis=0) - 45) < 12)
    # membership of one neuron is uniform over the groups (chi-square, 3 degrees of freedom)
    member = np.zeros(S)
    for s in range(trials):
        idx, off = O.partition_layer_iid(5000 + s, 1, N, S)
        member[np.searchsorted(off, np.where(idx == 17)[0][0], side="right") - 1] += 1
    chi2 = ((member - trials / S) ** 2 / (trials / S)).sum()
    assert chi2 < 16.3                                       # 0.1 % tail


def test_iid_round_reassembles_and_trains_like_the_balanced_one():
    # slicing and copy-back use only (idx, off): an untouched round is the identity, and with
    # S = 1 both rules give the same single group and therefore the same trained network
    dims = [6, 20, 14, 4]
    W, b, X, y = _tiny(dims, 3, 5, 2)
    o = O.IstOracle(dims, 3, partition_rule="iid")
    o.bind_weights(W, b)
    o.partition(4)
    sizes = [np.diff(off) for _, off in o.parts]
    assert any(len(set(s.tolist())) > 1 for s in sizes)     # truly unequal groups for this seed
    o.reassemble()
    for l in range(3):
        assert np.array_equal(o.W[l], W[l].astype(np.float64)) and np.array_equal(o.b[l], b[l].astype(np.float64))
    W1, b1, X1, y1 = _tiny(dims, 1, 5, 2)
    a = O.IstOracle(dims, 1, partition_rule="iid")
    c = O.IstOracle(dims, 1)
    for o2 in (a, c):
        o2.bind_weights(W1, b1)
        o2.round(7, X1, y1, 0.1, 2)
    for l in range(3):
        assert np.array_equal(a.W[l], c.W[l])
