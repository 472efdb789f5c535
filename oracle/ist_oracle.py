"""CPU oracle for one round of Independent Subnet Training (IST).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what one
IST round computes, written from the paper (arXiv 1910.02120) so that a reader
can check it against the text by eye.  It shares no code, layout, table or
helper with the CUDA library and must never be imported by it; only the tests,
the smoke check and the benchmark's CPU-baseline leg call it.

Everything is numpy; `@` (matmul), `lexsort` and `sort` are used as library
steps.  Storage and arithmetic are fp64 by default (`dtype=np.float32` gives
the secondary mode used to bound fp32 drift).  One subnet at a time, no
blocking, no fusion, no packed buffers.

What follows the paper, and what is a reading of it where the paper is silent:

* Sec. 2.1 "Constructing Subnets" / App. A: every hidden neuron goes to exactly
  one of the S subnets (sum_s m^(s)_{l,i} = 1), with marginal probability 1/S,
  independently per layer; input and output neurons belong to every subnet.
  READING (group sizes are never stated): a balanced random split, see
  `partition_layer`.
* Sec. 2.1, App. A footnote (weights are cut so that nothing belonging to a
  neuron outside the subnet is ever evaluated): subnet s owns
  W_l[G_{l-1}^s, G_l^s]; first layer sliced on columns only, last layer on
  rows only.
* App. A Eq. (2) with the n^2 factor removed, as Sec. 2.2 "Correcting
  Distributional Shift" does: f_l = S(W_l f_{l-1}) on the slice, scale 1.
  The batch standardisation of Sec. 2.2 is optional (`norm_eps`): off on the
  plain path, on in the *_norm functions.
* Sec. 2.1 "Training Subnets": J (= K here) iterations of local SGD per subnet,
  w <- w - eta * grad, no communication; then slices are copied back, with no
  collisions because the partition is disjoint.
* READING (the paper names no loss and no biases): softmax cross-entropy, mean
  over the minibatch; hidden biases travel with their neurons; the output bias
  is the one parameter every subnet holds, each trains its own copy and the
  copies are averaged at reassembly (the local-SGD treatment of shared state).
* READING: ReLU with derivative 0 at 0.

Parity pins (tests/test_oracle_pins.py): SplitMix64 published outputs for the
key mixer; partition invariants; S = 1 equals plain SGD; finite differences;
torch autograd; one-hidden-layer separability; the traffic closed forms of
Sec. 2.3; untouched reassembly is the identity.  The output-bias averaging and
the choice of which batch each subnet sees have no counterpart in the paper:
parity unpinned by the paper for those two readings (they are pinned only by
special cases: S = 1 identity, mean of equal copies).
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import numpy as np

_U64 = np.uint64
PHI = 0x9E3779B97F4A7C15          # SplitMix64 state increment
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_MASK = (1 << 64) - 1


# ----------------------------------------------------------------------------
# Partition (Sec. 2.1 "Constructing Subnets"; App. A membership indicators)
# ----------------------------------------------------------------------------

def splitmix64_mix(z: int) -> int:
    """Output function of SplitMix64 (Steele, Lea, Flood, OOPSLA 2014), on Python ints."""
    z &= _MASK
    z = ((z ^ (z >> 30)) * _M1) & _MASK
    z = ((z ^ (z >> 27)) * _M2) & _MASK
    return z ^ (z >> 31)


def splitmix64_stream(seed: int, count: int) -> List[int]:
    """The first `count` outputs of a SplitMix64 generator whose state starts at `seed`."""
    out = []
    state = seed & _MASK
    for _ in range(count):
        state = (state + PHI) & _MASK
        out.append(splitmix64_mix(state))
    return out


def neuron_keys(seed: int, layer: int, N: int) -> List[int]:
    """Random 64-bit key of every neuron of hidden layer `layer` (1-based).

    The layer's stream seed is the `layer`-th output of SplitMix64 seeded with
    the round seed; the keys are the first N outputs of SplitMix64 seeded with
    that stream seed.  Different layers therefore get independent streams
    (App. A: sampling is independent at each layer).
    """
    layer_seed = splitmix64_stream(seed, layer)[-1]
    return splitmix64_stream(layer_seed, N)


def partition_layer(seed: int, layer: int, N: int, S: int) -> Tuple[np.ndarray, np.ndarray]:
    """Balanced random partition of {0..N-1} into S groups.

    Neurons are ordered by (key, index) ascending; group g takes the next
    floor(N/S) (+1 if g < N mod S) neurons of that order; inside a group the
    indices are then listed in ascending order.  Returns (idx [N] int32,
    group-major, and off [S+1] int32 with group g = idx[off[g]:off[g+1]]).
    """
    if not (1 <= S <= N):
        raise ValueError("need 1 <= S <= N")
    keys = neuron_keys(seed, layer, N)
    order = sorted(range(N), key=lambda i: (keys[i], i))
    idx = np.empty(N, dtype=np.int32)
    off = np.zeros(S + 1, dtype=np.int32)
    start = 0
    for g in range(S):
        cnt = N // S + (1 if g < N % S else 0)
        members = sorted(order[start:start + cnt])
        idx[start:start + cnt] = members
        start += cnt
        off[g + 1] = start
    return idx, off


def partition_layer_iid(seed: int, layer: int, N: int, S: int) -> Tuple[np.ndarray, np.ndarray]:
    """Independent uniform assignment (the other reading of Sec. 2.1 "uniform assignment to one
    of n possible compute nodes"; App. A: each neuron joins subnet s with probability 1/n,
    independently of the others): neuron i goes to group floor(key_i * S / 2^64) with the same
    keys as the balanced rule.  Group sizes are Binomial(N, 1/S), not fixed; a group may be
    empty.  Indices ascend inside a group.  Returns (idx, off) like partition_layer."""
    if S < 1 or N < 1:
        raise ValueError("need S >= 1 and N >= 1")
    keys = neuron_keys(seed, layer, N)
    grp = [(int(keys[i]) * S) >> 64 for i in range(N)]
    idx = np.empty(N, dtype=np.int32)
    off = np.zeros(S + 1, dtype=np.int32)
    at = 0
    for g in range(S):
        members = [i for i in range(N) if grp[i] == g]      # ascending by construction
        idx[at:at + len(members)] = members
        at += len(members)
        off[g + 1] = at
    return idx, off


PARTITION_RULES = {"balanced": partition_layer, "iid": partition_layer_iid}


def partition(seed: int, layer_dims: Sequence[int], S: int, rule: str = "balanced"):
    """One partition per hidden layer l = 1..t-1.  Returns a list of (idx, off)."""
    t = len(layer_dims) - 1
    if t == 1 and S != 1:
        raise ValueError("a network without hidden layers has nothing to partition: S must be 1")
    return [PARTITION_RULES[rule](seed, l, int(layer_dims[l]), S) for l in range(1, t)]


def group(parts, hidden_layer: int, s: int) -> np.ndarray:
    """Index set G_l^s (hidden_layer is 1-based)."""
    idx, off = parts[hidden_layer - 1]
    return idx[off[s]:off[s + 1]]


# ----------------------------------------------------------------------------
# Slicing and copy-back (Sec. 2.1; App. A footnote)
# ----------------------------------------------------------------------------

def slice_subnet(W: Sequence[np.ndarray], b: Sequence[np.ndarray], parts, s: int):
    """Parameters of subnet s, as fresh arrays.

    W[l-1] is W_l with shape [N_{l-1}][N_l].  First layer: all rows, columns
    G_1^s.  Middle layers: rows G_{l-1}^s, columns G_l^s.  Last layer: rows
    G_{t-1}^s, all columns.  Hidden biases follow their neurons; the output
    bias is copied whole.
    """
    t = len(W)
    Ws, bs = [], []
    for l in range(1, t + 1):
        rows = slice(None) if l == 1 else group(parts, l - 1, s)
        cols = slice(None) if l == t else group(parts, l, s)
        Wl = W[l - 1]
        Ws.append(np.array(Wl[rows, :][:, cols], copy=True))
        bs.append(np.array(b[l - 1][cols], copy=True))
    return Ws, bs


def reassemble(W: List[np.ndarray], b: List[np.ndarray], parts, subnets) -> None:
    """Copy every subnet's slices back into the full network, in place.

    Entries of middle layers whose row group differs from their column group
    belong to no subnet and are left as they are.  The output bias becomes the
    mean of the S trained copies, written as old + (sum_s (copy_s - old)) / S with
    the sum taken in subnet order, so that untouched copies give back `old` exactly.
    """
    t = len(W)
    S = len(subnets)
    for s, (Ws, bs) in enumerate(subnets):
        for l in range(1, t + 1):
            rows = np.arange(W[l - 1].shape[0]) if l == 1 else group(parts, l - 1, s)
            cols = np.arange(W[l - 1].shape[1]) if l == t else group(parts, l, s)
            W[l - 1][np.ix_(rows, cols)] = Ws[l - 1]
            if l < t:
                b[l - 1][cols] = bs[l - 1]
    old = b[t - 1].copy()
    acc = np.zeros_like(old)
    for s in range(S):
        acc = acc + (subnets[s][1][t - 1] - old)
    b[t - 1][:] = old + acc / S


# ----------------------------------------------------------------------------
# Forward, loss, backward, SGD (App. A Eq. (2) without the n^2 factor; Sec. 2.1)
# ----------------------------------------------------------------------------

class CsrRows:
    """A batch of sparse input rows: row_ptr [B+1], col [nnz], val [nnz]."""

    def __init__(self, row_ptr, col, val):
        self.row_ptr = np.asarray(row_ptr, dtype=np.int64)
        self.col = np.asarray(col, dtype=np.int64)
        self.val = np.asarray(val)
        self.B = self.row_ptr.size - 1

    def row(self, r):
        lo, hi = self.row_ptr[r], self.row_ptr[r + 1]
        return self.col[lo:hi], self.val[lo:hi]


def _first_layer_product(X, W1, dtype):
    """X @ W1 for dense X [B][N0] or sparse rows (sum over stored nonzeros only)."""
    if isinstance(X, CsrRows):
        out = np.zeros((X.B, W1.shape[1]), dtype=dtype)
        for r in range(X.B):
            c, v = X.row(r)
            out[r] = v.astype(dtype) @ W1[c, :]
        return out
    return X @ W1


def forward(Ws, bs, X, dtype=np.float64):
    """Pre-activations z_1..z_t and activations a_0..a_{t-1} of one (sub)network."""
    t = len(Ws)
    a = [X if isinstance(X, CsrRows) else np.asarray(X, dtype=dtype)]
    z = []
    for l in range(1, t + 1):
        prod = _first_layer_product(a[0], Ws[0], dtype) if l == 1 else a[l - 1] @ Ws[l - 1]
        zl = prod + bs[l - 1]
        z.append(zl)
        if l < t:
            a.append(np.maximum(zl, 0))
    return z, a


def softmax_xent(z_t: np.ndarray, y: np.ndarray):
    """Mean softmax cross-entropy over the batch and d(loss)/d(z_t).

    loss = (1/B) sum_b [logsumexp(z_b) - z_b[y_b]], computed with the row
    maximum subtracted; delta = (softmax(z) - onehot(y)) / B.
    """
    B = z_t.shape[0]
    m = z_t.max(axis=1, keepdims=True)
    e = np.exp(z_t - m)
    se = e.sum(axis=1, keepdims=True)
    rows = np.arange(B)
    loss = (np.log(se[:, 0]) + m[:, 0] - z_t[rows, y]).sum() / B
    delta = e / se
    delta[rows, y] -= 1
    delta /= B
    return loss, delta


def gradients(Ws, bs, X, y, dtype=np.float64):
    """Loss and gradients (dW_l, db_l) of one minibatch, all from the current parameters.

    delta_t = (softmax - onehot)/B; dW_l = a_{l-1}^T delta_l; db_l = sum_b delta_l;
    delta_{l-1} = (delta_l W_l^T) * [z_{l-1} > 0].
    For sparse X, dW_1 is returned as a list of (cols, block) per row instead of a
    dense matrix: row r contributes val_r (outer) delta_1[r] to the rows `cols`.
    """
    t = len(Ws)
    z, a = forward(Ws, bs, X, dtype)
    loss, delta = softmax_xent(z[t - 1], np.asarray(y, dtype=np.int64))
    dW = [None] * t
    db = [None] * t
    for l in range(t, 0, -1):
        db[l - 1] = delta.sum(axis=0)
        if l == 1 and isinstance(X, CsrRows):
            blocks = []
            for r in range(X.B):
                c, v = X.row(r)
                blocks.append((c, np.outer(v.astype(dtype), delta[r])))
            dW[0] = blocks
        else:
            dW[l - 1] = a[l - 1].T @ delta
        if l > 1:
            delta = (delta @ Ws[l - 1].T) * (z[l - 2] > 0)
    return loss, dW, db


def input_gradient(Ws, bs, X, y, dtype=np.float64):
    """d(loss)/dX of one minibatch at the current parameters: delta_1 W_1^T, where delta_1 is the
    gradient with respect to the first layer's pre-activations (back-propagated as in
    `gradients`).  Sec. 2.2, "IST for other architectures": when only the fully connected part of
    a network is partitioned, whatever produces its input (a convolutional trunk that every site
    holds whole) is trained from this gradient.  Dense X only."""
    t = len(Ws)
    z, a = forward(Ws, bs, X, dtype)
    _, delta = softmax_xent(z[t - 1], np.asarray(y, dtype=np.int64))
    for l in range(t, 1, -1):
        delta = (delta @ Ws[l - 1].T) * (z[l - 2] > 0)
    return delta @ Ws[0].T


# ----------------------------------------------------------------------------
# Sec. 2.2 "Correcting Distributional Shift": every hidden neuron's input is
# standardised with the mean and standard deviation over the minibatch before
# the non-linearity (no n^2 factor, no learned scale or shift).
# READING: the paper gives no epsilon and does not say which variance; this
# uses the biased (1/B) variance and sigma = sqrt(var + eps).
# ----------------------------------------------------------------------------

def forward_norm(Ws, bs, X, eps, dtype=np.float64):
    """Forward pass with per-neuron batch standardisation in the hidden layers.

    z_l = a_{l-1} W_l + b_l;  zh_l = (z_l - mean_b z_l) / sqrt(var_b z_l + eps);
    a_l = max(zh_l, 0).  Returns z_t, the activations a_0..a_{t-1}, zh_1..zh_{t-1}
    and 1/sigma_1..1/sigma_{t-1}.
    """
    t = len(Ws)
    a = [X if isinstance(X, CsrRows) else np.asarray(X, dtype=dtype)]
    zh, rstd = [], []
    z = None
    for l in range(1, t + 1):
        prod = _first_layer_product(a[0], Ws[0], dtype) if l == 1 else a[l - 1] @ Ws[l - 1]
        z = prod + bs[l - 1]
        if l < t:
            mu = z.mean(axis=0)
            var = ((z - mu) ** 2).mean(axis=0)
            r = 1.0 / np.sqrt(var + eps)
            h = (z - mu) * r
            zh.append(h)
            rstd.append(r)
            a.append(np.maximum(h, 0))
    return z, a, zh, rstd


def gradients_norm(Ws, bs, X, y, eps, dtype=np.float64):
    """Loss and gradients with the standardisation differentiated through:
    d_zh = (delta_{l+1} W_{l+1}^T) * [zh > 0];
    d_z  = (d_zh - mean_b d_zh - zh * mean_b(d_zh * zh)) / sigma.
    """
    t = len(Ws)
    z_t, a, zh, rstd = forward_norm(Ws, bs, X, eps, dtype)
    loss, delta = softmax_xent(z_t, np.asarray(y, dtype=np.int64))
    dW = [None] * t
    db = [None] * t
    for l in range(t, 0, -1):
        db[l - 1] = delta.sum(axis=0)
        if l == 1 and isinstance(X, CsrRows):
            dW[0] = [(X.row(r)[0], np.outer(X.row(r)[1].astype(dtype), delta[r])) for r in range(X.B)]
        else:
            dW[l - 1] = a[l - 1].T @ delta
        if l > 1:
            h = zh[l - 2]
            d_zh = (delta @ Ws[l - 1].T) * (h > 0)
            delta = (d_zh - d_zh.mean(axis=0) - h * (d_zh * h).mean(axis=0)) * rstd[l - 2]
    return loss, dW, db


def calibrate(W, b, X, eps, dtype=np.float64):
    """Deployment statistics (Sec. 2.2): mean and 1/sigma of every hidden neuron's input over a
    data subset, computed with the full network layer by layer."""
    _, _, zh, rstd = forward_norm(W, b, X, eps, dtype)
    # forward_norm standardised with exactly these statistics; recover the means from it
    stats = []
    a = X if isinstance(X, CsrRows) else np.asarray(X, dtype=dtype)
    for l in range(1, len(W)):
        prod = _first_layer_product(a, W[0], dtype) if l == 1 else a @ W[l - 1]
        z = prod + b[l - 1]
        mu = z.mean(axis=0)
        stats.append((mu, rstd[l - 1]))
        a = np.maximum((z - mu) * rstd[l - 1], 0)
    return stats


def evaluate_norm(W, b, X, y, stats, dtype=np.float64):
    """Full-width forward with stored statistics: mean loss and number of correct predictions."""
    a = X if isinstance(X, CsrRows) else np.asarray(X, dtype=dtype)
    t = len(W)
    for l in range(1, t + 1):
        prod = _first_layer_product(a, W[0], dtype) if l == 1 else a @ W[l - 1]
        z = prod + b[l - 1]
        if l < t:
            mu, r = stats[l - 1]
            a = np.maximum((z - mu) * r, 0)
    y = np.asarray(y, dtype=np.int64)
    loss, _ = softmax_xent(z, y)
    return float(loss), int((z.argmax(axis=1) == y).sum())


def sgd_step(Ws, bs, X, y, lr, dtype=np.float64, norm_eps=None):
    """One local SGD iteration, in place: w <- w - lr * grad.  Returns the pre-update loss."""
    if norm_eps is None:
        loss, dW, db = gradients(Ws, bs, X, y, dtype)
    else:
        loss, dW, db = gradients_norm(Ws, bs, X, y, norm_eps, dtype)
    lr = dtype(lr)
    for l in range(len(Ws)):
        if isinstance(dW[l], list):
            for c, block in dW[l]:
                Ws[l][c, :] -= lr * block
        else:
            Ws[l] -= lr * dW[l]
        bs[l] -= lr * db[l]
    return loss


def evaluate(W, b, X, y, dtype=np.float64):
    """Full-width forward: mean loss and number of correct argmax predictions
    (ties go to the lowest class index, numpy's argmax rule)."""
    z, _ = forward(W, b, X, dtype)
    y = np.asarray(y, dtype=np.int64)
    loss, _ = softmax_xent(z[-1], y)
    return float(loss), int((z[-1].argmax(axis=1) == y).sum())


# ----------------------------------------------------------------------------
# One round, in the order the paper gives it
# ----------------------------------------------------------------------------

class IstOracle:
    """partition -> slice -> K local steps per subnet -> copy back."""

    def __init__(self, layer_dims: Sequence[int], S: int, dtype=np.float64, norm_eps=None,
                 partition_rule: str = "balanced"):
        self.partition_rule = partition_rule
        self.norm_eps = norm_eps          # None: plain path; a float: Sec. 2.2 standardisation
        self.stats = None
        self.layer_dims = [int(d) for d in layer_dims]
        self.t = len(self.layer_dims) - 1
        if self.t < 1:
            raise ValueError("need at least one weight layer")
        self.S = int(S)
        self.dtype = dtype
        self.W: Optional[List[np.ndarray]] = None
        self.b: Optional[List[np.ndarray]] = None
        self.parts = None
        self.subnets = None

    def bind_weights(self, W, b):
        """Takes copies in the oracle's dtype (the caller's arrays are not modified)."""
        assert len(W) == self.t and len(b) == self.t
        for l in range(self.t):
            assert W[l].shape == (self.layer_dims[l], self.layer_dims[l + 1])
            assert b[l].shape == (self.layer_dims[l + 1],)
        self.W = [np.array(w, dtype=self.dtype, copy=True) for w in W]
        self.b = [np.array(v, dtype=self.dtype, copy=True) for v in b]

    def partition(self, seed: int):
        self.parts = partition(seed, self.layer_dims, self.S, self.partition_rule)
        self.subnets = [slice_subnet(self.W, self.b, self.parts, s) for s in range(self.S)]
        return self.parts

    def _batch(self, X, y, s, k):
        """Batch of subnet s at local step k.  Dense X is [S][K][B][N0]; sparse X is a
        (row_ptr, col, val) triple over S*K*B rows in the same order; y is [S][K][B]."""
        if isinstance(X, tuple):
            row_ptr, col, val = X
            B = y.shape[2]
            K = y.shape[1]
            r0 = (s * K + k) * B
            lo, hi = int(row_ptr[r0]), int(row_ptr[r0 + B])
            xb = CsrRows(np.asarray(row_ptr[r0:r0 + B + 1]) - lo, col[lo:hi],
                         np.asarray(val[lo:hi], dtype=self.dtype))
        else:
            xb = np.asarray(X[s, k], dtype=self.dtype)
        return xb, y[s, k]

    def local_steps(self, X, y, lr: float, K: int) -> np.ndarray:
        """K SGD steps on each subnet; returns loss[s][k] (loss before the update of step k)."""
        losses = np.zeros((self.S, K), dtype=np.float64)
        for s in range(self.S):
            Ws, bs = self.subnets[s]
            for k in range(K):
                xb, yb = self._batch(X, y, s, k)
                losses[s, k] = sgd_step(Ws, bs, xb, yb, lr, self.dtype, self.norm_eps)
        return losses

    def local_steps_dx(self, X, y, lr: float, K: int):
        """local_steps that also returns dX[s][k] = d(loss of step k)/d(batch of step k), taken at
        the parameters the step starts from (before its update).  Plain path, dense X."""
        assert self.norm_eps is None and not isinstance(X, tuple)
        losses = np.zeros((self.S, K), dtype=np.float64)
        dX = np.zeros(np.asarray(X).shape, dtype=self.dtype)
        for s in range(self.S):
            Ws, bs = self.subnets[s]
            for k in range(K):
                xb, yb = self._batch(X, y, s, k)
                dX[s, k] = input_gradient(Ws, bs, xb, yb, self.dtype)
                losses[s, k] = sgd_step(Ws, bs, xb, yb, lr, self.dtype, None)
        return losses, dX

    def reassemble(self):
        reassemble(self.W, self.b, self.parts, self.subnets)
        self.subnets = None

    def calibrate(self, X):
        if isinstance(X, tuple):
            X = CsrRows(X[0], X[1], np.asarray(X[2], dtype=self.dtype))
        self.stats = calibrate(self.W, self.b, X, self.norm_eps, self.dtype)
        return self.stats

    def eval(self, X, y):
        if isinstance(X, tuple):
            X = CsrRows(X[0], X[1], np.asarray(X[2], dtype=self.dtype))
        if self.norm_eps is not None:
            return evaluate_norm(self.W, self.b, X, y, self.stats, self.dtype)
        return evaluate(self.W, self.b, X, y, self.dtype)

    def round(self, seed, X, y, lr, K):
        self.partition(seed)
        losses = self.local_steps(X, y, lr, K)
        self.reassemble()
        return losses
