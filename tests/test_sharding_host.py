"""Subnets split over ranks (Sec. 2.1 / 2.3), host side, on CPU with two gloo ranks: the slab
arithmetic, the all-gather of packed slices, and the protocol itself run with the oracle: two ranks
that each train half of the subnets and exchange their slices end with the full network of the
single-process round."""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import ist_oracle as O
from paper_1910_02120_b200 import sharding, synth


def test_subnet_range_splits_evenly():
    assert sharding.subnet_range(8, 2, 0) == (0, 4)
    assert sharding.subnet_range(8, 2, 1) == (4, 4)
    assert sharding.subnet_range(8, 8, 5) == (5, 1)
    assert sharding.subnet_range(3, 1, 0) == (0, 3)
    with pytest.raises(ValueError):
        sharding.subnet_range(6, 4, 0)
    with pytest.raises(ValueError):
        sharding.subnet_range(4, 2, 2)


DIMS, S, K, B, LR, SEED = (12, 40, 36, 5), 4, 3, 8, 0.05, 21


def _problem():
    W, b = synth.make_weights(DIMS, 9, bias_scale=0.1)
    w = synth.Workload("sh", DIMS, S=S, B=B, K=K, rounds=1, precision="fp32", x_dist="normal", lr=LR, seed=9)
    data = synth.make_round_inputs(w)
    return W, b, data


def _pack(o):
    """Per layer: [S][rows*cols] and [S][cols] zero-padded slabs of the subnets' current parameters."""
    out = []
    for l in range(len(DIMS) - 1):
        rmax = max(o.subnets[s][0][l].shape[0] for s in range(S))
        cmax = max(o.subnets[s][0][l].shape[1] for s in range(S))
        Wp = torch.zeros(S, rmax * cmax, dtype=torch.float64)
        bp = torch.zeros(S, cmax, dtype=torch.float64)
        out.append((Wp, bp, rmax, cmax))
    return out


def _rank_main(rank, world, port, outdir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    first, count = sharding.subnet_range(S, world, rank)
    W, b, data = _problem()
    o = O.IstOracle(DIMS, S)
    o.bind_weights(W, b)
    o.partition(SEED)
    for s in range(first, first + count):               # this rank's sites only
        Ws, bs = o.subnets[s]
        for k in range(K):
            O.sgd_step(Ws, bs, data.X[s, k].astype(np.float64), data.y[s, k], LR)
    packed = _pack(o)
    for l, (Wp, bp, rmax, cmax) in enumerate(packed):   # only the trained slabs are filled in
        for s in range(first, first + count):
            Ws, bs = o.subnets[s]
            r, c = Ws[l].shape
            slab = np.zeros((rmax, cmax))
            slab[:r, :c] = Ws[l]
            Wp[s] = torch.from_numpy(slab.reshape(-1))
            bp[s, :c] = torch.from_numpy(bs[l])
    got = sharding.exchange_slices([t for Wp, bp, _, _ in packed for t in (Wp, bp)], first, count)
    assert got == (world - 1) * sum(Wp[first:first + count].numel() * 8 + bp[first:first + count].numel() * 8
                                    for Wp, bp, _, _ in packed)
    for l, (Wp, bp, rmax, cmax) in enumerate(packed):   # unpack everybody's slices, then copy back
        for s in range(S):
            Ws, bs = o.subnets[s]
            r, c = Ws[l].shape
            Ws[l][...] = Wp[s].numpy().reshape(rmax, cmax)[:r, :c]
            bs[l][...] = bp[s, :c].numpy()
    o.reassemble()
    np.savez(os.path.join(outdir, f"rank{rank}.npz"), *o.W, *o.b)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_process_round(tmp_path):
    port = 29700 + os.getpid() % 1000
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    W, b, data = _problem()
    o = O.IstOracle(DIMS, S)
    o.bind_weights(W, b)
    o.round(SEED, data.X, data.y, LR, K)
    want = o.W + o.b
    for rank in range(2):
        got = np.load(os.path.join(str(tmp_path), f"rank{rank}.npz"))
        for i, w in enumerate(want):
            assert np.array_equal(got[f"arr_{i}"], w), (rank, i)
