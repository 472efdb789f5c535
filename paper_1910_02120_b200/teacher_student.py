"""Multi-round IST training on a synthetic classification task (paper Sec. 2.1: partition,
K local steps, copy back, re-partition, repeat; Sec. 2.2: the deployed full network is scored
with statistics taken over a data subset).

    python -m paper_1910_02120_b200.teacher_student --rounds 40

Every step of a round runs in the CUDA library; this module draws the task, moves each round's
minibatch rows into place (a device-side row gather with torch) and reports, per round, the
mean subnet loss and the loss / accuracy of the reassembled full network on held-out rows.
One JSON line per evaluated round.
"""
from __future__ import annotations

import argparse
import json
from typing import List, Optional, Sequence

import torch

from . import api, synth


def train(layer_dims: Sequence[int], S: int, K: int, B: int, rounds: int, lr: float,
          norm_eps: Optional[float] = 1e-5, precision: str = "bf16", seed: int = 1,
          n_train: int = 8192, n_test: int = 2048, eval_every: int = 1, resample: bool = True,
          device: str = "cuda:0") -> List[dict]:
    """Runs `rounds` IST rounds; returns one record per evaluated round.

    resample=False keeps the first round's partition for all rounds (the subnets then never
    exchange parameters: the "ensemble" arrangement the paper compares against)."""
    dims = [int(d) for d in layer_dims]
    X_all, y_all = synth.make_teacher_task(n_train + n_test, dims[0], dims[-1], seed)
    W, b = synth.make_weights(dims, seed)
    dev = torch.device(device)
    Xtr = torch.from_numpy(X_all[:n_train]).to(dev)
    ytr = torch.from_numpy(y_all[:n_train]).to(dev)
    Xte = torch.from_numpy(X_all[n_train:]).to(dev)
    yte = torch.from_numpy(y_all[n_train:]).to(dev)
    Wd = [torch.from_numpy(x).to(dev) for x in W]
    bd = [torch.from_numpy(x).to(dev) for x in b]
    prec = api.IST_BF16 if precision == "bf16" else api.IST_FP32
    ctx = api.Ist(dims, S, prec, max(B, min(n_test, 1024)), device=device)
    ctx.bind_weights(Wd, bd)
    if norm_eps is not None:
        ctx.enable_normalization(norm_eps)
    n_cal = min(n_train, ctx.max_batch)
    records = []
    for r in range(rounds):
        rows = torch.from_numpy(synth.draw_round_rows(n_train, S, K, B, seed, r).reshape(-1)).to(dev)
        Xr = Xtr.index_select(0, rows)
        if precision == "bf16" and dims[0] % 8 == 0:
            Xr = Xr.to(torch.bfloat16)
        yr = ytr.index_select(0, rows).contiguous()
        loss = ctx.round(seed * 7919 + (r if resample else 0), Xr, yr, lr, K, B)
        if (r + 1) % eval_every == 0 or r + 1 == rounds:
            if norm_eps is not None:
                ctx.calibrate(Xtr, n_cal)
            tl, tc = ctx.eval(Xte, yte, n_test)
            ctx.sync_status()
            records.append({"round": r + 1, "subnet_loss": float(loss.mean().item()),
                            "test_loss": float(tl.item()), "test_acc": tc.item() / n_test})
    ctx.close()
    return records


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--dims", default="64,512,512,10")
    ap.add_argument("--S", type=int, default=4)
    ap.add_argument("--K", type=int, default=10)
    ap.add_argument("--B", type=int, default=64)
    ap.add_argument("--rounds", type=int, default=40)
    ap.add_argument("--lr", type=float, default=0.05)
    ap.add_argument("--norm-eps", type=float, default=1e-5)
    ap.add_argument("--no-norm", action="store_true")
    ap.add_argument("--precision", default="bf16", choices=["bf16", "fp32"])
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--eval-every", type=int, default=5)
    ap.add_argument("--fixed-partition", action="store_true")
    args = ap.parse_args()
    recs = train([int(x) for x in args.dims.split(",")], args.S, args.K, args.B, args.rounds, args.lr,
                 None if args.no_norm else args.norm_eps, args.precision, args.seed,
                 eval_every=args.eval_every, resample=not args.fixed_partition)
    for r in recs:
        print(json.dumps(r))


if __name__ == "__main__":
    main()
