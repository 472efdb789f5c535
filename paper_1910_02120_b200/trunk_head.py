"""IST on the fully connected head of a network with a convolutional trunk (paper Sec. 2.2, "IST for
other architectures": the trunk is held whole by every site and trained by local SGD, its copies
averaged when the subnets are copied back; only the fully connected part is partitioned).

    python -m paper_1910_02120_b200.trunk_head --rounds 30

The head (partition, local steps, reassembly) runs in the CUDA library; the trunk is the caller's
part and is a small torch module here: one copy per subnet, which turns its subnet's images into
the head's input rows, receives the loss gradient with respect to those rows from
ist_local_steps_dx (one local step per call) and takes its own SGD step.  Synthetic images, a
synthetic teacher: a demonstration that the pieces fit, one JSON line per round.
"""
from __future__ import annotations

import argparse
import copy
import json
from typing import List

import torch

from . import api


def make_task(n: int, classes: int, seed: int, device):
    """Images [n][1][12][12] ~ N(0,1); labels from a fixed random convolution + linear teacher."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    x = torch.randn(n, 1, 12, 12, generator=g)
    k = torch.randn(4, 1, 3, 3, generator=g)
    a = torch.randn(4 * 5 * 5, classes, generator=g)
    f = torch.nn.functional.avg_pool2d(torch.tanh(torch.nn.functional.conv2d(x, k)), 2).flatten(1)
    return x.to(device), (f @ a).argmax(1).to(torch.int32).to(device)


def make_trunk(features: int, seed: int, device):
    torch.manual_seed(seed)
    return torch.nn.Sequential(torch.nn.Conv2d(1, 8, 3), torch.nn.ReLU(), torch.nn.AvgPool2d(2),
                               torch.nn.Flatten(), torch.nn.Linear(8 * 5 * 5, features)).to(device)


def train(rounds: int = 30, S: int = 4, K: int = 10, B: int = 64, features: int = 64, hidden: int = 256,
          classes: int = 10, lr: float = 0.3, precision: str = "fp32", seed: int = 1,
          device: str = "cuda:0") -> List[dict]:
    """Runs `rounds` rounds; returns per round the mean loss of the subnets' local steps."""
    dev = torch.device(device)
    n = S * K * B * 4
    x_all, y_all = make_task(n, classes, seed, dev)
    dims = [features, hidden, hidden, classes]
    g = torch.Generator(device="cpu").manual_seed(seed + 1)
    Wd = [((torch.rand(dims[i], dims[i + 1], generator=g) * 2 - 1) * (6.0 / dims[i]) ** 0.5).to(dev) for i in range(3)]
    bd = [torch.zeros(dims[i + 1], device=dev) for i in range(3)]
    prec = api.IST_BF16 if precision == "bf16" else api.IST_FP32
    ctx = api.Ist(dims, S, prec, B, device=device)
    ctx.bind_weights(Wd, bd)
    trunk = make_trunk(features, seed, dev)
    records = []
    for r in range(rounds):
        perm = torch.randperm(n, generator=g)[: S * K * B].to(dev).view(S, K, B)
        copies = [copy.deepcopy(trunk) for _ in range(S)]      # the trunk goes to every site whole
        ctx.partition(seed * 7919 + r)
        losses = []
        for k in range(K):
            rows = perm[:, k, :].reshape(-1)                   # [S][1][B]: one local step per call
            feats = [copies[s](x_all[rows[s * B:(s + 1) * B]]) for s in range(S)]
            X = torch.cat(feats).detach().contiguous()
            Xin = X.to(torch.bfloat16) if precision == "bf16" and features % 8 == 0 else X
            dx = torch.empty(S * B, features, dtype=torch.float32, device=dev)
            loss = ctx.local_steps(Xin, y_all[rows].contiguous(), lr, 1, B, dx_out=dx)
            losses.append(loss.mean().item())
            for s in range(S):                                 # each site's trunk: local SGD from its dX
                copies[s].zero_grad()
                feats[s].backward(dx[s * B:(s + 1) * B])
                with torch.no_grad():
                    for p in copies[s].parameters():
                        p -= lr * p.grad
        ctx.reassemble()
        ctx.sync_status()
        with torch.no_grad():                                  # the trunk's copies are averaged
            for p, *ps in zip(trunk.parameters(), *[c.parameters() for c in copies]):
                p.copy_(torch.stack(ps).mean(0))
        records.append({"round": r + 1, "subnet_loss": sum(losses) / len(losses)})
    ctx.close()
    return records


def main():
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--rounds", type=int, default=30)
    ap.add_argument("--S", type=int, default=4)
    ap.add_argument("--K", type=int, default=10)
    ap.add_argument("--B", type=int, default=64)
    ap.add_argument("--lr", type=float, default=0.3)
    ap.add_argument("--precision", default="fp32", choices=["bf16", "fp32"])
    args = ap.parse_args()
    for rec in train(args.rounds, args.S, args.K, args.B, lr=args.lr, precision=args.precision):
        print(json.dumps(rec))


if __name__ == "__main__":
    main()
