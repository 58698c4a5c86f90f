"""Block momentum against the number of learners, and against the averaging interval K, on the
CIFAR-shaped synthetic workload.

A synthetic stand-in for the paper's Section 4 study (validation accuracy for P in {6, 12, 24, 48}
and mu from 0 to 0.9 on an image benchmark): the same sweep on teacher-labelled Gaussian inputs,
with the total number of processed samples N*P*B*K held fixed as in the paper's tuning guideline
for "more processors".  The second table varies K in {1, 4, 16, 64} at mu = 0 (K-AVG) and at one
positive mu, again at a fixed sample budget: the quantity Lemma 5 is about (the best K with
momentum is not larger than the best K without).  Training runs entirely in the CUDA library;
this script only evaluates the global model on held-out samples with plain torch and prints the
tables.

    python -m paper_2110_00625_b200.examples.mu_sweep [--sweep mu|K|both] [--budget SAMPLES]
"""
import argparse

import numpy as np
import torch

import paper_2110_00625_b200 as m


def accuracy(dims, w, x, y):
    off, a = 0, x
    L = len(dims) - 1
    for l in range(L):
        W = w[off:off + dims[l + 1] * dims[l]].view(dims[l + 1], dims[l]); off += W.numel()
        b = w[off:off + dims[l + 1]]; off += dims[l + 1]
        a = torch.nn.functional.linear(a, W, b)
        if l < L - 1:
            a = torch.relu(a)
    return (a.argmax(dim=1) == y).float().mean().item()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--budget", type=int, default=1_500_000, help="samples processed per run")
    ap.add_argument("--width", type=int, default=512)
    ap.add_argument("--K", type=int, default=8)
    ap.add_argument("--B", type=int, default=64)
    ap.add_argument("--lr", type=float, default=0.02)
    ap.add_argument("--sweep", default="both", choices=["mu", "K", "both"])
    ap.add_argument("--P", type=int, default=12, help="learners of the K sweep")
    ap.add_argument("--mu", type=float, default=0.7, help="the positive momentum of the K sweep")
    args = ap.parse_args()
    W = m.workloads
    dims = [3072, args.width, args.width, 10]
    x, y = W.cifar_shaped(S=60000)
    xtr, ytr, xva, yva = x[:50000], y[:50000], x[50000:], y[50000:]
    dev = torch.device("cuda:0")
    xv = torch.from_numpy(xva).to(dev)
    yv = torch.from_numpy(yva).to(dev).long()
    w1 = W.mlp_init(dims)

    def train(P, K, mu):
        rounds = max(1, args.budget // (P * K * args.B))
        g = m.Mavg(w1, P=P, K=K, local_lr=args.lr, mu=mu, B=args.B, seed=W.BASE_SEED,
                   objective=m.OBJ_MLP, dims=dims, gemm_bf16=1, x=xtr, y=ytr, x_bf16=True)
        loss = float("nan")
        for r in range(rounds):
            if r == rounds - 1:
                loss = g.round(want_loss=True)
            else:
                g.round()
        g.sync()
        acc = accuracy(dims, g.w, xv, yv) if np.isfinite(loss) else float("nan")
        g.close()
        return rounds, f"{acc:.3f}/{loss:.3f}"

    if args.sweep in ("mu", "both"):
        mus = [0.0, 0.3, 0.5, 0.7, 0.9]
        print(f"model {dims}, K={args.K}, B={args.B}, lr={args.lr}, {args.budget} samples per run")
        print("P    rounds  " + "  ".join(f"mu={mu:<4}" for mu in mus) +
              "   (validation accuracy / last loss)")
        for P in (6, 12, 24, 48):
            cells = [train(P, args.K, mu) for mu in mus]
            print(f"{P:<4d} {cells[0][0]:<7d} " + "  ".join(c for _, c in cells))
    if args.sweep in ("K", "both"):
        mus = [0.0, args.mu]
        print(f"model {dims}, P={args.P}, B={args.B}, lr={args.lr}, {args.budget} samples per run")
        print("K    rounds  " + "  ".join(f"mu={mu:<4}" for mu in mus) +
              "   (validation accuracy / last loss)")
        for K in (1, 4, 16, 64):
            cells = [train(args.P, K, mu) for mu in mus]
            print(f"{K:<4d} {cells[0][0]:<7d} " + "  ".join(c for _, c in cells))


if __name__ == "__main__":
    main()
