"""Writes the stored expected values under tests/golden/ that come from the CPU oracle.

Calls only oracle/.  Run from the repository root:  python tests/golden/make_golden.py
"""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))

from oracle import oracle as O  # noqa: E402

SEED = 0x211000625


def main():
    # minibatch index streams: first 16 indices for (round, learner, step) = (1, 0, 1) and
    # (3, P-1, K) on the shapes of the small MLP workload (P=4, K=4, S=4096) and of the
    # CIFAR-shaped one (P=8, K=8, S=50000).
    lines = ["# seed round P learner step S : first 16 sample indices (oracle/batch_indices)"]
    for (P, K, S) in [(4, 4, 4096), (8, 8, 50000), (32, 16, 50000)]:
        for (n, j, k) in [(1, 0, 1), (3, P - 1, K)]:
            idx = O.batch_indices(SEED, n, P, j, k, S, 16)
            lines.append(f"{SEED} {n} {P} {j} {k} {S} : " + " ".join(str(int(i)) for i in idx))
    with open(os.path.join(HERE, "batch_indices.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")
    # synthetic gradients: bit patterns of the first 8 elements for two (round, learner, step)
    lines = ["# seed round learner step sigma : fp32 bit patterns (hex) of elements 0..7 "
             "(oracle/pseudograd)"]
    sigma = 0.0316227766
    for (n, j, k) in [(1, 0, 1), (2, 15, 64)]:
        g = O.pseudograd(SEED, n, j, k, 0, 8, sigma)
        lines.append(f"{SEED} {n} {j} {k} {sigma} : " +
                     " ".join(f"{int(b):08x}" for b in g.view("uint32")))
    with open(os.path.join(HERE, "pseudograd_bits.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
