"""Seeded synthetic inputs for the M-AVG workloads.

This module only produces input arrays (datasets, labels, initial weights, perturbed replicas) and
the table of workload shapes.  It contains none of the method's arithmetic and is the one module
that both the CUDA path's callers and the CPU checker's callers may use, so that both sides are
fed identical bytes.  numpy only.

The image-classification benchmarks the paper trains on (Section 4) are replaced by synthetic data
that keeps only their shapes: 3x32x32 inputs, 10 classes, 50 000 samples; parameter vectors of
11.2 M and 25.6 M elements.
"""
import numpy as np

BASE_SEED = 0x211000625

# name -> workload description.  gamma/rounds are this build's choices where the source of the
# workload list is silent.
CONFIGS = {
    "C1": dict(kind="mlp", dims=[32, 64, 10], bf16=False, P=4, K=4, B=32, gamma=0.05, mu=0.9,
               zeta=1.0, rounds=10, S=4096, data="gaussian_mixture"),
    "C2": dict(kind="mlp", dims=[3072, 512, 512, 10], bf16=True, P=8, K=8, B=128, gamma=0.05,
               mu=0.9, zeta=1.0, rounds=20, S=50000, data="cifar_shaped"),
    "C3": dict(kind="meta", n=11_200_000, P=[4, 16, 64], mu=[0.0, 0.9], zeta=1.0, updates=5,
               w_std=0.05, perturb_std=0.1),
    "C4": dict(kind="mlp", dims=[3072, 2048, 2048, 2048, 10], bf16=True, P=32, K=16, B=64,
               gamma=0.05, mu=0.9, zeta=1.0, rounds=20, S=50000, data="cifar_shaped"),
    "C5": dict(kind="pseudograd", n=25_600_000, P=16, K=[1, 4, 16, 64], gamma=0.05,
               mu=[0.0, 0.9], zeta=1.0, sigma=float(np.sqrt(1e-3)), w_std=0.05),
}


def _rng(seed, *tags):
    return np.random.Generator(np.random.Philox(key=np.random.SeedSequence([seed, *tags])
                                                .generate_state(2, dtype=np.uint64)))


def gaussian_mixture(seed=BASE_SEED, S=4096, d=32, classes=10):
    """S points in R^d from `classes` unit-variance clusters whose means are N(0, 4 I)."""
    r = _rng(seed, 101)
    means = 2.0 * r.standard_normal((classes, d))
    y = r.integers(0, classes, size=S).astype(np.int32)
    x = (means[y] + r.standard_normal((S, d))).astype(np.float32)
    return x, y


def cifar_shaped(seed=BASE_SEED, S=50000, d=3072, classes=10, teacher_hidden=256):
    """N(0,1) inputs of dimension d with labels from a fixed random ReLU teacher d-256-classes
    (weights N(0, 1/fan_in); label = argmax logit, ties to the lowest class)."""
    r = _rng(seed, 202)
    x = r.standard_normal((S, d), dtype=np.float32)
    t1 = (r.standard_normal((d, teacher_hidden)) / np.sqrt(d)).astype(np.float32)
    t2 = (r.standard_normal((teacher_hidden, classes)) / np.sqrt(teacher_hidden)).astype(
        np.float32)
    y = np.empty(S, dtype=np.int32)
    for lo in range(0, S, 8192):
        h = np.maximum(x[lo:lo + 8192] @ t1, 0.0)
        y[lo:lo + 8192] = np.argmax(h @ t2, axis=1).astype(np.int32)
    return x, y


def mlp_param_count(dims):
    return int(sum(dims[l + 1] * dims[l] + dims[l + 1] for l in range(len(dims) - 1)))


def mlp_init(dims, seed=BASE_SEED):
    """Flat [W_1 (out x in, row-major), b_1, W_2, b_2, ...]; W ~ N(0, 2/fan_in), b = 0."""
    r = _rng(seed, 303)
    parts = []
    for l in range(len(dims) - 1):
        fan_in, out = dims[l], dims[l + 1]
        parts.append((r.standard_normal(out * fan_in) * np.sqrt(2.0 / fan_in)).astype(np.float32))
        parts.append(np.zeros(out, dtype=np.float32))
    return np.concatenate(parts)


def global_model(n, std=0.05, seed=BASE_SEED):
    r = _rng(seed, 404)
    return (std * r.standard_normal(n, dtype=np.float32)).astype(np.float32)


def perturbed_replicas(w, P, std, update, seed=BASE_SEED, stride=None):
    """[P, stride] array with row j = w + N(0, std^2) noise; a fresh draw per `update`."""
    n = w.size
    stride = stride or n
    out = np.zeros((P, stride), dtype=np.float32)
    for j in range(P):
        r = _rng(seed, 505, update, j)
        out[j, :n] = w + std * r.standard_normal(n, dtype=np.float32)
    return out


def make_dataset(cfg, seed=BASE_SEED, S=None):
    S = S or cfg["S"]
    if cfg["data"] == "gaussian_mixture":
        return gaussian_mixture(seed, S=S, d=cfg["dims"][0], classes=cfg["dims"][-1])
    return cifar_shaped(seed, S=S, d=cfg["dims"][0], classes=cfg["dims"][-1])
