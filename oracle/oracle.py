"""numpy-facing wrapper of the CPU oracle (oracle/mavg_oracle.cpp).

TEST INFRASTRUCTURE: only tests, the smoke check and the benchmark's CPU-baseline leg may import
this module.  It imports nothing from the CUDA package and the CUDA package imports nothing from
here.

What pins each oracle function (tests/test_oracle_pins.py):
  mix64 / stream values   published SplitMix64 outputs for seed 1234567
  shard bounds, indices   cover [0,S) disjointly; every index inside its shard; uniformity
  pseudograd (Irwin-Hall) integer lane sums recomputed with Python big ints; mean, variance,
                          kurtosis 2.7 of the four-lane sum; range
  bf16 rounding           torch's float32 -> bfloat16 conversion on every upper half-word
  mlp_loss_grad           torch.autograd in float64 (fp32 mode); central differences; ln(C) at
                          zero weights; bf16 mode: an independent float64 restatement that applies
                          torch's bf16 conversion to W, activations and dZ where the products read
                          them (leaving any one rounding out is detected), bias gradient from the
                          unrounded dZ
  meta_update             mu = 0 is K-AVG (plain mean); identical replicas; the auxiliary
                          sequence z_n; unrolled momentum sum by brute force; first round
  local_steps + round     closed-form two-term recurrence on a diagonal quadratic; P=K=1, mu=0 is
                          plain SGD; K=1, mu=0 is synchronous SGD; d = -gamma G_n (Eq. 2)
  free-running MLP trajectories (losses, weights after many rounds): parity unpinned -- the paper
                          prints no value for any workload; they rest on the pins above.
"""
import ctypes as C
import os

import numpy as np

from . import build as _build

OBJ_PSEUDOGRAD, OBJ_MLP, OBJ_QUADRATIC = 1, 2, 3
TAG_BATCH, TAG_PSEUDOGRAD = 1, 2


class _Problem(C.Structure):
    _fields_ = [
        ("P", C.c_int32), ("K", C.c_int32), ("B", C.c_int32),
        ("gamma", C.c_float), ("zeta", C.c_float), ("mu", C.c_float),
        ("seed", C.c_uint64),
        ("objective", C.c_int32),
        ("n", C.c_int64), ("stride", C.c_int64),
        ("n_layers", C.c_int32), ("dims", C.c_int32 * 9), ("bf16", C.c_int32),
        ("x", C.c_void_p), ("y", C.c_void_p), ("S", C.c_int64),
        ("sigma", C.c_float),
        ("quad_a", C.c_void_p),
        ("threads", C.c_int32),
        ("beta", C.c_float), ("reset_u", C.c_int32), ("u", C.c_void_p),
    ]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        L = _lib
        L.orc_mix64.restype = C.c_uint64
        L.orc_mix64.argtypes = [C.c_uint64]
        L.orc_splitmix64_output.restype = C.c_uint64
        L.orc_splitmix64_output.argtypes = [C.c_uint64, C.c_uint64]
        L.orc_stream_key.restype = C.c_uint64
        L.orc_stream_key.argtypes = [C.c_uint64] * 5
        L.orc_bf16_round.restype = C.c_float
        L.orc_bf16_round.argtypes = [C.c_float]
        L.orc_bf16_round_array.argtypes = [C.c_void_p, C.c_void_p, C.c_int64]
        L.orc_shard_bounds.argtypes = [C.c_int64, C.c_int32, C.c_int32,
                                       C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
        L.orc_batch_indices.argtypes = [C.c_uint64, C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                        C.c_int64, C.c_int32, C.c_void_p]
        L.orc_pseudograd.argtypes = [C.c_uint64, C.c_int64, C.c_int32, C.c_int32, C.c_int64,
                                     C.c_int64, C.c_float, C.c_void_p]
        L.orc_mlp_param_count.restype = C.c_int64
        L.orc_mlp_param_count.argtypes = [C.c_int32, C.c_void_p]
        L.orc_mlp_loss_grad.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_int32, C.c_int32, C.c_void_p,
                                        C.POINTER(C.c_double)]
        L.orc_local_steps.argtypes = [C.POINTER(_Problem), C.c_int64, C.c_void_p, C.c_void_p,
                                      C.c_void_p]
        L.orc_meta_update.argtypes = [C.c_int32, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_float, C.c_float]
        L.orc_init.argtypes = [C.c_int32, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p,
                               C.c_void_p]
        L.orc_round.argtypes = [C.POINTER(_Problem), C.c_int64, C.c_void_p, C.c_void_p,
                                C.c_void_p, C.POINTER(C.c_double), C.c_void_p]
        L.orc_max_threads.restype = C.c_int32
    return _lib


def _ptr(a):
    return a.ctypes.data_as(C.c_void_p)


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def mix64(z):
    return int(lib().orc_mix64(z & 0xFFFFFFFFFFFFFFFF))


def splitmix64_output(state0, i):
    return int(lib().orc_splitmix64_output(state0, i))


def stream_key(seed, tag, n, j, k):
    return int(lib().orc_stream_key(seed, tag, n, j, k))


def bf16_round(a):
    a = _f32(a)
    out = np.empty_like(a)
    lib().orc_bf16_round_array(_ptr(a), _ptr(out), a.size)
    return out


def shard_bounds(S, P, j):
    lo, hi = C.c_int64(), C.c_int64()
    lib().orc_shard_bounds(S, P, j, C.byref(lo), C.byref(hi))
    return lo.value, hi.value


def batch_indices(seed, n, P, j, k, S, B):
    out = np.empty(B, dtype=np.int32)
    lib().orc_batch_indices(seed, n, P, j, k, S, B, _ptr(out))
    return out


def pseudograd(seed, n, j, k, i0, count, sigma):
    out = np.empty(count, dtype=np.float32)
    lib().orc_pseudograd(seed, n, j, k, i0, count, sigma, _ptr(out))
    return out


def mlp_param_count(dims):
    d = np.asarray(dims, dtype=np.int32)
    return int(lib().orc_mlp_param_count(len(dims) - 1, _ptr(d)))


def mlp_loss_grad(dims, w, X, y, bf16=False):
    d = np.asarray(dims, dtype=np.int32)
    w = _f32(w)
    X = _f32(X)
    y = np.ascontiguousarray(y, dtype=np.int32)
    assert w.size == mlp_param_count(dims) and X.shape == (y.size, dims[0])
    grad = np.empty_like(w)
    loss = C.c_double()
    lib().orc_mlp_loss_grad(len(dims) - 1, _ptr(d), _ptr(w), _ptr(X), _ptr(y), y.size,
                            int(bool(bf16)), _ptr(grad), C.byref(loss))
    return loss.value, grad


class Mavg:
    """Algorithm 1 held as plain numpy state: w (global model), v (block momentum),
    replicas [P, stride]."""

    def __init__(self, w1, P, K, gamma, mu, zeta=1.0, B=1, seed=0, objective=OBJ_PSEUDOGRAD,
                 dims=None, bf16=False, x=None, y=None, sigma=0.0, quad_a=None, stride=None,
                 threads=0, beta=0.0, reset_u=False):
        self.w = _f32(w1).copy()
        n = self.w.size
        self.stride = int(stride) if stride else n
        self.v = np.empty(n, dtype=np.float32)
        self.replicas = np.zeros((P, self.stride), dtype=np.float32)
        self._keep = []
        pb = _Problem()
        pb.P, pb.K, pb.B = P, K, B
        pb.gamma, pb.zeta, pb.mu = gamma, zeta, mu
        pb.seed = seed
        pb.objective = objective
        pb.n, pb.stride = n, self.stride
        if objective == OBJ_MLP:
            pb.n_layers = len(dims) - 1
            for i, d in enumerate(dims):
                pb.dims[i] = d
            assert mlp_param_count(dims) == n
            pb.bf16 = int(bool(bf16))
            x = _f32(x)
            y = np.ascontiguousarray(y, dtype=np.int32)
            assert x.shape == (y.size, dims[0])
            self._keep += [x, y]
            pb.x, pb.y, pb.S = x.ctypes.data, y.ctypes.data, y.size
        if objective == OBJ_QUADRATIC:
            a = _f32(quad_a)
            assert a.size == n
            self._keep.append(a)
            pb.quad_a = a.ctypes.data
        pb.sigma = sigma
        pb.threads = threads
        # learner-level momentum buffers u^j (all zero at the start, like v)
        self.u = np.zeros((P, self.stride), dtype=np.float32)
        pb.beta, pb.reset_u, pb.u = beta, int(bool(reset_u)), self.u.ctypes.data
        self.pb = pb
        self.round = 0
        lib().orc_init(P, n, self.stride, _ptr(self.replicas), _ptr(self.w), _ptr(self.v))

    @property
    def n(self):
        return self.w.size

    def set_hparams(self, K=None, gamma=None, zeta=None, mu=None):
        if K is not None:
            self.pb.K = K
        if gamma is not None:
            self.pb.gamma = gamma
        if zeta is not None:
            self.pb.zeta = zeta
        if mu is not None:
            self.pb.mu = mu

    def local_steps(self, want_G=False):
        """K local SGD steps of round self.round + 1 on every replica.  Returns (losses [P,K], G)."""
        losses = np.zeros((self.pb.P, self.pb.K), dtype=np.float64)
        G = np.zeros(self.n, dtype=np.float64) if want_G else None
        lib().orc_local_steps(C.byref(self.pb), self.round + 1, _ptr(self.replicas),
                              _ptr(losses), _ptr(G) if want_G else None)
        return losses, G

    def meta_update(self):
        lib().orc_meta_update(self.pb.P, self.n, self.stride, _ptr(self.replicas), _ptr(self.w),
                              _ptr(self.v), self.pb.mu, self.pb.zeta)
        self.round += 1

    def run_round(self, want_G=False):
        losses, G = self.local_steps(want_G)
        self.meta_update()
        return float(losses.mean()), G


def max_threads():
    return int(lib().orc_max_threads())
