"""ctypes binding of libmavg.so: argument marshalling only.

The functions of `Lib` carry the C names of include/mavg.h.  `Mavg` is a thin convenience class
that owns the torch tensors handed to the library (PyTorch is used for device memory and the
stream, nothing else) and forwards each method to the C entry point of the same name.  There is
no CPU fallback: if the shared library is missing, loading raises.
"""
import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
OBJ_NONE, OBJ_PSEUDOGRAD, OBJ_MLP = 0, 1, 2
SCHED_GRAPH, SCHED_GRAPH_TC = 0, 2
X_F32, X_BF16 = 0, 1
MAX_LAYERS = 8

STATUS = {0: "MAVG_OK", 1: "MAVG_ERR_INVALID_ARG", 2: "MAVG_ERR_BAD_BUFFER", 3: "MAVG_ERR_STATE",
          4: "MAVG_ERR_UNSUPPORTED", 5: "MAVG_ERR_CUDA", 6: "MAVG_ERR_TIMEOUT"}

EXPORTS = ["mavg_workspace_bytes", "mavg_create", "mavg_local_steps", "mavg_meta_update",
           "mavg_materialize_replicas", "mavg_round", "mavg_round_host", "mavg_set_hparams",
           "mavg_set_learner_momentum", "mavg_get_batch_indices",
           "mavg_get_losses", "mavg_get_round", "mavg_set_round", "mavg_get_launch_count",
           "mavg_get_step_plan", "mavg_set_profiling", "mavg_set_schedule", "mavg_get_profile", "mavg_sync",
           "mavg_set_wait_limit", "mavg_selftest_wait", "mavg_cache_release", "mavg_last_error",
           "mavg_batch_indices_noalloc", "mavg_destroy"]
KERNEL_CLASSES = ["meta_update", "broadcast", "pseudograd_steps", "batch_gather", "fwd_gemm",
                  "loss", "dgrad_gemm", "wgrad_sgd_gemm", "aux"]


class Config(C.Structure):
    _fields_ = [
        ("P", C.c_int32), ("K", C.c_int32), ("B", C.c_int32),
        ("local_lr", C.c_float), ("block_lr", C.c_float), ("mu", C.c_float),
        ("seed", C.c_uint64),
        ("objective", C.c_int32),
        ("n", C.c_int64),
        ("n_layers", C.c_int32), ("dims", C.c_int32 * (MAX_LAYERS + 1)), ("gemm_bf16", C.c_int32),
        ("pseudo_grad_sigma", C.c_float),
        ("x", C.c_void_p), ("x_dtype", C.c_int32), ("y", C.c_void_p), ("n_samples", C.c_int64),
        ("stream", C.c_void_p),
        ("defer_broadcast", C.c_int32),
        ("learner_momentum", C.c_float), ("learner_momentum_reset", C.c_int32),
        ("l2_keep", C.c_int32),
    ]


class Buffers(C.Structure):
    _fields_ = [
        ("replicas", C.c_void_p), ("replica_stride", C.c_int64),
        ("global_w", C.c_void_p), ("momentum", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
        ("learner_u", C.c_void_p),
    ]


class MavgError(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"{STATUS.get(status, status)}: {message}")
        self.status = status


def library_path():
    return os.path.join(HERE, "libmavg.so")


_lib = None


def load_library():
    """Loads libmavg.so and declares the prototypes.  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise OSError(f"{path} is missing: build it with `python -m paper_2110_00625_b200.build`; "
                      "there is no fallback path")
    L = C.CDLL(path)
    H = C.c_void_p
    L.mavg_workspace_bytes.argtypes = [C.POINTER(Config), C.POINTER(C.c_size_t)]
    L.mavg_create.argtypes = [C.POINTER(Config), C.POINTER(Buffers), C.POINTER(H)]
    L.mavg_local_steps.argtypes = [H]
    L.mavg_meta_update.argtypes = [H]
    L.mavg_round.argtypes = [H, C.POINTER(C.c_float)]
    L.mavg_round_host.argtypes = [H, C.c_void_p, C.c_void_p, C.POINTER(C.c_float)]
    L.mavg_set_hparams.argtypes = [H, C.c_int32, C.c_float, C.c_float, C.c_float]
    L.mavg_set_learner_momentum.argtypes = [H, C.c_float, C.c_int32]
    L.mavg_get_batch_indices.argtypes = [H, C.c_int64, C.c_int32, C.c_int32, C.c_void_p]
    L.mavg_get_losses.argtypes = [H, C.c_void_p]
    L.mavg_get_round.argtypes = [H, C.POINTER(C.c_int64)]
    L.mavg_set_round.argtypes = [H, C.c_int64]
    L.mavg_get_launch_count.argtypes = [H, C.POINTER(C.c_int64)]
    L.mavg_get_step_plan.argtypes = [H, C.POINTER(C.c_int32)]
    L.mavg_set_profiling.argtypes = [H, C.c_int32]
    L.mavg_set_schedule.argtypes = [H, C.c_int32]
    L.mavg_get_profile.argtypes = [H, C.c_void_p, C.c_void_p, C.c_int32]
    L.mavg_batch_indices_noalloc.argtypes = [C.c_uint64, C.c_int64, C.c_int32, C.c_int32,
                                             C.c_int32, C.c_int64, C.c_int32, C.c_void_p,
                                             C.c_void_p]
    L.mavg_materialize_replicas.argtypes = [H]
    L.mavg_sync.argtypes = [H]
    L.mavg_set_wait_limit.argtypes = [H, C.c_int32]
    L.mavg_selftest_wait.argtypes = [H]
    L.mavg_cache_release.argtypes = [H]
    L.mavg_last_error.argtypes = [H]
    L.mavg_last_error.restype = C.c_char_p
    L.mavg_destroy.argtypes = [H]
    for name in EXPORTS:
        if name != "mavg_last_error":
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


def make_config(P, K, local_lr, mu, block_lr=1.0, B=1, seed=0, objective=OBJ_NONE, n=0, dims=None,
                gemm_bf16=0, sigma=0.0, x_ptr=0, x_dtype=X_F32, y_ptr=0, n_samples=0, stream=0,
                defer_broadcast=False, learner_momentum=0.0, learner_momentum_reset=False,
                l2_keep=False):
    cfg = Config()
    cfg.P, cfg.K, cfg.B = P, K, B
    cfg.local_lr, cfg.block_lr, cfg.mu = local_lr, block_lr, mu
    cfg.seed = seed
    cfg.objective = objective
    cfg.n = n
    if dims is not None:
        cfg.n_layers = len(dims) - 1
        for i, d in enumerate(dims[:MAX_LAYERS + 1]):
            cfg.dims[i] = d
    cfg.gemm_bf16 = gemm_bf16
    cfg.pseudo_grad_sigma = sigma
    cfg.x, cfg.x_dtype, cfg.y, cfg.n_samples = x_ptr, x_dtype, y_ptr, n_samples
    cfg.stream = stream
    cfg.defer_broadcast = 1 if defer_broadcast else 0
    cfg.learner_momentum = learner_momentum
    cfg.learner_momentum_reset = 1 if learner_momentum_reset else 0
    cfg.l2_keep = int(l2_keep)
    return cfg


def batch_indices_noalloc(seed, round_, P, learner, step, n_samples, B, stream=0):
    """mavg_batch_indices_noalloc: the B sample indices of (round, learner, step) computed on the
    current CUDA device without a handle, a workspace or any allocation by the library."""
    import numpy as np
    L = load_library()
    out = np.empty(max(B, 1), dtype=np.int32)
    st = L.mavg_batch_indices_noalloc(seed, round_, P, learner, step, n_samples, B, stream,
                                      out.ctypes.data)
    if st != 0:
        raise MavgError(st, L.mavg_last_error(None).decode())
    return out[:B]


class Mavg:
    """Owns the device tensors of one M-AVG problem and forwards to the C ABI.

    w1: 1-D float32 tensor or array with the initial global model w~_1.  x, y: the dataset
    (MLP objective), moved to the device; x is stored as bf16 there when x_bf16 is set.
    """

    def __init__(self, w1, P, K, local_lr, mu, block_lr=1.0, B=1, seed=0, objective=OBJ_NONE,
                 dims=None, gemm_bf16=0, sigma=0.0, x=None, y=None, x_bf16=False, stride=None,
                 device="cuda:0", stream=None, defer_broadcast=False, learner_momentum=0.0,
                 learner_momentum_reset=False, with_learner_u=None, l2_keep=False):
        import torch
        self._torch = torch
        self.lib = load_library()
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        w1 = torch.as_tensor(w1, dtype=torch.float32).reshape(-1)
        n = w1.numel()
        self.n, self.P, self.K, self.B = n, P, K, B
        self.stride = int(stride) if stride else (n + 31) // 32 * 32
        self.w = w1.to(self.device).contiguous().clone()
        self.v = torch.empty(n, dtype=torch.float32, device=self.device)
        self.replicas = torch.empty((P, self.stride), dtype=torch.float32, device=self.device)
        self.x = self.y = None
        x_ptr = y_ptr = n_samples = 0
        if objective == OBJ_MLP:
            self.x = torch.as_tensor(x).to(self.device,
                                           torch.bfloat16 if x_bf16 else torch.float32).contiguous()
            self.y = torch.as_tensor(y).to(self.device, torch.int32).contiguous()
            x_ptr, y_ptr, n_samples = self.x.data_ptr(), self.y.data_ptr(), self.y.numel()
        self.stream = stream
        sptr = stream.cuda_stream if stream is not None else torch.cuda.current_stream().cuda_stream
        self.cfg = make_config(P, K, local_lr, mu, block_lr, B, seed, objective, n, dims, gemm_bf16,
                               sigma, x_ptr, X_BF16 if x_bf16 else X_F32, y_ptr, n_samples, sptr,
                               defer_broadcast, learner_momentum, learner_momentum_reset,
                               l2_keep)
        # learner momentum buffers u^j [P, stride]: allocated when beta != 0 or on request (a
        # handle that switches the momentum on later with set_learner_momentum)
        if with_learner_u is None:
            with_learner_u = learner_momentum != 0.0
        self.u = (torch.empty((P, self.stride), dtype=torch.float32, device=self.device)
                  if with_learner_u else None)
        nbytes = C.c_size_t()
        st = self.lib.mavg_workspace_bytes(C.byref(self.cfg), C.byref(nbytes))
        if st != 0:
            raise MavgError(st, self.lib.mavg_last_error(None).decode())
        self.workspace = torch.empty(max(nbytes.value, 256), dtype=torch.uint8, device=self.device)
        self.buf = Buffers(self.replicas.data_ptr(), self.stride, self.w.data_ptr(),
                           self.v.data_ptr(), self.workspace.data_ptr(), self.workspace.numel(),
                           self.u.data_ptr() if self.u is not None else None)
        self.handle = C.c_void_p()
        st = self.lib.mavg_create(C.byref(self.cfg), C.byref(self.buf), C.byref(self.handle))
        if st != 0:
            raise MavgError(st, self.lib.mavg_last_error(None).decode())

    def _check(self, st):
        if st != 0:
            raise MavgError(st, self.lib.mavg_last_error(self.handle).decode())

    def local_steps(self):
        self._check(self.lib.mavg_local_steps(self.handle))

    def meta_update(self):
        self._check(self.lib.mavg_meta_update(self.handle))

    def materialize_replicas(self):
        self._check(self.lib.mavg_materialize_replicas(self.handle))

    def round(self, want_loss=False):
        if want_loss:
            loss = C.c_float()
            self._check(self.lib.mavg_round(self.handle, C.byref(loss)))
            return loss.value
        self._check(self.lib.mavg_round(self.handle, None))
        return None

    def round_host(self, w_host, v_host):
        """w_host, v_host: pinned or pageable CPU float32 tensors of n elements, updated in place."""
        loss = C.c_float()
        self._check(self.lib.mavg_round_host(self.handle, w_host.data_ptr(), v_host.data_ptr(),
                                             C.byref(loss)))
        return loss.value

    def set_hparams(self, K, local_lr, block_lr, mu):
        self._check(self.lib.mavg_set_hparams(self.handle, K, local_lr, block_lr, mu))
        self.K = K

    def set_learner_momentum(self, beta, reset=False):
        self._check(self.lib.mavg_set_learner_momentum(self.handle, beta, int(bool(reset))))

    def get_batch_indices(self, round_, learner, step):
        import numpy as np
        out = np.empty(self.B, dtype=np.int32)
        self._check(self.lib.mavg_get_batch_indices(self.handle, round_, learner, step,
                                                    out.ctypes.data))
        return out

    def get_losses(self):
        import numpy as np
        out = np.empty((self.P, self.K), dtype=np.float32)
        self._check(self.lib.mavg_get_losses(self.handle, out.ctypes.data))
        return out

    def get_round(self):
        r = C.c_int64()
        self._check(self.lib.mavg_get_round(self.handle, C.byref(r)))
        return r.value

    def set_round(self, r):
        self._check(self.lib.mavg_set_round(self.handle, r))

    def launch_count(self):
        r = C.c_int64()
        self.lib.mavg_get_launch_count(self.handle, C.byref(r))
        return r.value

    def get_step_plan(self):
        """How a local step is laid out in launches: tensor_path, wgrad_merged, fwd_with_wgrad
        (layers 1..m whose next-step forward product rides on their weight-gradient launch) and
        fwd_run_tiles (per such layer, column tiles per partial sum), fwd_whole_rows (per such
        layer, the (learner, row tile) pairs taken as one run, without partial sums), dense_first_step (hidden
        layers whose first-step forward is one dense product over all learners' batch rows)."""
        out = (C.c_int32 * (4 + 2 * MAX_LAYERS))()
        self._check(self.lib.mavg_get_step_plan(self.handle, out))
        return {"tensor_path": out[0], "wgrad_merged": out[1], "fwd_with_wgrad": out[2],
                "fwd_run_tiles": list(out[3:3 + out[2]]),
                "fwd_whole_rows": list(out[4 + MAX_LAYERS:4 + MAX_LAYERS + out[2]]),
                "dense_first_step": [l + 1 for l in range(MAX_LAYERS) if out[3 + MAX_LAYERS] >> l & 1]}

    def set_profiling(self, on):
        self._check(self.lib.mavg_set_profiling(self.handle, int(bool(on))))

    def set_schedule(self, mode):
        """0: CUDA graph with the fused last layer and cluster-split forward where they pay
        (default); 2: CUDA graph with every product as plain tensor-core tiles."""
        self._check(self.lib.mavg_set_schedule(self.handle, int(mode)))

    def get_profile(self, reset=True):
        """{kernel class: (milliseconds, launches)} since the last reset."""
        ms = (C.c_float * len(KERNEL_CLASSES))()
        cnt = (C.c_int64 * len(KERNEL_CLASSES))()
        self._check(self.lib.mavg_get_profile(self.handle, ms, cnt, int(bool(reset))))
        return {k: (ms[i], cnt[i]) for i, k in enumerate(KERNEL_CLASSES)}

    def sync(self):
        self._check(self.lib.mavg_sync(self.handle))

    def set_wait_limit(self, microseconds):
        self._check(self.lib.mavg_set_wait_limit(self.handle, int(microseconds)))

    def selftest_wait(self):
        """Launches the kernel whose wait cannot be satisfied (see mavg_selftest_wait)."""
        self._check(self.lib.mavg_selftest_wait(self.handle))

    def l2_release(self):
        """Wait for the stream and give up the L2 lines kept for the masters (cold-cache timing)."""
        self._check(self.lib.mavg_cache_release(self.handle))

    def close(self):
        if getattr(self, "handle", None) is not None and self.handle:
            self.lib.mavg_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
