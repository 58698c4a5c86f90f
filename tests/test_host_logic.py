"""CPU-only checks of the product side: the shared library loads without a GPU and exports every
symbol the header declares, argument checking happens before any device work, and the workload
generators are seeded and shaped as documented."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2110_00625_b200 import build as B
    B.build()
    import paper_2110_00625_b200 as m
    return m.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "mavg.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mavg_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    import paper_2110_00625_b200 as m
    names = _declared()
    assert "mavg_create" in names and "mavg_round" in names and len(names) >= 15
    for name in names:
        assert hasattr(lib, name), name
    assert sorted(m.EXPORTS) == names


def _cfg(**kw):
    from paper_2110_00625_b200.binding import make_config
    base = dict(P=4, K=4, local_lr=0.05, mu=0.9, n=100)
    base.update(kw)
    return make_config(**base)


@pytest.mark.parametrize("kw,status", [
    (dict(P=0), 1), (dict(K=0), 1), (dict(mu=1.0), 1), (dict(mu=-0.1), 1),
    (dict(mu=float("nan")), 1), (dict(local_lr=float("inf")), 1), (dict(block_lr=float("nan")), 1),
    (dict(n=0), 1), (dict(objective=7), 1),
    (dict(objective=1, learner_momentum=1.0), 1), (dict(objective=1, learner_momentum=-0.5), 1),
    (dict(learner_momentum=0.5), 1),      # no learner level to apply it to
    (dict(objective=1, sigma=-1.0), 1),
    (dict(objective=2, dims=[4, 3], n=15, B=0, x_ptr=256, y_ptr=256, n_samples=10), 1),
    (dict(objective=2, dims=[4, 3], n=14, B=2, x_ptr=256, y_ptr=256, n_samples=10), 1),
    (dict(objective=2, dims=[4, 3], n=15, B=2, x_ptr=0, y_ptr=256, n_samples=10), 2),
    (dict(objective=2, dims=[4, 3], n=15, B=2, x_ptr=256, y_ptr=256, n_samples=2), 1),
    (dict(objective=2, dims=[4, 3], n=15, B=2, x_ptr=264, y_ptr=256, n_samples=10), 2),
    (dict(objective=2, dims=[4, 3], n=15, B=2, x_ptr=256, y_ptr=256, n_samples=10, gemm_bf16=3), 1),
    (dict(l2_keep=2), 1),                 # a flag: 0 or 1
    # widths that are not multiples of 8 are outside the tensor-core path
    (dict(objective=2, dims=[4, 3], n=15, B=2, x_ptr=256, y_ptr=256, n_samples=10, gemm_bf16=1), 4),
])
def test_bad_configs_are_rejected_on_the_host(lib, kw, status):
    cfg = _cfg(**kw)
    nb = C.c_size_t(123)
    assert lib.mavg_workspace_bytes(C.byref(cfg), C.byref(nb)) == status
    assert nb.value == 0
    assert len(lib.mavg_last_error(None)) > 0


def test_workspace_size_and_buffer_checks(lib):
    from paper_2110_00625_b200.binding import Buffers
    cfg = _cfg()
    nb = C.c_size_t()
    assert lib.mavg_workspace_bytes(C.byref(cfg), C.byref(nb)) == 0 and nb.value >= 256
    assert lib.mavg_workspace_bytes(None, C.byref(nb)) == 1
    assert lib.mavg_workspace_bytes(C.byref(cfg), None) == 1
    h = C.c_void_p(1)
    # NULL / misaligned / undersized buffers: rejected before any device call
    for buf, st in [
        (Buffers(0, 100, 256, 256, 256, 1 << 20), 2),
        (Buffers(256, 100, 256, 256, 260, 1 << 20), 2),
        (Buffers(256, 98, 256, 256, 256, 1 << 20), 2),
        (Buffers(256, 96, 256, 256, 256, 1 << 20), 2),
        (Buffers(256, 100, 256, 256, 256, 16), 2),
        (Buffers(264, 100, 256, 256, 256, 1 << 20), 2),
        (Buffers(256, 100, 256, 256, 256, 1 << 20, 264), 2),   # misaligned learner_u
    ]:
        assert lib.mavg_create(C.byref(cfg), C.byref(buf), C.byref(h)) == st
        assert h.value is None
        h = C.c_void_p(1)
    # learner momentum without its buffer
    cfg_m = _cfg(objective=1, learner_momentum=0.5)
    assert lib.mavg_create(C.byref(cfg_m), C.byref(Buffers(256, 100, 256, 256, 256, 1 << 20)),
                           C.byref(h)) == 2
    assert b"learner_u" in lib.mavg_last_error(None)
    h = C.c_void_p(1)
    assert lib.mavg_create(C.byref(cfg), None, C.byref(h)) == 1
    assert lib.mavg_create(C.byref(cfg), C.byref(Buffers(256, 100, 256, 256, 256, 1 << 20)), None) == 1
    # NULL handles
    assert lib.mavg_destroy(None) == 0
    assert lib.mavg_round(None, None) == 1
    assert lib.mavg_sync(None) == 1
    assert lib.mavg_set_wait_limit(None, 100) == 1
    assert lib.mavg_selftest_wait(None) == 1
    assert lib.mavg_set_schedule(None, 0) == 1
    assert lib.mavg_get_step_plan(None, (C.c_int32 * 20)()) == 1


def test_create_without_a_device_fails_cleanly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    from paper_2110_00625_b200.binding import Buffers
    cfg = _cfg()
    h = C.c_void_p()
    st = lib.mavg_create(C.byref(cfg), C.byref(Buffers(256, 100, 256, 256, 256, 1 << 20)), C.byref(h))
    assert st == 5 and h.value is None
    assert b"CUDA" in lib.mavg_last_error(None) or b"device" in lib.mavg_last_error(None)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    from paper_2110_00625_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "HERE", str(tmp_path))
    with pytest.raises(OSError, match="no fallback"):
        binding.load_library()


def test_workloads_are_seeded_and_shaped():
    from paper_2110_00625_b200 import workloads as W
    x, y = W.gaussian_mixture()
    x2, y2 = W.gaussian_mixture()
    assert x.shape == (4096, 32) and y.shape == (4096,) and x.dtype == np.float32
    assert np.array_equal(x, x2) and np.array_equal(y, y2)
    assert set(np.unique(y)) == set(range(10))
    xs, ys = W.cifar_shaped(S=2000)
    assert xs.shape == (2000, 3072) and abs(xs.std() - 1.0) < 0.01 and abs(xs.mean()) < 0.01
    assert ys.min() >= 0 and ys.max() <= 9 and len(np.unique(ys)) >= 5
    for name, n in [("C2", 1_841_162), ("C4", 14_706_698), ("C1", 2762)]:
        assert W.mlp_param_count(W.CONFIGS[name]["dims"]) == n
    w = W.mlp_init([32, 64, 10])
    assert w.size == 2762 and not w[2048:2112].any() and abs(w[:2048].std() - 0.25) < 0.02
    reps = W.perturbed_replicas(np.zeros(10000, np.float32), 3, 0.1, update=0, stride=10016)
    assert reps.shape == (3, 10016) and abs(reps[:, :10000].std() - 0.1) < 0.005
    assert not reps[:, 10000:].any()
    assert not np.array_equal(reps[0], reps[1])
    assert not np.array_equal(reps, W.perturbed_replicas(np.zeros(10000, np.float32), 3, 0.1, update=1, stride=10016))
