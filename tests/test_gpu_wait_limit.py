"""Failure detection of the engine itself: a device-side wait that can never be satisfied must run
out after the handle's limit, the kernel must return by itself, mavg_sync must report
MAVG_ERR_TIMEOUT exactly once, and the same handle must then compute what an untouched handle
computes (and what the CPU oracle computes).  The wait is made to run out by a barrier nobody
arrives on -- nothing traps, faults or spins without a limit."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

SEED = 0x211000625


def _mavg():
    import paper_2110_00625_b200 as m
    return m


def _pair():
    m = _mavg()
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(dims=[3072, 256, 128, 10], P=3, K=2, B=64, S=2048)
    x, y = m.workloads.make_dataset(cfg, S=cfg["S"])
    w1 = m.workloads.mlp_init(cfg["dims"])
    mk = lambda: m.Mavg(w1, P=cfg["P"], K=cfg["K"], local_lr=cfg["gamma"], mu=cfg["mu"], B=cfg["B"],
                        seed=SEED, objective=m.OBJ_MLP, dims=cfg["dims"], gemm_bf16=1, x=x, y=y)
    return m, cfg, x, y, w1, mk


def test_wait_runs_out_is_reported_once_and_the_handle_stays_usable(oracle):
    m, cfg, x, y, w1, mk = _pair()
    a, b = mk(), mk()
    o = oracle.Mavg(w1, P=cfg["P"], K=cfg["K"], gamma=cfg["gamma"], mu=cfg["mu"], B=cfg["B"],
                    seed=SEED, objective=oracle.OBJ_MLP, dims=cfg["dims"], bf16=True, x=x, y=y,
                    stride=a.stride)
    a.round(); b.round(); o.run_round()
    a.sync()
    a.set_wait_limit(30_000)                       # 30 ms instead of the default 2 s
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    a.selftest_wait()
    t1.record()
    with pytest.raises(m.MavgError) as err:
        a.sync()
    assert err.value.status == 6                   # MAVG_ERR_TIMEOUT
    ms = t0.elapsed_time(t1)
    assert 25.0 <= ms <= 1000.0, ms                # the kernel returned by itself, after the limit
    a.sync()                                       # the record was cleared: no second report
    a.set_wait_limit(0)                            # back to the default
    for _ in range(2):
        la, lb = a.round(want_loss=True), b.round(want_loss=True)
        lo, _ = o.run_round()
        assert la == lb
        assert abs(la - lo) <= 2e-2 * abs(lo)
    a.sync(); b.sync()
    assert torch.equal(a.w, b.w) and torch.equal(a.v, b.v)
    a.close(); b.close()


def test_wait_limit_arguments():
    m, cfg, x, y, w1, mk = _pair()
    g = mk()
    with pytest.raises(m.MavgError):
        g.set_wait_limit(-1)
    g.set_wait_limit(500_000)                      # half a second: no wait of a round comes near it
    g.round()
    g.sync()
    g.set_wait_limit(0)
    g.close()
