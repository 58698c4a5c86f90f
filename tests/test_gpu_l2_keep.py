"""The L2 set-aside for the learners' masters (tensor-core MLP handles whose P master copies fit in
half the L2): it may change speed only.  Rounds with lines released in between give the same bits
as rounds without, and closing the handle puts the context's limit back."""
import numpy as np
import pytest

pytestmark = pytest.mark.gpu

SEED = 0x211000625


def _handle(m, cfg, x, y, w1):
    return m.Mavg(w1, P=cfg["P"], K=cfg["K"], local_lr=cfg["gamma"], mu=cfg["mu"], B=cfg["B"],
                  seed=SEED, objective=m.OBJ_MLP, dims=cfg["dims"], gemm_bf16=1, x=x, y=y)


def _limit():
    cudart = pytest.importorskip("cuda.cudart")
    err, val = cudart.cudaDeviceGetLimit(cudart.cudaLimit.cudaLimitPersistingL2CacheSize)
    assert int(err) == 0
    return int(val)


def test_release_keeps_the_bits_and_close_restores_the_limit():
    import torch
    import paper_2110_00625_b200 as m
    torch.zeros(1, device="cuda")          # the context exists before the limit is read
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(dims=[3072, 256, 128, 10], P=3, K=3, B=64, S=2048)
    x, y = m.workloads.make_dataset(cfg, S=cfg["S"])
    w1 = m.workloads.mlp_init(cfg["dims"])
    before = _limit()
    a = _handle(m, cfg, x, y, w1)
    assert _limit() >= before
    b = _handle(m, cfg, x, y, w1)
    for _ in range(3):
        a.round()
        b.round()
        b.l2_release()
    a.sync(); b.sync()
    assert np.array_equal(a.w.cpu().numpy(), b.w.cpu().numpy())
    assert np.array_equal(a.v.cpu().numpy(), b.v.cpu().numpy())
    b.close()
    a.close()
    assert _limit() == before


def test_release_is_a_no_op_without_a_learner_level():
    import paper_2110_00625_b200 as m
    w1 = m.workloads.global_model(10_001, seed=1)
    g = m.Mavg(w1, P=4, K=1, local_lr=0.05, mu=0.9, seed=3, objective=m.OBJ_NONE)
    g.l2_release()
    g.meta_update()
    g.sync()
    g.close()
