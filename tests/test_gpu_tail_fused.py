"""The fused last-layer kernel of the default schedule (forward product, softmax cross-entropy,
dZ_L, the data gradient through the layer and the bias steps of the last two layers on CUDA
cores) against the CPU oracle and against the schedule that runs the same products on tensor
cores.  The two GPU schedules differ only in the order of fp32 sums inside the last layer, so
after one step from identical weights they must agree far more tightly than the bf16 gates
(loss 2e-2, parameters 5e-2) that hold against the oracle."""
import numpy as np
import pytest

from tests.util import assert_tiles_close, l2_rel, outlier_fraction, rel_err

pytestmark = pytest.mark.gpu

SEED = 0x211000625


def _mavg():
    import paper_2110_00625_b200 as m
    return m


def _cfg(**over):
    m = _mavg()
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(S=2048, gamma=0.05)
    cfg.update(over)
    return cfg


def _make(cfg, schedule, **kw):
    m = _mavg()
    x, y = m.workloads.make_dataset(cfg, S=cfg["S"])
    w1 = m.workloads.mlp_init(cfg["dims"])
    g = m.Mavg(w1, P=cfg["P"], K=cfg["K"], local_lr=cfg["gamma"], mu=cfg["mu"], B=cfg["B"],
               seed=SEED, objective=m.OBJ_MLP, dims=cfg["dims"], gemm_bf16=1, x=x, y=y, **kw)
    g.set_schedule(schedule)
    return g, x, y, w1


SHAPES = [
    dict(dims=[3072, 256, 128, 10], P=4, K=1, B=64),
    dict(dims=[512, 10], P=3, K=1, B=32),                  # one layer: no data gradient to take
    dict(dims=[256, 136, 32], P=5, K=1, B=16),             # 32 classes, one block per learner
    dict(dims=[3072, 2048, 10], P=2, K=1, B=48),           # wide last layer, ragged batch tiles
]


@pytest.mark.parametrize("shape", SHAPES)
def test_one_step_agrees_with_the_tensor_core_last_layer(shape):
    cfg = _cfg(**shape)
    a, *_ = _make(cfg, 0)
    b, *_ = _make(cfg, 2)
    a.local_steps(); b.local_steps()
    a.sync(); b.sync()
    la, lb = a.get_losses(), b.get_losses()
    assert np.abs(la - lb).max() <= 1e-5 * np.abs(lb).max()
    ra, rb = a.replicas.cpu().numpy()[:, :a.n], b.replicas.cpu().numpy()[:, :b.n]
    for j in range(cfg["P"]):
        # the step itself (the difference to the common starting point) in the 2-norm: a changed
        # summation order moves single bf16 roundings of dZ, nothing systematic
        w0 = a.w.cpu().numpy()
        assert l2_rel(ra[j] - w0, rb[j] - w0) <= 5e-3, j
        assert rel_err(ra[j], rb[j]) <= 1e-3, j
        assert_tiles_close(ra[j] - w0, rb[j] - w0, cfg["dims"], what=f"learner {j}")
    a.close(); b.close()


@pytest.mark.parametrize("dims,P,B", [([512, 10], 3, 32), ([960, 200, 10], 3, 48)])
def test_rounds_against_the_oracle(oracle, dims, P, B):
    cfg = _cfg(dims=dims, P=P, K=4, B=B)
    g, x, y, w1 = _make(cfg, 0)
    o = oracle.Mavg(w1, P=P, K=4, gamma=cfg["gamma"], mu=cfg["mu"], B=B, seed=SEED,
                    objective=oracle.OBJ_MLP, dims=dims, bf16=True, x=x, y=y, stride=g.stride)
    for r in range(3):
        lg = g.round(want_loss=True)
        lo, _ = o.run_round()
        assert abs(lg - lo) <= 2e-2 * abs(lo), (r, lg, lo)
        assert rel_err(g.w.cpu().numpy(), o.w) <= 5e-2, r
        assert l2_rel(g.v.cpu().numpy(), o.v) <= 5e-2, r
        assert outlier_fraction(g.v.cpu().numpy(), o.v, 5e-2) <= 0.15, r
        assert_tiles_close(g.v.cpu().numpy(), o.v, dims, l2_tol=1e-1, frac=1.0,
                           what=f"v after round {r + 1}")
    g.close()


def test_bias_steps_with_learner_momentum(oracle):
    # the bias steps of the last two layers are taken inside the fused kernel, with u^j if asked
    cfg = _cfg(dims=[960, 256, 10], P=3, K=3, B=32, gamma=0.01)
    g, x, y, w1 = _make(cfg, 0, learner_momentum=0.9)
    o = oracle.Mavg(w1, P=3, K=3, gamma=cfg["gamma"], mu=cfg["mu"], B=32, seed=SEED,
                    objective=oracle.OBJ_MLP, dims=cfg["dims"], bf16=True, x=x, y=y,
                    stride=g.stride, beta=0.9)
    for r in range(2):
        g.round(); o.run_round()
    g.sync()
    n = g.n
    nb = 256 + 10          # both bias vectors: [.. W1 | b1 | W2 | b2]
    b1 = slice(960 * 256, 960 * 256 + 256)
    b2 = slice(n - 10, n)
    gu, gw = g.u.cpu().numpy(), g.w.cpu().numpy()
    for j in range(3):
        for sl in (b1, b2):
            assert l2_rel(gu[j, sl], o.u[j, sl]) <= 5e-2, (j, sl)
    for sl in (b1, b2):
        assert rel_err(gw[sl], o.w[sl]) <= 5e-2
    assert nb == (b1.stop - b1.start) + (b2.stop - b2.start)
    g.close()
