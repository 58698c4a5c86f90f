"""GPU parity of learner-level momentum (momentum SGD inside each learner, the variant the paper
names after Eq. 2 and in its conclusion: u <- beta u - gamma g, w <- w + u) against the CPU
oracle, through the C ABI, for every kernel that takes the local step: the K-fused
pseudo-gradient pass, the CUDA-core MLP kernels and the tensor-core weight-gradient kernel with the
bias steps of the GEMM tails.  Both readings of what happens to u^j at a round boundary (kept, or
reset when the learners restart from the global model) are covered.  Tolerances as for the plain
local step: fp32 1e-5 (pseudo-gradients) / 1e-3 (fp32 MLP), bf16 operands 5e-2."""
import numpy as np
import pytest

from tests.util import l2_rel, rel_err

pytestmark = pytest.mark.gpu

SEED = 0x211000625


def _mavg():
    import paper_2110_00625_b200 as m
    return m


@pytest.mark.parametrize("reset", [False, True])
@pytest.mark.parametrize("K,defer", [(1, False), (5, True), (2100, False)])
def test_pseudograd_rounds(oracle, K, defer, reset):
    # n with a ragged tail; K = 2100 exceeds the number of steps one launch fuses
    m = _mavg()
    n = 40_003 if K > 100 else 300_007
    w1 = m.workloads.global_model(n, seed=5)
    kw = dict(P=3, K=K, mu=0.9, seed=9)
    g = m.Mavg(w1, local_lr=0.05, objective=m.OBJ_PSEUDOGRAD, sigma=0.03, defer_broadcast=defer,
               learner_momentum=0.8, learner_momentum_reset=reset, **kw)
    o = oracle.Mavg(w1, gamma=0.05, objective=oracle.OBJ_PSEUDOGRAD, sigma=0.03, stride=g.stride,
                    beta=0.8, reset_u=reset, **kw)
    for r in range(3):
        g.local_steps()
        o.local_steps()
        g.sync()
        gr, gu = g.replicas.cpu().numpy(), g.u.cpu().numpy()
        for j in range(3):
            assert rel_err(gr[j, :n], o.replicas[j, :n]) <= 1e-5, (r, j)
            assert rel_err(gu[j, :n], o.u[j, :n]) <= 1e-5, (r, j)
        g.meta_update()
        o.meta_update()
    g.sync()
    assert rel_err(g.w.cpu().numpy(), o.w) <= 1e-5
    assert rel_err(g.v.cpu().numpy(), o.v) <= 1e-5
    g.close()


def test_beta_zero_with_buffer_equals_plain_sgd():
    # a handle that owns u^j but runs with beta = 0 takes Algorithm 1's plain step, bit for bit,
    # and switching the momentum on later changes the result
    m = _mavg()
    n = 50_001
    w1 = m.workloads.global_model(n, seed=2)
    kw = dict(P=4, K=3, local_lr=0.05, mu=0.9, seed=4, objective=m.OBJ_PSEUDOGRAD, sigma=0.03)
    a = m.Mavg(w1, **kw)
    b = m.Mavg(w1, with_learner_u=True, **kw)
    for _ in range(2):
        a.round()
        b.round()
    a.sync(); b.sync()
    assert np.array_equal(a.w.cpu().numpy(), b.w.cpu().numpy())
    b.set_learner_momentum(0.9, reset=True)
    a.round(); b.round()
    a.sync(); b.sync()
    assert not np.array_equal(a.w.cpu().numpy(), b.w.cpu().numpy())
    with pytest.raises(Exception, match="learner_u"):
        a.set_learner_momentum(0.5)
    a.close(); b.close()


def _mlp_pair(oracle, cfg, mode, beta, reset, defer=False):
    m = _mavg()
    x, y = m.workloads.make_dataset(cfg, S=cfg["S"])
    w1 = m.workloads.mlp_init(cfg["dims"])
    g = m.Mavg(w1, P=cfg["P"], K=cfg["K"], local_lr=cfg["gamma"], mu=cfg["mu"], B=cfg["B"],
               seed=SEED, objective=m.OBJ_MLP, dims=cfg["dims"], gemm_bf16=mode, x=x, y=y,
               learner_momentum=beta, learner_momentum_reset=reset, defer_broadcast=defer)
    o = oracle.Mavg(w1, P=cfg["P"], K=cfg["K"], gamma=cfg["gamma"], mu=cfg["mu"], B=cfg["B"],
                    seed=SEED, objective=oracle.OBJ_MLP, dims=cfg["dims"], bf16=mode != 0, x=x,
                    y=y, stride=g.stride, beta=beta, reset_u=reset)
    return g, o


@pytest.mark.parametrize("reset", [False, True])
def test_fp32_mlp_trajectory(oracle, reset):
    m = _mavg()
    cfg = dict(m.workloads.CONFIGS["C1"])
    cfg.update(gamma=0.02)
    g, o = _mlp_pair(oracle, cfg, 0, 0.9, reset)
    for r in range(5):
        lg = g.round(want_loss=True)
        lo, _ = o.run_round()
        assert abs(lg - lo) <= 1e-4 * abs(lo) + 1e-6, (r, lg, lo)
        assert rel_err(g.w.cpu().numpy(), o.w) <= 1e-3, r
        assert rel_err(g.v.cpu().numpy(), o.v) <= 1e-3, r
    gu = g.u.cpu().numpy()
    for j in range(cfg["P"]):
        assert rel_err(gu[j, :g.n], o.u[j, :g.n]) <= 1e-3
    g.close()


@pytest.mark.parametrize("mode,reset,defer", [(2, False, False), (1, False, True), (1, True, False)])
def test_bf16_mlp_rounds(oracle, mode, reset, defer):
    # CIFAR-shaped workload with narrower layers; mode 2 = CUDA cores, mode 1 = tensor cores
    m = _mavg()
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(dims=[3072, 256, 128, 10], P=3, K=4, B=64, S=2048, gamma=0.01)
    g, o = _mlp_pair(oracle, cfg, mode, 0.9, reset, defer)
    for r in range(3):
        lg = g.round(want_loss=True)
        lo, _ = o.run_round()
        assert abs(lg - lo) <= 2e-2 * abs(lo), (r, lg, lo)
        assert rel_err(g.w.cpu().numpy(), o.w) <= 5e-2, r
        assert l2_rel(g.v.cpu().numpy(), o.v) <= 5e-2, r
    gu = g.u.cpu().numpy()
    for j in range(cfg["P"]):
        assert l2_rel(gu[j, :g.n], o.u[j, :g.n]) <= 5e-2
    g.close()


def test_tensor_core_first_step_per_learner(oracle):
    # one step from identical replicas, ragged widths (edge tiles of the u and master maps)
    m = _mavg()
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(dims=[3072, 200, 72, 10], P=2, K=2, B=48, S=1024, gamma=0.01)
    g, o = _mlp_pair(oracle, cfg, 1, 0.7, False)
    g.local_steps()
    o.local_steps()
    g.sync()
    gr, gu = g.replicas.cpu().numpy(), g.u.cpu().numpy()
    for j in range(cfg["P"]):
        assert rel_err(gr[j, :g.n], o.replicas[j, :g.n]) <= 5e-2
        assert l2_rel(gu[j, :g.n], o.u[j, :g.n]) <= 2e-2
    g.close()
