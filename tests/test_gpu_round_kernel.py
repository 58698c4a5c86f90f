"""The whole-round kernel (all K local steps of a round in one persistent launch, blocks handing
work to each other through counters) against the per-launch schedule and against the CPU oracle.
Both schedules run the same tiles with the same arithmetic, so their results must agree bit for
bit; the oracle comparison uses the bf16 gates (loss 2e-2, parameters 5e-2)."""
import numpy as np
import pytest

from tests.util import l2_rel, rel_err

pytestmark = pytest.mark.gpu

SEED = 0x211000625


def _mavg():
    import paper_2110_00625_b200 as m
    return m


def _make(cfg, round_kernel, defer=False):
    m = _mavg()
    x, y = m.workloads.make_dataset(cfg, S=cfg["S"])
    w1 = m.workloads.mlp_init(cfg["dims"])
    g = m.Mavg(w1, P=cfg["P"], K=cfg["K"], local_lr=cfg["gamma"], mu=cfg["mu"], B=cfg["B"],
               seed=SEED, objective=m.OBJ_MLP, dims=cfg["dims"], gemm_bf16=1, x=x, y=y,
               x_bf16=cfg.get("x_bf16", False), defer_broadcast=defer)
    g.set_schedule(1 if round_kernel else 2)
    return g, x, y, w1


def _cfg(**over):
    m = _mavg()
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(S=2048, gamma=0.05)
    cfg.update(over)
    return cfg


# Shapes the whole-round kernel covers (no product of theirs splits its contraction over blocks).
SHAPES = [
    dict(dims=[3072, 256, 128, 10], P=64, K=4, B=64),           # three layers, many learners
    dict(dims=[3072, 512, 512, 10], P=8, K=3, B=128),           # the benchmark's shape
    dict(dims=[960, 200, 10], P=3, K=5, B=48),                  # two layers, ragged widths and batch
    dict(dims=[512, 384, 264, 136, 10], P=5, K=3, B=32, x_bf16=True),   # four layers
    dict(dims=[512, 256, 128, 10], P=1, K=1, B=16),             # degenerate: one learner, one step
    dict(dims=[256, 128, 32], P=150, K=2, B=16),                # more learners than SMs, 32 classes
]
SMALL = dict(dims=[3072, 256, 128, 10], P=64, K=4, B=64)


def _local_step_launches(g):
    g.sync()
    before = g.launch_count()
    g.local_steps()
    g.sync()
    return g.launch_count() - before


@pytest.mark.parametrize("shape", SHAPES)
def test_same_bits_as_the_per_launch_schedule(shape):
    cfg = _cfg(**shape)
    a, *_ = _make(cfg, True)
    b, *_ = _make(cfg, False)
    for r in range(3):
        la = a.round(want_loss=True)
        lb = b.round(want_loss=True)
        assert la == lb, r
        assert np.array_equal(a.get_losses(), b.get_losses()), r
    a.sync(); b.sync()
    assert np.array_equal(a.w.cpu().numpy(), b.w.cpu().numpy())
    assert np.array_equal(a.v.cpu().numpy(), b.v.cpu().numpy())
    # the learners' own models after local steps only; one launch on the one side, many on the other
    assert _local_step_launches(a) == 1
    assert _local_step_launches(b) > cfg["K"]
    assert np.array_equal(a.replicas.cpu().numpy()[:, :a.n], b.replicas.cpu().numpy()[:, :b.n])
    # local steps twice in a row: the second call starts from the learners' models, not from w~
    a.local_steps(); b.local_steps()
    a.sync(); b.sync()
    assert np.array_equal(a.replicas.cpu().numpy()[:, :a.n], b.replicas.cpu().numpy()[:, :b.n])
    a.close(); b.close()


def test_shapes_that_split_a_contraction_keep_the_per_launch_schedule():
    # few learners and a long contraction: the forward product is split over blocks, which the
    # whole-round kernel does not do; the handle falls back to the per-launch graph by itself
    cfg = _cfg(dims=[3072, 256, 128, 10], P=4, K=4, B=64)
    g, *_ = _make(cfg, True, defer=True)
    g.round()
    assert _local_step_launches(g) > cfg["K"]
    g.close()


@pytest.mark.parametrize("defer", [False, True])
def test_rounds_against_the_oracle(oracle, defer):
    cfg = _cfg(dims=[3072, 256, 128, 10], P=16, K=4, B=64)
    cfg.update(dims=[960, 256, 128, 10])
    g, x, y, w1 = _make(cfg, True, defer=defer)
    o = oracle.Mavg(w1, P=cfg["P"], K=cfg["K"], gamma=cfg["gamma"], mu=cfg["mu"], B=cfg["B"],
                    seed=SEED, objective=oracle.OBJ_MLP, dims=cfg["dims"], bf16=True, x=x, y=y,
                    stride=g.stride)
    for r in range(3):
        lg = g.round(want_loss=True)
        lo, _ = o.run_round()
        assert abs(lg - lo) <= 2e-2 * abs(lo), (r, lg, lo)
        assert rel_err(g.w.cpu().numpy(), o.w) <= 5e-2, r
        assert l2_rel(g.v.cpu().numpy(), o.v) <= 5e-2, r
    assert _local_step_launches(g) == 1
    g.close()


def test_hyper_parameter_change_between_rounds():
    # K and the learning rate may change between rounds; the kernel takes them per launch
    cfg = _cfg(K=6, **{k: v for k, v in SMALL.items() if k != "K"})
    a, *_ = _make(cfg, True)
    b, *_ = _make(cfg, False)
    for K, lr in [(6, 0.05), (2, 0.02), (5, 0.01)]:
        a.set_hparams(K, lr, 1.0, 0.9)
        b.set_hparams(K, lr, 1.0, 0.9)
        assert a.round(want_loss=True) == b.round(want_loss=True)
    assert np.array_equal(a.w.cpu().numpy(), b.w.cpu().numpy())
    a.close(); b.close()
