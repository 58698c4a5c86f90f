"""GPU parity of the MLP learner level and of whole rounds against the CPU oracle, through the
C ABI.  Gates: index streams bit-exact; fp32 model: per-round loss within 1e-4 relative (plus
1e-6 absolute: logits of magnitude ~20 carry ~2e-6 of fp32 rounding, which is all that is left of
a loss that has fallen to 1e-4) and parameters within 1e-3; bf16-operand model: loss within 2e-2
relative, parameters within 5e-2."""
import numpy as np
import pytest
import torch

from tests.util import assert_tiles_close, l2_rel, outlier_fraction, rel_err

pytestmark = pytest.mark.gpu


def _mavg():
    import paper_2110_00625_b200 as m
    return m


def _pair(oracle, cfg, S=None, rounds=None, gemm_bf16=None, x_bf16=False, seed=0x211000625, **over):
    m = _mavg()
    c = dict(cfg)
    c.update(over)
    x, y = m.workloads.make_dataset(c, S=S or c["S"])
    w1 = m.workloads.mlp_init(c["dims"])
    mode = gemm_bf16 if gemm_bf16 is not None else (1 if c["bf16"] else 0)
    g = m.Mavg(w1, P=c["P"], K=c["K"], local_lr=c["gamma"], mu=c["mu"], block_lr=c["zeta"],
               B=c["B"], seed=seed, objective=m.OBJ_MLP, dims=c["dims"], gemm_bf16=mode, x=x, y=y,
               x_bf16=x_bf16)
    o = oracle.Mavg(w1, P=c["P"], K=c["K"], gamma=c["gamma"], mu=c["mu"], zeta=c["zeta"],
                    B=c["B"], seed=seed, objective=oracle.OBJ_MLP, dims=c["dims"],
                    bf16=bool(c["bf16"]), x=x, y=y, stride=g.stride)
    return g, o, c


def test_batch_indices_bit_exact(oracle):
    m = _mavg()
    for name in ("C1", "C2", "C4"):
        cfg = dict(m.workloads.CONFIGS[name])
        cfg["dims"] = [32, 16, 10]     # the index stream does not depend on the model
        cfg["bf16"] = False
        cfg["data"] = "gaussian_mixture"
        g, o, c = _pair(oracle, cfg)
        for (n, j, k) in [(1, 0, 1), (3, c["P"] - 1, c["K"]), (2, c["P"] // 2, 2)]:
            got = g.get_batch_indices(n, j, k)
            want = oracle.batch_indices(0x211000625, n, c["P"], j, k, c["S"], c["B"])
            assert np.array_equal(got, want)
        g.close()


def test_c1_fp32_full_trajectory(oracle):
    m = _mavg()
    g, o, c = _pair(oracle, m.workloads.CONFIGS["C1"])
    for r in range(c["rounds"]):
        lg = g.round(want_loss=True)
        lo, _ = o.run_round()
        assert abs(lg - lo) <= 1e-4 * abs(lo) + 1e-6, (r, lg, lo)
        assert rel_err(g.w.cpu().numpy(), o.w) <= 1e-3, r
        assert rel_err(g.v.cpu().numpy(), o.v) <= 1e-3, r
    g.sync()


def test_c1_first_local_steps_per_learner(oracle):
    # replicas after the K local steps of round 1, learner by learner, and every minibatch loss
    m = _mavg()
    g, o, c = _pair(oracle, m.workloads.CONFIGS["C1"])
    g.local_steps()
    losses_o, _ = o.local_steps()
    g.sync()
    gr = g.replicas.cpu().numpy()
    for j in range(c["P"]):
        assert rel_err(gr[j, :g.n], o.replicas[j, :g.n]) <= 1e-4
    assert np.abs(g.get_losses() - losses_o).max() <= 1e-4 * losses_o.max()


@pytest.mark.parametrize("dims,B,P,K", [([40, 24, 10], 7, 3, 2), ([33, 70, 65, 5], 20, 2, 3),
                                        ([16, 3], 1, 1, 1)])
def test_fp32_odd_shapes(oracle, dims, B, P, K):
    m = _mavg()
    cfg = dict(kind="mlp", dims=dims, bf16=False, P=P, K=K, B=B, gamma=0.05, mu=0.9, zeta=1.0,
               rounds=3, S=512, data="gaussian_mixture")
    g, o, c = _pair(oracle, cfg)
    for r in range(3):
        lg = g.round(want_loss=True)
        lo, _ = o.run_round()
        assert abs(lg - lo) <= 1e-4 * abs(lo) + 1e-6
        assert rel_err(g.w.cpu().numpy(), o.w) <= 1e-3


def test_p1_k1_mu0_is_plain_sgd_on_gpu(oracle):
    m = _mavg()
    cfg = dict(kind="mlp", dims=[32, 64, 10], bf16=False, P=1, K=1, B=32, gamma=0.05, mu=0.0,
               zeta=1.0, rounds=3, S=256, data="gaussian_mixture")
    g, o, c = _pair(oracle, cfg)
    x, y = m.workloads.make_dataset(c, S=256)
    w = o.w.copy()
    for r in range(1, 4):
        idx = oracle.batch_indices(0x211000625, r, 1, 0, 1, 256, 32)
        _, grad = oracle.mlp_loss_grad(c["dims"], w, x[idx], y[idx])
        w = (w.astype(np.float64) - np.float64(np.float32(0.05)) * grad).astype(np.float32)
        g.round()
    g.sync()
    assert rel_err(g.w.cpu().numpy(), w) <= 1e-4


@pytest.mark.parametrize("mode", [2, 1])
def test_bf16_small_cifar_shaped(oracle, mode):
    # CIFAR-shaped workload with narrower layers: several tiles per GEMM, bf16 operands.
    # mode 2 = CUDA-core arithmetic, mode 1 = tensor cores.
    m = _mavg()
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(dims=[3072, 256, 128, 10], P=4, K=4, B=64, S=2048, rounds=3)
    g, o, c = _pair(oracle, cfg, gemm_bf16=mode)
    for r in range(3):
        lg = g.round(want_loss=True)
        lo, _ = o.run_round()
        assert abs(lg - lo) <= 2e-2 * abs(lo), (r, lg, lo)
        assert rel_err(g.w.cpu().numpy(), o.w) <= 5e-2, r
        # free-running rounds: the drift of single bf16 roundings adds up over the steps, so v is
        # held in the 2-norm and, element by element, to a bounded share of outliers -- overall
        # and inside every output tile
        _check_update(g.v.cpu().numpy(), o.v, l2_tol=5e-2, frac=0.15)
        assert_tiles_close(g.v.cpu().numpy(), o.v, c["dims"], l2_tol=1e-1, frac=1.0,
                           what=f"v after round {r + 1}")
    g.sync()


def _check_update(got, want, l2_tol=2e-2, frac=0.02):
    """v and single steps are differences of weights, some 100 times smaller than the weights the
    5e-2 gate is stated for, and they feel the ReLU kink: when a pre-activation sits within
    rounding of zero the two sides may take different branches, which moves one sample's
    contribution (about 1/sqrt(B) of that weight row's update) and nothing else.  So: overall
    agreement in the 2-norm, and after a single step from identical weights all but a few rows
    (< 2 % of the elements) within 5e-2; over free-running rounds the flips compound, so only the
    2-norm is held there."""
    assert l2_rel(got, want) <= l2_tol
    if frac is not None:
        assert outlier_fraction(got, want, 5e-2) <= frac


def test_bf16_teacher_forced_step(oracle):
    # one local step from identical replicas, learner by learner: kernel error without drift
    m = _mavg()
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(dims=[3072, 256, 128, 10], P=3, K=1, B=128, S=2048)
    for mode in (2, 1):
        g, o, c = _pair(oracle, cfg, gemm_bf16=mode)
        g.local_steps()
        losses_o, _ = o.local_steps()
        g.sync()
        gr = g.replicas.cpu().numpy()
        for j in range(c["P"]):
            # compare the step taken, w_after - w_before, which is -gamma * grad
            step_g = gr[j, :g.n].astype(np.float64) - o.w
            step_o = o.replicas[j, :g.n].astype(np.float64) - o.w
            _check_update(step_g, step_o)
            assert_tiles_close(step_g, step_o, c["dims"], what=f"mode {mode} learner {j}")
        assert np.abs(g.get_losses() - losses_o).max() <= 2e-3 * losses_o.max()
        g.close()


def _tc_handle(cfg_over=None, K=3):
    m = _mavg()
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(dims=[3072, 256, 128, 10], P=4, K=K, B=64, S=2048)
    if cfg_over:
        cfg.update(cfg_over)
    x, y = m.workloads.make_dataset(cfg, S=cfg["S"])
    w1 = m.workloads.mlp_init(cfg["dims"])
    g = m.Mavg(w1, P=cfg["P"], K=cfg["K"], local_lr=cfg["gamma"], mu=cfg["mu"], B=cfg["B"],
               seed=m.workloads.BASE_SEED, objective=m.OBJ_MLP, dims=cfg["dims"], gemm_bf16=1,
               x=x, y=y, x_bf16=True)
    return g


def test_tc_path_is_deterministic_and_graph_equals_launch_by_launch():
    # two runs give the same bits (fixed reduction orders, no atomics on the value path), and the
    # replayed CUDA graph with its overlapped branches computes exactly what the serial,
    # launch-by-launch schedule (taken while per-launch profiling is on) computes
    outs = []
    for profiled in (False, False, True):
        g = _tc_handle()
        g.set_profiling(profiled)
        losses = [g.round(want_loss=True) for _ in range(3)]
        g.sync()
        outs.append((g.w.cpu().numpy(), g.v.cpu().numpy(), losses))
        if profiled:
            prof = g.get_profile()
            # rounds x steps launches: one launch takes the weight gradients of all three layers
            assert prof["wgrad_sgd_gemm"][1] == 3 * 3 and prof["meta_update"][1] == 3
        g.close()
    for other in outs[1:]:
        assert np.array_equal(outs[0][0], other[0]) and np.array_equal(outs[0][1], other[1])
        assert outs[0][2] == other[2]


def test_tc_hparam_change_and_repeated_local_steps():
    # K and the learning rate may change between rounds (the recorded graph is rebuilt)
    a = _tc_handle(K=2)
    a.round(); a.set_hparams(3, 0.02, 1.0, 0.5); a.round(); a.round()
    a.sync()
    b = _tc_handle(K=2)
    b.set_profiling(True)           # launch-by-launch reference for the same schedule of calls
    b.round(); b.set_hparams(3, 0.02, 1.0, 0.5); b.round(); b.round()
    b.sync()
    assert np.array_equal(a.w.cpu().numpy(), b.w.cpu().numpy())
    assert a.get_round() == 3
    # a second call without a meta-update in between starts from diverged replicas: it must take
    # the per-learner weight copies, not the shared copy of w~ -- compare graph and serial paths
    c = _tc_handle(K=2)
    c.local_steps(); c.local_steps(); c.sync()
    d = _tc_handle(K=2)
    d.set_profiling(True)
    d.local_steps(); d.local_steps(); d.sync()
    rc = c.replicas.cpu().numpy()[:, :c.n]      # columns n..stride are padding, never written
    assert np.array_equal(rc, d.replicas.cpu().numpy()[:, :d.n]) and np.isfinite(rc).all()
    assert not np.array_equal(rc[0], rc[1])
    # K lowered through set_hparams gives the same steps as a handle created with that K
    e = _tc_handle(K=2)
    e.local_steps(); e.sync()
    f = _tc_handle(K=4)
    f.set_hparams(2, 0.05, 1.0, 0.9)
    f.local_steps(); f.sync()
    assert np.array_equal(e.replicas.cpu().numpy()[:, :e.n], f.replicas.cpu().numpy()[:, :f.n])
    with pytest.raises(_mavg().MavgError):
        a.set_hparams(0, 0.05, 1.0, 0.9)
    with pytest.raises(_mavg().MavgError):
        a.set_hparams(2, 0.05, 1.0, 1.0)
    with pytest.raises(_mavg().MavgError):
        a.set_schedule(1)               # only MAVG_SCHED_GRAPH (0) and MAVG_SCHED_GRAPH_TC (2) exist


@pytest.mark.parametrize("dims,B,P,K", [
    ([64, 10], 16, 1, 2),                    # one layer, smallest batch
    ([72, 40, 24, 10], 48, 3, 2),            # widths that are multiples of 8 only; ragged tiles
    ([200, 136, 10], 32, 2, 3),              # in/out not multiples of 64 or 128
    ([1024, 384, 32], 256, 2, 2),            # largest batch, 32 classes, 3 row tiles
    ([4104, 128, 128, 128, 128, 8], 64, 2, 2),   # long contraction (65 slabs, ragged), 5 layers
    ([512, 1152, 16], 128, 5, 2),            # 9 row tiles x 5 learners
    # more 128-row tiles than SMs (two blocks per SM), ragged contraction (264, 648 = k x 64 + 8)
    # and a last row tile with 8 of 128 rows
    ([264, 648, 648, 10], 32, 25, 2),
    ([512, 2048, 1024, 10], 64, 10, 1),
])
def test_tc_shapes_teacher_forced(oracle, dims, B, P, K):
    # tensor-core path on shapes that exercise ragged tiles, contraction tails, batch tiling and
    # contraction splits; K local steps from identical replicas against the oracle, per learner
    m = _mavg()
    S = max(4 * P * B, 512)
    r = np.random.default_rng(17)
    x = r.standard_normal((S, dims[0])).astype(np.float32)
    y = r.integers(0, dims[-1], S).astype(np.int32)
    w1 = m.workloads.mlp_init(dims, seed=5)
    g = m.Mavg(w1, P=P, K=K, local_lr=0.05, mu=0.9, B=B, seed=99, objective=m.OBJ_MLP, dims=dims,
               gemm_bf16=1, x=x, y=y)
    o = oracle.Mavg(w1, P=P, K=K, gamma=0.05, mu=0.9, B=B, seed=99, objective=oracle.OBJ_MLP,
                    dims=dims, bf16=True, x=x, y=y, stride=g.stride)
    g.local_steps()
    losses_o, _ = o.local_steps()
    g.sync()
    gr = g.replicas.cpu().numpy()
    assert np.abs(g.get_losses() - losses_o).max() <= 2e-2 * losses_o.max()
    for j in range(P):
        step_g = gr[j, :g.n].astype(np.float64) - w1
        step_o = o.replicas[j, :g.n].astype(np.float64) - w1
        assert l2_rel(step_g, step_o) <= 3e-2, j
        # every 128 x 32 output tile of every layer and every bias vector on its own: a wrong
        # edge tile, contraction tail or split fix-up cannot hide in the norm of the whole step
        assert_tiles_close(step_g, step_o, dims, what=f"learner {j}")
    lg = g.round(want_loss=True)       # and a full round on top: finite, graph path
    assert np.isfinite(lg) and torch.isfinite(g.w).all()
    g.close()


def test_training_converges_and_block_momentum_accelerates():
    # end-to-end sanity on the CIFAR-shaped data: the training loss falls over the rounds, and
    # with the same number of rounds M-AVG (mu = 0.7) is ahead of K-AVG (mu = 0), the paper's
    # central claim (qualitative: no number of the paper is reproduced here)
    m = _mavg()
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(dims=[3072, 256, 256, 10], P=12, K=8, B=64, S=20000)
    x, y = m.workloads.make_dataset(cfg, S=cfg["S"])
    w1 = m.workloads.mlp_init(cfg["dims"])
    final = {}
    for mu in (0.0, 0.7):
        g = m.Mavg(w1, P=cfg["P"], K=cfg["K"], local_lr=0.02, mu=mu, B=cfg["B"],
                   seed=m.workloads.BASE_SEED, objective=m.OBJ_MLP, dims=cfg["dims"], gemm_bf16=1,
                   x=x, y=y, x_bf16=True)
        losses = [g.round(want_loss=True) for _ in range(60)]
        assert np.isfinite(losses).all()
        assert losses[-1] < 0.8 * losses[0]
        final[mu] = float(np.mean(losses[-5:]))
        g.close()
    assert final[0.7] < final[0.0]


def test_tc_mixed_call_sequences_keep_the_same_bits():
    # The default schedule keeps two bf16 copies of one layer's weights and alternates between
    # them from step to step, but only in its overlapped (graph) form.  Whatever mixture of graph
    # rounds, launch-by-launch rounds, repeated local steps, resumes and schedule changes a caller
    # makes, the result must be that of the same calls issued launch by launch.
    def run(profiled):
        g = _tc_handle(K=3)               # odd K: the current copy changes from round to round
        g.set_profiling(profiled)
        g.round()
        g.set_profiling(True); g.round(); g.set_profiling(profiled)
        g.local_steps(); g.local_steps(); g.meta_update()
        g.set_schedule(2); g.round(); g.set_schedule(0)
        g.round()
        g.set_round(g.get_round())        # resume: re-broadcast, next step starts from w~ again
        g.set_hparams(2, 0.02, 1.0, 0.9)
        g.round(); g.round()
        g.sync()
        out = (g.w.cpu().numpy(), g.v.cpu().numpy(), g.replicas.cpu().numpy()[:, :g.n])
        g.close()
        return out
    a, b = run(False), run(True)
    for x, y in zip(a, b):
        assert np.array_equal(x, y)


# Models whose first layer has more weight tiles than the one-launch-for-all-layers form takes
# (13 x 8 x 96 > 64 per SM): every layer's weight gradient is a launch of its own, and the launches
# of the hidden layers also form the NEXT step's forward product of their layer from the updated
# tiles (steps 1..K-1): one hidden layer, and two (the second one's launch reads the activations
# the first one's has just produced, and still writes its bf16 copy for the dgrad product); and one
# with more (learner, row tile) pairs than SMs (13 x 16 = 208), whose plan takes the first 148 pairs
# as whole rows and cuts the other 60 into two runs each (both kinds of work item in one launch).
FUSED_SHAPES = [[3072, 1024, 10], [3072, 1024, 512, 10], [3072, 2048, 10]]
FUSED_P, FUSED_B = 13, 16


def _fused_handle(dims, K, **kw):
    m = _mavg()
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(dims=dims, P=FUSED_P, K=K, B=FUSED_B, S=4096)
    x, y = m.workloads.make_dataset(cfg, S=cfg["S"])
    w1 = m.workloads.mlp_init(cfg["dims"])
    g = m.Mavg(w1, P=FUSED_P, K=K, local_lr=cfg["gamma"], mu=cfg["mu"], B=FUSED_B,
               seed=m.workloads.BASE_SEED, objective=m.OBJ_MLP, dims=dims, gemm_bf16=1,
               x=x, y=y, x_bf16=True, **kw)
    return g, cfg, x, y, w1


# Per-tile bounds: with 16 samples per batch a single ReLU decision that differs between the two
# roundings moves a whole weight row's gradient by 1/16 of itself, and three steps through two
# hidden layers collect more of those than the one-hidden-layer model (measured: the schedule that
# does not ride shows the same per-tile distances to the oracle, worst 0.033 against 0.034, and the
# two schedules are 0.004 apart); a wrong tile is off by ~1.
FUSED_TILE_TOL = {2: dict(l2_tol=2e-2, frac=0.05), 3: dict(l2_tol=5e-2, frac=0.15)}
FUSED_STEP_TOL = {2: 3e-2, 3: 5e-2}        # whole step of a learner; 5e-2 is the bf16 gate


@pytest.mark.parametrize("dims", FUSED_SHAPES)
@pytest.mark.parametrize("beta", [0.0, 0.9])
def test_forward_riding_on_the_weight_gradient_against_the_oracle(oracle, dims, beta):
    # K = 3 local steps from identical replicas: step 1 plain, steps 2 and 3 take their hidden
    # layers' forward products from the partial sums the step before left; per learner, per tile
    g, cfg, x, y, w1 = _fused_handle(dims, 3, learner_momentum=beta)
    plan = g.get_step_plan()
    assert plan["tensor_path"] == 1 and plan["wgrad_merged"] == 0
    assert plan["fwd_with_wgrad"] == len(dims) - 2
    assert all(16 <= r <= d // 32 for r, d in zip(plan["fwd_run_tiles"], dims))
    rows = [FUSED_P * -(-d // 128) for d in dims[1:-1]]
    assert all(0 <= wr <= n for wr, n in zip(plan["fwd_whole_rows"], rows))
    if dims[1] == 2048:
        assert 0 < plan["fwd_whole_rows"][0] < rows[0]
    xq = oracle.bf16_round(x)             # the GPU holds the dataset in bf16
    o = oracle.Mavg(w1, P=FUSED_P, K=3, gamma=cfg["gamma"], mu=cfg["mu"], B=FUSED_B,
                    seed=_mavg().workloads.BASE_SEED, objective=oracle.OBJ_MLP, dims=dims,
                    bf16=True, x=xq, y=y, stride=g.stride, beta=beta)
    g.local_steps()
    losses_o, _ = o.local_steps()
    g.sync()
    gr = g.replicas.cpu().numpy()
    assert np.abs(g.get_losses() - losses_o).max() <= 2e-2 * losses_o.max()
    for j in range(FUSED_P):
        step_g = gr[j, :g.n].astype(np.float64) - w1
        step_o = o.replicas[j, :g.n].astype(np.float64) - w1
        assert l2_rel(step_g, step_o) <= FUSED_STEP_TOL[len(dims) - 1], j
        assert_tiles_close(step_g, step_o, dims, what=f"learner {j}", **FUSED_TILE_TOL[len(dims) - 1])
    # the bf16 copy of layer 1 is valid again after the call's last step: a second call without a
    # meta-update in between starts from the learners' own weights and must agree as well
    g.local_steps()
    losses_o, _ = o.local_steps()
    g.sync()
    assert np.abs(g.get_losses() - losses_o).max() <= 2e-2 * losses_o.max()
    g.close()


@pytest.mark.parametrize("dims", FUSED_SHAPES)
def test_forward_riding_on_the_weight_gradient_graph_equals_launch_by_launch(dims):
    outs = []
    for profiled in (False, False, True):
        g, *_ = _fused_handle(dims, 4)
        g.set_profiling(profiled)
        losses = [g.round(want_loss=True) for _ in range(2)]
        g.local_steps(); g.local_steps(); g.meta_update()      # a call that starts from diverged replicas
        g.sync()
        outs.append((g.w.cpu().numpy(), g.v.cpu().numpy(), losses, g.get_losses()))
        g.close()
    # the same calls with the re-broadcast left to the next round's first step
    g, *_ = _fused_handle(dims, 4, defer_broadcast=True)
    losses = [g.round(want_loss=True) for _ in range(2)]
    g.local_steps(); g.local_steps(); g.meta_update()
    g.sync()
    outs.append((g.w.cpu().numpy(), g.v.cpu().numpy(), losses, g.get_losses()))
    g.close()
    for other in outs[1:]:
        assert np.array_equal(outs[0][0], other[0]) and np.array_equal(outs[0][1], other[1])
        assert outs[0][2] == other[2] and np.array_equal(outs[0][3], other[3])
    # and it computes what the plain-tiles schedule computes, to rounding order
    a, *_, a_w1 = _fused_handle(dims, 4)
    b, *_ = _fused_handle(dims, 4)
    b.set_schedule(2)
    la, lb = a.round(want_loss=True), b.round(want_loss=True)
    a.sync(); b.sync()
    assert abs(la - lb) <= 1e-3 * abs(lb)
    assert l2_rel(a.v.cpu().numpy(), b.v.cpu().numpy()) <= 2e-2
    ra, rb = a.replicas.cpu().numpy(), b.replicas.cpu().numpy()    # re-broadcast: all rows = w~
    assert_tiles_close(ra[0, :a.n].astype(np.float64) - a_w1, rb[0, :a.n].astype(np.float64) - a_w1,
                       dims, what="riding against plain tiles", l2_tol=2e-2, frac=0.05)
    a.close(); b.close()


def test_dense_first_step_forward_against_the_oracle(oracle):
    # At the first step of a round all learners hold w~ and the hidden layers' forward products
    # run as one dense product over the batch rows of all learners (128 x 256 tiles).  Shape with
    # a contraction tail (200 = 3 x 64 + 8), a ragged last row tile (520 = 4 x 128 + 8) and a last
    # batch tile that is three quarters full (39 x 64 = 9.75 x 256); K = 2, so that the second
    # step (per-learner weights, per-learner tiles) starts from what the dense step produced.
    m = _mavg()
    dims, B, P, K = [200, 1024, 520, 10], 64, 39, 2
    S = 4 * P * B
    r = np.random.default_rng(23)
    x = r.standard_normal((S, dims[0])).astype(np.float32)
    y = r.integers(0, dims[-1], S).astype(np.int32)
    w1 = m.workloads.mlp_init(dims, seed=6)
    g = m.Mavg(w1, P=P, K=K, local_lr=0.05, mu=0.9, B=B, seed=77, objective=m.OBJ_MLP, dims=dims,
               gemm_bf16=1, x=x, y=y)
    assert g.get_step_plan()["dense_first_step"] == [1, 2]
    o = oracle.Mavg(w1, P=P, K=K, gamma=0.05, mu=0.9, B=B, seed=77, objective=oracle.OBJ_MLP,
                    dims=dims, bf16=True, x=x, y=y, stride=g.stride)
    g.local_steps()
    losses_o, _ = o.local_steps()
    g.sync()
    gr = g.replicas.cpu().numpy()
    # the first step's losses depend on nothing but the dense products and the last layer
    assert np.abs(g.get_losses()[:, 0] - losses_o[:, 0]).max() <= 2e-3 * losses_o[:, 0].max()
    assert np.abs(g.get_losses() - losses_o).max() <= 2e-2 * losses_o.max()
    for j in (0, 3, 17, P - 2, P - 1):          # first and last learners of full and ragged tiles
        step_g = gr[j, :g.n].astype(np.float64) - w1
        step_o = o.replicas[j, :g.n].astype(np.float64) - w1
        assert l2_rel(step_g, step_o) <= 3e-2, j
        assert_tiles_close(step_g, step_o, dims, what=f"learner {j}")
    # the plain-tiles schedule forms the same first-step products per learner: same losses
    h = m.Mavg(w1, P=P, K=K, local_lr=0.05, mu=0.9, B=B, seed=77, objective=m.OBJ_MLP, dims=dims,
               gemm_bf16=1, x=x, y=y)
    h.set_schedule(2)
    h.local_steps()
    h.sync()
    assert np.abs(h.get_losses()[:, 0] - g.get_losses()[:, 0]).max() <= 1e-4 * losses_o[:, 0].max()
    g.close(); h.close()


@pytest.mark.parametrize("dims,B", [([3072, 1024, 10], 48), ([3072, 1024, 10], 128),
                                    ([3048, 1000, 10], 64)])
def test_forward_riding_other_batch_sizes_and_ragged_edges(oracle, dims, B):
    # B = 48: the forward accumulator's last 16 columns are read on their own (the batch is not a
    # multiple of 32); B = 128: two 64-wide contraction slabs, the bf16 tile on top of the dead
    # operand slabs, 256 columns of tensor memory.  Two local steps from identical replicas: the
    # second step's hidden activations come out of the first step's weight-gradient launch.
    # Against the plain-tiles schedule per tile (itself checked against the oracle at these batch
    # sizes by the shape tests above), and for B = 48 against the oracle directly.
    # 3048 x 1000: the last column tile has 8 of 32 columns and the last row tile 104 of 128 rows
    # (zero-filled operand tiles, clipped stores, rows beyond the layer not written).
    m = _mavg()
    P, K = 13, 2
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(dims=dims, P=P, K=K, B=B, S=4096)
    x, y = m.workloads.make_dataset(cfg, S=cfg["S"])
    w1 = m.workloads.mlp_init(dims)

    def run(schedule):
        g = m.Mavg(w1, P=P, K=K, local_lr=cfg["gamma"], mu=cfg["mu"], B=B,
                   seed=m.workloads.BASE_SEED, objective=m.OBJ_MLP, dims=dims, gemm_bf16=1,
                   x=x, y=y, x_bf16=True)
        assert g.get_step_plan()["fwd_with_wgrad"] == 1
        g.set_schedule(schedule)
        g.local_steps()
        g.sync()
        out = g.replicas.cpu().numpy()[:, :g.n].astype(np.float64), g.get_losses(), g.stride
        g.close()
        return out

    ra, la, stride = run(0)
    rb, lb, _ = run(2)
    assert np.abs(la - lb).max() <= 2e-3 * np.abs(lb).max()
    for j in (0, P // 2, P - 1):
        assert_tiles_close(ra[j] - w1, rb[j] - w1, dims, what=f"learner {j}, riding against plain")
    if B != 128:
        o = oracle.Mavg(w1, P=P, K=K, gamma=cfg["gamma"], mu=cfg["mu"], B=B,
                        seed=m.workloads.BASE_SEED, objective=oracle.OBJ_MLP, dims=dims, bf16=True,
                        x=oracle.bf16_round(x), y=y, stride=stride)
        losses_o, _ = o.local_steps()
        assert np.abs(la - losses_o).max() <= 2e-2 * losses_o.max()
        for j in (0, P - 1):
            step_o = o.replicas[j, :len(w1)].astype(np.float64) - w1
            assert l2_rel(ra[j] - w1, step_o) <= 3e-2, j
            assert_tiles_close(ra[j] - w1, step_o, dims, what=f"learner {j}")
