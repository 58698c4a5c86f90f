"""Deferred re-broadcast (Algorithm 1, "set w^j = w~" folded into the next round's first local
step): the engine must reach bit-identical (w~, v, replicas after the local steps, losses) with
and without it, on every objective, and agree with the CPU oracle."""
import numpy as np
import pytest
import torch

from tests.util import rel_err

pytestmark = pytest.mark.gpu


def _mavg():
    import paper_2110_00625_b200 as m
    return m


def _same(a, b):
    return torch.equal(a, b)


@pytest.mark.parametrize("n,P,K", [(5, 3, 2), (100_003, 4, 3), (1_200_000, 16, 4)])
def test_pseudograd_deferred_equals_eager(oracle, n, P, K):
    m = _mavg()
    w1 = m.workloads.global_model(n, seed=3)
    kw = dict(P=P, K=K, local_lr=0.05, mu=0.9, seed=99, objective=m.OBJ_PSEUDOGRAD, sigma=0.03)
    a = m.Mavg(w1, **kw)
    b = m.Mavg(w1, defer_broadcast=True, **kw)
    o = oracle.Mavg(w1, P=P, K=K, gamma=0.05, mu=0.9, seed=99, objective=oracle.OBJ_PSEUDOGRAD,
                    sigma=0.03, stride=a.stride)
    for r in range(3):
        a.local_steps()
        b.local_steps()
        a.sync(); b.sync()
        assert _same(a.replicas[:, :n], b.replicas[:, :n])
        learners = b.replicas[:, :n].clone()
        a.meta_update()
        b.meta_update()
        o.run_round()
        a.sync(); b.sync()
        assert _same(a.w, b.w) and _same(a.v, b.v)
        # the copies were not written: the array still holds this round's learner models
        assert _same(b.replicas[:, :n], learners)
        assert rel_err(b.w.cpu().numpy(), o.w) <= 1e-5
        assert rel_err(b.v.cpu().numpy(), o.v) <= 1e-5
    b.materialize_replicas()
    b.sync()
    for j in range(P):
        assert _same(b.replicas[j, :n], b.w)
    # once written, a second request is a no-op and the next round is unchanged
    b.materialize_replicas()
    a.round(); b.round()
    a.sync(); b.sync()
    assert _same(a.w, b.w) and _same(a.v, b.v)
    a.close(); b.close()


def test_meta_update_right_after_create_and_twice_in_a_row():
    # no local step in between: all learners equal w~, so d = 0, v <- mu v, w~ <- w~ + v
    m = _mavg()
    n, P = 4099, 5
    w1 = m.workloads.global_model(n, seed=5)
    kw = dict(P=P, K=2, local_lr=0.05, mu=0.5, seed=1, objective=m.OBJ_PSEUDOGRAD, sigma=0.1)
    a = m.Mavg(w1, **kw)
    b = m.Mavg(w1, defer_broadcast=True, **kw)
    b.replicas.fill_(123.0)          # must never be read as learner models
    for g in (a, b):
        g.meta_update()
        g.round()
        g.meta_update()
        g.meta_update()
        g.sync()
    assert _same(a.w, b.w) and _same(a.v, b.v)
    assert a.get_round() == b.get_round() == 4
    a.close(); b.close()


def test_meta_only_handle_leaves_replicas_alone(oracle):
    m = _mavg()
    n, P = 50_001, 6
    w1 = m.workloads.global_model(n, seed=8)
    g = m.Mavg(w1, P=P, K=1, local_lr=0.1, mu=0.9, objective=m.OBJ_NONE, defer_broadcast=True)
    o = oracle.Mavg(w1, P=P, K=1, gamma=0.1, mu=0.9, zeta=1.0, stride=g.stride)
    for u in range(3):
        reps = m.workloads.perturbed_replicas(o.w, P, 0.1, update=u, seed=11, stride=g.stride)
        o.replicas[:] = reps
        g.replicas.copy_(torch.from_numpy(reps))
        g.meta_update()
        o.meta_update()
        g.sync()
        assert rel_err(g.w.cpu().numpy(), o.w) <= 1e-5
        assert rel_err(g.v.cpu().numpy(), o.v) <= 1e-5
        assert np.array_equal(g.replicas.cpu().numpy()[:, :n], reps[:, :n])
    g.close()


def _mlp_pair(m, mode, dims, B, P, K, S=4000, **kw):
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(dims=dims, P=P, K=K, B=B, S=S)
    x, y = m.workloads.make_dataset(cfg, S=S)
    w1 = m.workloads.mlp_init(dims)
    common = dict(P=P, K=K, local_lr=0.05, mu=0.9, B=B, seed=m.workloads.BASE_SEED,
                  objective=m.OBJ_MLP, dims=dims, gemm_bf16=mode, x=x, y=y, x_bf16=(mode == 1))
    common.update(kw)
    return m.Mavg(w1, **common), m.Mavg(w1, defer_broadcast=True, **common)


@pytest.mark.parametrize("mode,dims,B,P,K", [
    (1, [512, 256, 128, 10], 64, 4, 3),      # tensor-core path, graph replay
    (1, [3072, 512, 512, 10], 128, 8, 2),    # the benchmark's shapes
    (1, [264, 200, 10], 48, 3, 1),           # ragged tiles, K = 1
    (0, [40, 24, 10], 7, 3, 2),              # CUDA-core fp32 path
    (2, [64, 48, 10], 16, 2, 2),             # CUDA-core path with rounded operands
])
def test_mlp_deferred_equals_eager(mode, dims, B, P, K):
    m = _mavg()
    a, b = _mlp_pair(m, mode, dims, B, P, K)
    n = a.n
    for r in range(3):
        a.local_steps(); b.local_steps()
        a.sync(); b.sync()
        assert _same(a.replicas[:, :n], b.replicas[:, :n])
        assert np.array_equal(a.get_losses(), b.get_losses())
        a.meta_update(); b.meta_update()
        a.sync(); b.sync()
        assert _same(a.w, b.w) and _same(a.v, b.v)
    la, lb = a.round(want_loss=True), b.round(want_loss=True)
    assert la == lb
    assert _same(a.w, b.w) and _same(a.v, b.v)
    a.close(); b.close()


def test_mlp_deferred_launch_by_launch_and_round_host():
    # profiled rounds take the launch-by-launch schedule; round_host starts from host copies
    m = _mavg()
    a, b = _mlp_pair(m, 1, [512, 256, 10], 64, 4, 2)
    b.set_profiling(True)
    for r in range(2):
        a.round(); b.round()
    a.sync(); b.sync()
    assert _same(a.w, b.w) and _same(a.v, b.v)
    b.set_profiling(False)
    wa, va = a.w.cpu().clone(), a.v.cpu().clone()
    wb, vb = wa.clone(), va.clone()
    la = a.round_host(wa, va)
    lb = b.round_host(wb, vb)
    assert la == lb
    assert torch.equal(wa, wb) and torch.equal(va, vb)
    # resume from a saved state
    a.set_round(7); b.set_round(7)
    a.round(); b.round()
    a.sync(); b.sync()
    assert _same(a.w, b.w) and _same(a.v, b.v)
    a.close(); b.close()


@pytest.mark.parametrize("mode", [0, 2])
def test_cuda_core_graph_recorded_after_materialize(mode):
    # CUDA-core path with deferred copies: the graph of a round's local steps is first recorded in
    # a round whose copies had been written on request just before.  Every later replay must still
    # start the learners from w~ (the copies are made outside the recorded graph), bit for bit
    # like a handle that always writes them.
    m = _mavg()
    dims = [40, 24, 10] if mode == 0 else [64, 48, 10]
    a, b = _mlp_pair(m, mode, dims, 16, 3, 2)
    b.materialize_replicas()          # copies exist when the first round records the graph
    for r in range(3):
        a.round(); b.round()
        a.sync(); b.sync()
        assert _same(a.w, b.w) and _same(a.v, b.v), r
    a.close(); b.close()
