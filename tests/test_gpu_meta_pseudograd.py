"""GPU parity of the meta-update and of the pseudo-gradient learner level against the CPU oracle,
through the C ABI.  fp32 meta-update gate: relative error <= 1e-5 (metric of tests/util.py)."""
import numpy as np
import pytest
import torch

from tests.util import rel_err

pytestmark = pytest.mark.gpu

META_TOL = 1e-5


def _mavg():
    import paper_2110_00625_b200 as m
    return m


@pytest.mark.parametrize("n", [1, 3, 4, 5, 1023, 2762, 100_003])
@pytest.mark.parametrize("P", [1, 2, 3, 9, 64])
def test_meta_update_small_and_ragged(oracle, n, P):
    m = _mavg()
    W = m.workloads
    w1 = W.global_model(n, seed=7)
    for mu, zeta in [(0.9, 1.0), (0.0, 1.0), (0.5, 0.7)]:
        g = m.Mavg(w1, P=P, K=1, local_lr=0.1, mu=mu, block_lr=zeta, objective=m.OBJ_NONE)
        o = oracle.Mavg(w1, P=P, K=1, gamma=0.1, mu=mu, zeta=zeta, stride=g.stride)
        for u in range(3):
            reps = W.perturbed_replicas(o.w, P, 0.1, update=u, seed=11, stride=g.stride)
            o.replicas[:] = reps
            g.replicas.copy_(torch.from_numpy(reps))
            g.meta_update()
            o.meta_update()
            g.sync()
            assert rel_err(g.w.cpu().numpy(), o.w) <= META_TOL
            assert rel_err(g.v.cpu().numpy(), o.v) <= META_TOL
            gr = g.replicas.cpu().numpy()
            gw = g.w.cpu().numpy()
            for j in range(P):   # the re-broadcast is exact
                assert np.array_equal(gr[j, :n], gw)
        assert g.get_round() == 3
        g.close()


def test_meta_update_mu0_is_the_mean():
    # K-AVG: with mu = 0 and block learning rate 1 the new global model is the replica mean
    m = _mavg()
    n, P = 50_000, 16
    w1 = m.workloads.global_model(n, seed=3)
    g = m.Mavg(w1, P=P, K=1, local_lr=0.1, mu=0.0, objective=m.OBJ_NONE)
    reps = m.workloads.perturbed_replicas(w1, P, 0.1, update=0, seed=5, stride=g.stride)
    g.replicas.copy_(torch.from_numpy(reps))
    g.meta_update()
    g.sync()
    mean = reps[:, :n].astype(np.float64).mean(axis=0)
    assert rel_err(g.w.cpu().numpy(), mean) <= META_TOL


@pytest.mark.parametrize("P,mu", [(4, 0.9), (16, 0.0), (64, 0.9)])
def test_meta_update_c3_shape_reduced(oracle, P, mu):
    # the bandwidth-sweep workload at 1/8 of its length (the oracle side stays in seconds):
    # several thousand tiles per replica and a ragged tail
    m = _mavg()
    n = 1_400_003
    w1 = m.workloads.global_model(n)
    g = m.Mavg(w1, P=P, K=1, local_lr=0.1, mu=mu, objective=m.OBJ_NONE)
    o = oracle.Mavg(w1, P=P, K=1, gamma=0.1, mu=mu, stride=g.stride)
    for u in range(5):
        reps = m.workloads.perturbed_replicas(o.w, P, 0.1, update=u, stride=g.stride)
        o.replicas[:] = reps
        g.replicas.copy_(torch.from_numpy(reps))
        g.meta_update()
        o.meta_update()
    g.sync()
    assert rel_err(g.w.cpu().numpy(), o.w) <= META_TOL
    assert rel_err(g.v.cpu().numpy(), o.v) <= META_TOL


@pytest.mark.parametrize("n,P,mu,defer", [
    (6_000_001, 3, 0.9, False),     # ring of 4 replica tiles x 3 stages (P <= 4), n % 4 = 1
    (2_500_003, 8, 0.0, False),     # ring of 6 x 2 (5 <= P <= 8), v not read, n % 4 = 3
    (2_500_003, 12, 0.9, True),     # ring of 3 x 2 with 4096-element tiles, copies deferred
    (2_500_002, 26, 0.9, False),    # ring of 6 x 2 (P >= 24), last group of 2 replicas
])
def test_meta_update_bulk_kernel_rings_and_ragged_end(oracle, n, P, mu, defer):
    # replica sets larger than the L2 with at least 2.4 M elements take the bulk-copy kernel; its
    # three ring shapes, a last group with fewer replicas than the ring's width, and the end of
    # the vector that is not a whole tile (nor a whole float4), done inside the same launch
    m = _mavg()
    w1 = m.workloads.global_model(n, seed=9)
    g = m.Mavg(w1, P=P, K=1, local_lr=0.1, mu=mu, objective=m.OBJ_NONE, defer_broadcast=defer)
    o = oracle.Mavg(w1, P=P, K=1, gamma=0.1, mu=mu, stride=g.stride)
    for u in range(2):
        reps = m.workloads.perturbed_replicas(o.w, P, 0.1, update=u, seed=21, stride=g.stride)
        o.replicas[:] = reps
        g.replicas.copy_(torch.from_numpy(reps))
        g.meta_update()
        o.meta_update()
    g.sync()
    assert rel_err(g.w.cpu().numpy(), o.w) <= META_TOL
    assert rel_err(g.v.cpu().numpy(), o.v) <= META_TOL
    got = g.replicas.cpu().numpy()
    if defer:       # the copies are left to the next local step: the array is untouched
        assert np.array_equal(got[:, :n], reps[:, :n])
    else:           # every replica is an exact copy of the new global model, ragged end included
        assert all(np.array_equal(got[j, :n], g.w.cpu().numpy()) for j in (0, P // 2, P - 1))
    g.close()


@pytest.mark.parametrize("K", [1, 4, 16, 64])
@pytest.mark.parametrize("mu", [0.0, 0.9])
def test_pseudograd_rounds(oracle, K, mu):
    m = _mavg()
    n, P, gamma, sigma = 300_001, 16, 0.05, float(np.sqrt(1e-3))
    w1 = m.workloads.global_model(n)
    g = m.Mavg(w1, P=P, K=K, local_lr=gamma, mu=mu, seed=99, objective=m.OBJ_PSEUDOGRAD,
               sigma=sigma)
    o = oracle.Mavg(w1, P=P, K=K, gamma=gamma, mu=mu, seed=99,
                    objective=oracle.OBJ_PSEUDOGRAD, sigma=sigma, stride=g.stride)
    for r in range(3):
        g.local_steps()
        o.local_steps()
        g.sync()
        gr = g.replicas.cpu().numpy()
        for j in (0, P - 1):
            assert rel_err(gr[j, :n], o.replicas[j, :n]) <= META_TOL
        g.meta_update()
        o.meta_update()
    g.sync()
    assert rel_err(g.w.cpu().numpy(), o.w) <= META_TOL
    assert rel_err(g.v.cpu().numpy(), o.v) <= META_TOL


def test_pseudograd_single_step_is_bit_exact(oracle):
    # one step from the broadcast state: w - gamma*g with a fused multiply-add on both sides can
    # differ only by the double-rounding of the oracle; the variates themselves must be bit-equal,
    # which shows as exact equality of (w1 - w_after) wherever no rounding tie occurs -- check the
    # variates through the K=1, gamma=1, w=0 case, where w_after = -g exactly.
    m = _mavg()
    n, P, sigma = 10_007, 3, 0.25
    w1 = np.zeros(n, dtype=np.float32)
    g = m.Mavg(w1, P=P, K=1, local_lr=1.0, mu=0.0, seed=5, objective=m.OBJ_PSEUDOGRAD, sigma=sigma)
    g.local_steps()
    g.sync()
    gr = g.replicas.cpu().numpy()
    for j in range(P):
        want = -oracle.pseudograd(5, 1, j, 1, 0, n, sigma)
        assert np.array_equal(gr[j, :n].view(np.uint32), want.view(np.uint32))
    g.close()


def test_k1_mu0_is_synchronous_sgd(oracle):
    # the full-round workload's identity: K = 1, mu = 0 equals SGD with the learner-averaged gradient
    m = _mavg()
    n, P, gamma, sigma = 200_000, 16, 0.05, float(np.sqrt(1e-3))
    w1 = m.workloads.global_model(n)
    g = m.Mavg(w1, P=P, K=1, local_lr=gamma, mu=0.0, seed=42, objective=m.OBJ_PSEUDOGRAD,
               sigma=sigma)
    w = w1.astype(np.float64)
    for r in range(1, 4):
        grads = np.stack([oracle.pseudograd(42, r, j, 1, 0, n, sigma) for j in range(P)])
        w = w - np.float64(np.float32(gamma)) * grads.astype(np.float64).mean(axis=0)
        g.round()
    g.sync()
    assert rel_err(g.w.cpu().numpy(), w) <= META_TOL


def test_round_host_and_resume(oracle):
    m = _mavg()
    n, P, K, gamma, sigma = 50_001, 4, 3, 0.05, 0.1
    w1 = m.workloads.global_model(n)
    a = m.Mavg(w1, P=P, K=K, local_lr=gamma, mu=0.9, seed=8, objective=m.OBJ_PSEUDOGRAD, sigma=sigma)
    for _ in range(4):
        a.round()
    a.sync()
    # same four rounds with the model living in host memory
    b = m.Mavg(w1, P=P, K=K, local_lr=gamma, mu=0.9, seed=8, objective=m.OBJ_PSEUDOGRAD, sigma=sigma)
    wh = torch.from_numpy(w1.copy()).pin_memory()
    vh = torch.zeros(n).pin_memory()
    for _ in range(4):
        b.round_host(wh, vh)
    assert np.array_equal(wh.numpy(), a.w.cpu().numpy())
    assert np.array_equal(vh.numpy(), a.v.cpu().numpy())
    # resume from (w~, v, round) after two rounds reproduces rounds three and four
    c = m.Mavg(w1, P=P, K=K, local_lr=gamma, mu=0.9, seed=8, objective=m.OBJ_PSEUDOGRAD, sigma=sigma)
    c.round(); c.round(); c.sync()
    w2, v2 = c.w.clone(), c.v.clone()
    d = m.Mavg(w1, P=P, K=K, local_lr=gamma, mu=0.9, seed=8, objective=m.OBJ_PSEUDOGRAD, sigma=sigma)
    d.w.copy_(w2); d.v.copy_(v2); d.set_round(2)
    d.round(); d.round(); d.sync()
    assert np.array_equal(d.w.cpu().numpy(), a.w.cpu().numpy())
    assert d.get_round() == 4


def test_determinism():
    m = _mavg()
    n, P = 123_457, 16
    w1 = m.workloads.global_model(n)
    outs = []
    for _ in range(2):
        g = m.Mavg(w1, P=P, K=4, local_lr=0.05, mu=0.9, seed=1, objective=m.OBJ_PSEUDOGRAD, sigma=0.1)
        for _ in range(3):
            g.round()
        g.sync()
        outs.append((g.w.cpu().numpy(), g.v.cpu().numpy()))
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])


def test_losses_exist_for_the_mlp_objective_only():
    # a pseudo-gradient handle may raise K far beyond the K its loss buffer was sized for; asking
    # it for losses must be refused, not served from beyond the buffer
    m = _mavg()
    w1 = m.workloads.global_model(1000, seed=2)
    g = m.Mavg(w1, P=16, K=1, local_lr=0.05, mu=0.9, seed=5, objective=m.OBJ_PSEUDOGRAD, sigma=0.03)
    g.set_hparams(64, 0.05, 1.0, 0.9)
    g.round()
    g.sync()
    with pytest.raises(m.MavgError) as err:
        g.get_losses()
    assert err.value.status == 3          # MAVG_ERR_STATE
    g.round()                             # the handle is not poisoned by the refusal
    g.sync()
    g.close()
