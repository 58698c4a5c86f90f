"""Pins of the CPU oracle to things other than itself: published generator outputs, library
routines (torch autograd, torch's bf16 conversion, numpy means), closed forms and identities the
paper states (mu = 0 is K-AVG; Eq. 2; the auxiliary sequence z_n of the convergence proof; the
unrolled momentum sum), brute force on tiny sizes.  CPU only."""
import math
import os

import numpy as np
import pytest
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
M64 = (1 << 64) - 1
GAMMA = 0x9E3779B97F4A7C15


# ------------------------------------------------------------------------------ random numbers
def test_splitmix64_published_vector(oracle):
    want = [int(l) for l in open(os.path.join(GOLDEN, "splitmix64_seed1234567.txt"))
            if l.strip() and not l.startswith("#")]
    got = [oracle.splitmix64_output(1234567, i) for i in range(1, 6)]
    assert got == want


def test_stream_key_is_a_chain_of_generator_steps(oracle):
    # fold(s, c) is "the (c+1)-th SplitMix64 output from state s"; check the chain through the
    # exported generator primitive only.
    seed, tag, n, j, k = 99, oracle.TAG_BATCH, 7, 3, 2
    s = seed
    for c in (tag, n, j, k):
        s = oracle.splitmix64_output(s, c + 1)
    assert oracle.stream_key(seed, tag, n, j, k) == s
    # distinct counters give distinct keys
    keys = {oracle.stream_key(seed, t, a, b, c) for t in (1, 2) for a in range(4)
            for b in range(4) for c in range(4)}
    assert len(keys) == 2 * 4 * 4 * 4


@pytest.mark.parametrize("S,P", [(4096, 4), (50000, 8), (50000, 32), (7, 3), (5, 5)])
def test_shards_partition_the_dataset(oracle, S, P):
    bounds = [oracle.shard_bounds(S, P, j) for j in range(P)]
    assert bounds[0][0] == 0 and bounds[-1][1] == S
    for j in range(P - 1):
        assert bounds[j][1] == bounds[j + 1][0]
    for j, (lo, hi) in enumerate(bounds):
        assert lo == (j * S) // P and hi == ((j + 1) * S) // P and hi > lo


def test_batch_indices_stay_in_shard_and_are_uniform(oracle):
    S, P, B = 50000, 32, 64
    for j in (0, 5, 31):
        lo, hi = oracle.shard_bounds(S, P, j)
        allidx = np.concatenate([oracle.batch_indices(11, n, P, j, k, S, B)
                                 for n in range(1, 40) for k in range(1, 17)])
        assert allidx.min() >= lo and allidx.max() < hi
        # chi-square against uniform over 16 equal bins of the shard
        bins = np.floor((allidx - lo) * 16.0 / (hi - lo)).astype(int)
        cnt = np.bincount(bins, minlength=16)
        chi2 = ((cnt - cnt.mean()) ** 2 / cnt.mean()).sum()
        assert chi2 < 45.0  # 15 dof: P(chi2 > 45) < 1e-4
    # (round, learner, step) select different streams
    a = oracle.batch_indices(11, 1, 4, 0, 1, 4096, 32)
    assert not np.array_equal(a, oracle.batch_indices(11, 2, 4, 0, 1, 4096, 32))
    assert not np.array_equal(a, oracle.batch_indices(11, 1, 4, 0, 2, 4096, 32))
    assert not np.array_equal(a, oracle.batch_indices(12, 1, 4, 0, 1, 4096, 32))
    # a prefix of a longer batch is the shorter batch (index s depends on s only)
    assert np.array_equal(a[:8], oracle.batch_indices(11, 1, 4, 0, 1, 4096, 8))


def test_batch_index_formula_by_big_integers(oracle):
    seed, n, P, j, k, S, B = 0x211000625, 3, 8, 7, 8, 50000, 16
    lo, hi = (j * S) // P, ((j + 1) * S) // P
    key = oracle.stream_key(seed, oracle.TAG_BATCH, n, j, k)
    want = []
    for s in range(B):
        h = oracle.splitmix64_output(key, s + 1)
        want.append(lo + (((h >> 32) * (hi - lo)) >> 32))
    assert list(oracle.batch_indices(seed, n, P, j, k, S, B)) == want


def test_golden_index_and_gradient_files_match(oracle):
    for line in open(os.path.join(GOLDEN, "batch_indices.txt")):
        if line.startswith("#"):
            continue
        head, vals = line.split(":")
        seed, n, P, j, k, S = (int(t) for t in head.split())
        want = [int(t) for t in vals.split()]
        assert list(oracle.batch_indices(seed, n, P, j, k, S, len(want))) == want
    for line in open(os.path.join(GOLDEN, "pseudograd_bits.txt")):
        if line.startswith("#"):
            continue
        head, vals = line.split(":")
        t = head.split()
        seed, n, j, k, sigma = int(t[0]), int(t[1]), int(t[2]), int(t[3]), float(t[4])
        want = [int(x, 16) for x in vals.split()]
        got = oracle.pseudograd(seed, n, j, k, 0, len(want), sigma).view(np.uint32)
        assert list(got) == want


def test_pseudograd_is_scaled_irwin_hall(oracle):
    seed, n, j, k, sigma = 5, 2, 3, 4, 0.25
    g = oracle.pseudograd(seed, n, j, k, 0, 400000, sigma).astype(np.float64)
    assert abs(g.mean()) < 4 * sigma / math.sqrt(g.size)
    assert abs(g.var() / sigma ** 2 - 1.0) < 0.01
    kurt = ((g - g.mean()) ** 4).mean() / g.var() ** 2
    assert abs(kurt - 2.7) < 0.03          # Irwin-Hall(4): 3 - 6/(5*4)
    bound = sigma * 131070 / math.sqrt(4 * (65536.0 ** 2 - 1) / 12)
    assert np.abs(g).max() <= bound * (1 + 1e-6)
    # element i by big integers: lanes of the (i+1)-th generator output of the stream key
    key = oracle.stream_key(seed, oracle.TAG_PSEUDOGRAD, n, j, k)
    c = np.float32(sigma / math.sqrt(4 * (65536.0 ** 2 - 1) / 12))
    for i in (0, 1, 77, 399999):
        h = oracle.splitmix64_output(key, i + 1)
        s = sum((h >> sh) & 0xFFFF for sh in (0, 16, 32, 48)) - 131070
        assert np.float32(g[i]) == np.float32(s) * c
    # windows of the same stream agree
    assert np.array_equal(oracle.pseudograd(seed, n, j, k, 1000, 50, sigma),
                          oracle.pseudograd(seed, n, j, k, 0, 1050, sigma)[1000:])


def test_bf16_rounding_against_torch(oracle):
    hi = np.arange(1 << 16, dtype=np.uint32) << 16
    lows = np.array([0, 1, 0x7FFF, 0x8000, 0x8001, 0xFFFF, 0x1234], dtype=np.uint32)
    bits = (hi[:, None] | lows[None, :]).reshape(-1)
    x = bits.view(np.float32)
    finite = np.isfinite(x)
    got = oracle.bf16_round(x)
    want = torch.from_numpy(x.copy()).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(got[finite].view(np.uint32), want[finite].view(np.uint32))
    assert np.isnan(got[np.isnan(x)]).all()


# ----------------------------------------------------------------------------------- objective
def _torch_mlp_loss(dims, w, X, y, dtype=torch.float64):
    off, a = 0, X
    L = len(dims) - 1
    for l in range(L):
        W = w[off:off + dims[l + 1] * dims[l]].view(dims[l + 1], dims[l]); off += W.numel()
        b = w[off:off + dims[l + 1]]; off += dims[l + 1]
        a = torch.nn.functional.linear(a, W, b)
        if l < L - 1:
            a = torch.relu(a)
    return torch.nn.functional.cross_entropy(a, y, reduction="mean")


@pytest.mark.parametrize("dims,B", [([32, 64, 10], 32), ([7, 5, 6, 3], 9), ([4, 3], 1)])
def test_mlp_gradient_against_autograd(oracle, dims, B):
    r = np.random.default_rng(1)
    n = oracle.mlp_param_count(dims)
    w = (0.3 * r.standard_normal(n)).astype(np.float32)
    X = r.standard_normal((B, dims[0])).astype(np.float32)
    y = r.integers(0, dims[-1], B).astype(np.int32)
    loss, grad = oracle.mlp_loss_grad(dims, w, X, y)
    wt = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    lt = _torch_mlp_loss(dims, wt, torch.tensor(X, dtype=torch.float64),
                         torch.tensor(y, dtype=torch.long))
    lt.backward()
    assert abs(loss - lt.item()) < 2e-6 * max(1.0, abs(lt.item()))
    g = wt.grad.numpy()
    assert np.abs(grad - g).max() < 2e-6 * max(1.0, np.abs(g).max())


def test_mlp_gradient_central_differences(oracle):
    dims, B = [6, 5, 4], 8
    r = np.random.default_rng(2)
    n = oracle.mlp_param_count(dims)
    w = (0.5 * r.standard_normal(n)).astype(np.float32)
    X = r.standard_normal((B, dims[0])).astype(np.float32)
    y = r.integers(0, dims[-1], B).astype(np.int32)
    _, grad = oracle.mlp_loss_grad(dims, w, X, y)
    h = 2.0 ** -7
    for i in range(n):
        wp, wm = w.copy(), w.copy()
        wp[i] += h
        wm[i] -= h
        fd = (oracle.mlp_loss_grad(dims, wp, X, y)[0] -
              oracle.mlp_loss_grad(dims, wm, X, y)[0]) / float(np.float64(wp[i]) - wm[i])
        assert abs(fd - grad[i]) < 2e-3 * max(1.0, abs(fd)), i


def test_mlp_loss_at_zero_weights_is_log_classes(oracle):
    dims = [32, 64, 10]
    w = np.zeros(oracle.mlp_param_count(dims), dtype=np.float32)
    X = np.random.default_rng(3).standard_normal((16, 32)).astype(np.float32)
    y = np.arange(16, dtype=np.int32) % 10
    loss, grad = oracle.mlp_loss_grad(dims, w, X, y)
    assert abs(loss - math.log(10.0)) < 1e-12
    # only the last bias sees a gradient: mean over the batch of (1/10 - onehot)
    nb = grad[-10:]
    want = 0.1 - np.bincount(y, minlength=10) / 16.0
    assert np.abs(nb - want).max() < 1e-7 and np.abs(grad[:-10]).max() == 0.0


def test_mlp_bf16_mode(oracle):
    dims, B = [16, 24, 5], 8
    r = np.random.default_rng(4)
    n = oracle.mlp_param_count(dims)
    w = (0.3 * r.standard_normal(n)).astype(np.float32)
    X = r.standard_normal((B, dims[0])).astype(np.float32)
    y = r.integers(0, dims[-1], B).astype(np.int32)
    l32, g32 = oracle.mlp_loss_grad(dims, w, X, y, bf16=False)
    l16, g16 = oracle.mlp_loss_grad(dims, w, X, y, bf16=True)
    # rounding the operands moves the result by O(2^-8), no more, and does move it (a hidden unit
    # whose pre-activation changes sign moves its own row by more: look at the median)
    assert 0 < abs(l16 - l32) < 0.03 * abs(l32)
    assert 0 < np.median(np.abs(g16 - g32)) < 0.01 * np.abs(g32).max()
    # single layer, operands already bf16-exact and a one-hot-free check: bf16 mode only differs
    # through the rounding of dZ, so the forward loss is identical
    dims1 = [16, 5]
    n1 = oracle.mlp_param_count(dims1)
    wq = oracle.bf16_round((0.3 * r.standard_normal(n1)).astype(np.float32))
    Xq = oracle.bf16_round(X)
    la, ga = oracle.mlp_loss_grad(dims1, wq, Xq, y, bf16=False)
    lb, gb = oracle.mlp_loss_grad(dims1, wq, Xq, y, bf16=True)
    assert la == lb
    # bias gradient uses the unrounded dZ
    assert np.array_equal(ga[-5:], gb[-5:])
    assert np.abs(ga - gb).max() < 2.0 ** -8 * np.abs(ga).max()


def _q_torch(a):
    """fp32 -> bf16 -> fp32 through torch's conversion (round to nearest even), as float64."""
    t = torch.tensor(np.asarray(a, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy().astype(np.float64)


def _mlp_bf16_restated(dims, w, X, y, drop=None):
    """The bf16-operand minibatch gradient written out again in numpy float64: every operand of a
    matrix product (weights, activations, dZ) is passed through torch's bf16 conversion at the
    place the workload statement puts it; the bias add, ReLU, softmax, dZ_L and the bias gradient
    use unrounded values.  Stored quantities (pre-activations, dZ) are fp32 like the oracle's.
    drop names ONE rounding to leave out (None: the statement itself) -- used to show that each
    rounding moves the result far beyond the comparison tolerance."""
    def q(a, name):
        return np.asarray(a, dtype=np.float64) if drop == name else _q_torch(a)
    L, B = len(dims) - 1, len(y)
    Ws, bs, off = [], [], 0
    for l in range(L):
        Ws.append(w[off:off + dims[l + 1] * dims[l]].reshape(dims[l + 1], dims[l])); off += Ws[-1].size
        bs.append(w[off:off + dims[l + 1]].astype(np.float64)); off += dims[l + 1]
    act = [q(X, "x")]
    zs = [None]
    for l in range(1, L + 1):
        z = (act[l - 1] @ q(Ws[l - 1], "w_fwd").T + bs[l - 1]).astype(np.float32)
        zs.append(z)
        act.append(q(np.maximum(z, 0), "act") if l < L else z.astype(np.float64))
    zL = zs[L].astype(np.float64)
    lse = np.log(np.exp(zL - zL.max(1, keepdims=True)).sum(1)) + zL.max(1)
    loss = float(np.mean(lse - zL[np.arange(B), y]))
    onehot = np.eye(dims[-1])[y]
    dz = ((np.exp(zL - lse[:, None]) - onehot) / B).astype(np.float32)
    gW, gb = [None] * L, [None] * L
    for l in range(L, 0, -1):
        gb[l - 1] = dz.astype(np.float64).sum(0)                       # from the unrounded dZ
        gW[l - 1] = q(dz, "dz_wgrad").T @ act[l - 1]
        if l > 1:
            da = q(dz, "dz_dgrad") @ q(Ws[l - 1], "w_dgrad")
            dz = np.where(zs[l - 1] > 0, da, 0.0).astype(np.float32)   # ReLU'(0) = 0
    grad = np.concatenate([np.concatenate([gW[l].reshape(-1), gb[l]]) for l in range(L)])
    return loss, grad


@pytest.mark.parametrize("dims,B", [([16, 24, 5], 8), ([24, 16, 8, 4], 12)])
def test_mlp_bf16_operand_rounding_restated(oracle, dims, B):
    # Which operands the bf16 mode rounds, and where, pinned by an independent restatement that
    # calls torch's conversion explicitly.  Inputs are generic fp32 values (not bf16-exact), so
    # that every rounding matters.
    r = np.random.default_rng(11)
    n = oracle.mlp_param_count(dims)
    w = (0.4 * r.standard_normal(n)).astype(np.float32)
    X = r.standard_normal((B, dims[0])).astype(np.float32)
    y = r.integers(0, dims[-1], B).astype(np.int32)
    loss, grad = oracle.mlp_loss_grad(dims, w, X, y, bf16=True)
    want_loss, want = _mlp_bf16_restated(dims, w, X, y)
    scale = np.abs(want).max()
    tol = 2e-6
    assert abs(loss - want_loss) < tol * max(1.0, abs(want_loss))
    assert np.abs(grad - want).max() < tol * scale
    # the bias gradients come from the unrounded dZ: they agree with a rounding-free sum of the
    # restatement's dZ to fp32 resolution (checked inside `want` above), and no weight gradient
    # of a hidden layer equals its fp32-mode value
    _, g32 = oracle.mlp_loss_grad(dims, w, X, y, bf16=False)
    assert np.abs(grad - g32).max() > 100 * tol * scale
    # Each single rounding left out of the restatement moves it away from the oracle by far more
    # than the tolerance: the comparison above would fail if the oracle dropped that rounding.
    for name in ("x", "w_fwd", "act", "dz_wgrad", "dz_dgrad", "w_dgrad"):
        _, mut = _mlp_bf16_restated(dims, w, X, y, drop=name)
        assert np.abs(grad - mut).max() > 50 * tol * scale, name


def test_mlp_bf16_bias_gradient_is_not_rounded(oracle):
    # dZ_L values are chosen by construction to sit far from bf16 grid points: one layer, zero
    # weights => p = 1/C for every class, dZ = (1/C - onehot)/B, which is not bf16-exact for
    # C = 10, B = 3.  The bias gradient must be the exact column sum of those values.
    dims, B = [8, 10], 3
    w = np.zeros(oracle.mlp_param_count(dims), dtype=np.float32)
    X = np.random.default_rng(5).standard_normal((B, 8)).astype(np.float32)
    y = np.array([1, 1, 7], dtype=np.int32)
    _, grad = oracle.mlp_loss_grad(dims, w, X, y, bf16=True)
    dz = ((0.1 - np.eye(10)[y]) / B).astype(np.float32).astype(np.float64)
    assert np.abs(grad[-10:] - dz.sum(0)).max() < 1e-7     # stored in fp32
    rounded = _q_torch(dz).sum(0)
    assert np.abs(rounded - dz.sum(0)).max() > 1e-5       # rounding dZ first would have shown
    # and the weight gradient does use the rounded dZ (and the rounded inputs)
    want = _q_torch(dz).T @ _q_torch(X)
    assert np.abs(grad[:-10].reshape(10, 8) - want).max() < 1e-7


# ---------------------------------------------------------------------------------- meta level
def _state(oracle, n=257, P=5, mu=0.9, zeta=1.0, seed=0, stride=None):
    r = np.random.default_rng(seed)
    w1 = r.standard_normal(n).astype(np.float32)
    m = oracle.Mavg(w1, P=P, K=1, gamma=0.1, mu=mu, zeta=zeta, stride=stride)
    return m, r


def test_init_sets_v_zero_and_broadcasts(oracle):
    m, _ = _state(oracle, stride=264)
    assert not m.v.any()
    for j in range(5):
        assert np.array_equal(m.replicas[j, :m.n], m.w)


def test_mu_zero_is_kavg(oracle):
    # Remark after Theorem 1: mu = 0 reduces M-AVG to K-AVG, i.e. w~ <- mean of the replicas.
    m, r = _state(oracle, mu=0.0)
    for _ in range(3):
        m.replicas[:, :m.n] += r.standard_normal((5, m.n)).astype(np.float32)
        w_old = m.w.copy()
        mean = m.replicas[:, :m.n].astype(np.float64).mean(axis=0)
        m.meta_update()
        assert np.abs(m.w - mean).max() < 1e-6
        assert np.abs(m.v - (mean - w_old)).max() < 1e-6
        assert all(np.array_equal(m.replicas[j, :m.n], m.w) for j in range(5))


def test_first_round_ignores_mu(oracle):
    outs = []
    for mu in (0.0, 0.5, 0.9):
        m, r = _state(oracle, mu=mu, seed=7)
        m.replicas[:, :m.n] += r.standard_normal((5, m.n)).astype(np.float32)
        m.meta_update()
        outs.append(m.w.copy())
    assert np.array_equal(outs[0], outs[1]) and np.array_equal(outs[0], outs[2])


def test_identical_replicas(oracle):
    m, r = _state(oracle, mu=0.9)
    rep = r.standard_normal(m.n).astype(np.float32)
    w_old = m.w.copy()
    m.replicas[:, :m.n] = rep
    m.meta_update()
    # a = rep exactly, d = rep - w~, v = d (v was 0), w~ = rep up to fp32 rounding of w~ + v
    assert np.abs(m.v - (rep.astype(np.float64) - w_old)).max() < 1e-6
    assert np.abs(m.w - rep).max() < 1e-6


@pytest.mark.parametrize("mu,zeta", [(0.9, 1.0), (0.5, 0.7), (0.0, 1.0)])
def test_auxiliary_sequence_and_unrolled_momentum(oracle, mu, zeta):
    # z_n = w~_n + mu/(1-mu) v_n obeys z_{n+1} - z_n = zeta d_n / (1-mu) (proof of Theorem 1), and
    # v_n = sum_i mu^i zeta d_{n-i}, hence w~_{N+1} = w~_1 + sum_n sum_{i<n} mu^i zeta d_{n-i}.
    n, P, N = 31, 3, 6
    m, r = _state(oracle, n=n, P=P, mu=mu, zeta=zeta, seed=11)
    w1 = m.w.astype(np.float64)
    ds = []
    for _ in range(N):
        m.replicas[:, :n] += 0.3 * r.standard_normal((P, n)).astype(np.float32)
        d = m.replicas[:, :n].astype(np.float64).mean(axis=0) - m.w
        z_old = m.w + mu / (1 - mu) * m.v.astype(np.float64)
        m.meta_update()
        z_new = m.w + mu / (1 - mu) * m.v.astype(np.float64)
        assert np.abs((z_new - z_old) - zeta * d / (1 - mu)).max() < 2e-5
        ds.append(d)
    v_want = sum(mu ** i * zeta * ds[N - 1 - i] for i in range(N))
    assert np.abs(m.v - v_want).max() < 5e-6
    w_want = w1 + sum(mu ** i * zeta * ds[k - i] for k in range(N) for i in range(k + 1))
    assert np.abs(m.w - w_want).max() < 2e-5


# --------------------------------------------------------------------------------- whole rounds
@pytest.mark.parametrize("P,K,mu,zeta", [(3, 4, 0.9, 1.0), (1, 1, 0.0, 1.0), (2, 7, 0.5, 0.8)])
def test_quadratic_closed_form(oracle, P, K, mu, zeta):
    # F(w) = 1/2 sum a_i w_i^2 with exact gradients: K local steps scale each coordinate by
    # rho_i = (1 - gamma a_i)^K, so d = (rho - 1) w~ and
    #   w~_{n+1} = (1 + mu - zeta (1 - rho)) w~_n - mu w~_{n-1},   w~_2 = (1 - zeta (1 - rho)) w~_1.
    n, gamma, N = 9, 0.1, 12
    r = np.random.default_rng(5)
    a = r.uniform(0.2, 3.0, n).astype(np.float32)
    w1 = r.standard_normal(n).astype(np.float32)
    m = oracle.Mavg(w1, P=P, K=K, gamma=gamma, mu=mu, zeta=zeta,
                    objective=oracle.OBJ_QUADRATIC, quad_a=a)
    rho = (1.0 - np.float64(np.float32(gamma)) * a.astype(np.float64)) ** K
    prev, cur = None, w1.astype(np.float64)
    for _ in range(N):
        m.run_round()
        if prev is None:
            nxt = (1 - zeta * (1 - rho)) * cur
        else:
            nxt = (1 + mu - zeta * (1 - rho)) * cur - mu * prev
        prev, cur = cur, nxt
        assert np.abs(m.w - cur).max() < 2e-5 * max(1.0, np.abs(cur).max())


def test_p1_k1_mu0_is_plain_sgd(oracle):
    dims, B, S = [8, 6, 3], 4, 40
    r = np.random.default_rng(6)
    x = r.standard_normal((S, dims[0])).astype(np.float32)
    y = r.integers(0, 3, S).astype(np.int32)
    w1 = (0.4 * r.standard_normal(oracle.mlp_param_count(dims))).astype(np.float32)
    m = oracle.Mavg(w1, P=1, K=1, gamma=0.2, mu=0.0, B=B, seed=21, objective=oracle.OBJ_MLP,
                    dims=dims, x=x, y=y)
    w = torch.tensor(w1, dtype=torch.float64)
    for n in range(1, 4):
        idx = oracle.batch_indices(21, n, 1, 0, 1, S, B)
        wt = w.clone().requires_grad_(True)
        _torch_mlp_loss(dims, wt, torch.tensor(x[idx], dtype=torch.float64),
                        torch.tensor(y[idx], dtype=torch.long)).backward()
        w = w - np.float64(np.float32(0.2)) * wt.grad
        m.run_round()
        assert np.abs(m.w - w.numpy()).max() < 1e-5


def test_k1_mu0_is_synchronous_sgd(oracle):
    # K = 1, mu = 0: w~ <- w~ - gamma * mean_j g_j (averaged-gradient SGD).
    n, P, gamma, sigma = 1000, 6, 0.05, 0.1
    w1 = np.random.default_rng(8).standard_normal(n).astype(np.float32)
    m = oracle.Mavg(w1, P=P, K=1, gamma=gamma, mu=0.0, seed=33,
                    objective=oracle.OBJ_PSEUDOGRAD, sigma=sigma)
    w = w1.astype(np.float64)
    for rnd in range(1, 4):
        g = np.stack([oracle.pseudograd(33, rnd, j, 1, 0, n, sigma) for j in range(P)])
        w = w - np.float64(np.float32(gamma)) * g.astype(np.float64).mean(axis=0)
        m.run_round()
        assert np.abs(m.w - w).max() < 1e-6


@pytest.mark.parametrize("objective", ["mlp", "pseudograd"])
def test_d_equals_minus_gamma_G(oracle, objective):
    # Eq. 2: the block "gradient" d of Algorithm 1 is -gamma G_n, G_n the learner-mean of the K
    # summed minibatch-mean gradients (no division by K).
    r = np.random.default_rng(9)
    if objective == "mlp":
        dims, B, S, P, K = [8, 6, 3], 4, 64, 3, 5
        x = r.standard_normal((S, 8)).astype(np.float32)
        y = r.integers(0, 3, S).astype(np.int32)
        w1 = (0.4 * r.standard_normal(oracle.mlp_param_count(dims))).astype(np.float32)
        m = oracle.Mavg(w1, P=P, K=K, gamma=0.1, mu=0.9, B=B, seed=3, objective=oracle.OBJ_MLP,
                        dims=dims, x=x, y=y)
    else:
        P, K = 4, 6
        w1 = r.standard_normal(500).astype(np.float32)
        m = oracle.Mavg(w1, P=P, K=K, gamma=0.1, mu=0.9, seed=3,
                        objective=oracle.OBJ_PSEUDOGRAD, sigma=0.3)
    for _ in range(2):
        w_old = m.w.astype(np.float64)
        _, G = m.local_steps(want_G=True)
        d = m.replicas[:, :m.n].astype(np.float64).mean(axis=0) - w_old
        assert np.abs(d + np.float64(np.float32(0.1)) * G).max() < 1e-6 * K
        assert np.abs(G).max() > 1e-3
        m.meta_update()


def test_learners_with_identical_data_stay_identical(oracle):
    # the learners are i.i.d. given w~; with a one-sample shard each they see the same data every
    # step only if the samples are equal -- build that case and check a = w^j.
    dims, P, K = [5, 4, 3], 3, 4
    r = np.random.default_rng(10)
    x1 = r.standard_normal((1, 5)).astype(np.float32)
    x = np.repeat(x1, P, axis=0)
    y = np.full(P, 2, dtype=np.int32)
    w1 = (0.4 * r.standard_normal(oracle.mlp_param_count(dims))).astype(np.float32)
    m = oracle.Mavg(w1, P=P, K=K, gamma=0.1, mu=0.0, B=2, seed=1, objective=oracle.OBJ_MLP,
                    dims=dims, x=x, y=y)
    m.local_steps()
    for j in range(1, P):
        assert np.array_equal(m.replicas[j], m.replicas[0])
    rep = m.replicas[0, :m.n].copy()
    m.meta_update()
    assert np.abs(m.w - rep).max() < 1e-6


def test_learner_order_does_not_matter(oracle):
    n, P = 100, 4
    r = np.random.default_rng(12)
    w1 = r.standard_normal(n).astype(np.float32)
    reps = w1 + r.standard_normal((P, n)).astype(np.float32)
    outs = []
    for perm in ([0, 1, 2, 3], [3, 1, 0, 2]):
        m = oracle.Mavg(w1, P=P, K=1, gamma=0.1, mu=0.9)
        m.replicas[:, :n] = reps[perm]
        m.meta_update()
        outs.append(m.w.copy())
    assert np.abs(outs[0] - outs[1]).max() < 1e-6


# -------------------------------------------------------------------- learner-level momentum
def test_beta_zero_is_algorithm_1_as_printed(oracle):
    n, P, K = 500, 3, 4
    w1 = np.random.default_rng(12).standard_normal(n).astype(np.float32)
    kw = dict(P=P, K=K, gamma=0.05, mu=0.7, seed=5, objective=oracle.OBJ_PSEUDOGRAD, sigma=0.2)
    a = oracle.Mavg(w1, **kw)
    b = oracle.Mavg(w1, beta=0.0, reset_u=True, **kw)
    for _ in range(3):
        a.run_round(); b.run_round()
    assert np.array_equal(a.w, b.w) and np.array_equal(a.v, b.v)
    assert not b.u.any()


@pytest.mark.parametrize("beta", [0.5, 0.9])
def test_learner_momentum_unrolled_sum(oracle, beta):
    # u_k = -gamma sum_{i<k} beta^i g_{k-i}  and  w_K = w_0 + sum_k u_k, by brute force in fp64
    n, K, gamma, sigma = 300, 6, 0.05, 0.3
    w1 = np.random.default_rng(13).standard_normal(n).astype(np.float32)
    m = oracle.Mavg(w1, P=2, K=K, gamma=gamma, mu=0.0, seed=17, objective=oracle.OBJ_PSEUDOGRAD,
                    sigma=sigma, beta=beta)
    m.local_steps()
    g32, b32 = np.float64(np.float32(gamma)), np.float64(np.float32(beta))
    for j in range(2):
        g = [oracle.pseudograd(17, 1, j, k, 0, n, sigma).astype(np.float64) for k in range(1, K + 1)]
        us = [-g32 * sum(b32 ** i * g[k - 1 - i] for i in range(k)) for k in range(1, K + 1)]
        assert np.abs(m.u[j, :n] - us[-1]).max() < 1e-6
        assert np.abs(m.replicas[j, :n] - (w1.astype(np.float64) + sum(us))).max() < 2e-6


@pytest.mark.parametrize("beta,gamma", [(0.5, 0.1), (0.9, 0.3)])
def test_learner_momentum_heavy_ball_closed_form(oracle, beta, gamma):
    # on F = 1/2 a w^2 the steps are the two-term recurrence w_{k+1} = (1 + beta - gamma a) w_k
    # - beta w_{k-1}, w_1 = (1 - gamma a) w_0, whose solution is c1 r1^k + c2 r2^k with r1, r2 the
    # (possibly complex) roots of r^2 - (1 + beta - gamma a) r + beta = 0
    n, K = 7, 9
    r = np.random.default_rng(14)
    a = r.uniform(0.3, 2.5, n).astype(np.float32)
    w0 = r.standard_normal(n).astype(np.float32)
    m = oracle.Mavg(w0, P=1, K=K, gamma=gamma, mu=0.0, objective=oracle.OBJ_QUADRATIC, quad_a=a,
                    beta=beta)
    m.local_steps()
    g32, b32 = np.float64(np.float32(gamma)), np.float64(np.float32(beta))
    t = (1 + b32 - g32 * a.astype(np.float64)).astype(np.complex128)
    disc = np.sqrt(t * t - 4 * b32)
    r1, r2 = (t + disc) / 2, (t - disc) / 2
    w_0 = w0.astype(np.complex128)
    w_1 = (1 - g32 * a.astype(np.float64)) * w_0
    c1 = (w_1 - r2 * w_0) / (r1 - r2)
    c2 = w_0 - c1
    want = (c1 * r1 ** K + c2 * r2 ** K).real
    assert np.abs(m.replicas[0, :n] - want).max() < 5e-6 * max(1.0, np.abs(want).max())


@pytest.mark.parametrize("reset", [False, True])
def test_learner_momentum_against_torch_sgd(oracle, reset):
    # P = 1, mu = 0, zeta = 1: the global model follows the single learner, so the rounds are one
    # run of momentum SGD -- torch's optimizer (buf <- beta buf + g, p <- p - lr buf, the same
    # sequence as u = -lr buf) with its buffer kept over the rounds, or re-made every round
    dims, B, S, K, beta, lr = [8, 6, 3], 4, 40, 3, 0.8, 0.1
    r = np.random.default_rng(15)
    x = r.standard_normal((S, dims[0])).astype(np.float32)
    y = r.integers(0, 3, S).astype(np.int32)
    w1 = (0.4 * r.standard_normal(oracle.mlp_param_count(dims))).astype(np.float32)
    m = oracle.Mavg(w1, P=1, K=K, gamma=lr, mu=0.0, B=B, seed=23, objective=oracle.OBJ_MLP,
                    dims=dims, x=x, y=y, beta=beta, reset_u=reset)
    w = torch.tensor(w1, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([w], lr=float(np.float32(lr)), momentum=float(np.float32(beta)))
    for n in range(1, 4):
        if reset:
            opt = torch.optim.SGD([w], lr=float(np.float32(lr)), momentum=float(np.float32(beta)))
        for k in range(1, K + 1):
            idx = oracle.batch_indices(23, n, 1, 0, k, S, B)
            opt.zero_grad()
            _torch_mlp_loss(dims, w, torch.tensor(x[idx], dtype=torch.float64),
                            torch.tensor(y[idx], dtype=torch.long)).backward()
            opt.step()
        m.run_round()
        assert np.abs(m.w - w.detach().numpy()).max() < 2e-5
