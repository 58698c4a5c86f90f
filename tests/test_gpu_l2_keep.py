"""The opt-in L2 set-aside for the learners' masters (l2_keep = 1; tensor-core MLP handles whose P
master copies fit in half the L2): it may change speed only, and a handle that does not ask for it
leaves the context's limit alone.  Rounds with lines released in between give the same bits
as rounds without; the context's limit follows the largest request among the live handles and is
back at its old value when the last of them is closed (checked in a process of its own, where no
other test's handle is alive)."""
import subprocess
import sys
import textwrap

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

SEED = 0x211000625


def _handle(m, cfg, x, y, w1, P=None, l2_keep=True):
    return m.Mavg(w1, P=P or cfg["P"], K=cfg["K"], local_lr=cfg["gamma"], mu=cfg["mu"], B=cfg["B"],
                  seed=SEED, objective=m.OBJ_MLP, dims=cfg["dims"], gemm_bf16=1, x=x, y=y,
                  l2_keep=l2_keep)


def _small():
    import paper_2110_00625_b200 as m
    cfg = dict(m.workloads.CONFIGS["C2"])
    cfg.update(dims=[3072, 256, 128, 10], P=3, K=3, B=64, S=2048)
    x, y = m.workloads.make_dataset(cfg, S=cfg["S"])
    w1 = m.workloads.mlp_init(cfg["dims"])
    return m, cfg, x, y, w1


def test_release_keeps_the_bits():
    m, cfg, x, y, w1 = _small()
    a = _handle(m, cfg, x, y, w1)
    b = _handle(m, cfg, x, y, w1)
    c = _handle(m, cfg, x, y, w1, l2_keep=False)
    for _ in range(3):
        a.round()
        b.round()
        b.l2_release()
        c.round()
    a.sync(); b.sync(); c.sync()
    for other in (b, c):
        assert np.array_equal(a.w.cpu().numpy(), other.w.cpu().numpy())
        assert np.array_equal(a.v.cpu().numpy(), other.v.cpu().numpy())
    c.close()
    b.close()
    a.close()


CHILD = textwrap.dedent("""
    import sys
    import torch
    from cuda import cudart
    sys.path.insert(0, {root!r})
    from tests.test_gpu_l2_keep import _small, _handle

    def limit():
        err, val = cudart.cudaDeviceGetLimit(cudart.cudaLimit.cudaLimitPersistingL2CacheSize)
        assert int(err) == 0
        return int(val)

    torch.zeros(1, device="cuda")          # the context exists before the limit is read
    err, most = cudart.cudaDeviceGetAttribute(cudart.cudaDeviceAttr.cudaDevAttrMaxPersistingL2CacheSize, 0)
    m, cfg, x, y, w1 = _small()
    before = limit()
    z = _handle(m, cfg, x, y, w1, P=3, l2_keep=False)   # the default: limit untouched
    assert limit() == before
    z.round(); z.sync(); z.close()
    assert limit() == before
    a = _handle(m, cfg, x, y, w1, P=3)
    la = limit()
    b = _handle(m, cfg, x, y, w1, P=8)
    lb = limit()
    a.close()                              # not the order of creation
    lb2 = limit()
    b.close()
    after = limit()
    print("LIMITS", most, before, la, lb, lb2, after)
    if most > 0:
        assert la >= before and lb > before and lb >= la and lb2 == lb, (before, la, lb, lb2)
    assert after == before, (before, after)
""")


def test_limit_follows_the_live_handles_and_is_restored():
    pytest.importorskip("cuda.cudart")
    import os
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", CHILD.format(root=root)], capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-2000:]
    assert "LIMITS" in out.stdout


def test_release_is_a_no_op_without_a_learner_level():
    import paper_2110_00625_b200 as m
    w1 = m.workloads.global_model(10_001, seed=1)
    g = m.Mavg(w1, P=4, K=1, local_lr=0.05, mu=0.9, seed=3, objective=m.OBJ_NONE)
    g.l2_release()
    g.meta_update()
    g.sync()
    g.close()
