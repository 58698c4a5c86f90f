"""The per-tile comparison the tensor-core parity tests use, tested on the host: a result with one
wrong 128 x 32 tile (an edge tile of a large layer) must be rejected although it passes a check in
the 2-norm of the whole update.  No kernel is involved."""
import numpy as np
import pytest

from tests.util import assert_tiles_close, l2_rel, mlp_layout, tile_errors


def _step(dims, seed=0):
    r = np.random.default_rng(seed)
    n = sum(o * i + o for _, o, i, _ in mlp_layout(dims))
    want = 1e-3 * r.standard_normal(n)
    got = want * (1.0 + 1e-3 * r.standard_normal(n))
    return got, want


def test_close_results_pass():
    dims = [3072, 200, 72, 10]               # ragged tiles in both directions
    got, want = _step(dims)
    assert_tiles_close(got, want, dims)
    assert max(e for _, e, _ in tile_errors(got, want, dims)) < 2e-3


@pytest.mark.parametrize("where", ["last_row_tile", "last_col_tile", "bias"])
def test_one_wrong_tile_is_rejected(where):
    dims = [3072, 2048, 2048, 10]           # a tile is 0.04 % of the update
    got, want = _step(dims, seed=1)
    (w_off, o, i, b_off) = mlp_layout(dims)[0]
    G = got[w_off:w_off + o * i].reshape(o, i)     # a view: edits land in got
    r = np.random.default_rng(2)
    if where == "last_row_tile":
        G[o - 128:o, 64:96] = r.permutation(G[o - 128:o, 64:96].reshape(-1)).reshape(128, 32)
    elif where == "last_col_tile":
        G[128:256, i - 32:i] = r.permutation(G[128:256, i - 32:i].reshape(-1)).reshape(128, 32)
    else:
        got[b_off:b_off + o] = r.permutation(got[b_off:b_off + o])
    # the whole-update 2-norm check of old does not see it ...
    assert l2_rel(got, want) < 3e-2
    # ... the per-tile check does
    with pytest.raises(AssertionError):
        assert_tiles_close(got, want, dims)


def test_zero_tiles_do_not_divide_by_nothing():
    dims = [256, 256, 10]
    got, want = _step(dims, seed=3)
    (w_off, o, i, b_off) = mlp_layout(dims)[0]
    for a in (got, want):                    # dead hidden units: exact zeros on both sides
        a[w_off:w_off + 128 * i] = 0.0
        a[b_off:b_off + 128] = 0.0
    assert_tiles_close(got, want, dims)
    got[w_off + 5] = 1e-3                    # but a non-zero where zero is expected is an error
    with pytest.raises(AssertionError):
        assert_tiles_close(got, want, dims, frac=0.0, skip_rows=0)
