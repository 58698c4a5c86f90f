"""Helpers shared by the tests: the error metric and problem builders that hand the same seeded
inputs to the CUDA library and to the CPU oracle."""
import numpy as np


def rel_err(x, y):
    """max_i |x_i - y_i| / max(|y_i|, rms(y)) -- relative error that stays defined where the
    reference element is near zero (y is the oracle's value)."""
    x = np.asarray(x, dtype=np.float64).reshape(-1)
    y = np.asarray(y, dtype=np.float64).reshape(-1)
    rms = float(np.sqrt(np.mean(y * y))) if y.size else 0.0
    den = np.maximum(np.abs(y), max(rms, 1e-30))
    return float((np.abs(x - y) / den).max()) if y.size else 0.0


def outlier_fraction(x, y, tol):
    """Fraction of elements whose error (same metric as rel_err) exceeds tol."""
    x = np.asarray(x, dtype=np.float64).reshape(-1)
    y = np.asarray(y, dtype=np.float64).reshape(-1)
    rms = float(np.sqrt(np.mean(y * y)))
    den = np.maximum(np.abs(y), max(rms, 1e-30))
    return float(np.mean(np.abs(x - y) / den > tol))


def l2_rel(x, y):
    x = np.asarray(x, dtype=np.float64).reshape(-1)
    y = np.asarray(y, dtype=np.float64).reshape(-1)
    return float(np.linalg.norm(x - y) / max(np.linalg.norm(y), 1e-30))


def mlp_layout(dims):
    """[(w_off, out, in, b_off)] of the flat per-replica layout [W_1 (out x in), b_1, W_2, ...]."""
    out, off = [], 0
    for l in range(len(dims) - 1):
        i, o = dims[l], dims[l + 1]
        out.append((off, o, i, off + o * i))
        off += o * i + o
    return out


def tile_errors(got, want, dims, tile=(128, 32), out_tol=5e-2, skip_rows=6):
    """Per output tile of every weight matrix (tile[0] rows x tile[1] columns, the unit a block of
    the tensor-core kernels produces) and per bias vector: (label, l2 error, outlier fraction).
    The l2 error of a tile is ||got - want|| over max(||want||, a quarter of what a tile of the
    layer's rms magnitude would weigh) -- the floor keeps tiles that are (nearly) all zero, e.g.
    rows of dead hidden units, from dividing by nothing.  The `skip_rows` rows of the tile with the
    largest error are left out of the norm: a hidden unit's pre-activation that lies within
    rounding of zero for one sample may take the other ReLU branch on the other side, which moves
    that one weight row by one sample's contribution (about 1/sqrt(B) of the row's update) and
    is a difference between two valid results, not a kernel error; a wrong tile is wrong in all
    its rows.  (Six rows of 128 is 5 %: with 64 to 128 samples and a few thousand units a learner's
    step sees a handful of such flips, and they cluster by row block, since a flipped unit moves
    its whole weight row, i.e. every column tile of that block.)  Outliers are elements whose error exceeds out_tol of max(|want_i|, rms of the
    layer); they are counted over the whole tile, skipped rows included."""
    got = np.asarray(got, dtype=np.float64).reshape(-1)
    want = np.asarray(want, dtype=np.float64).reshape(-1)
    res = []
    for l, (w_off, o, i, b_off) in enumerate(mlp_layout(dims), start=1):
        G = got[w_off:w_off + o * i].reshape(o, i)
        W = want[w_off:w_off + o * i].reshape(o, i)
        rms = max(float(np.sqrt(np.mean(W * W))), 1e-30)
        for r0 in range(0, o, tile[0]):
            for c0 in range(0, i, tile[1]):
                g = G[r0:r0 + tile[0], c0:c0 + tile[1]]
                w = W[r0:r0 + tile[0], c0:c0 + tile[1]]
                den = max(float(np.linalg.norm(w)), 0.25 * rms * np.sqrt(w.size))
                frac = float(np.mean(np.abs(g - w) / np.maximum(np.abs(w), rms) > out_tol))
                row_err = np.sort(((g - w) ** 2).sum(axis=1))
                keep = row_err[:max(len(row_err) - skip_rows, 1)]
                res.append((f"W{l}[{r0}:{r0 + tile[0]},{c0}:{c0 + tile[1]}]",
                            float(np.sqrt(keep.sum())) / den, frac))
        gb, wb = got[b_off:b_off + o], want[b_off:b_off + o]
        rb = max(float(np.sqrt(np.mean(wb * wb))), 1e-30)
        den = max(float(np.linalg.norm(wb)), 0.25 * rb * np.sqrt(o))
        frac = float(np.mean(np.abs(gb - wb) / np.maximum(np.abs(wb), rb) > out_tol))
        el_err = np.sort((gb - wb) ** 2)
        keep = el_err[:max(len(el_err) - skip_rows * max(1, o // tile[0]), 1)]
        res.append((f"b{l}", float(np.sqrt(keep.sum())) / den, frac))
    return res


def assert_tiles_close(got, want, dims, l2_tol=2e-2, out_tol=5e-2, frac=0.05, tile=(128, 32),
                       what="", skip_rows=6):
    """Every tile and every bias vector within l2_tol in the 2-norm (its skip_rows worst rows left
    out, see tile_errors) and with at most `frac` of its elements beyond out_tol: one wrong edge
    tile fails, however small its share of the layer."""
    bad = [(lab, e, f) for lab, e, f in tile_errors(got, want, dims, tile, out_tol, skip_rows)
           if e > l2_tol or f > frac]
    assert not bad, f"{what}: {len(bad)} tile(s) off, worst first: " + \
        ", ".join(f"{lab} l2={e:.3g} out={f:.3g}" for lab, e, f in
                  sorted(bad, key=lambda t: -t[1])[:4])
