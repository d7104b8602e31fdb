"""Pins of the oracle's grid-constrained DD-n construction (Section "Per-Layer Pair Search", steps 1 and 3:
histogram-DP cluster selection on the grid points of the LUT value format): exhaustive search over every way of
cutting a small histogram into runs, the optimality of the dynamic programme against other tables on the same
histogram, and data that already lies on 2^n grid points."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2605_14929_b200 import inputs as I

FIX = 16777216.0


def histogram(W, c, fmt, k):
    """Per cell (H, S, Q) as Python integers, from the layer's elements with every block in the pool: the same
    definition as the oracle's, written with numpy fp32 operations."""
    Wf = W.to(torch.float32).numpy()
    M, K = Wf.shape
    om = (c / c.max()).astype(np.float32)
    H, S, Q = {}, {}, {}
    for m in range(M):
        for j in range(K // 16):
            w = Wf[m, 16 * j:16 * j + 16]
            s_hat = np.float32(oracle.scale_quantize(fmt, float(np.abs(w).max()), k)[0])
            rcp = np.float32(1.0) / s_hat if s_hat > 0 else np.float32(0.0)
            u = (w * rcp).astype(np.float32)
            o = om[16 * j:16 * j + 16]
            cell = np.clip(np.rint(u.astype(np.float64) * 256.0), -320, 320).astype(int)
            ou = np.clip((o * u).astype(np.float32), np.float32(-256), np.float32(256))
            ouu = (ou * u).astype(np.float32)
            for r in range(16):
                t = int(cell[r])
                H[t] = H.get(t, 0) + int(np.rint(np.float64(o[r]) * FIX))
                S[t] = S.get(t, 0) + int(np.rint(np.float64(ou[r]) * FIX))
                Q[t] = Q.get(t, 0) + int(np.rint(np.float64(ouu[r]) * FIX))
    cells = sorted(t for t in H if H[t] > 0)
    return [(H[t], S[t], Q[t]) for t in cells]


def run_cost(cells):
    """Code point and cost of one run of cells, with the oracle's operations in Python floats (IEEE double)."""
    h = float(sum(x[0] for x in cells)); s = float(sum(x[1] for x in cells)); q2 = float(sum(x[2] for x in cells))
    q = float(I.snap_bf16(np.float32(s / h)))
    q = min(1.25, max(-1.25, q))
    return q, (q2 - (2.0 * q) * s) + (q * q) * h


def brute_force(hist, n_runs):
    B = len(hist)
    best = None
    for cuts in itertools.combinations(range(1, B), n_runs - 1):
        edges = (0,) + cuts + (B,)
        qs, total = [], 0.0
        # the same association as the dynamic programme: the runs' costs added from the first run on
        for a, b in zip(edges[:-1], edges[1:]):
            q, cst = run_cost(hist[a:b])
            qs.append(q)
            total = total + cst if qs[:-1] else cst
        if best is None or total < best[0]:
            best = (total, sorted(qs))
    return best


def eighths_layer(seed, M, K):
    """Weights that are multiples of 1/8 with a block maximum of exactly 1, so that u = w and few cells are hit."""
    rng = np.random.default_rng(seed)
    w = rng.choice(np.arange(-8, 8) / 8.0, size=(M, K), p=None)
    w[:, ::16] = 1.0
    W = torch.from_numpy(w.astype(np.float32)).to(torch.bfloat16)
    c = np.exp(rng.normal(0, 0.7, K)).astype(np.float32)
    return W, c


@pytest.mark.parametrize("seed,n_values,n_entries", [(1, 9, 2), (2, 11, 3), (3, 12, 3), (4, 7, 4)])
def test_dynamic_programme_equals_exhaustive_search(seed, n_values, n_entries):
    W, c = eighths_layer(seed, 6, 64)
    vals = np.sort(np.random.default_rng(seed).choice(np.arange(-8, 8), n_values - 1, replace=False)) / 8.0
    Wf = W.to(torch.float32).numpy()
    keep = np.isin(Wf, vals) | (Wf == 1.0)
    Wf = np.where(keep, Wf, vals[0])
    W = torch.from_numpy(Wf.astype(np.float32)).to(torch.bfloat16)
    fmt = I.scale_format("E5M6")
    hist = histogram(W, c, fmt, 0)
    assert n_entries < len(hist) <= 12
    NB = W.shape[0] * W.shape[1] // 16
    lut, cost, cnt = oracle.dd_grid_dp(W, c, fmt, 0, np.ones(NB, np.float32), NB, n_entries)
    want_cost, want_lut = brute_force(hist, n_entries)
    assert cnt == NB
    assert cost == want_cost / FIX
    assert list(lut) == want_lut


def model_cost(hist, table):
    """Cost of a given table on the histogram when every cell goes to its best entry."""
    total = 0.0
    for h, s, q2 in hist:
        total += min((float(q2) - 2.0 * float(q) * float(s)) + float(q) * float(q) * float(h) for q in table)
    return total / FIX


@pytest.mark.parametrize("fmt_name,n_bits", [("UE4M4", 4), ("E5M6", 5)])
def test_dynamic_programme_beats_every_other_table_on_its_histogram(fmt_name, n_bits):
    L = I.config1()
    L = I.Layer(L.W[:24].contiguous(), L.X)
    fmt = I.scale_format(fmt_name)
    c = oracle.channel_norms(L.X.numpy())
    atoms = I.alphabet(["NF4" if n_bits == 4 else "NF5"], with_negations=False)
    r = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True)
    NB = r["block_cos"].shape[1]
    k = int(r["k"][0])
    lut, cost, cnt = oracle.dd_grid_dp(L.W, c, fmt, k, r["block_cos"][0], NB // 2, 1 << n_bits)
    assert np.all(np.diff(lut) >= 0) and np.array_equal(lut, I.snap_bf16(lut)) and np.abs(lut).max() <= 1.25
    # the histogram of the same pool, through the Lloyd construction's pool rule
    tau = np.sort(r["block_cos"][0])[NB // 2 - 1]
    pool = r["block_cos"][0] <= tau
    assert cnt == int(pool.sum())
    nbk = L.W.shape[1] // 16
    rows = [L.W[m, 16 * j:16 * j + 16] for m in range(L.W.shape[0]) for j in range(nbk) if pool[m * nbk + j]]
    cs = [c[16 * j:16 * j + 16] for m in range(L.W.shape[0]) for j in range(nbk) if pool[m * nbk + j]]
    Wp = torch.stack(rows)                     # one block per row: blocks keep their own maxima and channels
    hist = {}
    om_max = c.max()
    for w, cc in zip(Wp, cs):
        for h, s, q2, t in _cells_of_block(w, cc / om_max, fmt, k):
            a = hist.setdefault(t, [0, 0, 0])
            a[0] += h; a[1] += s; a[2] += q2
    hist = [tuple(hist[t]) for t in sorted(hist) if hist[t][0] > 0]
    assert cost <= model_cost(hist, lut) * (1 + 1e-12) + 1e-12
    lloyd = oracle.dd_lloyd(L.W, c, fmt, k, r["block_cos"][0], NB // 2, atoms[0].lut, 8)[0]
    rng = np.random.default_rng(3)
    others = [lloyd, atoms[0].lut] + [np.sort(I.snap_bf16(rng.uniform(-1, 1, 1 << n_bits))) for _ in range(20)]
    for t in others:
        assert cost <= model_cost(hist, t) + 1e-9


def _cells_of_block(w, om, fmt, k):
    w = w.to(torch.float32).numpy()
    s_hat = np.float32(oracle.scale_quantize(fmt, float(np.abs(w).max()), k)[0])
    rcp = np.float32(1.0) / s_hat if s_hat > 0 else np.float32(0.0)
    u = (w * rcp).astype(np.float32)
    om = om.astype(np.float32)
    cell = np.clip(np.rint(u.astype(np.float64) * 256.0), -320, 320).astype(int)
    ou = np.clip((om * u).astype(np.float32), np.float32(-256), np.float32(256))
    ouu = (ou * u).astype(np.float32)
    for r in range(16):
        yield (int(np.rint(np.float64(om[r]) * FIX)), int(np.rint(np.float64(ou[r]) * FIX)),
               int(np.rint(np.float64(ouu[r]) * FIX)), int(cell[r]))


def test_data_on_grid_points_is_reproduced():
    # sixteen grid points in sixteen cells, every block maximum 1 and a scale format that holds 1 exactly: u = w,
    # the table is those points and nothing is lost (up to the rounding of the fixed-point sums)
    pts = np.array([-1.0, -0.75, -0.5, -0.375, -0.25, -0.125, -0.0625, 0.0, 0.0625, 0.125, 0.25, 0.375, 0.5, 0.625, 0.75, 1.0], np.float32)
    rng = np.random.default_rng(0)
    w = rng.choice(pts, size=(8, 128))
    w[:, ::16] = 1.0
    W = torch.from_numpy(w).to(torch.bfloat16)
    c = np.exp(rng.normal(0, 0.5, 128)).astype(np.float32)
    NB = 8 * 8
    lut, cost, cnt = oracle.dd_grid_dp(W, c, I.scale_format("E5M6"), 0, np.zeros(NB, np.float32), NB, 16)
    assert np.array_equal(lut, pts) and cnt == NB
    assert abs(cost) < 1e-4
    # fewer distinct values than entries: the table is padded with its last entry
    w2 = np.where(np.isin(w, pts[::3]) | (w == 1.0), w, 0.0).astype(np.float32)
    lut2, _, _ = oracle.dd_grid_dp(torch.from_numpy(w2).to(torch.bfloat16), c, I.scale_format("E5M6"), 0, np.zeros(NB, np.float32), NB, 16)
    assert set(lut2) == set(np.unique(w2)) and np.all(np.diff(lut2) >= 0)
