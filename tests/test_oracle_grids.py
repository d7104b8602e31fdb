"""Pins for the oracle's parametric element grids (promotion-profile formats; HIF7 / HIF8).  The grid
is pinned to the numbers the paper prints (80 / 96 values, ratios 120 / 240, E2M5 tops out at 3.94),
to the two element formats that already have their own pinned quantiser (E2M3, E4M3), and to an
exact-rational nearest-value search over the enumerated grid."""
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2605_14929_b200 import inputs as I

GOLD = {}
with open(os.path.join(os.path.dirname(__file__), "golden", "hosting_ratios.txt")) as fh:
    for line in fh:
        if line.strip() and not line.startswith("#"):
            k, v, tol = line.split()
            GOLD[k] = (float(v), float(tol))


def two_complement_products(shifts):
    return sorted({c * (1 << s) for c in range(-16, 16) for s in shifts})


def grid_values(a):
    """Every value of the grid, ascending, from the oracle's own value function."""
    x, y, bias, neg_max = a.grid
    mags, j = [], 0
    while oracle.grid_value(a, j) <= neg_max:
        mags.append(oracle.grid_value(a, j))
        j += 1
    mags = np.array(mags)
    return np.concatenate([-mags[:0:-1], mags[mags <= a.tmax]])


@pytest.mark.parametrize("name,shifts", [("HIF7", range(4)), ("HIF8", range(5))])
def test_hif_grids_are_the_coefficient_times_shift_products(name, shifts):
    a = I.fp_atom(name)
    want = two_complement_products(shifts)            # tc5 coefficient times 2^shift, as the datapath forms them
    got = grid_values(a)
    assert list(got) == [float(v) for v in want]
    assert len(got) == GOLD[name + "_distinct_values"][0]
    normal = [v for v in want if v >= 8]              # the normal range starts where the coefficient has its top bit
    assert max(want) / 1.0 == GOLD[name + "_normal_ratio"][0] and min(abs(v) for v in want if v) == 1
    assert max(normal) == a.tmax and -min(want) == a.grid[3]


def test_e2m5_tops_out_where_the_paper_says():
    a = I.fp_atom("E2M5")
    v, tol = GOLD["E2M5_format_max"]
    assert abs(a.tmax - v) <= tol and grid_values(a).max() == a.tmax
    assert len(grid_values(a)) == 2 * (3 * 32 - 1) + 1        # three exponent codes in use, one shared zero


@pytest.mark.parametrize("kind,x,bias,vmax", [(I.KIND_FP_E2M3, 2, 1, 7.5), (I.KIND_FP_E4M3, 4, 7, 448.0)])
def test_parametric_grid_reproduces_the_two_named_formats(kind, x, bias, vmax):
    a = I.Atom("g", 1 + x + 3, I.KIND_FP_GRID, 0, I.SCOPE_BLOCK, vmax, None, (x, 3, bias, vmax))
    rng = np.random.default_rng(0)
    us = np.concatenate([rng.standard_normal(4000) * vmax / 3, rng.standard_normal(2000) * 2.0 ** -6,
                         np.linspace(-1.2 * vmax, 1.2 * vmax, 3001), [0.0, -0.0]]).astype(np.float32)
    # every midpoint between neighbouring values and its fp32 neighbours
    g = grid_values(a)
    mids = ((g[1:] + g[:-1]) / 2).astype(np.float32)
    us = np.concatenate([us, mids, np.nextafter(mids, np.float32(np.inf)), np.nextafter(mids, np.float32(-np.inf))])
    for u in us:
        q1, c1 = oracle.grid_quantize(a, float(u))
        q0, c0 = oracle.fp_quantize(kind, float(u))
        assert (q1, c1) == (q0, c0), u


@pytest.mark.parametrize("name", ["HIF7", "HIF8", "E3M4", "E2M5", "E3M6"])
def test_grid_quantiser_is_the_exact_nearest_value_with_ties_to_even(name):
    a = I.fp_atom(name)
    g = [Fraction(float(v)) for v in grid_values(a)]
    zero = g.index(0)
    rng = np.random.default_rng(1)
    us = np.concatenate([rng.standard_normal(600) * a.tmax / 2.5, rng.standard_normal(200) * a.tmax / 200,
                         [a.tmax * 1.01, -a.grid[3] * 1.01, a.tmax, -a.grid[3], 0.0]]).astype(np.float32)
    gf = np.array([float(v) for v in g])
    mids = ((gf[1:] + gf[:-1]) / 2).astype(np.float32)
    us = np.concatenate([us, mids[:: max(1, len(mids) // 120)]])
    for u in us:
        fu = Fraction(float(u))
        dist = [abs(fu - v) for v in g]
        dmin = min(dist)
        cands = [i for i, d in enumerate(dist) if d == dmin]
        if len(cands) == 2:                           # a tie: the even magnitude number wins
            cands = [i for i in cands if abs(i - zero) % 2 == 0]
        q, code = oracle.grid_quantize(a, float(u))
        assert Fraction(q) == g[cands[0]], (name, u)
        assert (code & ~(1 << (a.n_bits - 1 if a.grid[0] == 0 else a.grid[0] + a.grid[1]))) == abs(cands[0] - zero)
    # values on the grid are fixed points
    for v in gf:
        assert oracle.grid_quantize(a, float(v))[0] == v


def test_block_evaluation_on_a_grid_format():
    # a block whose elements sit on s * grid reconstructs exactly; the scale is taken against the positive maximum
    a = I.fp_atom("HIF7")
    fmt = I.scale_format("E5M6")
    vals = np.array([120, -128, 15, -16, 8, 1, 0, -1, 64, 72, -7, 30, 2, 3, -60, 104], dtype=np.float32) * 2.0 ** -9
    c = np.linspace(0.5, 2.0, 16).astype(np.float32)
    vals2 = vals.copy()
    vals2[1] = -120 * 2.0 ** -9                        # now absmax / tmax is a power of two: exact reconstruction
    ev = oracle.eval_block(vals2, c, a, fmt, 0)
    assert ev["s_hat"] == 2.0 ** -9 and ev["sse"] == 0.0 and ev["cos"] == pytest.approx(1.0, abs=2e-7)
    assert np.array_equal(ev["q"] * np.float32(ev["s_hat"]), vals2)
    # a finer grid never reconstructs a block worse than a coarser one with the same range (E3M6 refines E3M4)
    L = I.tiny_layer(2, 4, 64)
    cc = oracle.channel_norms(L.X.numpy())
    r = oracle.pair_search(L.W, cc, I.scale_format("UE4M4"), [I.fp_atom("E3M4"), I.fp_atom("E3M6")], want_blocks=True)
    assert r["pair"]["mse"][1, 1] < r["pair"]["mse"][0, 0]
