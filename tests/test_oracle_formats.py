"""Pins for the oracle's number formats: bpw arithmetic, scale-word layouts, the scale codec,
the F_layer shift and the FP element grids -- against values the paper prints and against
exact-rational brute force."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2605_14929_b200 import inputs as I

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                out.append(line.split())
    return out


# ------------------------------------------------------------------ bpw (paper's printed examples)
def test_bpw_examples_from_paper():
    for s, g, b, want in _rows("bpw_examples.txt"):
        assert oracle.bpw(int(s), int(g), int(b)) == float(want)


def test_payload_bytes_are_2n_at_g16():
    # Overview item 4: g = 16 makes n in {4, 5, 6} pack to 2n bytes of codes per block
    L = I.tiny_layer(1, 2, 32)
    c = np.ones(32, np.float32)
    fmt = I.scale_format("UE4M4")
    for name, n in (("NF4", 4), ("NF5", 5)):
        r = oracle.pack(L.W, c, fmt, I.rom_atom(name), 0, container_bits=8)
        assert r["rc"] == 0 and r["codes"].shape == (4, 2 * n)
    r = oracle.pack(L.W, c, fmt, I.fp_atom("E2M3"), 0, container_bits=8)
    assert r["codes"].shape == (4, 12)


def test_scale_traffic_fraction():
    # Section "Scaled Outer Product": 12*256 scale bits against 4*16*256 operand bits -> 15.8 %
    gold = {r[0]: (float(r[1]), float(r[2])) for r in _rows("hosting_ratios.txt")}
    scale_bits = 12 * 256
    operand_bits = oracle.bpw(0, 16, 4) * 16 * 256
    want, tol = gold["scale_traffic_fraction"]
    assert abs(scale_bits / (scale_bits + operand_bits) - want) <= tol


# ------------------------------------------------------------------ scale-word bit placement
@pytest.mark.parametrize("row", _rows("scale_word_layouts.txt"))
def test_scale_word_layout_examples(row):
    name, b, w, x, y, m, layout = row[0], *map(int, row[1:6]), row[6]
    assert len(layout) == b and b - w - x - y == m
    fmt = I.ScaleFormat(name, w, x, y, (1 << (x - 1)) - 1)
    # walk one bit at a time through every field and check where it lands
    pos = {ch: [b - 1 - i for i, c in enumerate(layout) if c == ch] for ch in "semu"}
    for i, p in enumerate(reversed(pos["m"])):          # mantissa bit i (LSB first)
        assert oracle.scale_word(fmt, b, w, 0, 0, 1 << i, 0) == 1 << p
    for i, p in enumerate(reversed(pos["e"])):
        assert oracle.scale_word(fmt, b, w, 0, 1 << i, 0, 0) == 1 << p
    if w:
        assert oracle.scale_word(fmt, b, w, 1, 0, 0, 0) == 1 << pos["s"][0]
    else:
        assert oracle.scale_word(fmt, b, w, 1, 0, 0, 0) == 0xFFFFFFFF   # no sign bit to use
    if m:
        sel = oracle.scale_word(fmt, b, w, 0, 0, 0, 1)
        first_meta = pos["u"][-1] if w else pos["u"][0]   # signed: LSB end; unsigned: bit b-1
        assert sel == 1 << first_meta
    else:
        assert oracle.scale_word(fmt, b, w, 0, 0, 0, 1) == 0xFFFFFFFF


# ------------------------------------------------------------------ scale codec
def _grid(fmt):
    """Every representable magnitude of the format, exactly, ascending, with its (E, M)."""
    out = []
    top = (1 << fmt.exp_bits) - (1 if fmt.top_exp_reserved else 0)
    for E in range(top):
        for M in range(1 << fmt.man_bits):
            if E == 0:
                v = Fraction(M, 1 << fmt.man_bits) * Fraction(2) ** (1 - fmt.bias)
            else:
                v = (1 + Fraction(M, 1 << fmt.man_bits)) * Fraction(2) ** (E - fmt.bias)
            out.append((v, E, M))
    return out


@pytest.mark.parametrize("name", ["UE4M4", "E4M3", "UE4M6", "E5M6", "UE5M7", "E4M7", "E8M7", "UE8M0", "UE5M3"])
def test_scale_codec_roundtrip_every_code(name):
    fmt = I.scale_format(name)
    grid = _grid(fmt)
    prev = Fraction(-1)
    for v, E, M in grid:
        if v == 0:
            continue
        assert v > prev          # monotone in the code
        prev = v
        f = float(v)
        if not (2.0 ** -126 <= f < 2.0 ** 127):
            continue             # outside fp32's normal range (E8M7 extremes)
        s_hat, e2, m2 = oracle.scale_quantize(fmt, f, 0)
        assert (e2, m2) == (E, M) and s_hat == f
        assert oracle.scale_decode(fmt, E, M, 0) == f


@pytest.mark.parametrize("name", ["UE4M4", "E4M3", "E5M6", "UE4M6"])
def test_scale_quantize_is_nearest_even_by_brute_force(name):
    fmt = I.scale_format(name)
    grid = [g for g in _grid(fmt) if g[0] > 0]
    rng = np.random.default_rng(5)
    lo, hi = float(grid[0][0]), float(grid[-1][0])
    samples = list(np.exp(rng.uniform(math.log(lo / 8), math.log(hi * 8), 400)).astype(np.float32))
    # adversarial: exact midpoints between neighbouring grid values
    for i in range(0, len(grid) - 1, max(1, len(grid) // 64)):
        samples.append(np.float32(float((grid[i][0] + grid[i + 1][0]) / 2)))
    for s in samples:
        v = Fraction(float(s))
        best = min(grid, key=lambda g: (abs(g[0] - v), g[2] & 1))   # nearest, ties to even mantissa
        if v > grid[-1][0]:
            best = grid[-1]                                           # saturate
        s_hat, E, M = oracle.scale_quantize(fmt, float(s), 0)
        assert (E, M) == (best[1], best[2]), (float(s), E, M, best)
        assert Fraction(s_hat) == best[0]


def test_scale_quantize_zero_and_tiny():
    fmt = I.scale_format("UE4M4")
    assert oracle.scale_quantize(fmt, 0.0, 3) == (0.0, 0, 0)
    s_hat, E, M = oracle.scale_quantize(fmt, 1e-12, 0)   # far below the smallest subnormal
    assert (E, M) == (0, 1) and s_hat == 2.0 ** (1 - 7 - 4)


def test_shift_is_exact_inside_normal_range():
    # paragraph "Per-layer scale shift (F_layer)": a format whose values are closed under scaling by powers of two
    # quantises a shifted scale to the shifted quantised scale, so the shift costs no accuracy
    fmt = I.scale_format("UE4M4")
    rng = np.random.default_rng(1)
    for s in rng.uniform(0.3, 3.0, 100).astype(np.float32):
        base, E0, M0 = oracle.scale_quantize(fmt, float(s), 0)
        for k in (-3, 2, 5):
            s_hat, E, M = oracle.scale_quantize(fmt, float(s) * 2.0 ** -k, k)
            assert (E, M) == (E0, M0) and s_hat == base * 2.0 ** -k


# ------------------------------------------------------------------ F_layer
def test_f_layer_returns_zero_when_everything_fits():
    fmt = I.scale_format("UE4M4")   # normal exponents -6 .. 8
    sig = np.exp2(np.random.default_rng(0).uniform(-6, 8.9, 1000)).astype(np.float32)
    assert oracle.f_layer(fmt, sig) == 0


def test_f_layer_shift_tracks_the_data():
    fmt = I.scale_format("UE4M4")
    sig = np.exp2(np.random.default_rng(0).normal(-12, 2.0, 5000)).astype(np.float32)
    k0 = oracle.f_layer(fmt, sig)
    assert k0 > 0
    for j in (-3, 4):
        assert oracle.f_layer(fmt, sig * np.float32(2.0 ** j)) == k0 - j
    # brute force over k: count exponents in range
    e = np.floor(np.log2(sig.astype(np.float64))).astype(int)
    counts = {k: int(((e + k >= -6) & (e + k <= 8)).sum()) for k in range(-64, 65)}
    best = max(counts.values())
    cands = [k for k, v in counts.items() if v == best]
    assert k0 == min(cands, key=lambda k: (abs(k), -k))


def test_f_layer_near_zero_for_five_exponent_bits():
    # the paper reports k* ~ 0 for E5-class scale formats and a positive shift for E4-class ones
    L = I.config1()
    w = L.W.float().numpy().reshape(-1, 16)
    sig = np.abs(w).max(axis=1) * np.float32(2.0 ** -4)   # small-magnitude layer
    assert oracle.f_layer(I.scale_format("E5M6"), sig) == 0
    assert oracle.f_layer(I.scale_format("UE4M4"), sig) > 0


# ------------------------------------------------------------------ FP element grids
def test_e2m3_grid_facts_from_paper():
    gold = {r[0]: float(r[1]) for r in _rows("hosting_ratios.txt")}
    vals = sorted({oracle.fp_grid_value(I.KIND_FP_E2M3, c) for c in range(64)})
    assert len(vals) == gold["E2M3_distinct_values"]
    mags = sorted(v for v in vals if v > 0)
    normals = [v for v in mags if v >= 1.0]
    assert max(mags) == 7.5
    assert max(normals) / min(normals) == gold["E2M3_normal_ratio"]
    assert max(mags) / min(mags) == gold["E2M3_subnormal_ratio"]


def test_e4m3_grid():
    vals = [oracle.fp_grid_value(I.KIND_FP_E4M3, c) for c in range(0x7F)]
    assert max(vals) == 448.0 and vals[1] == 2.0 ** -9 and vals[8] == 2.0 ** -6


@pytest.mark.parametrize("kind,ncode", [(I.KIND_FP_E2M3, 32), (I.KIND_FP_E4M3, 127)])
def test_fp_quantize_matches_rational_nearest_even(kind, ncode):
    grid = [(Fraction(oracle.fp_grid_value(kind, c)), c) for c in range(ncode)]
    rng = np.random.default_rng(3)
    top = float(grid[-1][0])
    xs = list(rng.uniform(-1.3 * top, 1.3 * top, 300).astype(np.float32))
    xs += list((rng.standard_normal(300) * 0.5).astype(np.float32))
    for i in range(len(grid) - 1):       # every midpoint, both signs
        mid = np.float32(float((grid[i][0] + grid[i + 1][0]) / 2))
        xs += [mid, -mid]
    for x in xs:
        v = abs(Fraction(float(x)))
        want = min(grid, key=lambda g: (abs(g[0] - v), g[1] & 1))
        q, code = oracle.fp_quantize(kind, float(x))
        sign_bit = ncode + 1 if kind == I.KIND_FP_E4M3 else ncode
        assert code & (sign_bit - 1) == want[1], (float(x), code, want)
        assert abs(Fraction(q)) == want[0]
        assert (q < 0) == (x < 0 and want[0] != 0) or q == 0


def test_layer_pot_scale_is_ceiling_power_of_two():
    for wmax in (0.37, 0.5, 448.0, 449.0, 3.1e-3):
        s = oracle.layer_pot_scale(wmax, 448.0)
        assert s == 2.0 ** math.ceil(math.log2(np.float32(wmax) / np.float32(448.0)))
        assert np.float32(wmax) / s <= 448.0      # never saturates
