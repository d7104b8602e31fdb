"""Pins for the oracle's per-block path: nearest-entry encoding, reconstruction, the c-weighted
block cosine and squared error -- against exact-rational brute force, closed forms and invariants."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2605_14929_b200 import inputs as I

ATOMS4 = ["NF4", "SH4", "BOF4", "Split87"]


def _bf16(x):
    return I.snap_bf16(np.asarray(x, dtype=np.float32))


# ------------------------------------------------------------------ nearest-entry encode
@pytest.mark.parametrize("name", ATOMS4 + ["NF5", "SH5", "E2M2"])
def test_encode_is_exact_nearest_with_lowest_index_ties(name):
    a = I.rom_atom(name)
    lut = [Fraction(float(v)) for v in a.lut]
    rng = np.random.default_rng(7)
    us = list((rng.standard_normal(300) * 0.5 * a.tmax).astype(np.float32))
    us += [np.float32(float((lut[j] + lut[j + 1]) / 2)) for j in range(len(lut) - 1)]   # exact ties
    us += [np.float32(v) for v in a.lut]
    us += [np.float32(1e-30), np.float32(-1e-30), np.float32(3 * a.tmax), np.float32(-3 * a.tmax)]
    for u in us:
        fu = Fraction(float(u))
        want = min(range(len(lut)), key=lambda j: (abs(fu - lut[j]), j))
        assert oracle.encode_lut(a.lut, float(u)) == want, (name, float(u))


def test_tiny_u_between_symmetric_entries_is_not_a_false_tie():
    lut = np.array([-0.5, 0.5], np.float32)     # midpoint 0: any positive u is closer to +0.5
    assert oracle.encode_lut(lut, 1e-38) == 1
    assert oracle.encode_lut(lut, -1e-38) == 0
    assert oracle.encode_lut(lut, 0.0) == 0      # exact tie -> lowest index


# ------------------------------------------------------------------ reconstruction on the grid
@pytest.mark.parametrize("name", ATOMS4)
def test_values_on_the_grid_reconstruct_exactly(name):
    a = I.rom_atom(name)
    fmt = I.scale_format("E5M6")
    s = np.float32(0.03125)                     # a power of two: representable in E5M6, keeps w in bf16
    codes = np.random.default_rng(2).integers(0, 16, 16)
    codes[3] = 15                               # make sure the block max is the table max (1.0)
    w = (a.lut[codes].astype(np.float32) * s).astype(np.float32)
    assert np.all(_bf16(w) == w)
    c = np.random.default_rng(3).uniform(0.5, 2.0, 16).astype(np.float32)
    r = oracle.eval_block(w, c, a, fmt, 0)
    assert r["s_hat"] == s and list(r["codes"]) == list(codes)
    assert r["sse"] == 0.0
    assert abs(r["cos"] - 1.0) <= 2e-7


@pytest.mark.parametrize("kind", ["E2M3", "E4M3"])
def test_fp_values_on_the_grid_reconstruct_exactly(kind):
    a = I.fp_atom(kind)
    fmt = I.scale_format("E5M6")
    s = np.float32(2.0 ** -9)
    ncode = 32 if kind == "E2M3" else 127
    grid = np.array([oracle.fp_grid_value(a.kind, c) for c in range(ncode)], np.float32)
    codes = np.random.default_rng(4).integers(ncode // 2, ncode, 16)
    codes[0] = ncode - 1
    sign = np.where(np.arange(16) % 3 == 0, -1.0, 1.0).astype(np.float32)
    w = grid[codes] * s * sign
    r = oracle.eval_block(w, np.ones(16, np.float32), a, fmt, 0)
    assert r["sse"] == 0.0 and np.all(r["q"] == grid[codes] * sign)


# ------------------------------------------------------------------ block cosine
def test_single_nonzero_element_has_cosine_one():
    fmt = I.scale_format("E5M6")
    c = np.full(16, 0.7, np.float32)
    for name in ATOMS4:
        a = I.rom_atom(name)
        if 0.0 not in list(a.lut):
            continue
        for val in (0.5, -0.5):
            w = np.zeros(16, np.float32)
            w[5] = val
            cands = [a, a.negation()]
            got = [oracle.eval_block(w, c, x, fmt, 0)["cos"] for x in cands]
            # one of the two polarities maps the element onto an endpoint of magnitude 1
            assert max(got) == pytest.approx(1.0, abs=2e-7)


def test_zero_block_rules():
    fmt = I.scale_format("UE4M4")
    w = np.zeros(16, np.float32)
    c = np.ones(16, np.float32)
    r = oracle.eval_block(w, c, I.rom_atom("NF4"), fmt, 0)      # NF4 contains 0 -> q = 0 -> both norms zero
    assert r["cos"] == 1.0 and r["sse"] == 0.0 and r["s_hat"] == 0.0 and (r["E"], r["M"]) == (0, 0)
    r = oracle.eval_block(w, c, I.rom_atom("SH4"), fmt, 0)      # SH4 has no zero entry -> exactly one norm zero
    assert r["cos"] == 0.0


def test_block_cosine_matches_float64_definition_and_bounds():
    L = I.config1()
    c_all = oracle.channel_norms(L.X.numpy())
    W = L.W.float().numpy()
    fmt = I.scale_format("UE4M4")
    rng = np.random.default_rng(0)
    for name in ATOMS4 + ["E2M3"]:
        a = I.fp_atom(name) if name == "E2M3" else I.rom_atom(name)
        for _ in range(40):
            m, j = rng.integers(0, 256), rng.integers(0, 64)
            w = W[m, 16 * j:16 * j + 16]
            c = c_all[16 * j:16 * j + 16]
            r = oracle.eval_block(w, c, a, fmt, 1)
            q = r["q"].astype(np.float64)
            w64, c64 = w.astype(np.float64), c.astype(np.float64)
            cos = (c64 * w64 * q).sum() / np.sqrt((c64 * w64 * w64).sum() * (c64 * q * q).sum())
            sse = ((w64 - np.float64(r["s_hat"]) * q) ** 2).sum()
            assert r["cos"] == pytest.approx(cos, rel=2e-6)
            assert r["sse"] == pytest.approx(sse, rel=2e-5)
            assert abs(r["cos"]) <= 1.0 + 1e-6
            # reconstruction uses the table entry of the code
            if a.kind == I.KIND_LUT:
                assert np.all(r["q"] == a.lut[r["codes"]])
            # each code is the nearest entry to w / s_hat computed as w * (1 / s_hat)
            u = w * (np.float32(1.0) / np.float32(r["s_hat"]))
            if a.kind == I.KIND_LUT:
                assert [oracle.encode_lut(a.lut, float(x)) for x in u] == list(r["codes"])


def test_dropped_channel_weight_would_be_noticed():
    # the cosine must use c: with one dominant channel the value differs clearly from the unweighted one
    a = I.rom_atom("NF4")
    fmt = I.scale_format("E5M6")
    w = _bf16(np.random.default_rng(9).standard_normal(16) * 0.02)
    c1 = np.ones(16, np.float32)
    c2 = c1.copy()
    c2[int(np.argmin(np.abs(w)))] = 1000.0
    r1, r2 = oracle.eval_block(w, c1, a, fmt, 0), oracle.eval_block(w, c2, a, fmt, 0)
    assert list(r1["codes"]) == list(r2["codes"]) and r1["sse"] == r2["sse"]
    assert abs(r1["cos"] - r2["cos"]) > 1e-4


def test_power_of_two_rescaling_leaves_codes_and_cosine_unchanged():
    # per-block scale invariance: W * 2^j shifts the scale exponent only (F_layer shift k - j)
    a, fmt = I.rom_atom("SH4"), I.scale_format("UE4M4")
    w = _bf16(np.random.default_rng(11).standard_t(5, 16) * 0.02)
    c = np.random.default_rng(12).uniform(0.2, 3, 16).astype(np.float32)
    r0 = oracle.eval_block(w, c, a, fmt, 2)
    for j in (-3, 4):
        r = oracle.eval_block(w * np.float32(2.0 ** j), c, a, fmt, 2 - j)
        assert list(r["codes"]) == list(r0["codes"]) and (r["E"], r["M"]) == (r0["E"], r0["M"])
        assert r["cos"] == r0["cos"]
        assert r["sse"] == r0["sse"] * np.float32(4.0 ** j)


def test_negation_symmetry_per_block():
    # evaluating -a on -w gives the same codes, cosine and error as a on w, ties included
    fmt = I.scale_format("E5M6")
    rng = np.random.default_rng(21)
    for name in ATOMS4:
        a = I.rom_atom(name)
        for _ in range(20):
            w = _bf16(rng.standard_t(4, 16) * 0.015)
            c = rng.uniform(0.2, 3, 16).astype(np.float32)
            r0 = oracle.eval_block(w, c, a, fmt, 0)
            r1 = oracle.eval_block(-w, c, a.negation(), fmt, 0)
            assert list(r0["codes"]) == list(r1["codes"])
            assert r0["cos"] == r1["cos"] and r0["sse"] == r1["sse"]
            assert np.all(r0["q"] == -r1["q"])


def test_negated_candidate_equals_explicitly_negated_table():
    # -(lut) evaluated through the base table on -u reconstructs exactly like a table holding -lut
    fmt = I.scale_format("UE4M4")
    rng = np.random.default_rng(22)
    a = I.rom_atom("NF4")
    flipped = I.Atom("flipNF4", 4, I.KIND_LUT, 0, 16, 1.0, np.sort(-a.lut))
    for _ in range(30):
        w = _bf16(rng.standard_t(5, 16) * 0.02)
        c = rng.uniform(0.2, 3, 16).astype(np.float32)
        r0 = oracle.eval_block(w, c, a.negation(), fmt, 1)
        r1 = oracle.eval_block(w, c, flipped, fmt, 1)
        assert np.all(r0["q"] == r1["q"]) and r0["cos"] == r1["cos"] and r0["sse"] == r1["sse"]
