"""Pins for the oracle's layer-level steps: channel norms, the pair tables (brute force over all
selector vectors on tiny layers), sign-negation symmetry of the whole sweep, the DD-n Lloyd
iteration (fixed points, monotone distortion, exhaustive optimum) and the packer."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2605_14929_b200 import inputs as I


# ------------------------------------------------------------------ channel norms
def test_channel_norms_closed_forms():
    X = np.zeros((100, 4), np.float32)
    X[:, 0] = 3.0                       # constant column -> 3
    X[::2, 1] = 2.0                     # half the rows -> 2 / sqrt(2)
    X[:, 2] = np.where(np.arange(100) % 2, -1.5, 1.5)   # sign does not matter
    c = oracle.channel_norms(X)
    assert c[0] == 3.0 and c[2] == 1.5 and c[3] == 0.0
    assert c[1] == np.float32(np.sqrt(2.0))


def test_channel_norms_match_float64_rms():
    X = I.config1().X.numpy()
    c = oracle.channel_norms(X)
    ref = np.sqrt((X.astype(np.float64) ** 2).mean(axis=0))
    assert np.max(np.abs(c.astype(np.float64) - ref) / ref) < 1e-7
    assert c.shape == (1024,)


# ------------------------------------------------------------------ pair tables
def _tiny(seed, M=2, K=64):
    L = I.tiny_layer(seed, M, K)
    c = oracle.channel_norms(L.X.numpy())
    return L, c


def test_pair_table_equals_brute_force_over_selectors():
    # ACos is a mean of independent per-block terms, so the best selector vector is the per-block
    # best; enumerate all 2^Nb vectors on an 8-block layer and compare.
    L, c = _tiny(3)                                  # 2 x 64 -> 8 blocks
    fmt = I.scale_format("UE4M4")
    atoms = I.alphabet(["NF4", "SH4"])
    r = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True)
    bc, bs = r["block_cos"].astype(np.float64), r["block_sse"].astype(np.float64)
    nb = bc.shape[1]
    assert nb == 8
    for a, b in itertools.combinations(range(len(atoms)), 2):
        best = max(sum(bc[b if (sel >> i) & 1 else a, i] for i in range(nb)) for sel in range(1 << nb))
        assert r["pair"]["acos"][a, b] == pytest.approx(best / nb, rel=1e-12)
        mu = bc[b] > bc[a]
        assert r["pair"]["n_sel1"][a, b] == int(mu.sum())
        assert r["pair"]["mse"][a, b] == pytest.approx(np.where(mu, bs[b], bs[a]).sum() / (2 * 64), rel=1e-12)
        assert r["pair"]["acos"][a, b] >= max(r["pair"]["acos"][a, a], r["pair"]["acos"][b, b])
    for a in range(len(atoms)):
        assert r["pair"]["acos"][a, a] == pytest.approx(bc[a].mean(), rel=1e-12)
        assert r["pair"]["n_sel1"][a, a] == 0


def test_signed_table_is_best_of_four_and_contains_the_two_way_result():
    L, c = _tiny(4, 4, 64)
    fmt = I.scale_format("S1E4M4")
    atoms = I.alphabet(["NF4", "SH4", "BOF4"])
    r = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True)
    bc = r["block_cos"].astype(np.float64)
    for i, j in ((0, 2), (0, 4), (2, 4)):
        four = np.stack([bc[i], bc[i + 1], bc[j], bc[j + 1]])
        assert r["signed"]["acos"][i, j] == pytest.approx(four.max(axis=0).mean(), rel=1e-12)
        pick = four.argmax(axis=0)                  # numpy argmax keeps the first maximum: same priority
        assert r["signed"]["n_sel1"][i, j] == int((pick >= 2).sum())
        assert r["signed"]["n_neg"][i, j] == int((pick % 2 == 1).sum())
        assert r["signed"]["acos"][i, j] >= r["pair"]["acos"][i, j]
    assert r["signed"]["n_sel1"][1, 3] == -1        # negated entries are not bases
    # unsigned format: no signed table
    r2 = oracle.pair_search(L.W, c, I.scale_format("UE4M4"), atoms)
    assert np.all(r2["signed"]["n_sel1"] == -1)


def test_fp_candidates_are_singles_only_and_best_pair_rule():
    L, c = _tiny(5, 4, 64)
    atoms = I.alphabet(["NF4", "SH4"], fp=["E2M3", "E4M3", "E4M3^0"])
    r = oracle.pair_search(L.W, c, I.scale_format("UE4M4"), atoms)
    n = r["pair"]["n_sel1"]
    assert np.all(n[:4, 4:] == -1) and np.all(n[4:, 4:][~np.eye(3, dtype=bool)] == -1)
    assert np.all(np.diag(n) == 0)
    pairs = [(r["pair"]["acos"][a, b], -a, -b) for a in range(4) for b in range(a + 1, 4)]
    top = max(pairs)
    assert (r["best"][0], r["best"][1]) == (-top[1], -top[2])
    assert r["best"][2] == int(np.argmax(np.diag(r["pair"]["acos"])[:4]))
    # more element bits -> better fidelity on bell-shaped weights
    d = np.diag(r["pair"]["acos"])
    assert d[4] > d[0] and d[5] > d[0]


def test_sweep_of_negated_weights_swaps_each_atom_with_its_negation():
    L, c = _tiny(6, 8, 128)
    fmt = I.scale_format("E5M6")
    atoms = I.alphabet(["NF4", "SH4", "Split87"])
    r0 = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True)
    r1 = oracle.pair_search(-L.W, c, fmt, atoms, want_blocks=True)
    perm = [1, 0, 3, 2, 5, 4]
    assert np.array_equal(r0["block_cos"], r1["block_cos"][perm])
    assert np.array_equal(r0["block_sse"], r1["block_sse"][perm])
    assert np.array_equal(r0["k"], r1["k"])


def test_f_layer_shift_invariance_of_the_whole_sweep():
    # scaling W by 2^j moves k* by -j and leaves every cosine, and every count, unchanged
    L, c = _tiny(7, 8, 128)
    fmt = I.scale_format("UE4M4")
    atoms = I.alphabet(["NF4", "BOF4"])
    small = (L.W.float() * 2.0 ** -9).to(torch.bfloat16)
    r0 = oracle.pair_search(small, c, fmt, atoms, want_blocks=True)
    r1 = oracle.pair_search((small.float() * 8.0).to(torch.bfloat16), c, fmt, atoms, want_blocks=True)
    assert r0["k"][0] > 0 and np.array_equal(r1["k"], r0["k"] - 3)
    assert np.array_equal(r0["block_cos"], r1["block_cos"])
    assert np.array_equal(r0["pair"]["n_sel1"], r1["pair"]["n_sel1"])


def test_soft_checks_against_paper_ranges():
    # ACos at 4-bit pairs typically 0.997-0.999; block-scaled E2M3 beats layer-POT E4M3 in MSE
    L = I.config1()
    c = oracle.channel_norms(L.X.numpy())
    atoms = I.alphabet(["NF4", "SH4", "BOF4"], fp=["E2M3", "E4M3^0"])
    r = oracle.pair_search(L.W, c, I.scale_format("UE4M4"), atoms)
    best = r["pair"]["acos"][r["best"][0], r["best"][1]]
    assert 0.996 < best < 0.9995
    mse = np.diag(r["pair"]["mse"])
    assert mse[6] < mse[7]


# ------------------------------------------------------------------ Lloyd
def _grid_layer(lut, seed, M=8, K=64):
    """Weights lying exactly on s * lut with power-of-two block scales."""
    rng = np.random.default_rng(seed)
    codes = rng.integers(0, len(lut), (M, K))
    codes[:, ::16] = len(lut) - 1
    scale = np.exp2(rng.integers(-8, -3, (M, K // 16))).repeat(16, axis=1)
    return torch.from_numpy((lut[codes] * scale).astype(np.float32)).to(torch.bfloat16)


def test_lloyd_fixed_point_when_data_lies_on_the_table():
    lut = I.rom_atom("NF4").lut
    W = _grid_layer(lut, 0)
    NB = 8 * 4
    c = np.ones(64, np.float32)
    out, dist, cnt = oracle.dd_lloyd(W, c, I.scale_format("E5M6"), 0, np.zeros(NB, np.float32), NB, lut, 3)
    assert cnt == NB and np.array_equal(out, lut) and np.all(dist == 0.0)


def test_lloyd_pool_rule_and_distortion_decrease():
    L = I.config1()
    c = oracle.channel_norms(L.X.numpy())
    fmt = I.scale_format("UE4M4")
    nf4 = I.rom_atom("NF4")
    r = oracle.pair_search(L.W, c, fmt, [nf4], want_blocks=True)
    bc = r["block_cos"][0]
    NB = bc.size
    rank = NB // 2
    out, dist, cnt = oracle.dd_lloyd(L.W, c, fmt, int(r["k"][0]), bc, rank, nf4.lut, 8)
    tau = np.sort(bc)[rank - 1]
    assert cnt == int((bc <= tau).sum()) and cnt >= rank
    assert np.all(np.diff(out) >= 0) and np.all(I.snap_bf16(out) == out)
    # snapping to bf16 perturbs each step by < 2^-8 relative, far below the gains of early iterations
    assert dist[-1] < dist[0] * 0.9
    assert np.all(dist[1:] <= dist[:-1] * (1 + 1e-3))
    # the refined table reconstructs the pool better than the ROM table it started from
    dd = I.Atom("DD4", 4, I.KIND_LUT, 0, 16, 1.0, out)
    r2 = oracle.pair_search(L.W, c, fmt, [nf4, dd], k_mode=int(r["k"][0]), want_blocks=True)
    pool = bc <= tau
    assert r2["block_cos"][1][pool].mean() > r2["block_cos"][0][pool].mean()
    assert r2["pair"]["acos"][0, 1] > r2["pair"]["acos"][0, 0]


def test_lloyd_single_update_equals_weighted_means_and_bounds_exhaustive_optimum():
    # 12 points, 2 levels: one update from a given split must give the omega-weighted means of the
    # two cells (up to bf16 snapping), and no 2-level table can beat the exhaustive optimum.
    rng = np.random.default_rng(5)
    u = np.sort(I.snap_bf16(rng.uniform(-1, 1, 12)))
    u[-1] = 1.0
    w = np.zeros((1, 16), np.float32)
    w[0, :12] = u * 0.25                      # block absmax 0.25 -> scale 0.25 exactly, u recovered exactly
    W = torch.from_numpy(w).to(torch.bfloat16)
    c = np.ones(16, np.float32)
    c[:12] = rng.uniform(0.5, 1.0, 12).astype(np.float32)
    c[12:] = 1.0                              # four padding zeros carry weight too
    fmt = I.scale_format("E5M6")
    init = np.array([-0.5, 0.5], np.float32)
    out, dist, _ = oracle.dd_lloyd(W, c, fmt, 0, np.zeros(1, np.float32), 1, init, 1)
    pts = np.concatenate([u.astype(np.float64), np.zeros(4)])
    om = (c / c.max()).astype(np.float64)
    lo = pts <= 0.0                           # threshold of the initial table is 0; ties go low
    want = [np.sum(om[lo] * pts[lo]) / om[lo].sum(), np.sum(om[~lo] * pts[~lo]) / om[~lo].sum()]
    assert np.allclose(out, want, rtol=2 ** -8)
    d_before = np.sum(om * (pts - np.where(lo, -0.5, 0.5)) ** 2)
    assert dist[0] == pytest.approx(d_before, rel=1e-9)
    order = np.argsort(pts)
    p, o = pts[order], om[order]
    best = min(
        np.sum(o[:i] * (p[:i] - np.sum(o[:i] * p[:i]) / o[:i].sum()) ** 2)
        + np.sum(o[i:] * (p[i:] - np.sum(o[i:] * p[i:]) / o[i:].sum()) ** 2)
        for i in range(1, 16))
    out8, dist8, _ = oracle.dd_lloyd(W, c, fmt, 0, np.zeros(1, np.float32), 1, init, 8)
    assert dist8[-1] >= best * (1 - 1e-9)
    assert dist8[-1] <= dist8[0]


# ------------------------------------------------------------------ pack
def _unpack_codes(codes, n):
    bits = np.unpackbits(codes, axis=1, bitorder="little")
    return (bits.reshape(codes.shape[0], 16, n) * (1 << np.arange(n))).sum(axis=2)


def _unpack_words(words, b, count):
    bits = np.unpackbits(words, bitorder="little")[: count * b].reshape(count, b)
    return (bits.astype(np.int64) * (1 << np.arange(b))).sum(axis=1)


def test_pack_roundtrip_pair_with_sign_and_selector():
    L, c = _tiny(8, 4, 64)
    fmt = I.scale_format("S1E4M4")                 # "UE4M4 signed": 12-bit word, sign + selector
    a, b = I.rom_atom("NF4"), I.rom_atom("SH4")
    r = oracle.pack(L.W, c, fmt, a, 1, b, 1, use_sign=1, container_bits=12, word_sign_bits=1)
    assert r["rc"] == 0
    NB = 16
    assert r["codes"].shape == (NB, 8) and r["words"].size == NB * 12 // 8
    codes = _unpack_codes(r["codes"], 4)
    words = _unpack_words(r["words"], 12, NB)
    W = L.W.float().numpy().reshape(NB, 16)
    cb = np.tile(c.reshape(-1, 16), (4, 1))
    n1 = nneg = 0
    for i in range(NB):
        sign, sel = (words[i] >> 11) & 1, words[i] & 1
        E, M = (words[i] >> 7) & 15, (words[i] >> 3) & 15
        assert (words[i] >> 1) & 3 == 0            # unused metabits are zero
        n1 += sel
        nneg += sign
        base = b if sel else a
        cand = base.negation() if sign else base
        ev = oracle.eval_block(W[i], cb[i], cand, fmt, 1)
        assert (ev["E"], ev["M"]) == (E, M) and list(ev["codes"]) == list(codes[i])
        # decoder view: value = (+-s_hat) * lut[code]
        s = oracle.scale_decode(fmt, int(E), int(M), 1) * (-1.0 if sign else 1.0)
        assert np.array_equal(np.float32(s) * base.lut[codes[i]], np.float32(ev["s_hat"]) * ev["q"])
        # and the chosen candidate is the best of the four, earliest on ties
        four = [oracle.eval_block(W[i], cb[i], x, fmt, 1)["cos"] for x in (a, a.negation(), b, b.negation())]
        assert int(np.argmax(four)) == 2 * sel + sign
    assert (r["n_sel1"], r["n_neg"]) == (n1, nneg)


def test_pack_layouts_and_errors():
    L, c = _tiny(9, 2, 64)
    a, b = I.rom_atom("NF5"), I.rom_atom("SH5")
    ue = I.scale_format("UE4M4")
    # unsigned 8-bit word has no metabit: a pair cannot be packed into it
    assert oracle.pack(L.W, c, ue, a, 0, b, 0, container_bits=8)["rc"] == -1
    # sign requested from a word without a sign bit
    assert oracle.pack(L.W, c, ue, a, 0, None, 0, use_sign=1, container_bits=12)["rc"] == -1
    # S0E4M4 in 12 bits: selector at bit 11, magnitude at bits 3..10
    r = oracle.pack(L.W, c, ue, a, 0, b, 0, container_bits=12, word_sign_bits=0)
    assert r["rc"] == 0 and r["codes"].shape == (8, 10)
    words = _unpack_words(r["words"], 12, 8)
    assert np.all(words & 7 == 0)
    assert int(((words >> 11) & 1).sum()) == r["n_sel1"]
    # single FP6 atom with the byte-wide unsigned scale: 12 + 1 bytes per block -> 6.5 bpw
    r = oracle.pack(L.W, c, ue, I.fp_atom("E2M3"), 0, container_bits=8)
    assert (r["codes"].size + r["words"].size) * 8 / (2 * 64) == oracle.bpw(8, 16, 6) == 6.5
    codes = _unpack_codes(r["codes"], 6)
    W = L.W.float().numpy().reshape(8, 16)
    for i in range(8):
        ev = oracle.eval_block(W[i], np.tile(c.reshape(-1, 16), (2, 1))[i], I.fp_atom("E2M3"), ue, 0)
        assert list(ev["codes"]) == list(codes[i])
        vals = np.array([oracle.fp_grid_value(I.KIND_FP_E2M3, int(x)) for x in codes[i]], np.float32)
        assert np.array_equal(vals, ev["q"])
        assert r["words"][i] == (ev["E"] << 4) | ev["M"]
