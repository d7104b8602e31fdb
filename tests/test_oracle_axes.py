"""Pins for the oracle's design-axis options (paragraph "Pair-search design axes": partition metric,
reassignment metric, Lloyd weighting, pool definition).  Each option is checked against something
the mathematics fixes: brute force over selector vectors, optimality inequalities between the two
reassignment metrics, plain means for uniform weights, sorted ranks for the pool."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2605_14929_b200 import inputs as I


def _tiny(seed, M=2, K=64):
    L = I.tiny_layer(seed, M, K)
    return L, oracle.channel_norms(L.X.numpy())


# ------------------------------------------------------------------ axis (ii): reassignment metric
def test_error_selected_pair_table_equals_brute_force_minimum_error():
    # mse is a sum of independent per-block terms: the selector vector with the smallest total error is
    # the per-block smaller error.  Enumerate all 2^Nb vectors on an 8-block layer.
    L, c = _tiny(3)
    fmt = I.scale_format("UE4M4")
    atoms = I.alphabet(["NF4", "SH4"])
    r = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True, select_metric=1)
    bc, bs = r["block_cos"].astype(np.float64), r["block_sse"].astype(np.float64)
    nb = bc.shape[1]
    assert nb == 8
    for a, b in itertools.combinations(range(len(atoms)), 2):
        best = min(sum(bs[b if (sel >> i) & 1 else a, i] for i in range(nb)) for sel in range(1 << nb))
        assert r["pair"]["mse"][a, b] == pytest.approx(best / (2 * 64), rel=1e-12)
        mu = bs[b] < bs[a]                                   # a tie keeps the first codebook
        assert r["pair"]["n_sel1"][a, b] == int(mu.sum())
        assert r["pair"]["acos"][a, b] == pytest.approx(np.where(mu, bc[b], bc[a]).mean(), rel=1e-12)
    # the per-block values and the singles do not depend on the metric
    r0 = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True, select_metric=0)
    assert np.array_equal(r0["block_cos"], r["block_cos"]) and np.array_equal(r0["block_sse"], r["block_sse"])
    for a in range(len(atoms)):
        assert r["pair"]["acos"][a, a] == r0["pair"]["acos"][a, a] and r["pair"]["mse"][a, a] == r0["pair"]["mse"][a, a]


def test_each_reassignment_metric_is_optimal_for_its_own_objective():
    L = I.config1()
    L = I.Layer(L.W[:32].contiguous(), L.X)
    c = oracle.channel_norms(L.X.numpy())
    fmt = I.scale_format("S1E4M4")
    atoms = I.alphabet(["NF4", "SH4", "BOF4"])
    r_cos = oracle.pair_search(L.W, c, fmt, atoms, select_metric=0)
    r_err = oracle.pair_search(L.W, c, fmt, atoms, select_metric=1)
    differ = 0
    for tab in ("pair", "signed"):
        ok = r_cos[tab]["n_sel1"] >= 0
        assert np.array_equal(ok, r_err[tab]["n_sel1"] >= 0)
        assert np.all(r_cos[tab]["acos"][ok] >= r_err[tab]["acos"][ok] - 1e-15)
        assert np.all(r_err[tab]["mse"][ok] <= r_cos[tab]["mse"][ok] * (1 + 1e-12))
        differ += int((r_cos[tab]["n_sel1"][ok] != r_err[tab]["n_sel1"][ok]).sum())
    assert differ > 0                    # the two metrics do disagree on some blocks of a real-looking layer


def test_error_selected_signed_table_is_smallest_of_four():
    L, c = _tiny(4, 4, 64)
    fmt = I.scale_format("S1E4M4")
    atoms = I.alphabet(["NF4", "SH4", "BOF4"])
    r = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True, select_metric=1)
    bs, bc = r["block_sse"].astype(np.float64), r["block_cos"].astype(np.float64)
    for i, j in ((0, 2), (0, 4), (2, 4)):
        four = np.stack([bs[i], bs[i + 1], bs[j], bs[j + 1]])
        pick = four.argmin(axis=0)                  # numpy argmin keeps the first minimum: same priority
        assert r["signed"]["mse"][i, j] == pytest.approx(four.min(axis=0).sum() / (4 * 64), rel=1e-12)
        assert r["signed"]["n_sel1"][i, j] == int((pick >= 2).sum())
        assert r["signed"]["n_neg"][i, j] == int((pick % 2 == 1).sum())
        chosen = np.stack([bc[i], bc[i + 1], bc[j], bc[j + 1]])[pick, np.arange(pick.size)]
        assert r["signed"]["acos"][i, j] == pytest.approx(chosen.mean(), rel=1e-12)


def test_pack_by_error_picks_the_smallest_error_candidate():
    L, c = _tiny(8, 4, 64)
    fmt = I.scale_format("S1E4M4")
    a, b = I.rom_atom("NF4"), I.rom_atom("SH4")
    r = oracle.pack(L.W, c, fmt, a, 1, b, 1, use_sign=1, container_bits=12, word_sign_bits=1, select_metric=1)
    assert r["rc"] == 0
    NB = 16
    bits = np.unpackbits(r["words"], bitorder="little")[: NB * 12].reshape(NB, 12)
    words = (bits.astype(np.int64) * (1 << np.arange(12))).sum(axis=1)
    W = L.W.float().numpy().reshape(NB, 16)
    cb = np.tile(c.reshape(-1, 16), (4, 1))
    n1 = nneg = 0
    for i in range(NB):
        sign, sel = int((words[i] >> 11) & 1), int(words[i] & 1)
        four = [oracle.eval_block(W[i], cb[i], x, fmt, 1)["sse"] for x in (a, a.negation(), b, b.negation())]
        assert int(np.argmin(four)) == 2 * sel + sign
        n1 += sel
        nneg += sign
    assert (r["n_sel1"], r["n_neg"]) == (n1, nneg)


# ------------------------------------------------------------------ axes (i), (iv): the pool
def _nf4_blocks(rows=64):
    L = I.config1()
    L = I.Layer(L.W[:rows].contiguous(), L.X)
    c = oracle.channel_norms(L.X.numpy())
    fmt = I.scale_format("UE4M4")
    nf4 = I.rom_atom("NF4")
    r = oracle.pair_search(L.W, c, fmt, [nf4], want_blocks=True)
    return L, c, fmt, nf4, r


def test_pool_ranked_by_error_holds_the_largest_errors():
    L, c, fmt, nf4, r = _nf4_blocks()
    bs = r["block_sse"][0]
    NB = bs.size
    rank = NB // 4
    k = int(r["k"][0])
    out, dist, cnt = oracle.dd_lloyd(L.W, c, fmt, k, bs, rank, nf4.lut, 4, pool_by_error=True)
    tau = np.sort(bs)[::-1][rank - 1]
    assert cnt == int((bs >= tau).sum()) and cnt >= rank
    assert dist[-1] < dist[0]
    # a layer whose blocks are ranked identically by both metrics gives the same pool, hence the same table:
    # use a strictly decreasing function of the cosine as the "error"
    bc = r["block_cos"][0]
    fake_err = (2.0 - bc).astype(np.float32)
    out_c, dist_c, cnt_c = oracle.dd_lloyd(L.W, c, fmt, k, bc, rank, nf4.lut, 4)
    out_e, dist_e, cnt_e = oracle.dd_lloyd(L.W, c, fmt, k, fake_err, rank, nf4.lut, 4, pool_by_error=True)
    if np.unique(fake_err).size == np.unique(bc).size:       # the map did not merge distinct cosines
        assert cnt_c == cnt_e and np.array_equal(out_c, out_e) and np.array_equal(dist_c, dist_e)


def test_pool_by_threshold_equals_pool_by_rank_at_that_threshold():
    L, c, fmt, nf4, r = _nf4_blocks()
    bc = r["block_cos"][0]
    NB = bc.size
    k = int(r["k"][0])
    for rank in (1, NB // 3, NB):
        tau = float(np.sort(bc)[rank - 1])
        by_rank = oracle.dd_lloyd(L.W, c, fmt, k, bc, rank, nf4.lut, 3)
        by_thr = oracle.dd_lloyd(L.W, c, fmt, k, bc, 0, nf4.lut, 3, pool_threshold=tau)
        assert by_rank[2] == by_thr[2] == int((bc <= tau).sum())
        assert np.array_equal(by_rank[0], by_thr[0]) and np.array_equal(by_rank[1], by_thr[1])
    # a threshold below every cosine: empty pool, the table stays as it is
    out, dist, cnt = oracle.dd_lloyd(L.W, c, fmt, k, bc, 0, nf4.lut, 3, pool_threshold=-2.0)
    assert cnt == 0 and np.array_equal(out, nf4.lut) and np.all(dist == 0.0)
    # by error: threshold above / at the largest error
    bs = r["block_sse"][0]
    out, dist, cnt = oracle.dd_lloyd(L.W, c, fmt, k, bs, 0, nf4.lut, 3, pool_by_error=True, pool_threshold=float(bs.max()))
    assert cnt == int((bs >= bs.max()).sum())


# ------------------------------------------------------------------ axis (iii): Lloyd weighting
def test_uniform_weights_equal_weighted_when_all_channel_norms_are_equal():
    L, c, fmt, nf4, r = _nf4_blocks(32)
    flat = np.full_like(c, 0.37)
    r1 = oracle.pair_search(L.W, flat, fmt, [nf4], want_blocks=True)
    bc = r1["block_cos"][0]
    k = int(r1["k"][0])
    a = oracle.dd_lloyd(L.W, flat, fmt, k, bc, bc.size // 2, nf4.lut, 4)
    b = oracle.dd_lloyd(L.W, flat, fmt, k, bc, bc.size // 2, nf4.lut, 4, uniform_weights=True)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1]) and a[2] == b[2]
    # and with unequal norms the two weightings part ways
    a = oracle.dd_lloyd(L.W, c, fmt, int(r["k"][0]), r["block_cos"][0], bc.size // 2, nf4.lut, 4)
    b = oracle.dd_lloyd(L.W, c, fmt, int(r["k"][0]), r["block_cos"][0], bc.size // 2, nf4.lut, 4, uniform_weights=True)
    assert not np.array_equal(a[0], b[0])


def test_uniform_single_update_equals_plain_means():
    rng = np.random.default_rng(11)
    u = np.sort(I.snap_bf16(rng.uniform(-1, 1, 12)))
    u[-1] = 1.0
    w = np.zeros((1, 16), np.float32)
    w[0, :12] = u * 0.25                      # block absmax 0.25 -> scale 0.25 exactly, u recovered exactly
    W = torch.from_numpy(w).to(torch.bfloat16)
    c = rng.uniform(0.1, 3.0, 16).astype(np.float32)       # ignored by the uniform rule
    fmt = I.scale_format("E5M6")
    init = np.array([-0.5, 0.5], np.float32)
    out, dist, _ = oracle.dd_lloyd(W, c, fmt, 0, np.zeros(1, np.float32), 1, init, 1, uniform_weights=True)
    pts = np.concatenate([u.astype(np.float64), np.zeros(4)])
    lo = pts <= 0.0
    assert np.allclose(out, [pts[lo].mean(), pts[~lo].mean()], rtol=2 ** -8)
    assert dist[0] == pytest.approx(np.sum((pts - np.where(lo, -0.5, 0.5)) ** 2), rel=1e-9)
