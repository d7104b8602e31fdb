"""GPU parity on the benchmark configurations: the attention-projection layer at its full size in
the launch configuration that bench.py times (sampled blocks and rows against the oracle, the Lloyd
table and the ROM part of the pair tables in full), and reduced-row cases of the 7B-shaped
FP6-vs-FP8 comparison and of the 70B-shaped layer set at every scale format (the full-size cases of
those configurations are in test_gpu_fullsize.py)."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2605_14929_b200 import inputs as I

from . import oracle_pipeline
from .test_gpu_parity import B, REL, assert_tables, check_search, dev  # noqa: F401  (B is a fixture)

pytestmark = pytest.mark.gpu


def test_config2_full_size_in_the_bench_configuration(B):
    import bench
    from paper_2605_14929_b200.pipeline import LayerSweep
    Wl = bench.CONFIG2
    M, K, T = Wl["M"], Wl["K"], Wl["T"]
    fmt = I.scale_format(Wl["scale_format"])
    L = bench.make_layer(0)
    sw = LayerSweep(M, K, T, fmt, Wl["rom"], Wl["fp"], Wl["lloyd_iters"], device=dev())
    sw.run(L.W.to(dev()), L.X.to(dev()))
    got = sw.outputs()
    atoms = got.atoms
    A, NB, nbk = len(atoms), M * K // 16, K // 16

    # ---- channel norms: all of them
    c = oracle.channel_norms(L.X.numpy())
    assert np.array_equal(got.c.numpy().view(np.uint32), c.view(np.uint32))

    # ---- the ROM candidates over the whole layer: shifts, FMTa, single and pair entries, then the Lloyd table
    n_rom = 2 * len(Wl["rom"])
    rom = oracle.pair_search(L.W, c, fmt, atoms[:n_rom], want_blocks=True)
    assert np.array_equal(got.result["k"][:n_rom], rom["k"])
    fmta = int(rom["best"][2])
    assert got.rom_result["best"][2] == fmta
    for name in ("pair", "signed"):
        g, w = (got.pair_table if name == "pair" else got.signed_table)[:n_rom, :n_rom], rom[name]
        assert np.array_equal(g["n_sel1"], w["n_sel1"])
        ok = w["n_sel1"] >= 0
        assert np.array_equal(g["n_neg"][ok], w["n_neg"][ok])
        assert np.allclose(g["acos"][ok], w["acos"][ok], rtol=REL, atol=0) and np.allclose(g["mse"][ok], w["mse"][ok], rtol=REL, atol=0)
    full_cos = sw.full_cos.cpu().numpy()
    full_sse = sw.full_sse.cpu().numpy()
    assert np.array_equal(full_cos[:n_rom].view(np.uint32), rom["block_cos"].view(np.uint32))
    assert np.array_equal(full_sse[:n_rom].view(np.uint32), rom["block_sse"].view(np.uint32))
    a = atoms[fmta]
    init = np.sort(-a.lut) if a.negated else a.lut
    rank = max(1, min(NB, int(math.ceil(NB * 0.5))))
    lut, dist, cnt = oracle.dd_lloyd(L.W, c, fmt, int(rom["k"][fmta]), rom["block_cos"][fmta], rank, init, Wl["lloyd_iters"])
    assert np.array_equal(got.dd_lut[:16].view(np.uint32), lut.view(np.uint32))
    assert got.pool_count == cnt
    assert np.allclose(got.distortion, dist, rtol=REL, atol=0)

    # ---- the other candidates (DD4, -DD4, E2M3, E4M3): sampled blocks, one oracle block evaluation each
    rng = np.random.default_rng(5)
    W16 = L.W.view(torch.int16).numpy().view(np.uint16)
    Wf = (W16.astype(np.uint32) << 16).view(np.float32)
    sample = np.unique(np.concatenate([rng.integers(0, NB, 600), np.arange(0, 4 * nbk)]))   # random blocks + the first four rows
    dd = I.Atom("DD4", 4, I.KIND_LUT, 0, I.SCOPE_BLOCK, 1.0, lut)
    cand = {n_rom: dd, n_rom + 1: dd.negation()}
    for i in range(n_rom + 2, A):
        cand[i] = atoms[i]
    for i, atom in cand.items():
        k = int(got.result["k"][i])
        if atom.kind == I.KIND_LUT:
            assert k == int(rom["k"][0])          # same scale class (tmax 1) as the ROM atoms
        for blk in sample:
            m, j = divmod(int(blk), nbk)
            r = oracle.eval_block(Wf[m, 16 * j:16 * j + 16], c[16 * j:16 * j + 16], atom, fmt, k)
            assert np.float32(r["cos"]).view(np.uint32) == full_cos[i, blk].view(np.uint32), (i, blk)
            assert np.float32(r["sse"]).view(np.uint32) == full_sse[i, blk].view(np.uint32), (i, blk)
    # FP shifts: the oracle's F_layer on the layer's block scales
    amax = np.abs(Wf).reshape(M, nbk, 16).max(axis=2).ravel()
    for i in range(n_rom + 2, A):
        sigma = (amax / np.float32(atoms[i].tmax)).astype(np.float32)
        assert int(got.result["k"][i]) == oracle.f_layer(fmt, sigma)

    # ---- every table entry: what holds at any size
    P = got.pair_table
    for x in range(A):
        assert P["n_sel1"][x, x] == 0 and abs(P["acos"][x, x] - (1.0 - (1.0 - full_cos[x].astype(np.float64)).mean())) < 1e-9
        for y in range(x + 1, A):
            if P["n_sel1"][x, y] < 0:
                continue
            mu = full_cos[y] > full_cos[x]
            assert P["n_sel1"][x, y] == int(mu.sum())
            sel_cos = np.where(mu, full_cos[y], full_cos[x]).astype(np.float64)
            sel_sse = np.where(mu, full_sse[y], full_sse[x]).astype(np.float64)
            assert abs(P["acos"][x, y] - sel_cos.mean()) < 1e-9
            assert P["mse"][x, y] == pytest.approx(sel_sse.sum() / (M * K), rel=REL)
            assert P["acos"][x, y] >= max(P["acos"][x, x], P["acos"][y, y]) - 1e-12
    best = got.result["best"]
    sa, sb = int(best[3]), int(best[4])
    S = got.signed_table
    defined = S["n_sel1"] >= 0
    assert S["acos"][sa, sb] == S["acos"][defined].max()

    # ---- pack: the first four rows against the oracle's packer, counts against the signed table
    rows = 4
    pk = oracle.pack(L.W[:rows].contiguous(), c, fmt, cand.get(sa, atoms[sa]), int(got.result["k"][sa]),
                     cand.get(sb, atoms[sb]), int(got.result["k"][sb]), use_sign=1, container_bits=sw.container, word_sign_bits=1)
    assert pk["rc"] == 0 and sw.container == 16
    assert np.array_equal(got.codes.numpy().reshape(NB, 8)[:rows * nbk], pk["codes"])
    assert np.array_equal(got.words.numpy()[:rows * nbk * 2], pk["words"])
    assert (int(got.counts[0]), int(got.counts[1])) == (int(S["n_sel1"][sa, sb]), int(S["n_neg"][sa, sb]))


@pytest.mark.parametrize("which,rows", [(0, 96), (1, 64), (4, 40), (6, 24)])
def test_config3_fp6_block_scaled_against_fp8_layer_scaled(B, which, rows):
    # E2M3 with a UE4M4 scale per block (6.5 bpw) and E4M3 with one power-of-two scale per layer (8.0 bpw)
    L = I.config3_layer(0, 1, which, rows=rows)
    L = I.Layer(L.W, L.X[:128].contiguous())
    got, want = check_search(B, L, "UE4M4", [I.fp_atom("E2M3"), I.fp_atom("E4M3^0")])
    assert got["best"][0] == -1 and got["best"][2] == -1          # FP candidates are singles: no pair, no LUT single
    # the paper's table has the 6.5 bpw format ahead of the 8.0 bpw one on bell-shaped weights
    assert got["pair"]["mse"][0, 0] < got["pair"]["mse"][1, 1]


@pytest.mark.parametrize("fmt_name", I.TABLE_SCALE_FORMATS)
@pytest.mark.parametrize("which,rows", [(1, 24), (4, 8)])
def test_config5_layer_set_at_every_scale_format(B, fmt_name, which, rows):
    from paper_2605_14929_b200.pipeline import LayerSweep
    L = I.config5_layer(0, 2, which, rows=rows)
    L = I.Layer(L.W, L.X[:128].contiguous())
    fmt = I.scale_format(fmt_name)
    rom = ["NF4", "SH4", "BOF4", "Split87"]
    M, K = L.W.shape
    sw = LayerSweep(M, K, L.X.shape[0], fmt, rom, [], lloyd_iters=8)
    sw.run(L.W.to(dev()), L.X.to(dev()))
    got = sw.outputs()
    want = oracle_pipeline.run(L, fmt, rom, [], lloyd_iters=8, want_blocks=True)
    assert np.array_equal(got.c.numpy().view(np.uint32), want["c"].view(np.uint32))
    assert np.array_equal(got.dd_lut[:16].view(np.uint32), want["dd_lut"].view(np.uint32))
    assert got.pool_count == want["pool_count"]
    assert np.allclose(got.distortion, want["distortion"], rtol=REL, atol=0)
    A = len(want["atoms"])
    assert_tables(dict(pair=got.pair_table, signed=got.signed_table, k=got.result["k"], best=got.result["best"]), want["full"], A)
    assert np.array_equal(sw.full_cos.cpu().numpy().view(np.uint32), want["full"]["block_cos"].view(np.uint32))
    pk = want["pack"]
    assert np.array_equal(got.codes.numpy().reshape(pk["codes"].shape), pk["codes"])
    assert np.array_equal(got.words.numpy()[:pk["words"].size], pk["words"])
    assert (int(got.counts[0]), int(got.counts[1])) == (pk["n_sel1"], pk["n_neg"])
