"""GPU parity at the full size of the large benchmark configurations, in the launch configuration that
bench.py times: the MLP layers of the 7B-shaped FP6-vs-FP8 comparison (configuration 3), the n = 5 MLP pair with
DD5 at both of its scale formats (configuration 4), and the two largest layers of the 70B-shaped set at one
E4-class and one E5-class scale format (configuration 5).

What the oracle computes in full: the channel norms, the primary codebook's column of per-block cosines and
errors (its shift, its single-candidate table entry), the Lloyd table, pool count and distortion trace; for
configuration 3 both candidates in full.  Every other candidate is compared on sampled blocks and whole rows
through the oracle's one-block evaluation, every table entry is recomputed in float64 from the per-block arrays
(a property that holds at any size), and the packed stream is compared on row ranges at the start, in the middle
and at the end of the layer and through its counts.  Layers are generated on the device from their seed; the
oracle reads the same bytes from a host copy."""
import math
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle
from paper_2605_14929_b200 import inputs as I

from .test_gpu_parity import B, REL, dev  # noqa: F401  (B is a fixture)

pytestmark = pytest.mark.gpu


def _bits(a):
    return np.ascontiguousarray(a).view(np.uint32)


def _host_w(W):
    w16 = W.cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
    return w16, (w16.astype(np.uint32) << 16).view(np.float32)


def _sample_blocks(NB, nbk, M, n_random, rows, seed):
    rng = np.random.default_rng(seed)
    picks = [rng.integers(0, NB, n_random)]
    for m in rows:
        picks.append(np.arange(m * nbk, (m + 1) * nbk))
    return np.unique(np.concatenate(picks))


def _check_sampled_candidates(cand, sample, Wf, c, fmt, ks, nbk, full_cos, full_sse, pot=None):
    for i, atom in cand.items():
        for blk in sample:
            m, j = divmod(int(blk), nbk)
            r = oracle.eval_block(Wf[m, 16 * j:16 * j + 16], c[16 * j:16 * j + 16], atom, fmt, int(ks[i]),
                                  pot_scale=0.0 if pot is None else pot.get(i, 0.0))
            assert np.float32(r["cos"]).view(np.uint32) == full_cos[i, blk].view(np.uint32), (i, blk)
            assert np.float32(r["sse"]).view(np.uint32) == full_sse[i, blk].view(np.uint32), (i, blk)


def _check_tables_from_blocks(P, S, full_cos, full_sse, atoms, M, K, signed):
    """Every defined entry of the two tables against float64 sums of the per-block arrays (torch on the host)."""
    A = len(atoms)
    cos = torch.from_numpy(full_cos)
    sse = torch.from_numpy(full_sse)
    NB = cos.shape[1]

    def entry(ca, ea, cb, eb):
        mu = cb > ca
        sc = torch.where(mu, cb, ca).double().sum().item() / NB
        se = torch.where(mu, eb, ea).double().sum().item() / (M * K)
        return int(mu.sum().item()), sc, se

    for x in range(A):
        assert P["n_sel1"][x, x] == 0
        assert abs(P["acos"][x, x] - cos[x].double().mean().item()) < 1e-8
        assert P["mse"][x, x] == pytest.approx(sse[x].double().sum().item() / (M * K), rel=REL)
        for y in range(x + 1, A):
            if P["n_sel1"][x, y] < 0:
                continue
            n1, sc, se = entry(cos[x], sse[x], cos[y], sse[y])
            assert P["n_sel1"][x, y] == n1
            assert abs(P["acos"][x, y] - sc) < 1e-8 and P["mse"][x, y] == pytest.approx(se, rel=REL)
            assert P["acos"][x, y] >= max(P["acos"][x, x], P["acos"][y, y]) - 1e-12
    if not signed:
        assert (S["n_sel1"] < 0).all()
        return
    bases = [i for i in range(A - 1) if atoms[i].kind == I.KIND_LUT and not atoms[i].negated and atoms[i + 1].negated]
    best = {}
    for i in bases:                         # the better of (i, -i) per block, ties to i
        neg = cos[i + 1] > cos[i]
        best[i] = (torch.where(neg, cos[i + 1], cos[i]), torch.where(neg, sse[i + 1], sse[i]), neg)
    for i in bases:
        for j in bases:
            if j < i:
                continue
            ci, ei, ni = best[i]
            cj, ej, nj = best[j]
            n1, sc, se = entry(ci, ei, cj, ej)
            mu = cj > ci
            nneg = int(torch.where(mu, nj, ni).sum().item())
            assert S["n_sel1"][i, j] == n1 and S["n_neg"][i, j] == nneg, (i, j)
            assert abs(S["acos"][i, j] - sc) < 1e-8 and S["mse"][i, j] == pytest.approx(se, rel=REL)


def _words(stream, n_words, b):
    """The first n_words b-bit words of a little-endian bit stream (b in {8, 12, 16})."""
    if b == 8:
        return stream[:n_words].astype(np.uint32)
    if b == 16:
        return stream[:2 * n_words].view(np.uint16).astype(np.uint32)
    t = stream[:(n_words * 3 + 1) // 2 + 2].astype(np.uint32)
    n2 = (n_words + 1) // 2
    tri = t[:3 * n2].reshape(n2, 3)
    w = np.empty(2 * n2, np.uint32)
    w[0::2] = tri[:, 0] | ((tri[:, 1] & 15) << 8)
    w[1::2] = (tri[:, 1] >> 4) | (tri[:, 2] << 4)
    return w[:n_words]


def _run_on_gpu(L, fmt_name, rom, iters):
    """One layer through the whole hot path on the device; everything the comparison needs, on the host."""
    from paper_2605_14929_b200.pipeline import LayerSweep
    fmt = I.scale_format(fmt_name)
    M, K = L.W.shape
    sw = LayerSweep(M, K, L.X.shape[0], fmt, rom, [], iters, device=dev())
    sw.run(L.W, L.X)
    got = sw.outputs()
    return dict(fmt=fmt, got=got, full_cos=sw.full_cos.cpu().numpy(), full_sse=sw.full_sse.cpu().numpy(),
                use_sign=sw.use_sign, container=sw.container)


def _compare_with_oracle(run, w16, Wf, X, rom, iters, seed):
    """The results of ``_run_on_gpu`` against the oracle, as the module docstring says."""
    fmt, got, full_cos, full_sse = run["fmt"], run["got"], run["full_cos"], run["full_sse"]
    M, K = w16.shape
    nbk, NB = K // 16, M * K // 16
    atoms = got.atoms
    A, n_rom = len(atoms), 2 * len(rom)
    ne = 1 << atoms[0].n_bits

    c = oracle.channel_norms(X)
    assert np.array_equal(_bits(got.c.numpy()), _bits(c))
    # the shift of every scale class: the oracle's F_layer on the layer's block scales
    amax = np.abs(Wf).reshape(M, nbk, 16).max(axis=2).ravel()
    k_of = {}
    for i, a in enumerate(atoms):
        if a.tmax not in k_of:
            k_of[a.tmax] = oracle.f_layer(fmt, amax if a.tmax == 1.0 else (amax / np.float32(a.tmax)).astype(np.float32))
        assert int(got.result["k"][i]) == k_of[a.tmax], (i, a.name)

    # ---- the primary codebook over the whole layer, then the Lloyd refinement over its whole pool
    fmta = int(got.rom_result["best"][2])
    singles = [got.pair_table["acos"][i, i] for i in range(n_rom)]
    assert fmta == int(np.argmax(singles))                       # best single ROM candidate, ties to the lowest index
    col = oracle.pair_search(w16, c, fmt, [atoms[fmta]], want_blocks=True)
    k_rom = int(col["k"][0])
    assert k_rom == k_of[atoms[fmta].tmax]
    assert np.array_equal(_bits(full_cos[fmta]), _bits(col["block_cos"][0]))
    assert np.array_equal(_bits(full_sse[fmta]), _bits(col["block_sse"][0]))
    assert got.pair_table["acos"][fmta, fmta] == pytest.approx(col["pair"]["acos"][0, 0], rel=REL)
    assert got.pair_table["mse"][fmta, fmta] == pytest.approx(col["pair"]["mse"][0, 0], rel=REL)
    a = atoms[fmta]
    init = np.sort(-a.lut) if a.negated else a.lut
    rank = max(1, min(NB, int(math.ceil(NB * 0.5))))
    lut, dist, cnt = oracle.dd_lloyd(w16, c, fmt, k_rom, col["block_cos"][0], rank, init, iters)
    assert np.array_equal(_bits(got.dd_lut[:ne]), _bits(lut))
    assert got.pool_count == cnt
    assert np.allclose(got.distortion, dist, rtol=REL, atol=0)

    # ---- every other candidate: random blocks, the first two rows, one row in the middle and the last row
    sample = _sample_blocks(NB, nbk, M, 300, [0, 1, M // 2, M - 1], seed)
    dd = I.Atom("DD", atoms[0].n_bits, I.KIND_LUT, 0, I.SCOPE_BLOCK, 1.0, lut)
    cand = {i: atoms[i] for i in range(n_rom) if i != fmta}
    cand[n_rom], cand[n_rom + 1] = dd, dd.negation()
    _check_sampled_candidates(cand, sample, Wf, c, fmt, got.result["k"], nbk, full_cos, full_sse)

    # ---- every table entry from the per-block arrays; the best pair is the arg-max of its table
    P, S = got.pair_table, got.signed_table
    _check_tables_from_blocks(P, S, full_cos, full_sse, atoms, M, K, bool(fmt.sign_bits))
    best = got.result["best"]
    iu = [(x, y) for x in range(A) for y in range(x + 1, A) if P["n_sel1"][x, y] >= 0]
    assert (int(best[0]), int(best[1])) == max(iu, key=lambda xy: (P["acos"][xy], -xy[0], -xy[1]))
    if fmt.sign_bits:
        su = [(x, y) for x in range(A) for y in range(A) if S["n_sel1"][x, y] >= 0]
        assert (int(best[3]), int(best[4])) == max(su, key=lambda xy: (S["acos"][xy], -xy[0], -xy[1]))

    # ---- pack: row ranges at the start, in the middle and at the end of the layer, and the whole stream's counts
    sign = run["use_sign"]
    ia, ib = (int(best[3]), int(best[4])) if sign else (int(best[0]), int(best[1]))
    b = run["container"]
    codes = got.codes.numpy().reshape(NB, -1)
    words = got.words.numpy()
    pick = {n_rom: dd, n_rom + 1: dd.negation()}
    rows = 16
    for m0 in (0, (M // 2) & ~1, M - rows):
        pk = oracle.pack(w16[m0:m0 + rows], c, fmt, pick.get(ia, atoms[ia]), int(got.result["k"][ia]),
                         pick.get(ib, atoms[ib]), int(got.result["k"][ib]), use_sign=sign, container_bits=b, word_sign_bits=sign)
        assert pk["rc"] == 0
        assert np.array_equal(codes[m0 * nbk:(m0 + rows) * nbk], pk["codes"])
        o = m0 * nbk * b // 8                       # rows start on a byte boundary: nbk is even
        assert np.array_equal(words[o:o + pk["words"].size], pk["words"])
    tab = S if sign else P
    assert (int(got.counts[0]), int(got.counts[1])) == (int(tab["n_sel1"][ia, ib]), int(tab["n_neg"][ia, ib]) if sign else 0)
    wv = _words(words, NB, b)
    meta = b - sign - fmt.exp_bits - fmt.man_bits
    sel_bits = (wv & 1) if sign else (wv >> (b - 1))
    assert int(sel_bits.sum()) == int(got.counts[0])            # every word of the stream carries its selector
    if sign:
        assert int((wv >> (b - 1)).sum()) == int(got.counts[1])
    mag = (wv >> meta) & ((1 << (fmt.exp_bits + fmt.man_bits)) - 1) if sign else (wv >> (meta - 1)) & ((1 << (fmt.exp_bits + fmt.man_bits)) - 1)
    zero_blocks = int((np.abs(Wf).reshape(M, nbk, 16).max(axis=2) == 0).sum())
    assert int((mag == 0).sum()) == zero_blocks                 # a non-zero block never has a zero scale word
    return got


def _both_formats(B, make_layer, fmts, rom, iters):
    L = make_layer()
    runs = [_run_on_gpu(L, f, rom, iters) for f in fmts]         # the library is driven from one thread
    w16, Wf = _host_w(L.W)
    X = L.X.cpu().numpy()
    del L
    torch.cuda.empty_cache()
    with ThreadPoolExecutor(max_workers=len(fmts)) as ex:        # the oracle's passes for the formats run side by side
        futs = [ex.submit(_compare_with_oracle, r, w16, Wf, X, rom, iters, 11 + i) for i, r in enumerate(runs)]
        return [f.result() for f in futs]


@pytest.mark.parametrize("which", [3, 4])
def test_config5_largest_layers_at_an_e4_and_an_e5_scale_format(B, which):
    # 28672 x 8192 and 8192 x 28672 (235 M elements, 14.7 M blocks): K / 16 = 512 and 1792 column blocks with many
    # row iterations of the sweep, a Lloyd pool of 7.3 M blocks whose 28 672 cache tiles take several rounds per CTA, 12- and
    # 16-bit scale-word streams of 14.7 M words
    got = _both_formats(B, lambda: I.config5_layer(0, 0, which, device="cuda"), ["UE4M4", "E5M6"],
                        ["NF4", "SH4", "BOF4", "Split87"], 8)
    assert got[0].result["k"][0] > 0          # an E4-class scale needs a shift on weights of this size, an E5-class one does not
    assert got[1].result["k"][0] == 0


@pytest.mark.parametrize("which", [0, 1])
def test_config4_mlp_pair_with_dd5_at_both_scale_formats(B, which):
    # 14336 x 4096 and 4096 x 14336, 32-entry alphabet, DD5 by 16 Lloyd iterations, UE4M4 and E5M6
    _both_formats(B, lambda: I.config4_layer(0, which, device="cuda"), ["UE4M4", "E5M6"], ["NF5", "SH5", "BOF5", "E2M2"], 16)


@pytest.mark.parametrize("which", [4, 6])
def test_config3_mlp_layers_fp6_against_fp8_in_full(B, which):
    # gate 14336 x 4096 and down 4096 x 14336: E2M3 with a UE4M4 block scale against E4M3 with one power-of-two
    # scale per layer.  The block-scaled FP6 candidate goes through the oracle over the whole layer (row ranges
    # side by side, with the shift that the oracle's F_layer finds on the whole layer); the layer-scaled FP8
    # candidate, whose scale needs the whole layer's maximum, on sampled blocks and whole rows.
    L = I.config3_layer(0, 0, which, device="cuda")
    fmt = I.scale_format("UE4M4")
    atoms = [I.fp_atom("E2M3"), I.fp_atom("E4M3^0")]
    M, K = L.W.shape
    NB, nbk = M * K // 16, K // 16
    w16, Wf = _host_w(L.W)
    c = oracle.channel_norms(L.X.cpu().numpy())
    cd = torch.empty(K, dtype=torch.float32, device=dev())
    ws_norm = B.alloc_workspace(B.channel_norms_workspace(L.X.shape[0], K), dev())
    ws_search = B.alloc_workspace(B.pair_search_workspace(M, K, 2), dev())
    B.sop_channel_norms(L.X, cd, ws_norm)
    pt, res = B.new_pair_table(2, dev()), B.new_result(dev())
    bc = torch.empty((2, NB), dtype=torch.float32, device=dev())
    bs = torch.empty_like(bc)
    B.sop_pair_search(L.W, cd, fmt, atoms, pt, None, res, ws_search, block_cos=bc, block_sse=bs)
    torch.cuda.synchronize()
    assert np.array_equal(_bits(cd.cpu().numpy()), _bits(c))
    P, r = B.read_pair_table(pt, 2), B.read_result(res)
    full_cos, full_sse = bc.cpu().numpy(), bs.cpu().numpy()
    amax = np.abs(Wf).reshape(M, nbk, 16).max(axis=2).ravel()
    k0 = oracle.f_layer(fmt, (amax / np.float32(7.5)).astype(np.float32))
    assert int(r["k"][0]) == k0 and int(r["k"][1]) == 0 and r["best"][0] == -1 and r["best"][2] == -1
    assert r["layer_absmax"] == amax.max()
    n_part = 8
    edges = [M * i // n_part for i in range(n_part + 1)]
    with ThreadPoolExecutor(max_workers=n_part) as ex:
        parts = list(ex.map(lambda i: oracle.pair_search(w16[edges[i]:edges[i + 1]], c, fmt, atoms[:1], k_mode=k0, want_blocks=True),
                            range(n_part)))
    want_cos = np.concatenate([p["block_cos"][0] for p in parts])
    want_sse = np.concatenate([p["block_sse"][0] for p in parts])
    assert np.array_equal(_bits(full_cos[0]), _bits(want_cos)) and np.array_equal(_bits(full_sse[0]), _bits(want_sse))
    pot = oracle.layer_pot_scale(float(amax.max()), 448.0)
    sample = _sample_blocks(NB, nbk, M, 300, [0, M // 2, M - 1], 3)
    _check_sampled_candidates({1: atoms[1]}, sample, Wf, c, fmt, r["k"], nbk, full_cos, full_sse, pot={1: pot})
    for x in range(2):
        assert P["n_sel1"][x, x] == 0 and P["n_sel1"][0, 1] == -1
        assert abs(P["acos"][x, x] - full_cos[x].astype(np.float64).mean()) < 1e-8
        assert P["mse"][x, x] == pytest.approx(full_sse[x].astype(np.float64).sum() / (M * K), rel=REL)
    assert P["mse"][0, 0] < P["mse"][1, 1]          # the 6.5 bpw format ahead of the 8.0 bpw one, as in the paper's table
    # pack of the FP6 single (8-bit scale words, 12 bytes of codes per block): first and last rows
    codes = torch.empty(NB * 12, dtype=torch.uint8, device=dev())
    words = torch.empty(B.words_nbytes(NB, 8), dtype=torch.uint8, device=dev())
    B.sop_pack(L.W, cd, fmt, atoms, codes, words, index_a=0, index_b=B.NO_ATOM, search_result=res, container_bits=8)
    torch.cuda.synchronize()
    codes, words = codes.cpu().numpy().reshape(NB, 12), words.cpu().numpy()
    for m0 in (0, M - 8):
        pk = oracle.pack(w16[m0:m0 + 8], c, fmt, atoms[0], int(r["k"][0]), None, 0, container_bits=8)
        assert pk["rc"] == 0
        assert np.array_equal(codes[m0 * nbk:(m0 + 8) * nbk], pk["codes"])
        assert np.array_equal(words[m0 * nbk:(m0 + 8) * nbk], pk["words"])


def test_config5_attention_layer_with_both_sparse_streams_in_full(B):
    """The 8192x8192 layer at E5M6 with the outlier stream in front and the residual correction behind: 16384 tiles
    of 256 blocks per stream pass.  The outlier stream and the zeroed weights are compared in full; the correction is
    computed by the oracle in full from the pair, shifts and DD table that the device pipeline chose."""
    from paper_2605_14929_b200.pipeline import LayerSweep
    L = I.config5_layer(0, 0, 0, device=str(dev()))
    M, K = L.W.shape
    fmt = I.scale_format("E5M6")
    sw = LayerSweep(M, K, L.X.shape[0], fmt, ["NF4", "SH4", "BOF4", "Split87"], [], 8, device=dev(), opq_q=0.92, wr_sigma=0.001,
                    opq_capacity=M * K // 8)
    sw.run(L.W, L.X)
    out = sw.outputs()
    sp = sw.sparse_outputs()
    w16, _ = _host_w(L.W)
    W_host = torch.from_numpy(w16.view(np.int16).copy()).view(torch.bfloat16)
    o = oracle.opq_extract(W_host, oracle.opq_threshold(0.92, 16), capacity=M * K // 8)
    assert sp["opq"]["count"] == o["count"] <= M * K // 8
    assert np.array_equal(sp["opq"]["row_start"], o["row_start"]) and np.array_equal(sp["opq"]["records"], o["records"])
    assert np.array_equal(sp["opq"]["W_out"].view(torch.int16).numpy().view(np.uint16), o["W_out"])
    # the correction of the packed layer: the oracle re-evaluates the chosen pair on every block of the zeroed weights
    W2 = torch.from_numpy(o["W_out"].view(np.int16).copy()).view(torch.bfloat16)
    best = out.result["best"]
    assert sw.use_sign == 1
    ia, ib = int(best[3]), int(best[4])
    atoms = list(out.atoms)

    def atom(i):
        a = atoms[i]
        return I.Atom(a.name, a.n_bits, I.KIND_LUT, a.negated, I.SCOPE_BLOCK, 1.0, out.dd_lut[:16]) if (sw.dd_mask >> i) & 1 else a
    w = oracle.wr_extract(W2, out.c.numpy(), fmt, atom(ia), int(out.result["k"][ia]), atom(ib), int(out.result["k"][ib]), use_sign=1,
                          n_keep=sw.wr_keep, capacity=2 * sw.wr_keep + 1024)
    assert sp["wr"]["count"] == w["count"] >= sw.wr_keep and sp["wr"]["scale_exp"] == w["scale_exp"]
    assert np.float32(sp["wr"]["tau"]).view(np.uint32) == np.float32(w["tau"]).view(np.uint32)
    assert np.array_equal(sp["wr"]["row_start"], w["row_start"]) and np.array_equal(sp["wr"]["records"], w["records"])


def test_config5_attention_layer_at_the_other_six_scale_formats(B):
    # the 8192 x 8192 layer in full at the six scale formats of the paper's table that the largest layers above do not
    # take: the oracle's passes for the formats run side by side on the host
    got = _both_formats(B, lambda: I.config5_layer(0, 0, 0, device="cuda"), ["E4M3", "UE4M6", "E4M5", "UE5M7", "E4M7", "E8M7"],
                        ["NF4", "SH4", "BOF4", "Split87"], 8)
    assert len(got) == 6
