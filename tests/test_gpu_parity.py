"""GPU parity: every C-ABI entry point against the CPU oracle on the same seeded inputs.
Integers, codes, scale words, selectors, shifts and fp32 per-block values must match bit for bit;
per-layer ACos / MSE / distortion within 1e-6 relative (the sums are associated differently)."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2605_14929_b200 import inputs as I

from . import oracle_pipeline

pytestmark = pytest.mark.gpu
REL = 1e-6


@pytest.fixture(scope="module")
def B():
    from paper_2605_14929_b200 import build as libbuild
    libbuild.build()
    from paper_2605_14929_b200 import binding
    binding.lib()
    return binding


def dev():
    return torch.device("cuda:0")


def gpu_norms(B, X):
    Xd = X.to(dev())
    c = torch.empty(X.shape[1], dtype=torch.float32, device=dev())
    ws = B.alloc_workspace(B.channel_norms_workspace(*X.shape), dev())
    B.sop_channel_norms(Xd, c, ws)
    torch.cuda.synchronize()
    return c


def gpu_search(B, W, c, fmt, atoms, k_mode=None, dd_lut=None, dd_mask=0, two_calls_split=None, keep=False):
    M, K = W.shape
    A = len(atoms)
    NB = M * K // 16
    Wd, cd = W.to(dev()), torch.as_tensor(c).to(dev())
    pt, st, res = B.new_pair_table(A, dev()), B.new_pair_table(A, dev()), B.new_result(dev())
    bc = torch.full((A, NB), -7.0, dtype=torch.float32, device=dev())
    bs = torch.full((A, NB), -7.0, dtype=torch.float32, device=dev())
    ws = B.alloc_workspace(B.pair_search_workspace(M, K, A), dev())
    km = B.K_AUTO if k_mode is None else k_mode
    if two_calls_split is None:
        B.sop_pair_search(Wd, cd, fmt, atoms, pt, st, res, ws, k_mode=km, dd_lut=dd_lut, dd_mask=dd_mask, block_cos=bc,
                          block_sse=bs)
    else:
        # first the candidates in the mask (single-candidate reduction only), then the rest with the first ones loaded
        first = two_calls_split
        rest = ((1 << A) - 1) & ~first
        res1 = B.new_result(dev())
        # (keep: the first call forms every entry among its candidates and the second one keeps them)
        B.sop_pair_search(Wd, cd, fmt, atoms, pt, st, res1, ws, k_mode=km, dd_lut=dd_lut, dd_mask=dd_mask, block_cos=bc,
                          block_sse=bs, eval_mask=first, singles_only=not keep)
        torch.cuda.synchronize()
        first_pass = dict(pair=B.read_pair_table(pt, A).copy(), **B.read_result(res1))
        # the second call takes the shifts and max|W| from the first call's result instead of reading W again
        B.sop_pair_search(Wd, cd, fmt, atoms, pt, st, res, ws, k_mode=B.K_FROM_RESULT, prev_result=res1, dd_lut=dd_lut,
                          dd_mask=dd_mask, block_cos=bc, block_sse=bs, eval_mask=rest, load_mask=first, keep_loaded=keep)
    torch.cuda.synchronize()
    out = dict(pair=B.read_pair_table(pt, A), signed=B.read_pair_table(st, A), block_cos=bc.cpu().numpy(),
               block_sse=bs.cpu().numpy(), res_t=res, Wd=Wd, cd=cd, bc_t=bc, **B.read_result(res))
    if two_calls_split is not None:
        out["first_pass"] = first_pass
    return out


def assert_tables(got, want, A):
    for name in ("pair", "signed"):
        g, w = got[name], want[name]
        assert np.array_equal(g["n_sel1"], w["n_sel1"]), name
        defined = w["n_sel1"] >= 0
        assert np.array_equal(g["n_neg"][defined], w["n_neg"][defined]), name
        assert np.allclose(g["acos"][defined], w["acos"][defined], rtol=REL, atol=0)
        assert np.allclose(g["mse"][defined], w["mse"][defined], rtol=REL, atol=0)
        # the per-block cosines are identical, so the means agree far better than the bar
        # (fp32 partial sums of 8 gaps 1 - cos, then FP64: a few 1e-9 even when whole blocks have cos = 0)
        assert np.max(np.abs(g["acos"][defined] - w["acos"][defined]), initial=0.0) < 1e-8
    assert np.array_equal(got["k"][:A], want["k"])
    assert np.array_equal(got["best"], want["best"])


def check_search(B, layer, fmt_name, atoms, k_mode=None):
    fmt = I.scale_format(fmt_name)
    c = oracle.channel_norms(layer.X.numpy())
    want = oracle.pair_search(layer.W, c, fmt, atoms, k_mode=oracle.K_AUTO if k_mode is None else k_mode, want_blocks=True)
    got = gpu_search(B, layer.W, c, fmt, atoms, k_mode)
    A = len(atoms)
    assert np.array_equal(got["block_cos"].view(np.uint32), want["block_cos"].view(np.uint32))
    assert np.array_equal(got["block_sse"].view(np.uint32), want["block_sse"].view(np.uint32))
    assert_tables(got, want, A)
    return got, want


# ------------------------------------------------------------------ channel norms
@pytest.mark.parametrize("T,K", [(128, 1024), (1, 16), (65, 48), (200, 4096)])
def test_channel_norms_bit_exact(B, T, K):
    X = I.activations(3, 0, T, K)
    got = gpu_norms(B, X).cpu().numpy()
    assert np.array_equal(got.view(np.uint32), oracle.channel_norms(X.numpy()).view(np.uint32))


def test_channel_norms_strided_rows(B):
    X = I.activations(4, 0, 70, 96).to(dev())
    big = torch.zeros((70, 128), dtype=torch.float32, device=dev())
    big[:, :96] = X
    c = torch.empty(96, dtype=torch.float32, device=dev())
    ws = B.alloc_workspace(B.channel_norms_workspace(70, 96), dev())
    B.sop_channel_norms(big[:, :96], c, ws)
    torch.cuda.synchronize()
    assert np.array_equal(c.cpu().numpy(), oracle.channel_norms(X.cpu().numpy()))


# ------------------------------------------------------------------ the sweep
def test_config1_unsigned_and_signed(B):
    L = I.config1()
    atoms = I.alphabet(["NF4", "SH4", "BOF4"])
    check_search(B, L, "UE4M4", atoms)
    got, _ = check_search(B, L, "S1E4M4", atoms)
    assert got["best"][3] >= 0


@pytest.mark.parametrize("M,K", [(1, 16), (3, 48), (7, 1040), (33, 16), (600, 64)])
def test_ragged_and_tiny_shapes(B, M, K):
    L = I.tiny_layer(M * 1000 + K, M, K, T=5)
    check_search(B, L, "E5M6", I.alphabet(["NF4", "Split87"], fp=["E2M3"]))


# the eight formats of the paper's table, the two 8-bit GPU scale formats, and the 12-bit words with sign and
# metabits of the worked examples (Section "Scale Format and Metabit Allocation")
@pytest.mark.parametrize("fmt", I.TABLE_SCALE_FORMATS + ("UE8M0", "UE5M3", "S1E5M5", "S0E6M5", "S1E5M4", "S0E5M5"))
def test_every_scale_format(B, fmt):
    L = I.outlier_channel_layer(11, 96, 512, 64)
    check_search(B, L, fmt, I.alphabet(["NF4", "SH4"], fp=["E2M3", "E4M3", "E4M3^0"]))


def test_five_bit_alphabet(B):
    L = I.config4_layer(0, 0, rows=48)
    L = I.Layer(L.W[:, :2048].contiguous(), L.X[:256, :2048].contiguous())
    atoms = I.alphabet(["NF5", "SH5", "BOF5", "E2M2"])
    check_search(B, L, "UE4M4", atoms)
    check_search(B, L, "E5M6", atoms)


def test_explicit_shift_and_saturating_scales(B):
    # shifts that push most scales out of range: saturation and subnormal scale words on both sides
    L = I.config1()
    L = I.Layer(L.W[:64].contiguous(), L.X)
    atoms = I.alphabet(["NF4", "BOF4"], fp=["E2M3"])
    for k in (-12, 0, 14):
        check_search(B, L, "UE4M4", atoms, k_mode=k)


def test_zero_blocks_and_zero_rows(B):
    L = I.tiny_layer(5, 16, 256)
    W = L.W.clone()
    W[3] = 0
    W[:, 32:64] = 0
    check_search(B, I.Layer(W, L.X), "UE4M4", I.alphabet(["NF4", "SH4"], fp=["E4M3^0"]))


def test_tables_that_need_the_binary_search_path(B):
    # thresholds denser than any cell grid, non-bf16 entries, repeated entries: all must stay exact
    L = I.tiny_layer(6, 64, 256)
    dense = np.sort(np.concatenate([np.linspace(-1, 1, 12), [0.001, 0.0011, 0.00111, 0.3]])).astype(np.float32)
    a1 = I.Atom("dense", 4, I.KIND_LUT, 0, 16, 1.0, dense)
    dup = I.rom_atom("NF4").lut.copy()
    dup[8] = dup[7]
    a2 = I.Atom("dup", 4, I.KIND_LUT, 0, 16, 1.0, np.sort(dup))
    a3 = I.Atom("two", 4, I.KIND_LUT, 0, 16, 1.0, np.array([-0.5, 0.75], np.float32))
    check_search(B, L, "E5M6", [a1, a1.negation(), a2, a2.negation(), a3, I.rom_atom("E2M2")])


@pytest.mark.parametrize("fmt_name", ["UE4M4", "E5M6"])
def test_sweep_in_two_calls_equals_one_call(B, fmt_name):
    # "only the new columns": candidates evaluated by an earlier call are loaded, not evaluated again
    L = I.outlier_channel_layer(5, 200, 1024, 64)
    fmt = I.scale_format(fmt_name)
    atoms = I.alphabet(["NF4", "SH4", "BOF4"], fp=["E2M3", "E4M3^0"])
    c = oracle.channel_norms(L.X.numpy())
    want = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True)
    first = 0b01110011     # NF4, -NF4, BOF4, -BOF4, E2M3 first; SH4, -SH4, E4M3^0 in the second call
    got = gpu_search(B, L.W, c, fmt, atoms, two_calls_split=first)
    assert np.array_equal(got["block_cos"].view(np.uint32), want["block_cos"].view(np.uint32))
    assert np.array_equal(got["block_sse"].view(np.uint32), want["block_sse"].view(np.uint32))
    assert_tables(got, want, len(atoms))
    one = gpu_search(B, L.W, c, fmt, atoms)
    for name in ("pair", "signed"):
        assert np.array_equal(got[name]["n_sel1"], one[name]["n_sel1"])
    # the first call: diagonal entries of its candidates only, shifts of absent candidates reported as 0
    fp = got["first_pass"]
    A = len(atoms)
    for a in range(A):
        for b in range(A):
            defined = a == b and (first >> a) & 1
            assert (fp["pair"]["n_sel1"][a, b] >= 0) == bool(defined)
            if defined:
                assert np.isclose(fp["pair"]["acos"][a, a], want["pair"]["acos"][a, a], rtol=REL, atol=0)
    present = np.array([(first >> a) & 1 for a in range(A)], dtype=bool)
    assert np.array_equal(fp["k"][:A][present], want["k"][present]) and not fp["k"][:A][~present].any()
    lut_first = [a for a in range(A) if present[a] and atoms[a].kind == I.KIND_LUT]
    assert fp["best"][2] == max(lut_first, key=lambda a: (want["pair"]["acos"][a, a], -a))
    assert fp["best"][0] == -1 and fp["best"][3] == -1
    # the first call forms every entry among its candidates, the second keeps those and adds the entries of the new ones
    kept = gpu_search(B, L.W, c, fmt, atoms, two_calls_split=first, keep=True)
    assert_tables(kept, want, len(atoms))
    fp = kept["first_pass"]
    for a in range(A):
        for b in range(a, A):
            both = (first >> a) & 1 and (first >> b) & 1
            assert (fp["pair"]["n_sel1"][a, b] >= 0) == bool(both and want["pair"]["n_sel1"][a, b] >= 0)
            if fp["pair"]["n_sel1"][a, b] >= 0:
                assert fp["pair"]["n_sel1"][a, b] == want["pair"]["n_sel1"][a, b]


def test_negation_symmetry_on_gpu(B):
    L = I.tiny_layer(8, 32, 512)
    fmt = I.scale_format("E5M6")
    atoms = I.alphabet(["NF4", "SH4"])
    c = oracle.channel_norms(L.X.numpy())
    g0 = gpu_search(B, L.W, c, fmt, atoms)
    g1 = gpu_search(B, -L.W, c, fmt, atoms)
    assert np.array_equal(g0["block_cos"], g1["block_cos"][[1, 0, 3, 2]])


# ------------------------------------------------------------------ Lloyd
def gpu_lloyd(B, W, c, fmt, atoms, bc, rank, iters, k, fmta, **kw):
    M, K = W.shape
    out = torch.zeros(32, dtype=torch.float32, device=dev())
    dist = torch.zeros(iters + 1, dtype=torch.float64, device=dev())
    cnt = torch.zeros(1, dtype=torch.int64, device=dev())
    ws = B.alloc_workspace(B.dd4_lloyd_workspace(M, K), dev())
    B.sop_dd4_lloyd(W.to(dev()), torch.as_tensor(c).to(dev()), fmt, atoms, bc, rank, iters, out, dist, cnt, ws,
                    k_mode=k, fmta_index=fmta, **kw)
    torch.cuda.synchronize()
    return out.cpu().numpy(), dist.cpu().numpy(), int(cnt.item())


@pytest.mark.parametrize("fmt_name,names,iters", [("UE4M4", ["NF4", "SH4"], 8), ("E5M6", ["NF5", "SH5"], 16)])
def test_lloyd_matches_oracle(B, fmt_name, names, iters):
    L = I.config1()
    fmt = I.scale_format(fmt_name)
    atoms = I.alphabet(names)
    c = oracle.channel_norms(L.X.numpy())
    r = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True)
    NB = r["block_cos"].shape[1]
    for fmta in (0, 1):                     # a plain and a negated primary codebook
        for rank in (NB // 2, 1, NB):
            a = atoms[fmta]
            init = np.sort(-a.lut) if a.negated else a.lut
            want = oracle.dd_lloyd(L.W, c, fmt, int(r["k"][fmta]), r["block_cos"][fmta], rank, init, iters)
            bc = torch.from_numpy(r["block_cos"]).to(dev())
            ne = len(a.lut)
            # all iterations in one cooperative launch (the default where the grid fits), and one launch per iteration
            for per_iteration in (False, True):
                got = gpu_lloyd(B, L.W, c, fmt, atoms, bc, rank, iters, int(r["k"][fmta]), fmta, launch_per_iteration=per_iteration)
                assert np.array_equal(got[0][:ne].view(np.uint32), want[0].view(np.uint32))
                assert got[2] == want[2]
                assert np.allclose(got[1], want[1], rtol=REL, atol=0)
    M, K = L.W.shape
    assert B.dd4_lloyd_launches(M, K, iters, B.LLOYD_LAUNCH_PER_ITERATION) == 6 + iters + 1
    assert B.dd4_lloyd_launches(M, K, iters) in (7, 6 + iters + 1)


def test_lloyd_with_entries_closer_than_the_lookup_grid(B):
    # an initial table with several entries inside one cell of the iteration's lookup grid (width 2^-8):
    # those cells take the general search; zero rows and a zero column block are in the pool as well
    L = I.outlier_channel_layer(21, 160, 512, 64)
    W = L.W.clone()
    W[5] = 0
    W[:, 64:80] = 0
    L = I.Layer(W, L.X)
    fmt = I.scale_format("UE4M4")
    dense = np.sort(np.concatenate([np.linspace(-1, 1, 11), [0.001, 0.0011, 0.00111, 0.0028, 0.3]])).astype(np.float32)
    dense = I.snap_bf16(dense)
    atoms = [I.Atom("dense", 4, I.KIND_LUT, 0, 16, 1.0, np.sort(dense)), I.rom_atom("NF4")]
    c = oracle.channel_norms(L.X.numpy())
    r = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True)
    NB = r["block_cos"].shape[1]
    bc = torch.from_numpy(r["block_cos"]).to(dev())
    for rank in (NB, NB // 3):
        want = oracle.dd_lloyd(L.W, c, fmt, int(r["k"][0]), r["block_cos"][0], rank, atoms[0].lut, 6)
        got = gpu_lloyd(B, L.W, c, fmt, atoms, bc, rank, 6, int(r["k"][0]), 0)
        assert np.array_equal(got[0][:16].view(np.uint32), want[0].view(np.uint32))
        assert got[2] == want[2]
        assert np.allclose(got[1], want[1], rtol=REL, atol=0)


# ------------------------------------------------------------------ pack
def gpu_pack(B, W, c, fmt, atoms, ia, ib, k, use_sign, b, wsign, block_cos=None):
    M, K = W.shape
    NB = M * K // 16
    n = atoms[ia].n_bits
    codes = torch.zeros(NB * 2 * n, dtype=torch.uint8, device=dev())
    words = torch.full((B.words_nbytes(NB, b),), 0xAB, dtype=torch.uint8, device=dev())
    counts = torch.zeros(2, dtype=torch.int64, device=dev())
    B.sop_pack(W.to(dev()), torch.as_tensor(c).to(dev()), fmt, atoms, codes, words, index_a=ia, index_b=ib, k_mode=k,
               use_sign=use_sign, container_bits=b, word_sign_bits=wsign, counts=counts, block_cos=block_cos)
    torch.cuda.synchronize()
    return codes.cpu().numpy().reshape(NB, 2 * n), words.cpu().numpy(), counts.cpu().numpy()


@pytest.mark.parametrize("fmt_name,ia,ib,sign,b,wsign", [
    ("UE4M4", 0, 2, 0, 12, 0), ("S1E4M4", 0, 2, 1, 12, 1), ("E5M6", 1, 2, 0, 16, 1), ("E5M6", 0, 4, 1, 16, 1),
    ("UE4M4", 3, None, 0, 8, 0), ("UE5M3", 6, None, 0, 8, 0), ("E4M3", 0, None, 1, 8, 1),
    # the 12-bit worked examples: sign + selector (one metabit), no sign + selector, sign + selector + a spare metabit, selector alone
    ("S1E5M5", 0, 2, 1, 12, 1), ("S0E6M5", 0, 4, 0, 12, 0), ("S1E5M4", 2, 4, 1, 12, 1), ("S0E5M5", 1, 3, 0, 12, 0)])
def test_pack_matches_oracle(B, fmt_name, ia, ib, sign, b, wsign):
    L = I.config1()
    L = I.Layer(L.W[:96].contiguous(), L.X)
    fmt = I.scale_format(fmt_name)
    atoms = I.alphabet(["NF4", "SH4", "BOF4"], fp=["E2M3"])
    c = oracle.channel_norms(L.X.numpy())
    want = oracle.pack(L.W, c, fmt, atoms[ia], 1, None if ib is None else atoms[ib], 1, use_sign=sign, container_bits=b,
                       word_sign_bits=wsign)
    assert want["rc"] == 0
    codes, words, counts = gpu_pack(B, L.W, c, fmt, atoms, ia, B.NO_ATOM if ib is None else ib, 1, sign, b, wsign)
    assert np.array_equal(codes, want["codes"])
    assert np.array_equal(words[:want["words"].size], want["words"])
    assert (int(counts[0]), int(counts[1])) == (want["n_sel1"], want["n_neg"])
    # the same choice read off the per-block cosines of a sweep: identical bytes
    bc = gpu_search(B, L.W, c, fmt, atoms, k_mode=1)["bc_t"]
    codes2, words2, counts2 = gpu_pack(B, L.W, c, fmt, atoms, ia, B.NO_ATOM if ib is None else ib, 1, sign, b, wsign,
                                       block_cos=bc)
    assert np.array_equal(codes2, codes) and np.array_equal(words2, words) and np.array_equal(counts2, counts)


def test_pack_five_bit_pair(B):
    L = I.tiny_layer(12, 40, 256)
    fmt = I.scale_format("UE4M4")
    atoms = I.alphabet(["NF5", "SH5"])
    c = oracle.channel_norms(L.X.numpy())
    want = oracle.pack(L.W, c, fmt, atoms[0], 0, atoms[3], 0, container_bits=12)
    codes, words, counts = gpu_pack(B, L.W, c, fmt, atoms, 0, 3, 0, 0, 12, 0)
    assert np.array_equal(codes, want["codes"]) and np.array_equal(words[:want["words"].size], want["words"])


# ------------------------------------------------------------------ the whole layer pipeline
@pytest.mark.parametrize("fmt_name,rom,fp,iters,shape", [
    ("S1E4M4", ["NF4", "SH4", "BOF4"], [], 8, None),                               # configuration 1
    ("E5M6", ["NF4", "SH4", "BOF4", "Split87"], ["E2M3", "E4M3"], 8, (512, 1024)),   # configuration 2, reduced rows
    ("UE4M4", ["NF5", "SH5", "BOF5", "E2M2"], [], 16, (64, 4096)),                 # configuration 4, reduced rows
    ("E5M6", ["NF5", "SH5", "BOF5", "E2M2"], [], 16, (48, 4096)),                  # ... at its second scale format: DD5 Lloyd + pack
])
def test_pipeline_matches_oracle(B, fmt_name, rom, fp, iters, shape):
    from paper_2605_14929_b200.pipeline import LayerSweep
    fmt = I.scale_format(fmt_name)
    if shape is None:
        L = I.config1()
    elif rom[0] == "NF5":
        full = I.config4_layer(0, 0, rows=shape[0])
        L = I.Layer(full.W, full.X[:256].contiguous())
    else:
        L = I.outlier_channel_layer(0, shape[0], shape[1], 128)
    M, K = L.W.shape
    sw = LayerSweep(M, K, L.X.shape[0], fmt, rom, fp, lloyd_iters=iters, want_blocks=True)
    sw.run(L.W.to(dev()), L.X.to(dev()))
    got = sw.outputs()
    want = oracle_pipeline.run(L, fmt, rom, fp, lloyd_iters=iters, want_blocks=True)
    assert np.array_equal(got.c.numpy().view(np.uint32), want["c"].view(np.uint32))
    ne = len(want["dd_lut"])
    assert np.array_equal(got.dd_lut[:ne].view(np.uint32), want["dd_lut"].view(np.uint32))
    assert got.pool_count == want["pool_count"]
    assert np.allclose(got.distortion, want["distortion"], rtol=REL, atol=0)
    assert got.rom_result["best"][2] == want["rom"]["best"][2]   # the first pass reduces single candidates only: FMTa
    A = len(want["atoms"])
    full = dict(pair=got.pair_table, signed=got.signed_table, k=got.result["k"], best=got.result["best"])
    assert_tables(full, want["full"], A)
    assert np.array_equal(sw.full_cos.cpu().numpy().view(np.uint32), want["full"]["block_cos"].view(np.uint32))
    pk = want["pack"]
    assert np.array_equal(got.codes.numpy().reshape(pk["codes"].shape), pk["codes"])
    assert np.array_equal(got.words.numpy()[:pk["words"].size], pk["words"])
    assert (int(got.counts[0]), int(got.counts[1])) == (pk["n_sel1"], pk["n_neg"])


@pytest.mark.parametrize("graphs", [False, True])
def test_layer_stream_returns_each_layers_own_results(B, graphs):
    # five different layers through the overlapped host -> device -> host stream (every slot is used again): every
    # layer's results equal those of a plain run on that layer, launched call by call or as recorded CUDA graphs
    from paper_2605_14929_b200.pipeline import LayerStream, LayerSweep
    fmt = I.scale_format("S1E4M4")
    M, K, T = 48, 512, 64
    layers = [I.outlier_channel_layer(40 + i, M, K, T) for i in range(5)]
    sw = LayerSweep(M, K, T, fmt, ["NF4", "SH4"], [], 4, device=dev())
    want = []
    for L in layers:
        sw.run(L.W.to(dev()), L.X.to(dev()))
        torch.cuda.synchronize()
        want.append({k: getattr(sw, k).cpu().clone() for k in LayerStream.OUT})
    ls = LayerStream(sw, graphs=graphs)
    host = [(L.W.pin_memory(), L.X.pin_memory()) for L in layers]
    got = []
    for i, (Wh, Xh) in enumerate(host):
        ls.submit(i, Wh, Xh)
        if i:
            got.append({k: v.clone() for k, v in ls.collect(i - 1).items()})
    got.append({k: v.clone() for k, v in ls.collect(len(host) - 1).items()})
    assert ls.h2d_bytes == M * K * 2 + T * K * 4
    for i in range(5):
        for k in LayerStream.OUT:
            if k == "distortion":       # an FP64 sum in scheduling order: equal to rounding, not bit for bit
                assert torch.allclose(got[i][k], want[i][k], rtol=1e-9, atol=0), (i, k)
            else:
                assert torch.equal(got[i][k], want[i][k]), (i, k)
    assert not torch.equal(want[0]["codes"], want[1]["codes"])


def test_lloyd_without_iterations_reports_the_initial_table(B):
    # iters = 0: the table stays the primary codebook's, the one distortion entry is that of this table
    L = I.tiny_layer(17, 24, 256)
    fmt = I.scale_format("UE4M4")
    atoms = I.alphabet(["NF4"])
    c = oracle.channel_norms(L.X.numpy())
    r = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True)
    NB = r["block_cos"].shape[1]
    want = oracle.dd_lloyd(L.W, c, fmt, int(r["k"][0]), r["block_cos"][0], NB // 2, atoms[0].lut, 0)
    got = gpu_lloyd(B, L.W, c, fmt, atoms, torch.from_numpy(r["block_cos"]).to(dev()), NB // 2, 0, int(r["k"][0]), 0)
    assert np.array_equal(got[0][:16], atoms[0].lut) and np.array_equal(want[0], atoms[0].lut)
    assert got[2] == want[2] and np.allclose(got[1], want[1], rtol=REL, atol=0)
    assert B.dd4_lloyd_launches(24, 256, 0) == 7


def test_graph_replay_equals_the_calls(B):
    # the layer's calls captured into one CUDA graph: refilling the bound input tensors and replaying gives the
    # results of a plain run on the new layer
    from paper_2605_14929_b200.pipeline import LayerStream, LayerSweep
    fmt = I.scale_format("S1E4M4")
    M, K, T = 40, 512, 64
    a, b = I.outlier_channel_layer(50, M, K, T), I.outlier_channel_layer(51, M, K, T)
    sw = LayerSweep(M, K, T, fmt, ["NF4", "SH4"], [], 4, device=dev())
    sw.run(b.W.to(dev()), b.X.to(dev()))
    torch.cuda.synchronize()
    want = {k: getattr(sw, k).cpu().clone() for k in LayerStream.OUT}
    Wd, Xd = a.W.to(dev()), a.X.to(dev())
    sw.capture(Wd, Xd)
    Wd.copy_(b.W)
    Xd.copy_(b.X)
    sw.replay()
    torch.cuda.synchronize()
    for k in LayerStream.OUT:
        if k == "distortion":
            assert torch.allclose(sw.distortion.cpu(), want[k], rtol=1e-9, atol=0)
        else:
            assert torch.equal(getattr(sw, k).cpu(), want[k]), k


@pytest.mark.parametrize("graphs", [False, True])
def test_layer_stream_over_several_scale_formats(B, graphs):
    # one layer shape at three scale formats whose sweeps share the large buffers, the channel norms and the exponent
    # histogram: every (layer, format) result equals that of a sweep of its own
    from paper_2605_14929_b200.pipeline import LayerStream, LayerSweep
    M, K, T = 40, 768, 64
    fmts = [I.scale_format(f) for f in ("UE4M4", "E5M6", "E4M3")]
    layers = [I.student_layer(60 + i, 0, M, K, T, 4.0, channel_sigma=0.8) for i in range(3)]
    row, first = [], None
    for fmt in fmts:
        sw = LayerSweep(M, K, T, fmt, ["NF4", "SH4", "BOF4"], [], 3, device=dev(), share=first)
        first = first or sw
        row.append(sw)
    ls = LayerStream(row, graphs=graphs)
    host = [(L.W.pin_memory(), L.X.pin_memory()) for L in layers]
    got = []
    for i, (Wh, Xh) in enumerate(host):
        ls.submit(i, Wh, Xh)
        if i:
            got.append([{k: v.clone() for k, v in o.items()} for o in ls.collect(i - 1)])
    got.append([{k: v.clone() for k, v in o.items()} for o in ls.collect(len(host) - 1)])
    for i, L in enumerate(layers):
        for f, fmt in enumerate(fmts):
            own = LayerSweep(M, K, T, fmt, ["NF4", "SH4", "BOF4"], [], 3, device=dev())
            own.run(L.W.to(dev()), L.X.to(dev()))
            torch.cuda.synchronize()
            for k in LayerStream.OUT:
                w = getattr(own, k).cpu()
                if k == "distortion":
                    assert torch.allclose(got[i][f][k], w, rtol=1e-9, atol=0), (i, f, k)
                else:
                    assert torch.equal(got[i][f][k], w), (i, f, k)
