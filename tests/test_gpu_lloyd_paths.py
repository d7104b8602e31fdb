"""GPU parity on the paths of the Lloyd refinement and of the packer that ordinary sizes do not reach:
the transfer of a CTA's per-cell partial sums in the middle of its tile loop, several cache tiles per warp
of an iteration CTA, a status entry that says "not finished", a search result without a pair handed to the
packer, and an alphabet whose lookup tables do not fit the shared memory at their finest grid."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_14929_b200 import inputs as I

from .test_gpu_parity import B, REL, check_search, dev, gpu_lloyd  # noqa: F401  (B is a fixture)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("spill,ctas,per_warp,iter_ctas", [(1, 2, 1, 2), (3, 1, 4, 1), (5, 7, 2, 3)])
def test_lloyd_partial_sum_transfers_inside_the_tile_loop(B, spill, ctas, per_warp, iter_ctas):
    # 128 cache tiles over one, two or seven CTAs of the cache kernel with a transfer every 1, 3 or 5 tiles: every CTA
    # spills in the middle of its loop and (3, 5) once more for the remainder.  The iteration kernels run on one,
    # two or three CTAs, so a warp walks up to sixteen tiles and the CTA folds its 32-bit partial sums every
    # 1, 4 or 2 rounds.  The table, the pool count and the trace stay those of the oracle.  All blocks are in
    # the pool (rank = N_b) and half of them.
    L = I.outlier_channel_layer(31, 512, 1024, 64)
    fmt = I.scale_format("E5M6")
    atoms = I.alphabet(["NF4", "SH4"])
    c = oracle.channel_norms(L.X.numpy())
    r = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True)
    NB = r["block_cos"].shape[1]
    assert NB == 128 * 256
    bc = torch.from_numpy(r["block_cos"]).to(dev())
    B.dd4_lloyd_tuning(spill, ctas, per_warp, iter_ctas)
    try:
        for rank in (NB, NB // 2):
            want = oracle.dd_lloyd(L.W, c, fmt, int(r["k"][0]), r["block_cos"][0], rank, atoms[0].lut, 8)
            for per_iteration in (False, True):
                got = gpu_lloyd(B, L.W, c, fmt, atoms, bc, rank, 8, int(r["k"][0]), 0, launch_per_iteration=per_iteration)
                assert np.array_equal(got[0][:16].view(np.uint32), want[0].view(np.uint32))
                assert got[2] == want[2]
                assert np.allclose(got[1], want[1], rtol=REL, atol=0)
    finally:
        B.dd4_lloyd_tuning()
    with pytest.raises(B.SopError):
        B.dd4_lloyd_tuning(0, 0, 4, 0)
    with pytest.raises(B.SopError):
        B.dd4_lloyd_tuning(128, 0, 5, 0)


def test_outputs_refuse_a_codebook_from_an_unfinished_lloyd_call(B):
    # the status entry is planted on the host side of the API (no wait on the device is made to run out)
    from paper_2605_14929_b200.pipeline import LayerSweep
    L = I.tiny_layer(3, 32, 256)
    sw = LayerSweep(32, 256, L.X.shape[0], I.scale_format("UE4M4"), ["NF4", "SH4"], [], lloyd_iters=4, device=dev())
    sw.run(L.W.to(dev()), L.X.to(dev()))
    got = sw.outputs()
    assert got.distortion[4] >= 0.0 and np.all(got.distortion >= 0.0)
    sw.distortion[4] = -1.0
    with pytest.raises(B.LloydNotFinished):
        sw.outputs()


def test_pack_reports_a_result_block_without_a_pair(B):
    # a singles-only search leaves best_a / best_b at -1: the packer writes nothing and says so in the counts
    L = I.tiny_layer(4, 16, 256)
    fmt = I.scale_format("UE4M4")
    atoms = I.alphabet(["NF4", "SH4"])
    Wd, cd = L.W.to(dev()), torch.as_tensor(oracle.channel_norms(L.X.numpy())).to(dev())
    A, NB = len(atoms), 16 * 16
    pt, res = B.new_pair_table(A, dev()), B.new_result(dev())
    ws = B.alloc_workspace(B.pair_search_workspace(16, 256, A), dev())
    bc = torch.empty((A, NB), dtype=torch.float32, device=dev())
    B.sop_pair_search(Wd, cd, fmt, atoms, pt, None, res, ws, block_cos=bc, block_sse=torch.empty_like(bc), singles_only=True)
    codes = torch.full((NB * 8,), 0x5A, dtype=torch.uint8, device=dev())
    words = torch.zeros(B.words_nbytes(NB, 12), dtype=torch.uint8, device=dev())
    counts = torch.zeros(2, dtype=torch.int64, device=dev())
    for block_cos in (None, bc):
        B.sop_pack(Wd, cd, fmt, atoms, codes, words, search_result=res, container_bits=12, counts=counts, block_cos=block_cos)
        torch.cuda.synchronize()
        assert counts.tolist() == [-1, -1]
        assert bool((codes == 0x5A).all())
    # the same result block does hold a pair after a full search
    B.sop_pair_search(Wd, cd, fmt, atoms, pt, None, res, ws, block_cos=bc, block_sse=torch.empty_like(bc))
    B.sop_pack(Wd, cd, fmt, atoms, codes, words, search_result=res, container_bits=12, counts=counts, block_cos=bc)
    torch.cuda.synchronize()
    assert counts[0].item() >= 0 and not bool((codes == 0x5A).all())


def test_eight_fine_tables_beyond_the_shared_memory_are_swept_exactly(B):
    # eight distinct 16-entry tables with threshold gaps near 2^-7: at the finest lookup grid their cell tables need
    # more shared memory than a CTA has, so the grid is coarsened and the dense ones are searched exactly
    rng = np.random.default_rng(7)
    atoms = []
    for t in range(8):
        base = np.linspace(-1.0, 1.0, 16)
        base[7] = base[6] + 2.0 ** -6 * (1 + t % 3)          # two entries 1/64 .. 3/64 apart: thresholds 2^-7 apart at worst
        base[9] = base[8] + 2.0 ** -6
        lut = np.sort(I.snap_bf16(base + rng.uniform(-0.01, 0.01, 16) * (np.arange(16) % 5 == 0)))
        lut[0], lut[-1] = -1.0, 1.0
        atoms.append(I.Atom(f"fine{t}", 4, I.KIND_LUT, 0, 16, 1.0, np.sort(lut).astype(np.float32)))
    L = I.tiny_layer(9, 96, 512)
    check_search(B, L, "UE4M4", atoms)
    check_search(B, L, "E5M6", atoms + [atoms[0].negation(), atoms[3].negation()])


@pytest.mark.parametrize("fmt_name,names,layer", [("UE4M4", ["NF4", "SH4"], "config1"), ("E5M6", ["NF5", "SH5"], "config1"),
                                                  ("E5M6", ["NF4", "BOF4"], "outlier")])
def test_grid_constrained_dd_by_dynamic_programming(B, fmt_name, names, layer):
    # pair-search steps 1 and 3: cluster selection on the LUT value format's grid points; the table bit for bit, the
    # least total cost and the pool count, for a plain and a negated primary codebook and three pool sizes
    L = I.config1() if layer == "config1" else I.outlier_channel_layer(8, 320, 1024, 64)
    fmt = I.scale_format(fmt_name)
    atoms = I.alphabet(names)
    c = oracle.channel_norms(L.X.numpy())
    r = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True)
    NB = r["block_cos"].shape[1]
    bc = torch.from_numpy(r["block_cos"]).to(dev())
    ne = len(atoms[0].lut)
    for fmta in (0, 1):
        for rank in (NB // 2, 7, NB):
            want = oracle.dd_grid_dp(L.W, c, fmt, int(r["k"][fmta]), r["block_cos"][fmta], rank, ne)
            got = gpu_lloyd(B, L.W, c, fmt, atoms, bc, rank, 0, int(r["k"][fmta]), fmta, grid_dp=True)
            assert np.array_equal(got[0][:ne].view(np.uint32), want[0].view(np.uint32))
            assert got[2] == want[2]
            assert got[1][0] == pytest.approx(want[1], rel=REL, abs=1e-12)
    # the dynamic programme replaces the iterations: asking for both is refused
    with pytest.raises(B.SopError):
        gpu_lloyd(B, L.W, c, fmt, atoms, bc, NB // 2, 3, 0, 0, grid_dp=True)
    # axes (i), (iii), (iv) reach the construction like they reach the Lloyd one
    bs = torch.from_numpy(r["block_sse"]).to(dev())
    want = oracle.dd_grid_dp(L.W, c, fmt, int(r["k"][0]), r["block_sse"][0], NB // 3, ne, pool_by_error=True, uniform_weights=True)
    got = gpu_lloyd(B, L.W, c, fmt, atoms, bs, NB // 3, 0, int(r["k"][0]), 0, grid_dp=True, pool_by_error=True, uniform_weights=True)
    assert np.array_equal(got[0][:ne].view(np.uint32), want[0].view(np.uint32)) and got[2] == want[2]


def test_shifts_from_the_histogram_of_an_earlier_format():
    """A layer swept at several scale formats builds the exponent histogram of its block scales once: the sweeps of
    the later formats derive their shifts from the workspace (flag SOP_SEARCH_REUSE_PREPASS) and give what a sweep
    of their own gives, the layer-wide power-of-two scale of a ^0 candidate included."""
    from paper_2605_14929_b200.pipeline import LayerSweep
    d = torch.device("cuda:0")
    L = I.config5_layer(0, 1, 1, rows=48)
    L = I.Layer(L.W, L.X[:128].contiguous())
    M, K = L.W.shape
    Wd, Xd = L.W.to(d), L.X.to(d)
    rom, fp = ["NF4", "SH4", "BOF4"], ["E4M3^0", "E2M3"]
    fmts = [I.scale_format(f) for f in ("E5M6", "UE4M4", "E4M3", "UE8M0")]
    first = None
    shared = []
    for f, fmt in enumerate(fmts):
        sw = LayerSweep(M, K, 128, fmt, rom, fp, 3, device=d, share=first)
        first = first or sw
        sw.run(Wd, Xd, norms=(f == 0), reuse_prepass=(f > 0))
        shared.append(sw.outputs())
    ks = set()
    for fmt, got in zip(fmts, shared):
        own = LayerSweep(M, K, 128, fmt, rom, fp, 3, device=d)
        own.run(Wd, Xd)
        want = own.outputs()
        assert np.array_equal(got.result["k"], want.result["k"]) and np.array_equal(got.result["best"], want.result["best"])
        assert got.result["layer_absmax"] == want.result["layer_absmax"] > 0
        assert np.array_equal(got.pair_table["n_sel1"], want.pair_table["n_sel1"])
        assert np.array_equal(got.pair_table["acos"], want.pair_table["acos"], equal_nan=True)
        assert np.array_equal(got.dd_lut.view(np.uint32), want.dd_lut.view(np.uint32))
        assert torch.equal(got.codes, want.codes) and torch.equal(got.words, want.words)
        ks.add(int(want.result["k"][0]))
    assert len(ks) > 1          # the formats really need different shifts


def test_reduction_on_one_tile_and_on_two_tiles_at_a_time():
    """The reduction kernel's two launch shapes (two tiles of 256 blocks per step where the shared memory allows, one
    otherwise) make the same additions in the same order: every table entry is the same bit for bit, at a signed and
    an unsigned scale format, with a ragged last tile and an odd number of tiles per CTA."""
    from paper_2605_14929_b200 import binding as Bd
    from paper_2605_14929_b200.pipeline import LayerSweep
    d = torch.device("cuda:0")
    L = I.student_layer(71, 0, 1345, 1024, 64, 4.0, channel_sigma=0.6)      # 86080 blocks: 337 tiles, the last one ragged
    Wd, Xd = L.W.to(d), L.X.to(d)
    for fmt_name in ("E5M6", "UE4M4"):
        fmt = I.scale_format(fmt_name)
        got = []
        try:
            for pairs in (True, False):
                Bd.pair_search_tuning(pairs)
                sw = LayerSweep(1345, 1024, 64, fmt, ["NF4", "SH4", "BOF4", "Split87"], [], 3, device=d)
                sw.run(Wd, Xd)
                got.append(sw.outputs())
        finally:
            Bd.pair_search_tuning(True)
        a, b = got
        for name in ("pair_table", "signed_table"):
            for field in ("acos", "mse", "n_sel1", "n_neg"):
                assert np.array_equal(getattr(a, name)[field], getattr(b, name)[field], equal_nan=(field in ("acos", "mse"))), (fmt_name, name, field)
        assert np.array_equal(a.result["best"], b.result["best"])
