"""GPU parity for the design-axis options (paragraph "Pair-search design axes"): reassignment by block
error, pool ranked by error, pool by threshold, uniform Lloyd weights.  Same bar as the default path:
integers, tables and bytes bit for bit, layer sums within 1e-6 relative."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_14929_b200 import inputs as I

from .test_gpu_parity import B, REL, assert_tables, dev  # noqa: F401  (B is a fixture)

pytestmark = pytest.mark.gpu


def _search_mse(B, W, c, fmt, atoms, split=None, dd_lut=None, dd_mask=0):
    M, K = W.shape
    A = len(atoms)
    NB = M * K // 16
    Wd, cd = W.to(dev()), torch.as_tensor(c).to(dev())
    pt, st, res = B.new_pair_table(A, dev()), B.new_pair_table(A, dev()), B.new_result(dev())
    bc = torch.full((A, NB), -7.0, dtype=torch.float32, device=dev())
    bs = torch.full((A, NB), -7.0, dtype=torch.float32, device=dev())
    ws = B.alloc_workspace(B.pair_search_workspace(M, K, A), dev())
    if split is None:
        B.sop_pair_search(Wd, cd, fmt, atoms, pt, st, res, ws, block_cos=bc, block_sse=bs, select_mse=True,
                          dd_lut=dd_lut, dd_mask=dd_mask)
    else:
        res1 = B.new_result(dev())
        rest = ((1 << A) - 1) & ~split
        B.sop_pair_search(Wd, cd, fmt, atoms, pt, st, res1, ws, block_cos=bc, block_sse=bs, eval_mask=split,
                          singles_only=True, select_mse=True, dd_lut=dd_lut, dd_mask=dd_mask)
        B.sop_pair_search(Wd, cd, fmt, atoms, pt, st, res, ws, k_mode=B.K_FROM_RESULT, prev_result=res1, block_cos=bc,
                          block_sse=bs, eval_mask=rest, load_mask=split, select_mse=True, dd_lut=dd_lut, dd_mask=dd_mask)
    torch.cuda.synchronize()
    return dict(pair=B.read_pair_table(pt, A), signed=B.read_pair_table(st, A), block_cos=bc.cpu().numpy(),
                block_sse=bs.cpu().numpy(), bs_t=bs, **B.read_result(res))


@pytest.mark.parametrize("fmt_name,names,fp,split", [
    ("S1E4M4", ["NF4", "SH4", "BOF4"], [], None),
    ("E5M6", ["NF4", "SH4", "BOF4", "Split87"], ["E2M3", "E4M3"], None),
    ("E5M6", ["NF4", "SH4", "BOF4"], ["E2M3"], 0b1110011),     # SH4 and -SH4 in a second call
    ("UE4M4", ["NF5", "SH5"], [], None),
])
def test_sweep_with_error_reassignment_matches_oracle(B, fmt_name, names, fp, split):
    L = I.config1()
    L = I.Layer(L.W[:200].contiguous(), L.X)        # 200 x 1024: several tiles per CTA half and a ragged tail
    fmt = I.scale_format(fmt_name)
    atoms = I.alphabet(names, fp=fp)
    A = len(atoms)
    c = oracle.channel_norms(L.X.numpy())
    want = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True, select_metric=1)
    got = _search_mse(B, L.W, c, fmt, atoms, split=split)
    assert np.array_equal(got["block_cos"].view(np.uint32), want["block_cos"].view(np.uint32))
    assert np.array_equal(got["block_sse"].view(np.uint32), want["block_sse"].view(np.uint32))
    assert_tables(got, want, A)
    assert np.array_equal(got["k"][:A], want["k"])
    assert list(got["best"]) == list(want["best"])
    # the option changes the assignment on this layer (otherwise the test would not see it)
    base = oracle.pair_search(L.W, c, fmt, atoms)
    assert not np.array_equal(base["pair"]["n_sel1"], want["pair"]["n_sel1"])


def _lloyd(B, W, c, fmt, atoms, metric, rank, iters, k, fmta, **kw):
    M, K = W.shape
    out = torch.zeros(32, dtype=torch.float32, device=dev())
    dist = torch.zeros(iters + 1, dtype=torch.float64, device=dev())
    cnt = torch.zeros(1, dtype=torch.int64, device=dev())
    ws = B.alloc_workspace(B.dd4_lloyd_workspace(M, K), dev())
    B.sop_dd4_lloyd(W.to(dev()), torch.as_tensor(c).to(dev()), fmt, atoms, metric, rank, iters, out, dist, cnt, ws,
                    k_mode=k, fmta_index=fmta, **kw)
    torch.cuda.synchronize()
    return out.cpu().numpy(), dist.cpu().numpy(), int(cnt.item())


def _same(got, want, ne):
    assert np.array_equal(got[0][:ne].view(np.uint32), want[0].view(np.uint32))
    assert got[2] == want[2]
    assert np.allclose(got[1], want[1], rtol=REL, atol=0)


def test_lloyd_axes_match_oracle(B):
    L = I.config1()
    fmt = I.scale_format("UE4M4")
    atoms = I.alphabet(["NF4", "SH4"])
    c = oracle.channel_norms(L.X.numpy())
    r = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True)
    NB = r["block_cos"].shape[1]
    bc = torch.from_numpy(r["block_cos"]).to(dev())
    bs = torch.from_numpy(r["block_sse"]).to(dev())
    iters = 6
    for fmta in (0, 1):
        a = atoms[fmta]
        init = np.sort(-a.lut) if a.negated else a.lut
        k = int(r["k"][fmta])
        ne = len(a.lut)
        for rank in (NB // 2, 1, NB):
            # axis (i): pool ranked by block error
            want = oracle.dd_lloyd(L.W, c, fmt, k, r["block_sse"][fmta], rank, init, iters, pool_by_error=True)
            _same(_lloyd(B, L.W, c, fmt, atoms, bs, rank, iters, k, fmta, pool_by_error=True), want, ne)
            # axis (iii): uniform weights (with either pool metric)
            want = oracle.dd_lloyd(L.W, c, fmt, k, r["block_cos"][fmta], rank, init, iters, uniform_weights=True)
            _same(_lloyd(B, L.W, c, fmt, atoms, bc, rank, iters, k, fmta, uniform_weights=True), want, ne)
        want = oracle.dd_lloyd(L.W, c, fmt, k, r["block_sse"][fmta], NB // 3, init, iters, pool_by_error=True, uniform_weights=True)
        _same(_lloyd(B, L.W, c, fmt, atoms, bs, NB // 3, iters, k, fmta, pool_by_error=True, uniform_weights=True), want, ne)
        # axis (iv): pool by a threshold on the metric, including an empty and a full pool
        for q in (0.25, 0.6):
            tau = float(np.quantile(r["block_cos"][fmta], q))
            want = oracle.dd_lloyd(L.W, c, fmt, k, r["block_cos"][fmta], 0, init, iters, pool_threshold=tau)
            _same(_lloyd(B, L.W, c, fmt, atoms, bc, 1, iters, k, fmta, pool_threshold=tau), want, ne)
            tau_e = float(np.quantile(r["block_sse"][fmta], 1 - q))
            want = oracle.dd_lloyd(L.W, c, fmt, k, r["block_sse"][fmta], 0, init, iters, pool_by_error=True, pool_threshold=tau_e)
            _same(_lloyd(B, L.W, c, fmt, atoms, bs, 1, iters, k, fmta, pool_by_error=True, pool_threshold=tau_e), want, ne)
        for tau in (-2.0, 2.0):
            want = oracle.dd_lloyd(L.W, c, fmt, k, r["block_cos"][fmta], 0, init, iters, pool_threshold=tau)
            assert want[2] == (0 if tau < 0 else NB)
            _same(_lloyd(B, L.W, c, fmt, atoms, bc, 1, iters, k, fmta, pool_threshold=tau), want, ne)


@pytest.mark.parametrize("fmt_name,ia,ib,sign,b,wsign", [
    ("UE4M4", 0, 2, 0, 12, 0), ("S1E4M4", 0, 2, 1, 12, 1), ("E5M6", 0, 4, 1, 16, 1), ("E5M6", 1, 2, 0, 16, 1)])
def test_pack_with_error_reassignment_matches_oracle(B, fmt_name, ia, ib, sign, b, wsign):
    L = I.config1()
    L = I.Layer(L.W[:96].contiguous(), L.X)
    fmt = I.scale_format(fmt_name)
    atoms = I.alphabet(["NF4", "SH4", "BOF4"], fp=["E2M3"])
    c = oracle.channel_norms(L.X.numpy())
    want = oracle.pack(L.W, c, fmt, atoms[ia], 1, atoms[ib], 1, use_sign=sign, container_bits=b, word_sign_bits=wsign,
                       select_metric=1)
    assert want["rc"] == 0
    base = oracle.pack(L.W, c, fmt, atoms[ia], 1, atoms[ib], 1, use_sign=sign, container_bits=b, word_sign_bits=wsign)
    assert (want["n_sel1"], want["n_neg"]) != (base["n_sel1"], base["n_neg"])

    def run(block_metric):
        M, K = L.W.shape
        NB = M * K // 16
        codes = torch.zeros(NB * 8, dtype=torch.uint8, device=dev())
        words = torch.full((B.words_nbytes(NB, b),), 0xAB, dtype=torch.uint8, device=dev())
        counts = torch.zeros(2, dtype=torch.int64, device=dev())
        B.sop_pack(L.W.to(dev()), torch.as_tensor(c).to(dev()), fmt, atoms, codes, words, index_a=ia, index_b=ib, k_mode=1,
                   use_sign=sign, container_bits=b, word_sign_bits=wsign, counts=counts, block_cos=block_metric,
                   select_mse=True)
        torch.cuda.synchronize()
        return codes.cpu().numpy().reshape(NB, 8), words.cpu().numpy(), counts.cpu().numpy()

    codes, words, counts = run(None)                         # candidates evaluated by the pack kernel
    assert np.array_equal(codes, want["codes"])
    assert np.array_equal(words[:want["words"].size], want["words"])
    assert (int(counts[0]), int(counts[1])) == (want["n_sel1"], want["n_neg"])
    # the same choice read off the per-block errors of a sweep: identical bytes
    M, K = L.W.shape
    A = len(atoms)
    pt, st, res = B.new_pair_table(A, dev()), B.new_pair_table(A, dev()), B.new_result(dev())
    bc = torch.empty((A, M * K // 16), dtype=torch.float32, device=dev())
    bs = torch.empty_like(bc)
    ws = B.alloc_workspace(B.pair_search_workspace(M, K, A), dev())
    B.sop_pair_search(L.W.to(dev()), torch.as_tensor(c).to(dev()), fmt, atoms, pt, st, res, ws, k_mode=1, block_cos=bc,
                      block_sse=bs, select_mse=True)
    codes2, words2, counts2 = run(bs)
    assert np.array_equal(codes2, codes) and np.array_equal(words2, words) and np.array_equal(counts2, counts)
