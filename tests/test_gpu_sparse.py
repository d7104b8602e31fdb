"""GPU parity of the two sparse side streams against the oracle: outlier extraction before the search (Section
"Outlier Per-Quantum Extraction (OPQ)") and the sparse correction of the codebook residual (Section "Sparse
Residual Correction (Wr)").  Everything is integer or bit work: W_out, row starts, records, counts, the layer
exponent and the threshold are compared exactly."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2605_14929_b200 import binding as B
from paper_2605_14929_b200 import inputs as I
from paper_2605_14929_b200.pipeline import LayerSweep

from . import oracle_pipeline
from .test_gpu_parity import dev

pytestmark = pytest.mark.gpu


def run_opq(W: torch.Tensor, m: float, capacity=None, ldw=None):
    M, K = W.shape
    d = dev()
    if ldw:
        buf = torch.zeros(M, ldw, dtype=torch.bfloat16, device=d)
        buf[:, :K] = W.to(d)
        Wd = buf[:, :K]
        out = torch.full((M, ldw), 7.0, dtype=torch.bfloat16, device=d)[:, :K]
    else:
        Wd = W.to(d)
        out = torch.full((M, K), 7.0, dtype=torch.bfloat16, device=d)
    cap = M * K if capacity is None else capacity
    row_start = torch.zeros(M + 1, dtype=torch.int32, device=d)
    records = torch.zeros(max(cap, 1), dtype=torch.int32, device=d) if cap else None
    count = torch.zeros(1, dtype=torch.int64, device=d)
    ws = B.opq_workspace(M, K, d)
    B.sop_opq_extract(Wd, m, out, row_start, records, count, ws)
    torch.cuda.synchronize()
    n = int(count.item())
    rec = records.cpu().numpy().view(np.uint32)[:min(n, cap)] if cap else np.zeros(0, np.uint32)
    return dict(W_out=out.contiguous().cpu().view(torch.int16).numpy().view(np.uint16), row_start=row_start.cpu().numpy().view(np.uint32),
                records=rec, count=n)


def assert_opq(got, want):
    assert got["count"] == want["count"]
    assert np.array_equal(got["row_start"], want["row_start"])
    assert np.array_equal(got["records"], want["records"])
    assert np.array_equal(got["W_out"], want["W_out"])


@pytest.mark.parametrize("M,K,ldw", [(8, 64, None), (37, 1040, None), (300, 4096, None), (19, 208, 256), (1, 16, None)])
@pytest.mark.parametrize("q", [0.92, 0.5])
def test_opq_matches_oracle(M, K, ldw, q):
    L = I.laplace_outlier_layer(7, 1, M, K, 8)
    m = B.opq_threshold(q, 16)
    assert m == pytest.approx(oracle.opq_threshold(q, 16), rel=1e-12)
    got = run_opq(L.W, m, ldw=ldw)
    want = oracle.opq_extract(L.W, m)
    assert q > 0.9 or want["count"] > M * K // 100          # the lower quantile takes a real share
    assert_opq(got, want)


def test_opq_edge_cases():
    m = B.opq_threshold(0.92, 16)
    # zero layer, constant-magnitude layer: no outliers, W_out = W
    for W in (torch.zeros(5, 48, dtype=torch.bfloat16), torch.full((5, 48), -0.5, dtype=torch.bfloat16)):
        got = run_opq(W, m)
        assert got["count"] == 0 and not got["row_start"].any()
        assert np.array_equal(got["W_out"], W.view(torch.int16).numpy().view(np.uint16))
    # a capacity below the count: the count is reported, the records that fit are written, W_out is complete
    L = I.laplace_outlier_layer(3, 0, 64, 512, 8)
    want = oracle.opq_extract(L.W, 2.0)
    assert want["count"] > 40
    got = run_opq(L.W, 2.0, capacity=40)
    assert got["count"] == want["count"] and np.array_equal(got["records"], want["records"][:40]) and np.array_equal(got["W_out"], want["W_out"])
    got = run_opq(L.W, 2.0, capacity=0)
    assert got["count"] == want["count"] and np.array_equal(got["row_start"], want["row_start"])
    # an outlier in every block of a row, in the last column of the last row
    W = torch.ones(3, 64, dtype=torch.float32) * 0.01
    W[1, 5::16] = 3.0
    W[2, 63] = -2.0
    Wb = W.to(torch.bfloat16)
    assert_opq(run_opq(Wb, m), oracle.opq_extract(Wb, m))


def run_wr(L, fmt, rom, n_keep, use_sign, lloyd_iters=0, capacity=None, fp=()):
    """The layer through the pipeline (search, pack), then the correction of what was packed."""
    d = dev()
    M, K = L.W.shape
    sw = LayerSweep(M, K, L.X.shape[0], fmt, rom, list(fp), lloyd_iters, device=d)
    Wd, Xd = L.W.to(d), L.X.to(d)
    sw.run(Wd, Xd)
    out = sw.outputs()
    cap = M * K if capacity is None else capacity
    row_start = torch.zeros(M + 1, dtype=torch.int32, device=d)
    records = torch.zeros(max(cap, 1), dtype=torch.int32, device=d)
    count = torch.zeros(1, dtype=torch.int64, device=d)
    e = torch.zeros(1, dtype=torch.int32, device=d)
    tau = torch.zeros(1, dtype=torch.float32, device=d)
    ws = B.wr_workspace(M, K, d)
    B.sop_wr_extract(Wd, sw.c, sw.fmt_c, sw.atoms_c, sw.codes, sw._words_store, n_keep, row_start, records, count, e, ws, tau=tau,
                     index_a=0 if sw.single else B.PAIR_FROM_RESULT, index_b=B.NO_ATOM if sw.single else B.PAIR_FROM_RESULT,
                     search_result=sw.result, use_sign=sw.use_sign, container_bits=sw.container, word_sign_bits=sw.use_sign,
                     dd_lut=sw.dd_lut if sw.dd_mask else None, dd_mask=sw.dd_mask)
    torch.cuda.synchronize()
    n = int(count.item())
    got = dict(count=n, row_start=row_start.cpu().numpy().view(np.uint32), records=records.cpu().numpy().view(np.uint32)[:min(n, cap)],
               scale_exp=int(e.item()), tau=float(tau.item()))
    return sw, out, got


def oracle_wr(L, fmt, out, sw, n_keep):
    if sw.single:           # one element format packed alone
        return oracle.wr_extract(L.W, out.c.numpy(), fmt, out.atoms[0], int(out.result["k"][0]), None, 0, use_sign=0, n_keep=n_keep)
    best = out.result["best"]
    ia, ib = (int(best[3]), int(best[4])) if sw.use_sign else (int(best[0]), int(best[1]))
    atoms = list(out.atoms)
    dd = out.dd_lut[:1 << atoms[0].n_bits]

    def atom(i):
        a = atoms[i]
        if (sw.dd_mask >> i) & 1:
            a = I.Atom(a.name, a.n_bits, I.KIND_LUT, a.negated, I.SCOPE_BLOCK, 1.0, dd)
        return a
    c = out.c.numpy()
    return oracle.wr_extract(L.W, c, fmt, atom(ia), int(out.result["k"][ia]), atom(ib), int(out.result["k"][ib]),
                             use_sign=sw.use_sign, n_keep=n_keep)


@pytest.mark.parametrize("fmt_name,rows,K,iters", [("E5M6", 24, 512, 4), ("UE4M4", 40, 256, 0), ("S1E5M5", 9, 1024, 2), ("E4M3", 64, 128, 0)])
def test_wr_matches_oracle_on_the_packed_layer(fmt_name, rows, K, iters):
    L = I.student_layer(11, 2, rows, K, 64, 4.0)
    fmt = I.scale_format(fmt_name)
    for n_keep in (1, max(1, math.ceil(0.001 * rows * K)), rows * K // 50):
        sw, out, got = run_wr(L, fmt, ["NF4", "SH4", "BOF4"], n_keep, None, lloyd_iters=iters)
        want = oracle_wr(L, fmt, out, sw, n_keep)
        assert want["count"] >= n_keep
        assert got["count"] == want["count"] and got["scale_exp"] == want["scale_exp"]
        assert np.float32(got["tau"]).view(np.uint32) == np.float32(want["tau"]).view(np.uint32)
        assert np.array_equal(got["row_start"], want["row_start"])
        assert np.array_equal(got["records"], want["records"])


def test_wr_edge_cases():
    fmt = I.scale_format("E5M6")
    L = I.student_layer(5, 0, 16, 256, 64, 5.0)
    # every element asked for: everything with a residual is kept
    sw, out, got = run_wr(L, fmt, ["NF4", "SH4"], 16 * 256, None)
    want = oracle_wr(L, fmt, out, sw, 16 * 256)
    assert got["count"] == want["count"] <= 16 * 256 and np.array_equal(got["records"], want["records"])
    # a capacity below the count
    sw, out, got = run_wr(L, fmt, ["NF4", "SH4"], 100, None, capacity=10)
    want = oracle_wr(L, fmt, out, sw, 100)
    assert got["count"] == want["count"] >= 100 and np.array_equal(got["records"], want["records"][:10])
    assert np.array_equal(got["row_start"], want["row_start"])


def test_opq_then_search_then_wr_chain():
    """The three steps as the paper orders them: outliers out, the search on the rest, the correction of its residual."""
    L = I.laplace_outlier_layer(9, 0, 48, 512, 64)
    m = B.opq_threshold(0.92, 16)
    o = run_opq(L.W, m)
    assert o["count"] > 0
    W2 = torch.from_numpy(o["W_out"].view(np.int16).copy()).view(torch.bfloat16)
    L2 = I.Layer(W2, L.X)
    fmt = I.scale_format("E5M6")
    n_keep = math.ceil(0.001 * 48 * 512)
    sw, out, got = run_wr(L2, fmt, ["NF4", "SH4", "BOF4", "Split87"], n_keep, None, lloyd_iters=4)
    want = oracle_wr(L2, fmt, out, sw, n_keep)
    assert got["count"] == want["count"] and np.array_equal(got["records"], want["records"]) and got["scale_exp"] == want["scale_exp"]
    # an outlier position holds +0 in the search input: its residual is minus the table value nearest to zero, times the scale
    assert np.array_equal(o["W_out"], oracle.opq_extract(L.W, m)["W_out"])


@pytest.mark.parametrize("graph", [False, True])
def test_layer_sweep_with_both_streams(graph):
    """LayerSweep with opq_q and wr_sigma: the outlier stream, the search on the zeroed weights and the correction of
    the packed layer, call by call and replayed as one CUDA graph."""
    d = dev()
    L = I.laplace_outlier_layer(13, 2, 96, 1024, 64)
    fmt = I.scale_format("E5M6")
    rom = ["NF4", "SH4", "BOF4", "Split87"]
    sw = LayerSweep(96, 1024, 64, fmt, rom, [], 4, device=d, opq_q=0.92, wr_sigma=0.001)
    Wd, Xd = L.W.to(d), L.X.to(d)
    if graph:
        sw.capture(Wd, Xd)
        sw.replay()
    else:
        sw.run(Wd, Xd)
    out = sw.outputs()
    sp = sw.sparse_outputs()
    o = oracle.opq_extract(L.W, oracle.opq_threshold(0.92, 16))
    assert sp["opq"]["count"] == o["count"] > 0
    assert np.array_equal(sp["opq"]["records"], o["records"]) and np.array_equal(sp["opq"]["row_start"], o["row_start"])
    assert np.array_equal(sp["opq"]["W_out"].view(torch.int16).numpy().view(np.uint16), o["W_out"])
    W2 = torch.from_numpy(o["W_out"].view(np.int16).copy()).view(torch.bfloat16)
    L2 = I.Layer(W2, L.X)
    want = oracle_pipeline.run(L2, fmt, rom, [], lloyd_iters=4)
    assert np.array_equal(out.dd_lut[:16].view(np.uint32), want["dd_lut"].view(np.uint32))
    pk = want["pack"]
    assert np.array_equal(out.codes.numpy().reshape(pk["codes"].shape), pk["codes"])
    w = oracle_wr(L2, fmt, out, sw, sw.wr_keep)
    assert sp["wr"]["count"] == w["count"] >= sw.wr_keep == math.ceil(0.001 * 96 * 1024)
    assert np.array_equal(sp["wr"]["records"], w["records"]) and np.array_equal(sp["wr"]["row_start"], w["row_start"])
    assert sp["wr"]["scale_exp"] == w["scale_exp"]


def test_streams_beyond_one_round_of_the_tile_scan():
    """More than 1024 tiles of 256 blocks: the one-CTA scan carries its running sum from round to round."""
    M, K = 2304, 2048                                  # 294912 blocks = 1152 tiles
    L = I.laplace_outlier_layer(21, 3, M, K, 64)
    m = B.opq_threshold(0.92, 16)
    assert_opq(run_opq(L.W, m), oracle.opq_extract(L.W, m))
    fmt = I.scale_format("UE4M4")
    n_keep = math.ceil(0.001 * M * K)
    sw, out, got = run_wr(L, fmt, ["NF4", "SH4"], n_keep, None)
    want = oracle_wr(L, fmt, out, sw, n_keep)
    assert got["count"] == want["count"] >= n_keep and got["scale_exp"] == want["scale_exp"]
    assert np.array_equal(got["row_start"], want["row_start"]) and np.array_equal(got["records"], want["records"])


@pytest.mark.parametrize("rom,fp,fmt_name,iters", [(["NF5", "SH5", "BOF5"], (), "UE4M4", 0), (["NF5", "E2M2"], (), "E5M6", 3),
                                                  ([], ("E2M3",), "UE4M4", 0), ([], ("E4M3",), "E5M6", 0), ([], ("E3M4",), "UE4M4", 0)])
def test_wr_on_wider_codes_and_element_formats(rom, fp, fmt_name, iters):
    """The general decode: 5-bit table codes (ten bytes per block), and single element formats whose codes are the
    format's own bit pattern (6 and 8 bits)."""
    L = I.student_layer(17, 1, 20, 320, 64, 4.0)
    fmt = I.scale_format(fmt_name)
    n_keep = 40
    sw, out, got = run_wr(L, fmt, rom, n_keep, None, lloyd_iters=iters, fp=fp)
    want = oracle_wr(L, fmt, out, sw, n_keep)
    assert got["count"] == want["count"] >= n_keep and got["scale_exp"] == want["scale_exp"]
    assert np.array_equal(got["row_start"], want["row_start"]) and np.array_equal(got["records"], want["records"])


def test_wr_when_the_candidates_do_not_fit_their_list():
    """A layer whose residuals are all alike: every element lies in the bin of the block maxima, the candidate list
    (65536 entries here) overflows and the full decode passes take over.  The metrics differ through the channel
    norms only, so the threshold cuts between columns."""
    d = dev()
    M, K, T = 128, 2048, 16
    W = torch.full((M, K), 1.0078125, dtype=torch.bfloat16)            # 1 + 2^-7: the 6-bit scale mantissa rounds it to 1
    X = (1.0 + 0.2 * torch.arange(K, dtype=torch.float32) / K).repeat(T, 1).contiguous()
    L = I.Layer(W, X)
    fmt = I.scale_format("E5M6")
    n_keep = 5000
    sw, out, got = run_wr(L, fmt, ["NF4", "SH4"], n_keep, None)
    want = oracle_wr(L, fmt, out, sw, n_keep)
    assert want["count"] >= n_keep and want["count"] % M == 0 and want["count"] < M * K // 8        # whole columns, a small share
    assert got["count"] == want["count"] and got["scale_exp"] == want["scale_exp"]
    assert np.array_equal(got["row_start"], want["row_start"]) and np.array_equal(got["records"], want["records"])
    # the same layer with equal channel norms: every metric ties, everything is kept
    L1 = I.Layer(W, torch.ones(T, K))
    sw, out, got = run_wr(L1, fmt, ["NF4", "SH4"], 100, None)
    want = oracle_wr(L1, fmt, out, sw, 100)
    assert got["count"] == want["count"] == M * K and np.array_equal(got["records"], want["records"])


def test_layer_set_with_both_streams_shares_the_outlier_stream_between_formats():
    """A layer set at two scale formats with both streams: the outlier stream of a layer is extracted once (it does not
    depend on the scale format) and every (layer, format) correction equals that of a sweep of its own."""
    from paper_2605_14929_b200.pipeline import LayerSetSweep
    d = dev()
    shapes = [(48, 512, 64), (32, 768, 64), (48, 512, 64)]
    fmts = [I.scale_format("E5M6"), I.scale_format("UE4M4")]
    rom = ["NF4", "SH4", "BOF4"]
    layers = [I.laplace_outlier_layer(80 + i, i, M, K, T) for i, (M, K, T) in enumerate(shapes)]
    sset = LayerSetSweep(shapes, fmts, rom, [], 3, device=d, opq_q=0.92, wr_sigma=0.002)
    dev_layers = [(L.W.to(d), L.X.to(d)) for L in layers]
    got = {}
    for li, (row, (W, X)) in enumerate(zip(sset.sweeps, dev_layers)):       # layer by layer: the formats of a layer share its buffers
        for f, sw in enumerate(row):
            sw.run(W, X, norms=(f == 0), reuse_prepass=(f > 0))
            got[(li, f)] = (sw.outputs(), sw.sparse_outputs())
    for li, L in enumerate(layers):
        M, K, T = shapes[li]
        for f, fmt in enumerate(fmts):
            own = LayerSweep(M, K, T, fmt, rom, [], 3, device=d, opq_q=0.92, wr_sigma=0.002)
            own.run(*dev_layers[li])
            wo, ws = own.outputs(), own.sparse_outputs()
            go, gs = got[(li, f)]
            assert np.array_equal(gs["opq"]["records"], ws["opq"]["records"]) and gs["opq"]["count"] == ws["opq"]["count"] > 0
            assert torch.equal(go.codes, wo.codes) and torch.equal(go.words, wo.words)
            assert gs["wr"]["count"] == ws["wr"]["count"] and gs["wr"]["scale_exp"] == ws["wr"]["scale_exp"]
            assert np.array_equal(gs["wr"]["records"], ws["wr"]["records"]) and np.array_equal(gs["wr"]["row_start"], ws["wr"]["row_start"])
    # the whole set in one pass gives the last layer's results in the shared buffers, and runs without error
    sset.run(dev_layers)
    sset.check()


def test_wr_with_dead_channels_zero_blocks_and_large_rows():
    """Channels that never fire (c_k = 0: their residuals have no salience and are never kept), all-zero blocks, and
    rows scaled by 2^12 and 2^-12 (residuals far from 1: the layer exponent follows the largest kept residual)."""
    L = I.student_layer(31, 0, 24, 512, 64, 4.0)
    Wf = L.W.to(torch.float32).numpy().copy()
    Wf[3] *= 4096.0
    Wf[7] *= 1.0 / 4096.0
    Wf[5, 64:128] = 0.0
    X = L.X.clone()
    X[:, 16:48] = 0.0
    X[:, 300] = 0.0
    L2 = I.Layer(torch.from_numpy(Wf).to(torch.bfloat16), X)
    fmt = I.scale_format("E5M6")
    for n_keep in (5, 200, 24 * 512):
        sw, out, got = run_wr(L2, fmt, ["NF4", "SH4"], n_keep, None, lloyd_iters=2)
        want = oracle_wr(L2, fmt, out, sw, n_keep)
        assert got["count"] == want["count"] and got["scale_exp"] == want["scale_exp"] > 0
        assert np.array_equal(got["row_start"], want["row_start"]) and np.array_equal(got["records"], want["records"])
        cols = got["records"] & 0xFFFF
        assert not np.isin(cols, np.r_[16:48, 300]).any()              # dead channels are never kept
    assert got["count"] < 24 * 512                                       # ... even when everything is asked for
