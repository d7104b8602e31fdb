"""Pins of the oracle's two sparse side streams: outlier extraction before the search (Section "Outlier
Per-Quantum Extraction (OPQ)") and the sparse correction of the codebook residual (Section "Sparse Residual
Correction (Wr)").  The threshold is checked against the quantile it is defined by (another library's inverse normal
CDF, and a Monte-Carlo count), the outlier test against exact rational arithmetic and a closed-form boundary, the
residual against the packed stream decoded here, the selection against a sort, the stored values against a brute-force
search of the E3M4 grid."""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2605_14929_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "sparse_stream_costs.txt")


def bf16_bits(W: torch.Tensor) -> np.ndarray:
    return W.view(torch.int16).numpy().view(np.uint16)


def bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32)


def to_bf16(x) -> torch.Tensor:
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)


# ---------------------------------------------------------------- OPQ threshold

@pytest.mark.parametrize("q,M", [(0.92, 16), (0.5, 16), (0.99, 16), (0.92, 8), (0.92, 32), (0.999, 16)])
def test_threshold_is_the_quantile_of_the_block_maximum(q, M):
    from scipy.special import ndtri
    m = oracle.opq_threshold(q, M)
    # (2 Phi(m) - 1)^M = q  <=>  Phi(m) = (1 + q^(1/M)) / 2
    assert m == pytest.approx(float(ndtri((1.0 + q ** (1.0 / M)) / 2.0)), rel=1e-12)


def test_threshold_monte_carlo_and_the_papers_default():
    m = oracle.opq_threshold(0.92, 16)
    # the paper prints m "about 2.7" for q = 0.92 at g = 16; its formula gives 2.79
    assert 2.7 <= m <= 2.85
    rng = np.random.default_rng(11)
    n = 400_000
    z = rng.standard_normal((n, 16))
    frac = float((np.abs(z).max(axis=1) < m).mean())      # F_M(m): no element of the block beyond m
    assert abs(frac - 0.92) < 4.0 * np.sqrt(0.92 * 0.08 / n)
    # per element: 1 - q^(1/16) = 0.52 % for unit-variance Gaussian blocks
    assert float((np.abs(z) > m).mean()) == pytest.approx(1.0 - 0.92 ** (1.0 / 16.0), rel=0.02)


def test_stream_costs_printed_in_the_paper():
    rows = [ln.split("#")[0].split() for ln in open(GOLDEN) if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for name, bits, rate, bpw, tol in rows:
        assert int(bits) == 32                                  # 16-bit index + bf16 value; 16-bit index + 8-bit value + headers
        assert abs(int(bits) * float(rate) - float(bpw)) <= float(tol)


# ---------------------------------------------------------------- OPQ extraction

def exact_mask(w_block: np.ndarray, m: float) -> list:
    """|w_i| / sqrt(mean w^2) > m in exact rational arithmetic."""
    w = [Fraction(float(x)) for x in w_block]
    s2 = sum(x * x for x in w)
    m2 = Fraction(m) * Fraction(m)
    return [x * x * 16 > m2 * s2 for x in w]


def test_outlier_test_against_exact_rational_arithmetic():
    L = I.tiny_layer(3, 12, 96)
    W = L.W.clone()
    Wf = W.to(torch.float32).numpy()
    Wf[2, 5] *= 9.0; Wf[7, 40] *= -14.0; Wf[7, 41] *= 6.0; Wf[11, 95] *= 20.0      # a few planted spikes
    Wf[4, 16:32] = 0.0                                                                 # a zero block
    W = to_bf16(Wf)
    Wf = W.to(torch.float32).numpy()
    m = oracle.opq_threshold(0.92, 16)
    got = oracle.opq_extract(W, m)
    want = np.zeros(Wf.shape, dtype=bool)
    for r in range(Wf.shape[0]):
        for j in range(Wf.shape[1] // 16):
            want[r, 16 * j:16 * j + 16] = exact_mask(Wf[r, 16 * j:16 * j + 16], m)
    assert want[2, 5] and want[7, 40] and want[11, 95] and not want[4, 16:32].any()
    bits = bf16_bits(W)
    # W_out: outliers zeroed, everything else untouched
    assert np.array_equal(got["W_out"], np.where(want, np.uint16(0), bits))
    # stream: ascending by (row, column), the exact bf16 value kept
    rows, cols = np.nonzero(want)
    assert got["count"] == len(rows) == int(got["row_start"][-1])
    assert np.array_equal(got["records"] & 0xFFFF, cols.astype(np.uint32))
    assert np.array_equal(got["records"] >> 16, bits[rows, cols].astype(np.uint32))
    assert np.array_equal(got["row_start"], np.concatenate([[0], np.cumsum(want.sum(axis=1))]).astype(np.uint32))
    # zeroed input + scattered stream = the original, bit for bit
    back = got["W_out"].copy()
    for r in range(Wf.shape[0]):
        for rec in got["records"][got["row_start"][r]:got["row_start"][r + 1]]:
            back[r, rec & 0xFFFF] = rec >> 16
    assert np.array_equal(back, bits)


def test_outlier_boundary_closed_form():
    # fifteen ones and one x: x^2 16 > m^2 (15 + x^2)  <=>  x > m sqrt(15 / (16 - m^2));  m = 2: 2.2360...
    m = 2.0
    edge = m * np.sqrt(15.0 / (16.0 - m * m))
    assert 2.234375 < edge < 2.25                               # two neighbouring bf16 values
    for x, is_out in ((2.234375, False), (2.25, True), (-2.25, True), (-2.234375, False)):
        w = np.ones((1, 16), dtype=np.float32)
        w[0, 9] = x
        got = oracle.opq_extract(to_bf16(w), m)
        assert got["count"] == int(is_out)
        if is_out:
            assert got["records"][0] == (9 | (int(bf16_bits(to_bf16(np.float32([x])))[0]) << 16))
    # equal magnitudes: |w| / rms = 1, never beyond a threshold above 1
    assert oracle.opq_extract(to_bf16(np.full((2, 32), -0.37, dtype=np.float32)), 1.0001)["count"] == 0


def test_outlier_mask_is_scale_free_and_capacity_only_truncates():
    L = I.laplace_outlier_layer(5, 0, 16, 128, 8)
    m = 2.5
    a = oracle.opq_extract(L.W, m)
    assert a["count"] > 0
    scaled = to_bf16(L.W.to(torch.float32).numpy() * np.float32(2.0 ** -9))      # exact in bf16
    b = oracle.opq_extract(scaled, m)
    assert np.array_equal(a["records"] & 0xFFFF, b["records"] & 0xFFFF) and np.array_equal(a["row_start"], b["row_start"])
    cut = oracle.opq_extract(L.W, m, capacity=3)
    assert cut["count"] == a["count"] and np.array_equal(cut["records"], a["records"][:3]) and np.array_equal(cut["W_out"], a["W_out"])


# ---------------------------------------------------------------- Wr

E3M4 = [0.0] + [(mm / 16.0) * 2.0 ** -2 for mm in range(1, 16)] + [(1.0 + mm / 16.0) * 2.0 ** (e - 3) for e in range(1, 7) for mm in range(16)]


def e3m4_value(code: int) -> float:
    e, mm = (code >> 4) & 7, code & 15
    v = (mm / 16.0) * 2.0 ** -2 if e == 0 else (1.0 + mm / 16.0) * 2.0 ** (e - 3)
    return -v if code & 0x80 else v


def decode_packed(W, fmt, a, k_a, b, k_b, use_sign, pk, bits, sign_bits):
    """(s_hat, q) per element from the packed stream, decoded here: scale word fields by the bit placement
    (sign at the top, selector = metabit 0 with a sign bit and the top bit without), codes as 4-bit fields."""
    M, K = W.shape
    nbk = K // 16
    s_hat = np.zeros((M, K), dtype=np.float32)
    q = np.zeros((M, K), dtype=np.float32)
    stream = int.from_bytes(pk["words"].tobytes(), "little")
    y, x = fmt.man_bits, fmt.exp_bits
    meta = bits - sign_bits - x - y
    for blk in range(M * nbk):
        word = (stream >> (blk * bits)) & ((1 << bits) - 1)
        if sign_bits:
            sgn, sel, code = word >> (bits - 1), word & 1 if meta >= 1 else 0, (word >> meta) & ((1 << (x + y)) - 1)
        else:
            sgn, sel, code = 0, word >> (bits - 1) if meta >= 1 else 0, (word >> max(meta - 1, 0)) & ((1 << (x + y)) - 1)
        atom, k = (b, k_b) if sel else (a, k_a)
        s = oracle.scale_decode(fmt, code >> y, code & ((1 << y) - 1), k)
        lut = np.asarray(atom.lut, dtype=np.float32)
        neg = atom.negated ^ sgn
        payload = int.from_bytes(pk["codes"][blk].tobytes(), "little")
        r, j = divmod(blk, nbk)
        for i in range(16):
            cd = (payload >> (4 * i)) & 15
            s_hat[r, 16 * j + i] = s
            q[r, 16 * j + i] = -lut[cd] if neg else lut[cd]
    return s_hat, q


def wr_case(seed=2, M=8, K=64, fmt_name="S1E4M4", use_sign=1, n_keep=9):
    L = I.tiny_layer(seed, M, K)
    c = oracle.channel_norms(L.X.numpy())
    fmt = I.scale_format(fmt_name)
    a, b = I.rom_atom("NF4"), I.rom_atom("SH4")
    bits = 12 if use_sign else 8
    pk = oracle.pack(L.W, c, fmt, a, 0, b, 0, use_sign=use_sign, container_bits=12, word_sign_bits=use_sign)
    assert pk["rc"] == 0
    wr = oracle.wr_extract(L.W, c, fmt, a, 0, b, 0, use_sign=use_sign, n_keep=n_keep, want_resid=True)
    return L, c, fmt, a, b, pk, wr


@pytest.mark.parametrize("fmt_name,use_sign", [("S1E4M4", 1), ("UE4M4", 0)])
def test_residual_is_the_weight_minus_the_decoded_packed_stream(fmt_name, use_sign):
    L, c, fmt, a, b, pk, wr = wr_case(fmt_name=fmt_name, use_sign=use_sign)
    s_hat, q = decode_packed(L.W, fmt, a, 0, b, 0, use_sign, pk, 12, use_sign)
    Wf = L.W.to(torch.float32).numpy()
    E = wr["resid"]
    for r in range(Wf.shape[0]):
        for k in range(Wf.shape[1]):
            exact = Fraction(float(Wf[r, k])) - Fraction(float(s_hat[r, k])) * Fraction(float(q[r, k]))
            e = float(E[r, k])
            ulp = Fraction(float(np.spacing(np.float32(abs(e))))) if e != 0.0 else Fraction(2) ** -149
            assert abs(Fraction(e) - exact) <= ulp / 2            # one rounding of w - s_hat q


@pytest.mark.parametrize("n_keep", [1, 9, 64, 511])
def test_selection_is_the_top_of_a_sort_and_values_are_the_nearest_grid_points(n_keep):
    L, c, fmt, a, b, pk, wr = wr_case(n_keep=n_keep)
    E = wr["resid"]
    metric = (np.abs(E) * c[None, :].astype(np.float32)).astype(np.float32)
    order = np.sort(metric.ravel())[::-1]
    tau = order[n_keep - 1]
    assert np.float32(wr["tau"]) == tau
    keep = (metric >= tau) & (metric > 0)
    rows, cols = np.nonzero(keep)
    assert wr["count"] == len(rows) >= n_keep
    assert np.array_equal(wr["records"] & 0xFFFF, cols.astype(np.uint32))
    assert np.array_equal(wr["row_start"], np.concatenate([[0], np.cumsum(keep.sum(axis=1))]).astype(np.uint32))
    # nothing left out is more salient than anything kept
    assert metric[~keep].max() < metric[keep].min()
    # the layer exponent: the smallest power of two that brings the kept residuals inside the E3M4 range
    emax = float(np.abs(E[keep]).max())
    e = wr["scale_exp"]
    assert emax <= 15.5 * 2.0 ** e and emax > 15.5 * 2.0 ** (e - 1)
    # every stored value is the grid point nearest to E / 2^e (brute force over the 112 magnitudes), ties to the even number
    grid = np.array(E3M4)
    for rec, r, k in zip(wr["records"], rows, cols):
        code = int(rec >> 16)
        assert code < 256 and ((code >> 4) & 7) != 7
        x = float(E[r, k]) / 2.0 ** e
        v = e3m4_value(code)
        d = np.abs(grid - abs(x))
        assert abs(abs(v) - abs(x)) == d.min()
        if (d == d.min()).sum() == 2:
            assert (code & 0x7F) % 2 == 0
        assert (v < 0) == (x < 0) or v == 0.0
    # the correction lowers the activation-weighted error of the layer
    corr = np.zeros_like(E, dtype=np.float64)
    for rec, r, k in zip(wr["records"], rows, cols):
        corr[r, k] = e3m4_value(int(rec >> 16)) * 2.0 ** e
    c64 = c.astype(np.float64)[None, :]
    assert ((E - corr) ** 2 * c64 ** 2).sum() < (E.astype(np.float64) ** 2 * c64 ** 2).sum()


def test_ties_at_the_threshold_all_enter_and_zero_residuals_never_do():
    L = I.tiny_layer(4, 4, 64)
    W = torch.cat([L.W, L.W], dim=0)                     # every metric value appears twice
    c = oracle.channel_norms(L.X.numpy())
    fmt = I.scale_format("UE4M4")
    a = I.rom_atom("NF4")
    wr = oracle.wr_extract(W, c, fmt, a, 0, None, 0, use_sign=0, n_keep=5)
    assert wr["count"] == 6
    half = wr["row_start"][4]
    assert np.array_equal(wr["records"][:half], wr["records"][half:])
    # weights that the table represents exactly leave no residual: nothing is stored
    lut = np.asarray(a.lut, dtype=np.float32)
    rng = np.random.default_rng(0)
    idx = rng.integers(0, 16, (4, 64))
    idx[:, ::16] = 15                                    # the block maximum is the table's maximum: scale 1/4 exactly
    Wg = to_bf16(lut[idx] * np.float32(0.25))
    assert np.array_equal(Wg.to(torch.float32).numpy(), lut[idx] * np.float32(0.25))
    z = oracle.wr_extract(Wg, c, fmt, a, 0, None, 0, use_sign=0, n_keep=7, want_resid=True)
    assert not z["resid"].any() and z["count"] == 0 and z["scale_exp"] == 0


# ---------------------------------------------------------------- soft checks against the paper's claims

def block_acos(W, What, c):
    """Mean over blocks of the c-weighted cosine between w and its reconstruction (float64)."""
    M, K = W.shape
    w = W.astype(np.float64).reshape(M, K // 16, 16)
    q = What.astype(np.float64).reshape(M, K // 16, 16)
    cb = np.asarray(c, dtype=np.float64).reshape(1, K // 16, 16)
    dot = (cb * w * q).sum(axis=2)
    nw = (cb * w * w).sum(axis=2)
    nq = (cb * q * q).sum(axis=2)
    cos = np.where((nw > 0) & (nq > 0), dot / np.sqrt(np.where(nw * nq > 0, nw * nq, 1.0)), np.where((nw == 0) & (nq == 0), 1.0, 0.0))
    return float(cos.mean())


def test_wr_gains_a_few_ppm_of_acos_at_four_bits():
    # the paper: sparsity 0.001 costs about 0.032 bpw and typically gains 5-15 ppm of pair-mean ACos at 4-bit codebooks
    L = I.student_layer(23, 0, 96, 1024, 256, 5.0, channel_sigma=0.5)
    c = oracle.channel_norms(L.X.numpy())
    fmt = I.scale_format("S1E5M5")
    a, b = I.rom_atom("NF4"), I.rom_atom("SH4")
    n_keep = int(np.ceil(0.001 * 96 * 1024))
    wr = oracle.wr_extract(L.W, c, fmt, a, 0, b, 0, use_sign=1, n_keep=n_keep, want_resid=True)
    Wf = L.W.to(torch.float32).numpy()
    What = Wf.astype(np.float64) - wr["resid"].astype(np.float64)
    before = block_acos(Wf, What, c)
    corrected = What.copy()
    rs = wr["row_start"]
    for r in range(96):
        for rec in wr["records"][rs[r]:rs[r + 1]]:
            corrected[r, rec & 0xFFFF] += e3m4_value(int(rec >> 16)) * 2.0 ** wr["scale_exp"]
    after = block_acos(Wf, corrected, c)
    gain_ppm = (after - before) * 1e6
    assert 0.997 < before < 0.9995                 # the paper's typical range of 4-bit pairs is [0.997, 0.999]
    assert 1.0 < gain_ppm < 200.0                  # a few ppm to a few tens of ppm
    assert 32.0 * wr["count"] / (96 * 1024) == pytest.approx(0.032, abs=0.002)


def test_opq_makes_the_codebook_input_easier():
    # with the outliers stored exactly, the rest of the block concentrates inside the table's range: the best pair's
    # ACos on the zeroed weights is above that on the original ones, and the stream costs 32 bits per outlier
    L = I.laplace_outlier_layer(29, 0, 64, 1024, 128, frac=0.003)
    c = oracle.channel_norms(L.X.numpy())
    fmt = I.scale_format("S1E5M5")
    atoms = I.alphabet(["NF4", "SH4", "BOF4"])
    m = oracle.opq_threshold(0.92, 16)
    o = oracle.opq_extract(L.W, m)
    W2 = torch.from_numpy(o["W_out"].view(np.int16).copy()).view(torch.bfloat16)
    r0 = oracle.pair_search(L.W, c, fmt, atoms)
    r1 = oracle.pair_search(W2, c, fmt, atoms)
    best0 = r0["pair"]["acos"][r0["best"][0], r0["best"][1]]
    best1 = r1["pair"]["acos"][r1["best"][0], r1["best"][1]]
    assert best1 > best0
    rate = o["count"] / (64 * 1024)
    assert 0.003 <= rate < 0.05                    # at least the planted 8-sigma spikes
    assert 32.0 * rate < 1.6
