"""ctypes marshalling for the CPU oracle.  Argument conversion only; the arithmetic is all in
``sop_oracle.cpp``.  Atoms and scale formats are duck-typed (any object with the attributes of
``inputs.Atom`` / ``inputs.ScaleFormat``), so this file imports nothing from the product package."""
from __future__ import annotations

import ctypes as C
from typing import Optional, Sequence

import numpy as np

from . import build as _build

K_AUTO = -1000


class _Fmt(C.Structure):
    _fields_ = [("sign_bits", C.c_int), ("exp_bits", C.c_int), ("man_bits", C.c_int), ("bias", C.c_int),
                ("top_exp_reserved", C.c_int)]


class _Atom(C.Structure):
    _fields_ = [("n_bits", C.c_int), ("kind", C.c_int), ("negated", C.c_int), ("scope", C.c_int),
                ("tmax", C.c_float), ("n_entries", C.c_int), ("lut", C.c_float * 32),
                ("grid_exp_bits", C.c_int), ("grid_man_bits", C.c_int), ("grid_bias", C.c_int), ("grid_neg_max", C.c_float)]


class _PairStat(C.Structure):
    _fields_ = [("acos", C.c_double), ("mse", C.c_double), ("n_sel1", C.c_longlong), ("n_neg", C.c_longlong)]


PAIR_DTYPE = np.dtype([("acos", "f8"), ("mse", "f8"), ("n_sel1", "i8"), ("n_neg", "i8")])

_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.osop_bpw.restype = C.c_double
        _lib.osop_scale_decode.restype = C.c_float
        _lib.osop_scale_word.restype = C.c_uint
        _lib.osop_fp_quantize.restype = C.c_float
        _lib.osop_fp_grid_value.restype = C.c_double
        _lib.osop_layer_pot_scale.restype = C.c_float
        _lib.osop_grid_quantize.restype = C.c_float
        _lib.osop_grid_value.restype = C.c_double
        _lib.osop_opq_threshold.restype = C.c_double
        _lib.osop_opq_extract.restype = C.c_longlong
        _lib.osop_wr_extract.restype = C.c_longlong
    return _lib


def _fmt(f) -> _Fmt:
    return _Fmt(f.sign_bits, f.exp_bits, f.man_bits, f.bias, f.top_exp_reserved)


def _atom(a) -> _Atom:
    s = _Atom()
    s.n_bits, s.kind, s.negated, s.scope, s.tmax = a.n_bits, a.kind, a.negated, a.scope, a.tmax
    s.n_entries = 0
    if a.lut is not None:
        s.n_entries = len(a.lut)
        for i, v in enumerate(a.lut):
            s.lut[i] = float(v)
    g = getattr(a, "grid", None)
    if g is not None:
        s.grid_exp_bits, s.grid_man_bits, s.grid_bias, s.grid_neg_max = g
    return s


def _atoms(atoms: Sequence) -> C.Array:
    arr = (_Atom * len(atoms))()
    for i, a in enumerate(atoms):
        arr[i] = _atom(a)
    return arr


def _p(a: np.ndarray, t):
    return a.ctypes.data_as(C.POINTER(t))


def _w16(W) -> np.ndarray:
    """bf16 torch tensor or uint16 array -> contiguous uint16 numpy array of bf16 bit patterns."""
    if isinstance(W, np.ndarray):
        assert W.dtype == np.uint16
        return np.ascontiguousarray(W)
    import torch
    return W.contiguous().view(torch.int16).numpy().view(np.uint16)


def bpw(scale_bits: int, g: int, elem_bits: int) -> float:
    return lib().osop_bpw(scale_bits, g, elem_bits)


def channel_norms(X) -> np.ndarray:
    X = np.ascontiguousarray(np.asarray(X, dtype=np.float32))
    T, K = X.shape
    c = np.empty(K, dtype=np.float32)
    lib().osop_channel_norms(_p(X, C.c_float), C.c_longlong(T), C.c_longlong(K), C.c_longlong(K), _p(c, C.c_float))
    return c


def scale_quantize(fmt, sigma: float, k: int):
    s, E, M = C.c_float(), C.c_uint(), C.c_uint()
    lib().osop_scale_quantize(C.byref(_fmt(fmt)), C.c_float(sigma), k, C.byref(s), C.byref(E), C.byref(M))
    return s.value, E.value, M.value


def scale_decode(fmt, E: int, M: int, k: int) -> float:
    return lib().osop_scale_decode(C.byref(_fmt(fmt)), E, M, k)


def scale_word(fmt, b: int, w_word: int, sign: int, E: int, M: int, sel: int) -> int:
    return lib().osop_scale_word(C.byref(_fmt(fmt)), b, w_word, sign, E, M, sel)


def f_layer(fmt, sigma) -> int:
    s = np.ascontiguousarray(np.asarray(sigma, dtype=np.float32))
    return lib().osop_f_layer(C.byref(_fmt(fmt)), _p(s, C.c_float), C.c_longlong(s.size))


def encode_lut(lut, u: float) -> int:
    l = np.ascontiguousarray(np.asarray(lut, dtype=np.float32))
    return lib().osop_encode_lut(_p(l, C.c_float), len(l), C.c_float(u))


def fp_quantize(kind: int, u: float):
    code = C.c_int()
    q = lib().osop_fp_quantize(kind, C.c_float(u), C.byref(code))
    return q, code.value


def fp_grid_value(kind: int, code: int) -> float:
    return lib().osop_fp_grid_value(kind, code)


def grid_quantize(atom, u: float):
    """(value, code) of u on the parametric element grid of ``atom`` (kind 3)."""
    code = C.c_int()
    q = lib().osop_grid_quantize(C.byref(_atom(atom)), C.c_float(u), C.byref(code))
    return q, code.value


def grid_value(atom, j: int) -> float:
    return lib().osop_grid_value(C.byref(_atom(atom)), j)


def layer_pot_scale(wmax: float, tmax: float) -> float:
    return lib().osop_layer_pot_scale(C.c_float(wmax), C.c_float(tmax))


def eval_block(w, c, atom, fmt, k: int, pot_scale: float = 0.0):
    w = np.ascontiguousarray(np.asarray(w, dtype=np.float32))
    c = np.ascontiguousarray(np.asarray(c, dtype=np.float32))
    cs, se, sh, E, M = C.c_float(), C.c_float(), C.c_float(), C.c_uint(), C.c_uint()
    codes = np.zeros(16, dtype=np.int32)
    q = np.zeros(16, dtype=np.float32)
    lib().osop_eval_block(_p(w, C.c_float), _p(c, C.c_float), C.byref(_atom(atom)), C.byref(_fmt(fmt)), k,
                          C.c_float(pot_scale), C.byref(cs), C.byref(se), C.byref(sh), C.byref(E), C.byref(M),
                          _p(codes, C.c_int), _p(q, C.c_float))
    return dict(cos=cs.value, sse=se.value, s_hat=sh.value, E=E.value, M=M.value, codes=codes, q=q)


def pair_search(W, c, fmt, atoms, k_mode: int = K_AUTO, want_blocks: bool = False, select_metric: int = 0):
    """Returns dict(pair, signed, k, best, block_cos, block_sse).  select_metric: 0 = the block cosine decides
    the per-block reassignment, 1 = the block squared error does (design axis ii)."""
    w16 = _w16(W)
    M, K = w16.shape
    c = np.ascontiguousarray(np.asarray(c, dtype=np.float32))
    A = len(atoms)
    NB = M * (K // 16)
    pair = np.zeros((A, A), dtype=PAIR_DTYPE)
    sgn = np.zeros((A, A), dtype=PAIR_DTYPE)
    k_out = np.zeros(A, dtype=np.int32)
    best = np.zeros(5, dtype=np.int32)
    bc = np.zeros((A, NB), dtype=np.float32) if want_blocks else None
    bs = np.zeros((A, NB), dtype=np.float32) if want_blocks else None
    lib().osop_pair_search_axes(_p(w16, C.c_uint16), C.c_longlong(M), C.c_longlong(K), C.c_longlong(K), _p(c, C.c_float),
                           C.byref(_fmt(fmt)), k_mode, _atoms(atoms), A, int(select_metric), _p(pair, _PairStat), _p(sgn, _PairStat),
                           _p(k_out, C.c_int), _p(best, C.c_int),
                           _p(bc, C.c_float) if want_blocks else None, _p(bs, C.c_float) if want_blocks else None)
    return dict(pair=pair, signed=sgn, k=k_out, best=best, block_cos=bc, block_sse=bs)


def dd_lloyd(W, c, fmt, k: int, block_cos, pool_rank: int, init_lut, iters: int, pool_by_error: bool = False,
             pool_threshold: float = 0.0, uniform_weights: bool = False):
    """Returns (lut, distortion[iters + 1], pool_count).  block_cos holds the per-block metric that ranks the
    blocks: cosines, or squared errors with pool_by_error (axis i); pool_rank = 0 takes pool_threshold instead of
    a rank (axis iv); uniform_weights sets every Lloyd weight to 1 (axis iii)."""
    w16 = _w16(W)
    M, K = w16.shape
    c = np.ascontiguousarray(np.asarray(c, dtype=np.float32))
    bc = np.ascontiguousarray(np.asarray(block_cos, dtype=np.float32))
    init = np.ascontiguousarray(np.asarray(init_lut, dtype=np.float32))
    out = np.zeros(len(init), dtype=np.float32)
    dist = np.zeros(iters + 1, dtype=np.float64)
    cnt = C.c_longlong()
    lib().osop_dd_lloyd_axes(_p(w16, C.c_uint16), C.c_longlong(M), C.c_longlong(K), C.c_longlong(K), _p(c, C.c_float),
                             C.byref(_fmt(fmt)), k, _p(bc, C.c_float), int(bool(pool_by_error)), C.c_longlong(pool_rank),
                             C.c_float(pool_threshold), int(bool(uniform_weights)), _p(init, C.c_float),
                             len(init), iters, _p(out, C.c_float), _p(dist, C.c_double), C.byref(cnt))
    return out, dist, cnt.value


def dd_grid_dp(W, c, fmt, k: int, block_metric, pool_rank: int, n_entries: int, pool_by_error: bool = False,
               pool_threshold: float = 0.0, uniform_weights: bool = False):
    """Grid-constrained DD-n by dynamic programming over the cell histogram of the pool.
    Returns (lut[n_entries], cost, pool_count); the pool arguments are those of ``dd_lloyd``."""
    w16 = _w16(W)
    M, K = w16.shape
    c = np.ascontiguousarray(np.asarray(c, dtype=np.float32))
    bm = np.ascontiguousarray(np.asarray(block_metric, dtype=np.float32))
    out = np.zeros(n_entries, dtype=np.float32)
    cost = C.c_double()
    cnt = C.c_longlong()
    lib().osop_dd_grid_dp(_p(w16, C.c_uint16), C.c_longlong(M), C.c_longlong(K), C.c_longlong(K), _p(c, C.c_float),
                          C.byref(_fmt(fmt)), k, _p(bm, C.c_float), int(bool(pool_by_error)), C.c_longlong(pool_rank),
                          C.c_float(pool_threshold), int(bool(uniform_weights)), n_entries, _p(out, C.c_float),
                          C.byref(cost), C.byref(cnt))
    return out, cost.value, cnt.value


def pack(W, c, fmt, a, k_a: int, b=None, k_b: int = 0, use_sign: int = 0, container_bits: int = 8,
         word_sign_bits: int = 0, select_metric: int = 0):
    """Returns dict(rc, codes [N_b, 2n] uint8, words uint8 stream, n_sel1, n_neg)."""
    w16 = _w16(W)
    M, K = w16.shape
    c = np.ascontiguousarray(np.asarray(c, dtype=np.float32))
    NB = M * (K // 16)
    codes = np.zeros((NB, 2 * a.n_bits), dtype=np.uint8)
    words = np.zeros((NB * container_bits + 7) // 8, dtype=np.uint8)
    n1, nn = C.c_longlong(), C.c_longlong()
    rc = lib().osop_pack_axes(_p(w16, C.c_uint16), C.c_longlong(M), C.c_longlong(K), C.c_longlong(K), _p(c, C.c_float),
                         C.byref(_fmt(fmt)), C.byref(_atom(a)), k_a, C.byref(_atom(b)) if b is not None else None, k_b,
                         use_sign, container_bits, word_sign_bits, int(select_metric), _p(codes, C.c_ubyte), _p(words, C.c_ubyte),
                         C.byref(n1), C.byref(nn))
    return dict(rc=rc, codes=codes, words=words, n_sel1=n1.value, n_neg=nn.value)


def opq_threshold(q: float, max_order: int = 16) -> float:
    """m with (2 Phi(m) - 1)^M = q (Section "Outlier Per-Quantum Extraction (OPQ)")."""
    return float(lib().osop_opq_threshold(C.c_double(q), int(max_order)))


def opq_extract(W, m: float, capacity: int = None):
    """Returns dict(W_out [M, K] uint16 bf16 bits, row_start [M + 1] uint32, records uint32 (k | bf16 << 16), count)."""
    w16 = _w16(W)
    M, K = w16.shape
    cap = M * K if capacity is None else int(capacity)
    out = np.zeros_like(w16)
    row_start = np.zeros(M + 1, dtype=np.uint32)
    records = np.zeros(max(cap, 1), dtype=np.uint32)
    n = lib().osop_opq_extract(_p(w16, C.c_uint16), C.c_longlong(M), C.c_longlong(K), C.c_longlong(K), C.c_double(m),
                               _p(out, C.c_uint16), C.c_longlong(K), _p(row_start, C.c_uint), _p(records, C.c_uint), C.c_longlong(cap))
    return dict(W_out=out, row_start=row_start, records=records[:min(n, cap)].copy(), count=int(n))


def wr_extract(W, c, fmt, a, k_a: int, b=None, k_b: int = 0, use_sign: int = 0, n_keep: int = 1, select_metric: int = 0,
               capacity: int = None, want_resid: bool = False):
    """Returns dict(row_start, records uint32 (k | E3M4 code << 16), count, scale_exp, tau[, resid [M, K] float32])."""
    w16 = _w16(W)
    M, K = w16.shape
    c = np.ascontiguousarray(np.asarray(c, dtype=np.float32))
    cap = M * K if capacity is None else int(capacity)
    row_start = np.zeros(M + 1, dtype=np.uint32)
    records = np.zeros(max(cap, 1), dtype=np.uint32)
    resid = np.zeros((M, K), dtype=np.float32) if want_resid else None
    e, tau = C.c_int(), C.c_float()
    n = lib().osop_wr_extract(_p(w16, C.c_uint16), C.c_longlong(M), C.c_longlong(K), C.c_longlong(K), _p(c, C.c_float),
                              C.byref(_fmt(fmt)), C.byref(_atom(a)), k_a, C.byref(_atom(b)) if b is not None else None, k_b,
                              use_sign, int(select_metric), C.c_longlong(int(n_keep)), _p(row_start, C.c_uint), _p(records, C.c_uint),
                              C.c_longlong(cap), C.byref(e), C.byref(tau), _p(resid, C.c_float) if want_resid else None)
    out = dict(row_start=row_start, records=records[:min(n, cap)].copy(), count=int(n), scale_exp=e.value, tau=float(tau.value))
    if want_resid:
        out["resid"] = resid
    return out
