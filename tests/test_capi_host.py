"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, and rejects bad arguments on the host before anything is launched."""
import ctypes as C
import dataclasses
import os
import re

import numpy as np
import pytest

from paper_2605_14929_b200 import binding as B
from paper_2605_14929_b200 import build as libbuild
from paper_2605_14929_b200 import inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    libbuild.build()
    return B.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "sop.h")).read()
    declared = set(re.findall(r"\b(sop_[a-z0-9_]+)\s*\(", header))
    assert declared == set(B.exported_symbols())
    for name in declared:
        assert hasattr(lib, name), name
    assert lib.sop_version() >= 100


def test_struct_layouts_match_header():
    assert C.sizeof(B.AtomStruct) == 6 * 4 + 32 * 4 + 4 * 4
    assert C.sizeof(B.PairStat) == 32 and B.PAIR_DTYPE.itemsize == 32
    assert C.sizeof(B.SearchResult) == 16 * 4 + 5 * 4 + 4 + 8
    assert C.sizeof(B.ScaleFmt) == 20


def test_error_text(lib):
    for code in range(0, -8, -1):
        assert len(lib.sop_strerror(code)) > 1
    assert b"unknown" in lib.sop_strerror(-99)


FAKE = C.c_void_p(0x10000)     # never dereferenced: every call below fails validation first


def _search(lib, M=4, K=64, ldw=64, g=16, fmt=None, atoms=None, n=None, k=B.K_AUTO, W=FAKE, ws=FAKE, wsb=1 << 30,
            dd=None, mask=0, emask=0xFFFFFFFF, lmask=0, flags=0, bc=None, prev=None):
    fmt = fmt or I.scale_format("UE4M4")
    atoms = atoms if atoms is not None else I.alphabet(["NF4"])
    n = len(atoms) if n is None else n
    return lib.sop_pair_search(W, C.c_longlong(M), C.c_longlong(K), C.c_longlong(ldw), FAKE, g, C.byref(B.make_fmt(fmt)), k,
                               B.make_atoms(atoms), n, dd, C.c_uint(mask), C.c_uint(emask), C.c_uint(lmask), flags, prev, FAKE, None, FAKE, bc,
                               bc, ws,
                               C.c_size_t(wsb), None)


def test_pair_search_rejects_bad_arguments(lib):
    assert _search(lib, W=None) == -1
    assert _search(lib, K=60, ldw=60) == -2            # K % 16
    assert _search(lib, M=0) == -2
    assert _search(lib, ldw=32) == -2                  # ld < K
    assert _search(lib, g=32) == -2
    assert _search(lib, W=C.c_void_p(0x10004)) == -2   # W not 16-byte aligned
    bad = I.ScaleFormat("bad", 0, 9, 3, 7)
    assert _search(lib, fmt=bad) == -3
    assert _search(lib, fmt=I.ScaleFormat("bad", 0, 8, 7, 127, 0)) == -3   # largest scale not finite in fp32
    assert _search(lib, n=0) == -4 and _search(lib, n=17) == -4
    a = I.rom_atom("NF4")
    a.lut = a.lut[::-1].copy()
    assert _search(lib, atoms=[a]) == -4               # unsorted table
    a = I.rom_atom("NF4")
    a.tmax = 0.0
    assert _search(lib, atoms=[a]) == -4
    a = I.fp_atom("E2M3")
    a.n_bits = 5
    assert _search(lib, atoms=[a]) == -4
    assert _search(lib, k=65) == -7
    assert _search(lib, ws=None) == -5 and _search(lib, wsb=16) == -5
    assert _search(lib, ws=C.c_void_p(0x10010)) == -5  # workspace not 256-byte aligned
    assert _search(lib, mask=1) == -1                  # dd_mask without a device table
    assert _search(lib, mask=4, dd=FAKE) == -4         # mask bit beyond the alphabet
    assert _search(lib, emask=0) == -4                 # nothing evaluated and nothing loaded
    assert _search(lib, emask=1, lmask=1, bc=FAKE) == -4   # a candidate both evaluated and loaded
    assert _search(lib, emask=0, lmask=4, bc=FAKE) == -4   # load bit beyond the alphabet
    atoms2 = I.alphabet(["NF4"])
    assert _search(lib, atoms=atoms2, emask=1, lmask=2) == -1   # loading needs the per-block arrays
    assert _search(lib, flags=16) == -7                # unknown flag
    assert _search(lib, k=B.K_FROM_RESULT) == -1       # shifts from an earlier result need that result
    assert _search(lib, k=B.K_FROM_RESULT, prev=C.c_void_p(0x20000)) == -7   # ... and a loaded candidate in every class


def test_other_entry_points_reject_bad_arguments(lib):
    ll = C.c_longlong
    n = C.c_size_t()
    assert lib.sop_channel_norms_workspace(ll(0), ll(8), C.byref(n)) == -2
    assert lib.sop_channel_norms_workspace(ll(130), ll(8), C.byref(n)) == 0 and n.value == 3 * 8 * 8
    assert lib.sop_channel_norms(None, ll(4), ll(8), ll(8), FAKE, FAKE, C.c_size_t(1 << 20), None) == -1
    assert lib.sop_channel_norms(FAKE, ll(4), ll(8), ll(4), FAKE, FAKE, C.c_size_t(1 << 20), None) == -2
    assert lib.sop_channel_norms(FAKE, ll(4), ll(8), ll(8), FAKE, FAKE, C.c_size_t(8), None) == -5
    fmt = C.byref(B.make_fmt(I.scale_format("UE4M4")))
    atoms = I.alphabet(["NF4", "SH4"])
    arr = B.make_atoms(atoms)

    def lloyd(rank=1, iters=8, k=0, fmta=0, res=None, flags=0, thr=0.0):
        return lib.sop_dd4_lloyd(FAKE, ll(4), ll(64), ll(64), FAKE, 16, fmt, k, res, FAKE, ll(rank), C.c_float(thr), flags, arr,
                                 len(atoms), fmta, iters, FAKE, FAKE, FAKE, FAKE, C.c_size_t(1 << 20), None)
    assert lloyd(rank=0) == -7 and lloyd(rank=17) == -7 and lloyd(iters=65) == -7 and lloyd(k=99) == -7
    assert lloyd(flags=32) == -7                                          # unknown flag
    assert lloyd(flags=B.LLOYD_GRID_DP, iters=8) == -7                    # the dynamic programme replaces the iterations
    assert lloyd(flags=B.LLOYD_POOL_THRESHOLD, thr=float("nan")) == -7    # a NaN threshold orders nothing
    assert lloyd(rank=0, flags=B.LLOYD_POOL_THRESHOLD, iters=65) == -7    # the rank is ignored, the rest is still checked
    assert lloyd(fmta=9) == -7
    assert lloyd(k=B.K_FROM_RESULT) == -1 and lloyd(fmta=B.FMTA_FROM_RESULT) == -1

    def pack(ia=0, ib=2, k=0, sign=0, b=12, wsb=0, res=None, f=fmt, flags=0):
        return lib.sop_pack(FAKE, ll(4), ll(64), ll(64), FAKE, 16, f, arr, len(atoms), None, C.c_uint(0), ia, ib, k, res,
                            sign, b, wsb, FAKE, FAKE, None, None, flags, None)
    assert pack(flags=2) == -7
    assert pack(b=8) == -3                  # UE4M4 in 8 bits has no metabit for the selector
    assert pack(b=10) == -3
    assert pack(sign=1, wsb=0) == -3        # sign requested, word has no sign bit
    assert pack(ia=5) == -7 and pack(ib=7) == -7
    assert pack(ia=B.PAIR_FROM_RESULT) == -1
    assert pack(k=B.K_FROM_RESULT) == -1


def test_grid_arguments_are_checked_on_the_host(lib):
    FAKE = C.c_void_p(0x1000)
    ll = C.c_longlong
    fmt = C.byref(B.make_fmt(I.scale_format("UE4M4")))

    def search(atom):
        arr = B.make_atoms([atom])
        return lib.sop_pair_search(FAKE, ll(4), ll(64), ll(64), FAKE, 16, fmt, 0, arr, 1, None, C.c_uint(0), C.c_uint(1), C.c_uint(0), 0,
                                   None, FAKE, None, FAKE, None, None, None, C.c_size_t(0), None)

    good = I.fp_atom("HIF7")
    assert search(dataclasses.replace(good, tmax=121.0)) == -4                       # 121 is not a value of the grid
    assert search(dataclasses.replace(good, grid=(0, 3, -2, 100.0))) == -4           # negative end below the positive one
    assert search(dataclasses.replace(good, grid=(0, 11, -2, 128.0))) == -4          # too many mantissa bits
    assert search(dataclasses.replace(good, negated=1)) == -4
    assert search(good) == -5                                                          # passes the atom checks, stops at the workspace
    # a grid without a sign|E|M code, or wider than 8 bits, is not packed
    for atom in (I.fp_atom("HIF7"), I.fp_atom("E3M6")):
        arr = B.make_atoms([atom])
        rc = lib.sop_pack(FAKE, ll(4), ll(64), ll(64), FAKE, 16, fmt, arr, 1, None, C.c_uint(0), 0, B.NO_ATOM, 0, None, 0, 12, 0,
                          C.c_void_p(0x1000), FAKE, None, None, 0, None)
        assert rc == -4


def test_lloyd_status_entry_is_read_on_the_host(lib):
    # distortion[iters] < 0 marks a call that did not run to its end: the binding turns it into an exception
    import torch
    d = torch.tensor([3.0, 2.0, 1.5], dtype=torch.float64)
    B.check_lloyd_status(d, 2)
    d[2] = -1.0
    with pytest.raises(B.LloydNotFinished):
        B.check_lloyd_status(d, 2)
    B.check_lloyd_status(d, 1)


def test_lloyd_tuning_ranges(lib):
    assert lib.sop_dd4_lloyd_tuning(0, 0, 4, 0) == -7 and lib.sop_dd4_lloyd_tuning(129, 0, 4, 0) == -7
    assert lib.sop_dd4_lloyd_tuning(128, -1, 4, 0) == -7 and lib.sop_dd4_lloyd_tuning(128, 0, 4, -1) == -7
    assert lib.sop_dd4_lloyd_tuning(128, 0, 0, 0) == -7 and lib.sop_dd4_lloyd_tuning(128, 0, 5, 0) == -7
    assert lib.sop_dd4_lloyd_tuning(1, 2, 1, 3) == 0
    assert lib.sop_dd4_lloyd_tuning(128, 0, 4, 0) == 0      # the defaults again


def test_sparse_stream_entry_points_reject_bad_arguments(lib):
    ll = C.c_longlong
    m = C.c_double()
    assert lib.sop_pair_search_tuning(2) == -7 and lib.sop_pair_search_tuning(1) == 0
    assert lib.sop_opq_threshold(C.c_double(0.92), 16, C.byref(m)) == 0 and 2.79 < m.value < 2.80
    assert lib.sop_opq_threshold(C.c_double(0.92), 16, None) == -1
    assert lib.sop_opq_threshold(C.c_double(1.0), 16, C.byref(m)) == -7 and lib.sop_opq_threshold(C.c_double(0.5), 0, C.byref(m)) == -7
    n = C.c_size_t()
    assert lib.sop_opq_workspace(ll(4), ll(60), C.byref(n)) == -2 and lib.sop_wr_workspace(ll(0), ll(64), C.byref(n)) == -2
    assert lib.sop_opq_workspace(ll(4), ll(64), C.byref(n)) == 0 and n.value >= 4 * 4 * 2
    OUT = C.c_void_p(0x20000)

    def opq(W=FAKE, out=OUT, K=64, ldo=64, thr=2.8, cap=16, rec=FAKE, ws=FAKE, wsb=1 << 20, cnt=FAKE):
        return lib.sop_opq_extract(W, ll(4), ll(K), ll(K), 16, C.c_double(thr), out, ll(ldo), FAKE, rec, ll(cap), cnt, ws, C.c_size_t(wsb), None)
    assert opq(W=None) == -1 and opq(cnt=None) == -1 and opq(rec=None) == -1
    assert opq(out=FAKE) == -7                       # in place: the stream is read from the untouched input
    assert opq(thr=0.0) == -7 and opq(thr=float("nan")) == -7
    assert opq(ldo=60) == -2 and opq(K=65552) == -2  # the record holds the column in 16 bits
    assert opq(wsb=64) == -5 and opq(ws=None) == -5
    assert opq(cap=-1) == -1

    fmt = C.byref(B.make_fmt(I.scale_format("UE4M4")))
    atoms = I.alphabet(["NF4", "SH4"])
    arr = B.make_atoms(atoms)

    def wr(ia=0, ib=2, k=0, sign=0, b=12, wsb=0, res=None, keep=3, cap=8, rec=FAKE, exp=FAKE, ws=FAKE, wbytes=1 << 20):
        return lib.sop_wr_extract(FAKE, ll(4), ll(64), ll(64), FAKE, 16, fmt, arr, len(atoms), None, C.c_uint(0), ia, ib, k, res, sign, b, wsb,
                                  FAKE, FAKE, ll(keep), FAKE, rec, ll(cap), FAKE, exp, None, ws, C.c_size_t(wbytes), None)
    assert wr(keep=0) == -7 and wr(keep=4 * 64 + 1) == -7
    assert wr(b=8) == -3 and wr(sign=1, wsb=0) == -3
    assert wr(ia=5) == -7 and wr(ia=B.PAIR_FROM_RESULT) == -1 and wr(k=B.K_FROM_RESULT) == -1
    assert wr(exp=None) == -1 and wr(rec=None) == -1
    assert wr(wbytes=16) == -5
