"""ctypes binding of ``libsop.so``: the same entry points as ``include/sop.h``, with torch tensors
supplying device memory and streams.  Argument marshalling only -- every step of the sweep runs in
the library's CUDA kernels.  There is no CPU fallback: a missing library is an error.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

from . import build as _build

K_AUTO = -1000
K_FROM_RESULT = -1001
FMTA_FROM_RESULT = -1
PAIR_FROM_RESULT = -1
NO_ATOM = -2
MAX_ATOMS = 16
ALL_ATOMS = 0xFFFFFFFF
SEARCH_SINGLES_ONLY = 1
SEARCH_SELECT_MSE = 2
SEARCH_KEEP_LOADED_ENTRIES = 4
SEARCH_REUSE_PREPASS = 8
LLOYD_POOL_BY_ERROR, LLOYD_UNIFORM_WEIGHTS, LLOYD_POOL_THRESHOLD, LLOYD_LAUNCH_PER_ITERATION, LLOYD_GRID_DP = 1, 2, 4, 8, 16
PACK_SELECT_MSE = 1
MAX_ENTRIES = 32


class SopError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().sop_strerror(code).decode()
        if code == -6:
            msg += ": " + lib().sop_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({code})")


class ScaleFmt(C.Structure):
    _fields_ = [("sign_bits", C.c_int), ("exp_bits", C.c_int), ("man_bits", C.c_int), ("bias", C.c_int),
                ("top_exp_reserved", C.c_int)]


class AtomStruct(C.Structure):
    _fields_ = [("n_bits", C.c_int), ("kind", C.c_int), ("negated", C.c_int), ("scope", C.c_int),
                ("tmax", C.c_float), ("n_entries", C.c_int), ("lut", C.c_float * MAX_ENTRIES),
                ("grid_exp_bits", C.c_int), ("grid_man_bits", C.c_int), ("grid_bias", C.c_int), ("grid_neg_max", C.c_float)]


class PairStat(C.Structure):
    _fields_ = [("acos", C.c_double), ("mse", C.c_double), ("n_sel1", C.c_longlong), ("n_neg", C.c_longlong)]


class SearchResult(C.Structure):
    _fields_ = [("k", C.c_int * MAX_ATOMS), ("best_a", C.c_int), ("best_b", C.c_int), ("best_single", C.c_int),
                ("best_sa", C.c_int), ("best_sb", C.c_int), ("layer_absmax", C.c_float), ("reserved", C.c_int * 2)]


PAIR_DTYPE = np.dtype([("acos", "f8"), ("mse", "f8"), ("n_sel1", "i8"), ("n_neg", "i8")])
RESULT_BYTES = C.sizeof(SearchResult)

_lib = None


def lib_path() -> str:
    return _build.LIB


def lib():
    """The loaded C-ABI library.  Built in-tree by ``build.py``; never silently replaced."""
    global _lib
    if _lib is None:
        if not os.path.exists(_build.LIB):
            raise ImportError(f"{_build.LIB} is missing: run `python -m paper_2605_14929_b200.build` "
                              "(nvcc, sm_100a).  There is no CPU fallback.")
        _lib = C.CDLL(_build.LIB)
        _lib.sop_strerror.restype = C.c_char_p
        _lib.sop_last_cuda_error.restype = C.c_char_p
    return _lib


def exported_symbols():
    return ["sop_strerror", "sop_last_cuda_error", "sop_version", "sop_channel_norms_workspace", "sop_channel_norms",
            "sop_channel_norms_static",
            "sop_pair_search_workspace", "sop_pair_search_tuning", "sop_pair_search", "sop_dd4_lloyd_workspace", "sop_dd4_lloyd_launches", "sop_dd4_lloyd_tuning",
            "sop_dd4_lloyd", "sop_pack", "sop_opq_threshold", "sop_opq_workspace", "sop_opq_extract", "sop_wr_workspace",
            "sop_wr_extract",
            "sop_profile_enable", "sop_profile_ms", "sop_profile_last_ms", "sop_profile_last_sweep_ms"]


def _check(rc: int, where: str):
    if rc != 0:
        raise SopError(rc, where)


def make_fmt(f) -> ScaleFmt:
    """A ``ScaleFmt`` struct from a descriptor (a struct is passed through: marshal once, call often)."""
    if isinstance(f, ScaleFmt):
        return f
    return ScaleFmt(f.sign_bits, f.exp_bits, f.man_bits, f.bias, f.top_exp_reserved)


def make_atoms(atoms) -> C.Array:
    """An array of ``AtomStruct`` from a list of descriptors (an array is passed through)."""
    if isinstance(atoms, C.Array):
        return atoms
    arr = (AtomStruct * max(1, len(atoms)))()
    for i, a in enumerate(atoms):
        s = arr[i]
        s.n_bits, s.kind, s.negated, s.scope, s.tmax = a.n_bits, a.kind, a.negated, a.scope, a.tmax
        s.n_entries = 0 if a.lut is None else len(a.lut)
        if a.lut is not None:
            for j, v in enumerate(a.lut):
                s.lut[j] = float(v)
        g = getattr(a, "grid", None)
        if g is not None:
            s.grid_exp_bits, s.grid_man_bits, s.grid_bias, s.grid_neg_max = g
    return arr


def _ptr(t: Optional[torch.Tensor]):
    return C.c_void_p(0 if t is None else t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _ll(v) -> C.c_longlong:
    return C.c_longlong(int(v))


# ------------------------------------------------------------------ workspace queries
def channel_norms_workspace(T: int, K: int) -> int:
    n = C.c_size_t()
    _check(lib().sop_channel_norms_workspace(_ll(T), _ll(K), C.byref(n)), "sop_channel_norms_workspace")
    return n.value


def pair_search_workspace(M: int, K: int, n_atoms: int) -> int:
    n = C.c_size_t()
    _check(lib().sop_pair_search_workspace(_ll(M), _ll(K), n_atoms, C.byref(n)), "sop_pair_search_workspace")
    return n.value


def dd4_lloyd_workspace(M: int, K: int) -> int:
    n = C.c_size_t()
    _check(lib().sop_dd4_lloyd_workspace(_ll(M), _ll(K), C.byref(n)), "sop_dd4_lloyd_workspace")
    return n.value


def dd4_lloyd_launches(M: int, K: int, iters: int, flags: int = 0) -> int:
    """Kernel launches of one ``sop_dd4_lloyd`` call on the current device."""
    n = C.c_int()
    _check(lib().sop_dd4_lloyd_launches(_ll(M), _ll(K), iters, flags, C.byref(n)), "sop_dd4_lloyd_launches")
    return n.value


def dd4_lloyd_tuning(cell_spill_tiles: int = 128, cache_ctas: int = 0, tiles_per_warp: int = 4, iter_ctas: int = 0) -> None:
    """Launch-shape parameters of ``sop_dd4_lloyd`` (test aid; the defaults restore the library's own)."""
    _check(lib().sop_dd4_lloyd_tuning(cell_spill_tiles, cache_ctas, tiles_per_warp, iter_ctas), "sop_dd4_lloyd_tuning")


class LloydNotFinished(RuntimeError):
    """``sop_dd4_lloyd`` left its status entry negative: a bounded wait between iterations gave up (or the call
    never ran to its end), so the codebook it wrote must not be used."""


def check_lloyd_status(distortion: torch.Tensor, iters: int) -> None:
    """Reads the status entry ``distortion[iters]`` of a finished (synchronised) ``sop_dd4_lloyd`` call and
    raises ``LloydNotFinished`` when it is negative."""
    if float(distortion[iters].item()) < 0.0:
        raise LloydNotFinished(f"sop_dd4_lloyd did not finish: distortion[{iters}] = {float(distortion[iters].item())}")


def alloc_workspace(nbytes: int, device) -> torch.Tensor:
    """A 256-byte aligned device buffer (torch's caching allocator aligns to 512 bytes)."""
    return torch.empty(max(256, nbytes), dtype=torch.uint8, device=device)


# ------------------------------------------------------------------ entry points
def sop_channel_norms(X: torch.Tensor, c_out: torch.Tensor, workspace: torch.Tensor, stream=None) -> None:
    assert X.is_cuda and X.dtype == torch.float32 and X.dim() == 2 and X.stride(1) == 1
    assert c_out.is_cuda and c_out.dtype == torch.float32 and c_out.is_contiguous()
    T, K = X.shape
    _check(lib().sop_channel_norms(_ptr(X), _ll(T), _ll(K), _ll(X.stride(0)), _ptr(c_out), _ptr(workspace),
                                   C.c_size_t(workspace.numel()), _stream(stream)), "sop_channel_norms")


NORMS_STATIC_DOUBLES = 1 << 19


def sop_channel_norms_static(X: torch.Tensor, c_out: torch.Tensor, stream=None) -> None:
    """Channel norms with the library's built-in scratch instead of a caller workspace: for callers
    that must not allocate device memory.  Needs ceil(T / 64) * K <= NORMS_STATIC_DOUBLES; calls on
    one device share the scratch and must not overlap on the GPU."""
    assert X.is_cuda and X.dtype == torch.float32 and X.dim() == 2 and X.stride(1) == 1
    assert c_out.is_cuda and c_out.dtype == torch.float32 and c_out.is_contiguous()
    T, K = X.shape
    _check(lib().sop_channel_norms_static(_ptr(X), _ll(T), _ll(K), _ll(X.stride(0)), _ptr(c_out), _stream(stream)),
           "sop_channel_norms_static")


def sop_pair_search(W: torch.Tensor, c: torch.Tensor, fmt, atoms: Sequence, pair_table: torch.Tensor,
                    signed_table: Optional[torch.Tensor], result: torch.Tensor, workspace: torch.Tensor,
                    k_mode: int = K_AUTO, dd_lut: Optional[torch.Tensor] = None, dd_mask: int = 0,
                    block_cos: Optional[torch.Tensor] = None, block_sse: Optional[torch.Tensor] = None,
                    stream=None, g: int = 16, eval_mask: int = ALL_ATOMS, load_mask: int = 0,
                    singles_only: bool = False, prev_result: Optional[torch.Tensor] = None,
                    select_mse: bool = False, keep_loaded: bool = False, reuse_prepass: bool = False) -> None:
    """``keep_loaded``: the table entries among the candidates of ``load_mask`` stay as an earlier call wrote them
    into ``pair_table`` / ``signed_table``; only the entries with a newly evaluated candidate are formed."""
    assert W.is_cuda and W.dtype == torch.bfloat16 and W.dim() == 2 and W.stride(1) == 1
    M, K = W.shape
    _check(lib().sop_pair_search(_ptr(W), _ll(M), _ll(K), _ll(W.stride(0)), _ptr(c), g, C.byref(make_fmt(fmt)), k_mode,
                                 make_atoms(atoms), len(atoms), _ptr(dd_lut), C.c_uint(dd_mask), C.c_uint(eval_mask),
                                 C.c_uint(load_mask),
                                 (SEARCH_SINGLES_ONLY if singles_only else 0) | (SEARCH_SELECT_MSE if select_mse else 0)
                                 | (SEARCH_KEEP_LOADED_ENTRIES if keep_loaded else 0) | (SEARCH_REUSE_PREPASS if reuse_prepass else 0),
                                 _ptr(prev_result),
                                 _ptr(pair_table),
                                 _ptr(signed_table), _ptr(result), _ptr(block_cos), _ptr(block_sse), _ptr(workspace),
                                 C.c_size_t(workspace.numel()), _stream(stream)), "sop_pair_search")


def sop_dd4_lloyd(W: torch.Tensor, c: torch.Tensor, fmt, atoms: Sequence, block_cos: torch.Tensor, pool_rank: int,
                  iters: int, out_lut: torch.Tensor, distortion: torch.Tensor, pool_count: torch.Tensor,
                  workspace: torch.Tensor, k_mode: int = K_FROM_RESULT, search_result: Optional[torch.Tensor] = None,
                  fmta_index: int = FMTA_FROM_RESULT, stream=None, g: int = 16, pool_by_error: bool = False,
                  uniform_weights: bool = False, pool_threshold: Optional[float] = None,
                  launch_per_iteration: bool = False, grid_dp: bool = False) -> None:
    """``block_cos`` is the per-block metric that ranks the blocks: cosines, or errors with ``pool_by_error``.
    A ``pool_threshold`` replaces the rank.  ``grid_dp`` (with ``iters`` = 0) takes the grid-constrained construction
    by dynamic programming instead of Lloyd iterations; ``distortion[0]`` is then its least total cost."""
    assert W.is_cuda and W.dtype == torch.bfloat16 and W.dim() == 2 and W.stride(1) == 1
    M, K = W.shape
    _check(lib().sop_dd4_lloyd(_ptr(W), _ll(M), _ll(K), _ll(W.stride(0)), _ptr(c), g, C.byref(make_fmt(fmt)), k_mode,
                               _ptr(search_result), _ptr(block_cos), _ll(pool_rank),
                               C.c_float(0.0 if pool_threshold is None else pool_threshold),
                               (LLOYD_POOL_BY_ERROR if pool_by_error else 0) | (LLOYD_UNIFORM_WEIGHTS if uniform_weights else 0)
                               | (LLOYD_POOL_THRESHOLD if pool_threshold is not None else 0)
                               | (LLOYD_LAUNCH_PER_ITERATION if launch_per_iteration else 0) | (LLOYD_GRID_DP if grid_dp else 0),
                               make_atoms(atoms), len(atoms),
                               fmta_index, iters, _ptr(out_lut), _ptr(distortion), _ptr(pool_count), _ptr(workspace),
                               C.c_size_t(workspace.numel()), _stream(stream)), "sop_dd4_lloyd")


def sop_pack(W: torch.Tensor, c: torch.Tensor, fmt, atoms: Sequence, codes: torch.Tensor, words: torch.Tensor,
             index_a: int = PAIR_FROM_RESULT, index_b: int = PAIR_FROM_RESULT, k_mode: int = K_FROM_RESULT,
             search_result: Optional[torch.Tensor] = None, use_sign: int = 0, container_bits: int = 8,
             word_sign_bits: int = 0, counts: Optional[torch.Tensor] = None, dd_lut: Optional[torch.Tensor] = None,
             dd_mask: int = 0, stream=None, g: int = 16, block_cos: Optional[torch.Tensor] = None,
             select_mse: bool = False) -> None:
    """``block_cos``: per-block cosines of a sweep, or with ``select_mse`` its per-block errors."""
    assert W.is_cuda and W.dtype == torch.bfloat16 and W.dim() == 2 and W.stride(1) == 1
    M, K = W.shape
    _check(lib().sop_pack(_ptr(W), _ll(M), _ll(K), _ll(W.stride(0)), _ptr(c), g, C.byref(make_fmt(fmt)),
                          make_atoms(atoms), len(atoms), _ptr(dd_lut), C.c_uint(dd_mask), index_a, index_b, k_mode,
                          _ptr(search_result), use_sign, container_bits, word_sign_bits, _ptr(codes), _ptr(words),
                          _ptr(counts), _ptr(block_cos), PACK_SELECT_MSE if select_mse else 0, _stream(stream)), "sop_pack")


def opq_threshold(q: float = 0.92, max_order: int = 16) -> float:
    """The m with (2 Phi(m) - 1)^max_order = q."""
    m = C.c_double()
    _check(lib().sop_opq_threshold(C.c_double(q), int(max_order), C.byref(m)), "sop_opq_threshold")
    return m.value


def opq_workspace(M: int, K: int, device) -> torch.Tensor:
    n = C.c_size_t()
    _check(lib().sop_opq_workspace(_ll(M), _ll(K), C.byref(n)), "sop_opq_workspace")
    return torch.empty(n.value, dtype=torch.uint8, device=device)


def sop_opq_extract(W: torch.Tensor, m: float, W_out: torch.Tensor, row_start: torch.Tensor, records: Optional[torch.Tensor],
                    count: torch.Tensor, workspace: torch.Tensor, stream=None, g: int = 16) -> None:
    """``row_start``: M + 1 int32/uint32 words, ``records``: the capacity in 32-bit words (None: count only),
    ``count``: one int64."""
    assert W.is_cuda and W.dtype == torch.bfloat16 and W.dim() == 2 and W.stride(1) == 1 and W_out.stride(1) == 1
    M, K = W.shape
    _check(lib().sop_opq_extract(_ptr(W), _ll(M), _ll(K), _ll(W.stride(0)), g, C.c_double(m), _ptr(W_out), _ll(W_out.stride(0)),
                                 _ptr(row_start), _ptr(records), _ll(0 if records is None else records.numel()), _ptr(count),
                                 _ptr(workspace), C.c_size_t(workspace.numel()), _stream(stream)), "sop_opq_extract")


def wr_workspace(M: int, K: int, device) -> torch.Tensor:
    n = C.c_size_t()
    _check(lib().sop_wr_workspace(_ll(M), _ll(K), C.byref(n)), "sop_wr_workspace")
    return torch.empty(n.value, dtype=torch.uint8, device=device)


def sop_wr_extract(W: torch.Tensor, c: torch.Tensor, fmt, atoms: Sequence, codes: torch.Tensor, words: torch.Tensor, n_keep: int,
                   row_start: torch.Tensor, records: Optional[torch.Tensor], count: torch.Tensor, scale_exp: torch.Tensor,
                   workspace: torch.Tensor, tau: Optional[torch.Tensor] = None,
                   index_a: int = PAIR_FROM_RESULT, index_b: int = PAIR_FROM_RESULT, k_mode: int = K_FROM_RESULT,
                   search_result: Optional[torch.Tensor] = None, use_sign: int = 0, container_bits: int = 8,
                   word_sign_bits: int = 0, dd_lut: Optional[torch.Tensor] = None, dd_mask: int = 0, stream=None, g: int = 16) -> None:
    """The arguments from ``fmt`` to ``word_sign_bits`` are those given to ``sop_pack`` for this layer."""
    assert W.is_cuda and W.dtype == torch.bfloat16 and W.dim() == 2 and W.stride(1) == 1
    M, K = W.shape
    _check(lib().sop_wr_extract(_ptr(W), _ll(M), _ll(K), _ll(W.stride(0)), _ptr(c), g, C.byref(make_fmt(fmt)), make_atoms(atoms),
                                len(atoms), _ptr(dd_lut), C.c_uint(dd_mask), index_a, index_b, k_mode, _ptr(search_result), use_sign,
                                container_bits, word_sign_bits, _ptr(codes), _ptr(words), _ll(n_keep), _ptr(row_start),
                                _ptr(records), _ll(0 if records is None else records.numel()), _ptr(count), _ptr(scale_exp),
                                _ptr(tau), _ptr(workspace), C.c_size_t(workspace.numel()), _stream(stream)), "sop_wr_extract")


def pair_search_tuning(reduce_tile_pairs: bool = True) -> None:
    """Launch shape of the reduction kernel (results do not depend on it)."""
    _check(lib().sop_pair_search_tuning(1 if reduce_tile_pairs else 0), "sop_pair_search_tuning")


def profile_enable(on: bool) -> None:
    _check(lib().sop_profile_enable(1 if on else 0), "sop_profile_enable")


PROFILE_SWEEP, PROFILE_LLOYD, PROFILE_PACK, PROFILE_NORMS, PROFILE_REDUCE, PROFILE_POOL, PROFILE_PREPASS = 0, 1, 2, 3, 4, 5, 6
PROFILE_OPQ, PROFILE_WR = 7, 8


def profile_ms(which: int, back: int = 0) -> float:
    """Milliseconds of the main kernel(s) of the ``back``-th last call of that kind (waits for it)."""
    ms = C.c_float()
    _check(lib().sop_profile_ms(which, back, C.byref(ms)), "sop_profile_ms")
    return ms.value


def profile_last_ms(which: int) -> float:
    return profile_ms(which, 0)


def profile_last_sweep_ms() -> float:
    return profile_last_ms(PROFILE_SWEEP)


# ------------------------------------------------------------------ result readers (device -> host)
def read_pair_table(t: torch.Tensor, n_atoms: int) -> np.ndarray:
    return t.cpu().numpy().view(PAIR_DTYPE).reshape(n_atoms, n_atoms)


def read_result(t: torch.Tensor) -> dict:
    raw = t.cpu().numpy().tobytes()
    r = SearchResult.from_buffer_copy(raw)
    return dict(k=np.array(r.k[:], dtype=np.int32), best=np.array([r.best_a, r.best_b, r.best_single, r.best_sa, r.best_sb],
                                                               dtype=np.int32), layer_absmax=r.layer_absmax)


def new_pair_table(n_atoms: int, device) -> torch.Tensor:
    return torch.zeros(n_atoms * n_atoms * PAIR_DTYPE.itemsize, dtype=torch.uint8, device=device)


def new_result(device) -> torch.Tensor:
    return torch.zeros(RESULT_BYTES, dtype=torch.uint8, device=device)


def words_nbytes(n_blocks: int, container_bits: int) -> int:
    """Bytes to allocate for the scale-word stream (whole 32-bit words)."""
    return ((n_blocks * container_bits + 7) // 8 + 3) // 4 * 4
