"""Seeded synthetic inputs and codebook alphabets for the SOP candidate sweep.

This module is *data only*.  It produces the tensors a layer sweep consumes (bf16 weights ``W``
[M x K], fp32 calibration activations ``X`` [T x K]) and the alphabets of codebooks ("atoms") that
the sweep evaluates.  None of the method's arithmetic (scaling, encoding, cosine, Lloyd, packing)
lives here, so the CUDA path and the CPU oracle can both be fed from it without sharing any code.

Weights and activations follow the recipes of the five benchmark configurations: heavy-tailed
Student-t / Laplace entries with per-row or per-channel lognormal scales and a few outlier channels.
They stand in for the open-model weights and calibration text the paper measures on, which are not
available offline.

Atoms: the paper names its ROM codebooks (NF4, BOF4, Split87, SH4 and 32-entry versions) but prints
only the SH construction (Section "Primary Formats": sinh(alpha t) + c, alpha = 1.50, c = -0.02).
NF-k is rebuilt from its published Gaussian-quantile description; BOF-k and Split87 are *stand-ins*
fitted by a seeded Lloyd iteration and frozen in ``rom_tables.json`` beside this file.  The sweep
takes the alphabet as an input array, so no result depends on where the numbers came from.
"""
from __future__ import annotations

import dataclasses
import json
import math
import os
import re
from statistics import NormalDist
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

KIND_LUT = 0
KIND_FP_E2M3 = 1
KIND_FP_E4M3 = 2
KIND_FP_GRID = 3      # an element grid given by parameters: (exp_bits, man_bits, bias, largest negative magnitude)

SCOPE_BLOCK = 16
SCOPE_LAYER_POT = 0

_HERE = os.path.dirname(os.path.abspath(__file__))
ROM_TABLE_PATH = os.path.join(_HERE, "rom_tables.json")


# --------------------------------------------------------------------------------------------
# descriptors
# --------------------------------------------------------------------------------------------
@dataclasses.dataclass(frozen=True)
class ScaleFormat:
    """A scale word ``SwExMy`` (Section "Scale Format and Metabit Allocation").

    ``sign_bits`` w, ``exp_bits`` x, ``man_bits`` y; bias 2^(x-1)-1; ``top_exp_reserved`` = 1 makes
    the all-ones exponent code unavailable (IEEE-like, needed for E8M7 = bf16 so that the largest
    scale stays finite in fp32).
    """
    name: str
    sign_bits: int
    exp_bits: int
    man_bits: int
    bias: int
    top_exp_reserved: int = 0

    @property
    def logical_bits(self) -> int:
        return self.sign_bits + self.exp_bits + self.man_bits


def scale_format(name: str) -> ScaleFormat:
    """Parse ``UE4M4`` / ``E5M6`` / ``S1E4M4`` / ``S0E6M5`` into a descriptor."""
    m = re.fullmatch(r"(UE|E|S0E|S1E)(\d+)M(\d+)", name)
    if not m:
        raise ValueError(f"not a scale format name: {name!r}")
    w = 1 if m.group(1) in ("E", "S1E") else 0
    x, y = int(m.group(2)), int(m.group(3))
    if x < 1 or x > 8 or y < 0 or y > 10:
        raise ValueError(f"unsupported scale format {name!r}")
    return ScaleFormat(name, w, x, y, (1 << (x - 1)) - 1, 1 if x == 8 else 0)


# the eight formats of the paper's scale-format table
TABLE_SCALE_FORMATS = ("UE4M4", "E4M3", "UE4M6", "E4M5", "UE5M7", "E5M6", "E4M7", "E8M7")


@dataclasses.dataclass
class Atom:
    """One candidate of the alphabet.

    ``lut`` is ascending and bf16-representable (LUT kinds only).  ``negated`` marks the
    sign-negated variant: the candidate is -(lut).  ``tmax`` is the value the block absmax is
    divided by to form the scale.  ``scope`` is 16 (per-block scale) or 0 (one power-of-two scale
    per layer, the "^0" format suffix).
    """
    name: str
    n_bits: int
    kind: int = KIND_LUT
    negated: int = 0
    scope: int = SCOPE_BLOCK
    tmax: float = 1.0
    lut: Optional[np.ndarray] = None
    grid: Optional[tuple] = None      # KIND_FP_GRID: (exp_bits, man_bits, bias, neg_max); exp_bits 0 = no sign|E|M code

    def negation(self) -> "Atom":
        assert self.kind == KIND_LUT
        return dataclasses.replace(self, name="-" + self.name, negated=1 - self.negated)


def snap_bf16(x) -> np.ndarray:
    """Round fp32/fp64 values to the nearest bf16 (ties to even), returned as fp32."""
    t = torch.as_tensor(np.asarray(x, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy().copy()


def lut_ratio(lut: Sequence[float]) -> float:
    """max |entry| / min non-zero |entry| -- the "ratio" column of the hosting-capacity tables."""
    a = np.abs(np.asarray(lut, dtype=np.float64))
    return float(a.max() / a[a > 0].min())


# --------------------------------------------------------------------------------------------
# ROM atoms
# --------------------------------------------------------------------------------------------
def nf_values(k: int) -> np.ndarray:
    """Gaussian-quantile grid with 2^(k-1)-1 negative entries, zero, and 2^(k-1) positive entries.

    Positive side: 2^(k-1)+1 equally spaced probabilities from ``delta`` down to 1/2 pushed
    through the inverse normal CDF; negative side: 2^(k-1) of them, mirrored; one shared zero;
    divide by the largest value so the endpoints are -1 and +1.
    """
    nd = NormalDist()
    half = 1 << (k - 1)
    delta = 0.5 * ((1.0 - 1.0 / (2.0 * ((1 << k) - 1))) + (1.0 - 1.0 / (1 << (k + 1))))
    pos = [nd.inv_cdf(p) for p in np.linspace(delta, 0.5, half + 1)[:-1]]
    neg = [-nd.inv_cdf(p) for p in np.linspace(delta, 0.5, half)[:-1]]
    v = np.array(sorted(neg + [0.0] + pos), dtype=np.float64)
    return v / np.abs(v).max()


def sh_values(k: int, alpha: float = 1.50, c: float = -0.02) -> np.ndarray:
    """sinh(alpha t) + c for 2^k uniformly spaced t in [-1, 1], divided by the largest magnitude."""
    t = np.linspace(-1.0, 1.0, 1 << k)
    v = np.sinh(alpha * t) + c
    return v / np.abs(v).max()


def e2m2_rom_values() -> np.ndarray:
    """The 32 codes of an FP5 E2M2 grid (bias 1, subnormals, every code finite), ascending.

    -0 and +0 are both stored as 0, so the table has 31 distinct values and one duplicate.
    """
    vals = []
    for s in (1.0, -1.0):
        for e in range(4):
            for m in range(4):
                mag = (m / 4.0) if e == 0 else (1.0 + m / 4.0) * 2.0 ** (e - 1)
                vals.append(s * mag)
    return np.array(sorted(vals), dtype=np.float64)


def fit_block_lloyd_levels(n_levels: int, n_neg: int, pin_zero: bool, dist: str, seed: int,
                           n_blocks: int = 1 << 16, iters: int = 60) -> np.ndarray:
    """Seeded 1-D Lloyd fit used for the BOF-k / Split87 stand-ins.

    Samples blocks of 16 iid values (standard normal or Student-t with 5 degrees of freedom),
    divides each block by its largest magnitude, and fits ``n_levels`` levels with -1 and +1
    pinned (and 0 pinned when ``pin_zero``); ``n_neg`` of the free levels start below zero.
    """
    rng = np.random.Generator(np.random.Philox(seed))
    z = rng.standard_normal((n_blocks, 16)) if dist == "normal" else rng.standard_t(5.0, (n_blocks, 16))
    y = np.sort((z / np.abs(z).max(axis=1, keepdims=True)).ravel())
    n_pos = n_levels - n_neg - (1 if pin_zero else 0)
    neg = -np.linspace(1.0, 0.0, n_neg + 1)[:-1] ** 1.5 if n_neg else np.zeros(0)
    pos = np.linspace(0.0, 1.0, n_pos + 1)[1:] ** 1.5
    lv = np.concatenate([neg, [0.0] if pin_zero else [], pos])
    pinned = np.isin(np.arange(n_levels), [0, n_levels - 1] + ([n_neg] if pin_zero else []))
    csum = np.concatenate([[0.0], np.cumsum(y)])
    for _ in range(iters):
        edges = np.searchsorted(y, 0.5 * (lv[1:] + lv[:-1]))
        lo = np.concatenate([[0], edges])
        hi = np.concatenate([edges, [y.size]])
        cnt = hi - lo
        mean = (csum[hi] - csum[lo]) / np.maximum(cnt, 1)
        lv = np.where(pinned | (cnt == 0), lv, mean)
    return lv


def _rom_tables() -> dict:
    with open(ROM_TABLE_PATH) as f:
        return json.load(f)


def build_rom_tables() -> dict:
    """Recompute every frozen stand-in table (see ``make_rom_tables.py``)."""
    return {
        "BOF4": fit_block_lloyd_levels(16, 7, True, "normal", 41).tolist(),
        "BOF5": fit_block_lloyd_levels(32, 15, True, "normal", 42).tolist(),
        "Split87": fit_block_lloyd_levels(16, 7, True, "student5", 43).tolist(),
    }


def rom_atom(name: str) -> Atom:
    """A fixed-ROM atom by name: NF4 NF5 SH4 SH5 BOF4 BOF5 Split87 E2M2."""
    if name in ("NF4", "NF5"):
        v, n = nf_values(int(name[2])), int(name[2])
    elif name in ("SH4", "SH5"):
        v, n = sh_values(int(name[2])), int(name[2])
    elif name in ("BOF4", "BOF5", "Split87"):
        v = np.array(_rom_tables()[name], dtype=np.float64)
        n = 5 if name.endswith("5") else 4
    elif name == "E2M2":
        v, n = e2m2_rom_values(), 5
    else:
        raise KeyError(name)
    lut = np.sort(snap_bf16(v))
    return Atom(name=name, n_bits=n, kind=KIND_LUT, tmax=float(np.abs(lut).max()), lut=lut)


def fp_atom(name: str) -> Atom:
    """FP element formats evaluated as single candidates: E2M3, E4M3, and E4M3^0 (layer POT scale)."""
    if name == "E2M3":
        return Atom(name, 6, KIND_FP_E2M3, 0, SCOPE_BLOCK, 7.5)
    if name == "E4M3":
        return Atom(name, 8, KIND_FP_E4M3, 0, SCOPE_BLOCK, 448.0)
    if name == "E4M3^0":
        return Atom(name, 8, KIND_FP_E4M3, 0, SCOPE_LAYER_POT, 448.0)
    if name in GRID_FORMATS or (name.endswith("^0") and name[:-2] in GRID_FORMATS):
        return grid_atom(name)
    raise KeyError(name)


def ieee_like_grid(x: int, y: int) -> tuple:
    """(bias, largest value) of an ExMy element grid with bias 2^(x-1)-1 (at least 1) and the all-ones
    exponent code left out: the convention under which the paper's E2M5 tops out at 3.94."""
    bias = max(1, (1 << (x - 1)) - 1)
    top = (1 << x) - 2
    return bias, float((2.0 - 2.0 ** -y) * 2.0 ** (top - bias))


# promotion-profile element grids beyond E2M3 / E4M3: name -> (n_bits, exp_bits, man_bits, bias, tmax, neg_max).
# HIF7 / HIF8 are 5-bit two's-complement coefficients times 2^s (s up to 3 / 4): magnitudes 0..15 and then
# 8..15 times 2^s, with -16 * 2^s reaching one step further on the negative side.
def _grid_table():
    t = {}
    for nm, x, y in (("E3M4", 3, 4), ("E2M5", 2, 5), ("E5M2", 5, 2), ("E3M6", 3, 6), ("E4M5", 4, 5), ("E3M8", 3, 8),
                     ("E4M7", 4, 7), ("E5M6e", 5, 6)):
        bias, top = ieee_like_grid(x, y)
        t[nm] = (1 + x + y, x, y, bias, top, top)
    t["HIF7"] = (7, 0, 3, -2, 120.0, 128.0)
    t["HIF8"] = (8, 0, 3, -2, 240.0, 256.0)
    return t


GRID_FORMATS = _grid_table()


def grid_atom(name: str) -> Atom:
    scope = SCOPE_BLOCK
    base = name
    if name.endswith("^0"):
        scope, base = SCOPE_LAYER_POT, name[:-2]
    n, x, y, bias, tmax, neg_max = GRID_FORMATS[base]
    return Atom(name, n, KIND_FP_GRID, 0, scope, tmax, None, (x, y, bias, neg_max))


def alphabet(names: Sequence[str], with_negations: bool = True, fp: Sequence[str] = ()) -> List[Atom]:
    """ROM atoms in the given order, each followed by its negation, then the FP singles."""
    out: List[Atom] = []
    for nm in names:
        a = rom_atom(nm)
        out.append(a)
        if with_negations:
            out.append(a.negation())
    out.extend(fp_atom(f) for f in fp)
    return out


# --------------------------------------------------------------------------------------------
# layers
# --------------------------------------------------------------------------------------------
@dataclasses.dataclass
class Layer:
    W: torch.Tensor  # [M, K] bf16
    X: torch.Tensor  # [T, K] fp32
    name: str = ""


def _gen(seed: int, *stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=seed, counter=[*stream, 0, 0, 0, 0][:4]))


def _to_bf16(w: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(w, dtype=np.float32)).to(torch.bfloat16)


def activations(seed: int, layer_id: int, T: int, K: int, sigma: float = 1.0,
                outlier_cols: Optional[np.ndarray] = None, outlier_gain: float = 20.0) -> torch.Tensor:
    """X[t, k] = z[t, k] * exp(sigma * z'[k]): per-channel lognormal scales on iid normal tokens."""
    g = _gen(seed, layer_id, 2)
    ch = np.exp(sigma * g.standard_normal(K)).astype(np.float32)
    if outlier_cols is not None:
        ch[outlier_cols] *= outlier_gain
    x = g.standard_normal((T, K), dtype=np.float32) * ch[None, :]
    return torch.from_numpy(x)


def config1(seed: int = 0) -> Layer:
    """256 x 1024, Student-t(5) * 0.02 with lognormal(0, 0.3) row scales; X 128 x 1024."""
    M, K, T = 256, 1024, 128
    g = _gen(seed, 0, 1)
    w = 0.02 * g.standard_t(5.0, (M, K)) * np.exp(0.3 * g.standard_normal((M, 1)))
    return Layer(_to_bf16(w), activations(seed, 0, T, K), "config1")


def outlier_channel_layer(seed: int, M: int, K: int, T: int, nu: float = 4.0, sd: float = 0.015,
                          frac: float = 0.01, gain: float = 20.0, layer_id: int = 0) -> Layer:
    """Student-t(nu) * sd weights with a fixed ``frac`` of input channels scaled by ``gain``."""
    g = _gen(seed, layer_id, 1)
    cols = np.sort(g.choice(K, size=max(1, int(round(frac * K))), replace=False))
    w = (sd * g.standard_t(nu, (M, K))).astype(np.float32)
    w[:, cols] *= gain
    return Layer(_to_bf16(w), activations(seed, layer_id, T, K, 1.0, cols, gain), f"outlier_{M}x{K}")


def config2(seed: int = 0, M: int = 4096, K: int = 4096, T: int = 512) -> Layer:
    """Attention projection 4096 x 4096 with 1 % outlier channels (x20); X 512 x 4096."""
    return outlier_channel_layer(seed, M, K, T)


def student_layer(seed: int, layer_id: int, M: int, K: int, T: int, nu: float, sd: float = 0.02,
                  channel_sigma: float = 0.0, device: str = "cpu") -> Layer:
    """Student-t(nu) * sd weights, optional lognormal(0, channel_sigma) input-channel scales.

    ``device`` may name a CUDA device: large layers (7B / 70B shapes) are generated there with
    torch's seeded generator, one layer at a time, and only sampled rows travel to the host.
    """
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + layer_id) & 0x7FFFFFFFFFFF)
    z = torch.randn((M, K), generator=g, device=device, dtype=torch.float32)
    chi = torch.zeros((M, K), device=device, dtype=torch.float32)
    n_int = int(math.floor(nu))
    for _ in range(n_int):
        chi += torch.randn((M, K), generator=g, device=device, dtype=torch.float32) ** 2
    frac = nu - n_int
    if frac > 0:
        chi += frac * torch.randn((M, K), generator=g, device=device, dtype=torch.float32) ** 2
    w = sd * z / torch.sqrt(chi / nu)
    del z, chi
    ch = torch.exp(channel_sigma * torch.randn((K,), generator=g, device=device, dtype=torch.float32))
    if channel_sigma > 0:
        w = w * ch[None, :]
    x = torch.randn((T, K), generator=g, device=device, dtype=torch.float32)
    x = x * torch.exp(torch.randn((K,), generator=g, device=device, dtype=torch.float32))[None, :]
    if channel_sigma > 0:
        x = x * ch[None, :]
    return Layer(w.to(torch.bfloat16), x, f"student_{M}x{K}_nu{nu:g}")


def laplace_outlier_layer(seed: int, layer_id: int, M: int, K: int, T: int, b: float = 0.01,
                          frac: float = 0.001, k_sigma: float = 8.0, device: str = "cpu") -> Layer:
    """Laplace(0, b) weights with ``frac`` of the entries replaced by +-k_sigma standard deviations."""
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + layer_id) & 0x7FFFFFFFFFFF)
    u = torch.rand((M, K), generator=g, device=device, dtype=torch.float32) - 0.5
    w = -b * torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp(max=0.4999999))
    sel = torch.rand((M, K), generator=g, device=device) < frac
    sgn = torch.where(torch.rand((M, K), generator=g, device=device) < 0.5, -1.0, 1.0)
    w = torch.where(sel, sgn * (k_sigma * b * math.sqrt(2.0)), w)
    x = torch.randn((T, K), generator=g, device=device, dtype=torch.float32)
    x = x * torch.exp(torch.randn((K,), generator=g, device=device, dtype=torch.float32))[None, :]
    return Layer(w.to(torch.bfloat16), x, f"laplace_{M}x{K}")


# shapes of one transformer block of the 7B-shaped and 70B-shaped sweeps: (name, M, K)
SHAPES_7B = (("q", 4096, 4096), ("k", 1024, 4096), ("v", 1024, 4096), ("o", 4096, 4096),
             ("gate", 14336, 4096), ("up", 14336, 4096), ("down", 4096, 14336))
SHAPES_70B = (("qo", 8192, 8192), ("k", 1024, 8192), ("v", 1024, 8192),
              ("gate_up", 28672, 8192), ("down", 8192, 28672))


def config3_layer(seed: int, block: int, which: int, rows: Optional[int] = None, device: str = "cpu") -> Layer:
    """Layer ``which`` of transformer block ``block`` of the 7B-shaped sweep (nu ~ U[3, 8] per layer)."""
    _, M, K = SHAPES_7B[which]
    lid = block * len(SHAPES_7B) + which
    nu = 3.0 + 5.0 * float(_gen(seed, lid, 7).random())
    return student_layer(seed, lid, rows or M, K, 512, nu, 0.02, 0.0, device)


def config5_layer(seed: int, block: int, which: int, rows: Optional[int] = None, device: str = "cpu") -> Layer:
    """Layer of the 70B-shaped set: Student-t(5) with lognormal(0, 1.2) channel scales, X 1024 x K."""
    _, M, K = SHAPES_70B[which]
    lid = block * len(SHAPES_70B) + which
    return student_layer(seed, lid, rows or M, K, 1024, 5.0, 0.02, 1.2, device)


def config4_layer(seed: int, which: int, rows: Optional[int] = None, device: str = "cpu") -> Layer:
    """MLP pair of the n = 5 extension: 14336 x 4096 (which = 0) or 4096 x 14336 (which = 1), X 2048 tokens."""
    M, K = ((14336, 4096), (4096, 14336))[which]
    return laplace_outlier_layer(seed, which, rows or M, K, 2048, device=device)


def tiny_layer(seed: int, M: int, K: int, T: int = 8) -> Layer:
    """Small bell-shaped layer for brute-force tests."""
    g = _gen(seed, 99, 1)
    w = 0.02 * g.standard_t(5.0, (M, K))
    return Layer(_to_bf16(w), activations(seed, 99, T, K), f"tiny_{M}x{K}")
