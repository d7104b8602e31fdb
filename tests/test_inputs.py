"""The shared input module: atom alphabets against the facts the paper prints, and seeded layers."""
import os

import numpy as np
import torch

from paper_2605_14929_b200 import inputs as I

GOLD = {}
with open(os.path.join(os.path.dirname(__file__), "golden", "hosting_ratios.txt")) as f:
    for line in f:
        line = line.split("#")[0].split()
        if line:
            GOLD[line[0]] = (float(line[1]), float(line[2]))


def test_nf4_shape_and_ratio():
    # Section "Block Scaling": equal endpoints, seven negative entries against eight positive
    v = I.nf_values(4)
    assert (v < 0).sum() == 7 and (v > 0).sum() == 8 and (v == 0).sum() == 1
    assert v[0] == -1.0 and v[-1] == 1.0
    want, tol = GOLD["NF4_ratio"]
    assert abs(I.lut_ratio(v) - want) <= tol


def test_sh_ratios():
    for k, key in ((4, "SH4_ratio"), (5, "SH5_ratio")):
        want, tol = GOLD[key]
        assert abs(I.lut_ratio(I.sh_values(k)) - want) <= tol
    v = I.sh_values(4)
    assert 0.0 not in list(v) and abs(v).max() == 1.0


def test_rom_atoms_are_sorted_bf16_tables():
    for name in ("NF4", "SH4", "BOF4", "Split87", "NF5", "SH5", "BOF5", "E2M2"):
        a = I.rom_atom(name)
        assert len(a.lut) == 1 << a.n_bits and np.all(np.diff(a.lut) >= 0)
        assert np.array_equal(I.snap_bf16(a.lut), a.lut)
        assert a.tmax == float(np.abs(a.lut).max())
    assert len(set(I.rom_atom("E2M2").lut.tolist())) == 31     # -0 and +0 collapse


def test_frozen_tables_match_their_recipe():
    rebuilt = I.build_rom_tables()
    for k, v in I._rom_tables().items():
        assert np.allclose(rebuilt[k], v, rtol=0, atol=1e-12)


def test_layers_are_seeded_and_shaped():
    a, b = I.config1(0), I.config1(0)
    assert torch.equal(a.W, b.W) and torch.equal(a.X, b.X)
    assert a.W.shape == (256, 1024) and a.W.dtype == torch.bfloat16 and a.X.shape == (128, 1024)
    assert not torch.equal(a.W, I.config1(1).W)
    L = I.outlier_channel_layer(0, 64, 512, 32)
    col_rms = L.W.float().pow(2).mean(0).sqrt()
    assert int((col_rms > 5 * col_rms.median()).sum()) == 5     # 1 % of 512 channels scaled x20
    L4 = I.config4_layer(0, 0, rows=32)
    assert L4.W.shape == (32, 4096) and L4.X.shape == (2048, 4096)
    L5 = I.config5_layer(0, 0, 1, rows=16)
    assert L5.W.shape == (16, 8192)


def test_scale_format_names():
    f = I.scale_format("S1E4M4")
    assert (f.sign_bits, f.exp_bits, f.man_bits, f.bias) == (1, 4, 4, 7)
    assert I.scale_format("UE5M7").sign_bits == 0 and I.scale_format("E8M7").top_exp_reserved == 1
