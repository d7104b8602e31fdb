"""GPU parity for element grids given by parameters (promotion-profile formats, HIF7 / HIF8): the sweep's
per-block values bit for bit, layer sums within 1e-6 relative, packed bytes exact for the 8-bit grids."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_14929_b200 import inputs as I

from .test_gpu_parity import B, assert_tables, gpu_search, gpu_pack  # noqa: F401  (B is a fixture)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("fmt_name,fp", [
    ("UE4M6", ["HIF7", "HIF8", "E2M3"]),                   # the paper's HIF7-vs-E2M3 comparison at one scale format
    ("UE4M6", ["E2M5", "E3M4", "E4M3", "E5M2"]),           # the FP8-class grids of the appendix table
    ("E5M6", ["E3M6", "E4M5", "E3M8", "E4M7"]),            # FP10 / FP12-class grids
    ("UE8M0", ["E3M4^0", "E4M3^0", "HIF8^0"]),             # one power-of-two scale per layer
])
def test_profile_of_grid_formats_matches_oracle(B, fmt_name, fp):
    L = I.outlier_channel_layer(7, 72, 1024, 64)
    fmt = I.scale_format(fmt_name)
    atoms = I.alphabet(["NF4"], fp=fp)
    A = len(atoms)
    c = oracle.channel_norms(L.X.numpy())
    want = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True)
    got = gpu_search(B, L.W, c, fmt, atoms)
    assert np.array_equal(got["block_cos"].view(np.uint32), want["block_cos"].view(np.uint32))
    assert np.array_equal(got["block_sse"].view(np.uint32), want["block_sse"].view(np.uint32))
    assert_tables(got, want, A)
    assert np.array_equal(got["k"][:A], want["k"])
    assert list(got["best"]) == list(want["best"])
    # different grids give different profiles (the parameters reach the kernel)
    acos = [want["pair"]["acos"][a, a] for a in range(2, A)]
    assert len(set(acos)) == len(acos)


def test_zero_blocks_and_saturation_on_a_grid(B):
    # zero rows, a block that sits on the negative end of HIF7 (-128 against +120), layer-scope saturation
    L = I.tiny_layer(5, 24, 256)
    W = L.W.clone()
    W[3] = 0
    W[4, :16] = torch.tensor([-128, 120, 15, -16, 8, 1, 0, -1, 64, 72, -7, 30, 2, 3, -60, 104], dtype=torch.float32).to(torch.bfloat16) * 2.0 ** -7
    L = I.Layer(W, L.X)
    fmt = I.scale_format("E5M6")
    atoms = [I.fp_atom("HIF7"), I.fp_atom("HIF8"), I.fp_atom("E2M5"), I.fp_atom("E2M5^0")]
    c = oracle.channel_norms(L.X.numpy())
    want = oracle.pair_search(L.W, c, fmt, atoms, want_blocks=True)
    got = gpu_search(B, L.W, c, fmt, atoms)
    assert np.array_equal(got["block_cos"].view(np.uint32), want["block_cos"].view(np.uint32))
    assert np.array_equal(got["block_sse"].view(np.uint32), want["block_sse"].view(np.uint32))
    assert_tables(got, want, len(atoms))


@pytest.mark.parametrize("name,fmt_name,b", [("E3M4", "UE4M4", 8), ("E2M5", "UE4M6", 12), ("E5M2", "E5M6", 12)])
def test_pack_of_an_eight_bit_grid_matches_oracle(B, name, fmt_name, b):
    L = I.config1()
    L = I.Layer(L.W[:48].contiguous(), L.X)
    fmt = I.scale_format(fmt_name)
    atoms = [I.fp_atom(name), I.rom_atom("NF4")]
    c = oracle.channel_norms(L.X.numpy())
    wsign = fmt.sign_bits
    want = oracle.pack(L.W, c, fmt, atoms[0], 1, None, 1, container_bits=b, word_sign_bits=wsign)
    assert want["rc"] == 0
    codes, words, counts = gpu_pack(B, L.W, c, fmt, atoms, 0, B.NO_ATOM, 1, 0, b, wsign)
    assert np.array_equal(codes, want["codes"])
    assert np.array_equal(words[:want["words"].size], want["words"])
