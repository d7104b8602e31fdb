"""The layer pipeline written with oracle calls only (test infrastructure): the reference that the
CUDA pipeline is compared against, step for step."""
import math

import numpy as np

import oracle
from paper_2605_14929_b200 import inputs as I


def container_bits(fmt, need_sign, need_selector):
    need = fmt.exp_bits + fmt.man_bits + (1 if need_sign else 0) + (1 if need_selector else 0)
    return next(b for b in (8, 12, 16) if b >= need)


def run(layer, fmt, rom, fp=(), lloyd_iters=8, pool_percent=50.0, want_blocks=False):
    c = oracle.channel_norms(layer.X.numpy())
    rom_atoms = I.alphabet(rom, with_negations=True)
    n_bits = rom_atoms[0].n_bits
    out = dict(c=c, rom_atoms=rom_atoms)
    full = list(rom_atoms)
    if lloyd_iters > 0:
        r1 = oracle.pair_search(layer.W, c, fmt, rom_atoms, want_blocks=True)
        fmta = int(r1["best"][2])
        NB = r1["block_cos"].shape[1]
        rank = max(1, min(NB, int(math.ceil(NB * (100.0 - pool_percent) / 100.0))))
        a = rom_atoms[fmta]
        init = np.sort(-a.lut) if a.negated else a.lut
        lut, dist, cnt = oracle.dd_lloyd(layer.W, c, fmt, int(r1["k"][fmta]), r1["block_cos"][fmta], rank, init, lloyd_iters)
        dd = I.Atom(f"DD{n_bits}", n_bits, I.KIND_LUT, 0, I.SCOPE_BLOCK, 1.0, lut)
        full += [dd, dd.negation()]
        out.update(rom=r1, dd_lut=lut, distortion=dist, pool_count=cnt)
    full += [I.fp_atom(f) for f in fp]
    r2 = oracle.pair_search(layer.W, c, fmt, full, want_blocks=want_blocks)
    out.update(full=r2, atoms=full)
    sign = 1 if fmt.sign_bits and fmt.exp_bits + fmt.man_bits + 2 <= 16 else 0
    ia, ib = (int(r2["best"][3]), int(r2["best"][4])) if sign else (int(r2["best"][0]), int(r2["best"][1]))
    b = container_bits(fmt, bool(sign), True)
    pk = oracle.pack(layer.W, c, fmt, full[ia], int(r2["k"][ia]), full[ib], int(r2["k"][ib]), use_sign=sign,
                     container_bits=b, word_sign_bits=sign)
    out.update(pack=pk, pair=(ia, ib), container=b)
    return out
