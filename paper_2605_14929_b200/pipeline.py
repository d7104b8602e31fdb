"""The per-layer hot path as a sequence of C-ABI calls on one stream, with no host round trip
in between: channel norms -> sweep of every fixed candidate (ROM atoms, negations, FP singles;
single-candidate reduction only: it finds FMTa and leaves every candidate's per-block cosine and
error in device arrays) -> DD-n Lloyd refinement -> sweep of the two new columns (DD-n and its
negation) with the fixed candidates' per-block values loaded, reducing every pair -> pack of the
chosen pair.  This module only allocates buffers and orders the calls.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Sequence

import numpy as np
import torch

from . import binding as B
from . import inputs as I


def layers_for_rank(n_layers: int, rank: int, world: int) -> List[int]:
    """Layer-parallel sharding: layers are independent units of the sweep, layer l goes to rank
    l mod world; no data-path collective is involved."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("need 0 <= rank < world")
    return list(range(rank, n_layers, world))


def job_throughput(units_per_rank: float, local_seconds: float, group=None) -> float:
    """Whole-job throughput of a layer-parallel run: the units all ranks processed divided by the
    slowest rank's time (sum and max over the process group; a single process when no group is up)."""
    import torch.distributed as dist
    t = torch.tensor([units_per_rank, local_seconds], dtype=torch.float64)
    if dist.is_available() and dist.is_initialized():
        dev = torch.device("cuda", torch.cuda.current_device()) if dist.get_backend(group) == "nccl" else torch.device("cpu")
        units, secs = t[:1].to(dev), t[1:].to(dev)
        dist.all_reduce(units, op=dist.ReduceOp.SUM, group=group)
        dist.all_reduce(secs, op=dist.ReduceOp.MAX, group=group)
        return float(units.item() / secs.item())
    return float(t[0] / t[1])


def scale_word_container(fmt, need_sign: bool, need_selector: bool) -> int:
    """Smallest container b in {8, 12, 16} holding sign + exponent + mantissa + selector."""
    need = fmt.exp_bits + fmt.man_bits + (1 if need_sign else 0) + (1 if need_selector else 0)
    for b in (8, 12, 16):
        if b >= need:
            return b
    raise ValueError("scale word does not fit 16 bits")


@dataclasses.dataclass
class SweepOutputs:
    c: torch.Tensor
    pair_table: np.ndarray
    signed_table: np.ndarray
    result: dict
    rom_result: dict
    dd_lut: np.ndarray
    distortion: np.ndarray
    pool_count: int
    codes: torch.Tensor
    words: torch.Tensor
    counts: np.ndarray
    atoms: List[I.Atom]


class LayerSweep:
    """Buffers and call order for one layer shape.  ``rom`` are base ROM atom names; every ROM atom
    is followed by its negation; ``fp`` are FP singles; ``lloyd_iters`` = 0 disables the DD atom."""

    def __init__(self, M: int, K: int, T: int, fmt: I.ScaleFormat, rom: Sequence[str], fp: Sequence[str] = (),
                 lloyd_iters: int = 8, pool_percent: float = 50.0, device="cuda", want_blocks: bool = False):
        self.M, self.K, self.T, self.fmt = M, K, T, fmt
        self.dev = torch.device(device)
        self.iters = lloyd_iters
        self.rom_atoms = I.alphabet(rom, with_negations=True)
        n_bits = self.rom_atoms[0].n_bits
        self.full_atoms = list(self.rom_atoms)
        self.dd_mask = 0
        if lloyd_iters > 0:
            dd = I.Atom(f"DD{n_bits}", n_bits, I.KIND_LUT, 0, I.SCOPE_BLOCK, 1.0, np.zeros(1 << n_bits, np.float32))
            self.dd_mask = (1 << len(self.full_atoms)) | (1 << (len(self.full_atoms) + 1))
            self.full_atoms += [dd, dd.negation()]
        self.full_atoms += [I.fp_atom(f) for f in fp]
        # marshalled once: the calls of run() then cost no Python loops
        self.atoms_c = B.make_atoms(self.full_atoms)
        self.fmt_c = B.make_fmt(fmt)
        self.NB = M * (K // 16)
        self.pool_rank = int(math.ceil(self.NB * (100.0 - pool_percent) / 100.0))
        self.pool_rank = max(1, min(self.NB, self.pool_rank))
        nR, nF = len(self.rom_atoms), len(self.full_atoms)
        d = self.dev
        self.c = torch.empty(K, dtype=torch.float32, device=d)
        self.ws_norm = B.alloc_workspace(B.channel_norms_workspace(T, K), d)
        self.ws_search = B.alloc_workspace(B.pair_search_workspace(M, K, nF), d)
        self.ws_lloyd = B.alloc_workspace(B.dd4_lloyd_workspace(M, K), d)
        self.rom_table = B.new_pair_table(nF, d)
        self.rom_result = B.new_result(d)
        self.fixed_mask = ((1 << nF) - 1) & ~self.dd_mask
        self.dd_lut = torch.zeros(B.MAX_ENTRIES, dtype=torch.float32, device=d)
        self.distortion = torch.zeros(max(1, lloyd_iters + 1), dtype=torch.float64, device=d)
        self.pool_count = torch.zeros(1, dtype=torch.int64, device=d)
        self.pair_table = B.new_pair_table(nF, d)
        self.signed_table = B.new_pair_table(nF, d)
        self.result = B.new_result(d)
        # the packed word carries sign + selector when both fit 16 bits; a 16-bit signed format (E8M7) has no
        # metabit left, so its pair is packed without the sign (the selector takes the sign's bit)
        self.use_sign = 1 if fmt.sign_bits and fmt.exp_bits + fmt.man_bits + 2 <= 16 else 0
        self.container = scale_word_container(fmt, bool(self.use_sign), True)
        self.codes = torch.empty(self.NB * 2 * n_bits, dtype=torch.uint8, device=d)
        self.words = torch.empty(B.words_nbytes(self.NB, self.container), dtype=torch.uint8, device=d)
        self.counts = torch.zeros(2, dtype=torch.int64, device=d)
        self.full_cos = torch.empty((nF, self.NB), dtype=torch.float32, device=d)
        self.full_sse = torch.empty((nF, self.NB), dtype=torch.float32, device=d)
        self.kernel_launches_per_step = 0
        self.lloyd_launches = B.dd4_lloyd_launches(M, K, lloyd_iters) if lloyd_iters > 0 else 0

    def run(self, W: torch.Tensor, X: torch.Tensor, stream=None) -> None:
        """One pass of the whole hot path over device-resident W [M, K] bf16 and X [T, K] fp32."""
        n = 0
        B.sop_channel_norms(X, self.c, self.ws_norm, stream)
        n += 2
        if self.iters > 0:
            B.sop_pair_search(W, self.c, self.fmt_c, self.atoms_c, self.rom_table, None, self.rom_result, self.ws_search,
                              block_cos=self.full_cos, block_sse=self.full_sse, eval_mask=self.fixed_mask,
                              singles_only=True, stream=stream)
            n += 2
            B.sop_dd4_lloyd(W, self.c, self.fmt_c, self.atoms_c, self.full_cos, self.pool_rank, self.iters, self.dd_lut,
                            self.distortion, self.pool_count, self.ws_lloyd, search_result=self.rom_result, stream=stream)
            n += self.lloyd_launches
            B.sop_pair_search(W, self.c, self.fmt_c, self.atoms_c, self.pair_table, self.signed_table, self.result,
                              self.ws_search, dd_lut=self.dd_lut, dd_mask=self.dd_mask, block_cos=self.full_cos,
                              block_sse=self.full_sse, eval_mask=self.dd_mask, load_mask=self.fixed_mask,
                              k_mode=B.K_FROM_RESULT, prev_result=self.rom_result, stream=stream)
        else:
            B.sop_pair_search(W, self.c, self.fmt_c, self.atoms_c, self.pair_table, self.signed_table, self.result,
                              self.ws_search, block_cos=self.full_cos, block_sse=self.full_sse, stream=stream)
            n += 1
        n += 1
        B.sop_pack(W, self.c, self.fmt_c, self.atoms_c, self.codes, self.words, search_result=self.result,
                   use_sign=self.use_sign, container_bits=self.container, word_sign_bits=self.use_sign,
                   counts=self.counts, dd_lut=self.dd_lut if self.dd_mask else None, dd_mask=self.dd_mask,
                   block_cos=self.full_cos, stream=stream)
        n += 1
        self.kernel_launches_per_step = n

    def capture(self, W: torch.Tensor, X: torch.Tensor) -> None:
        """Record the calls of ``run(W, X)`` into a CUDA graph bound to these two tensors (refill them in place
        for the next layer); ``replay()`` then launches the whole pass at once, without the gaps between a
        dozen launches.  Profiling (``binding.profile_enable``) must be off: events recorded inside a graph
        cannot be read back."""
        self.run(W, X)                       # the library's one-time set-ups happen outside the capture
        torch.cuda.synchronize(self.dev)
        side = torch.cuda.Stream(self.dev)
        side.wait_stream(torch.cuda.current_stream(self.dev))
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            self.run(W, X, side)
        torch.cuda.current_stream(self.dev).wait_stream(side)
        self._graph, self._graph_inputs = graph, (W, X)

    def replay(self) -> None:
        self._graph.replay()

    def outputs(self) -> SweepOutputs:
        torch.cuda.synchronize(self.dev)
        nF, nR = len(self.full_atoms), len(self.rom_atoms)
        return SweepOutputs(
            c=self.c.cpu(), pair_table=B.read_pair_table(self.pair_table, nF),
            signed_table=B.read_pair_table(self.signed_table, nF), result=B.read_result(self.result),
            rom_result=B.read_result(self.rom_result) if self.iters > 0 else {},
            dd_lut=self.dd_lut.cpu().numpy(), distortion=self.distortion.cpu().numpy(),
            pool_count=int(self.pool_count.item()), codes=self.codes.cpu(), words=self.words.cpu(),
            counts=self.counts.cpu().numpy(), atoms=self.full_atoms)


class LayerStream:
    """Streams host-resident layers of one shape through a ``LayerSweep``.  While layer i is swept, the
    weights and activations of layer i + 1 travel host -> device and the results of layer i - 1 travel
    device -> host: two input slots, two output slots, three CUDA streams ordered by events.  The host
    tensors must be pinned for the copies to overlap.

        stream = LayerStream(sweep)
        for i, (W_host, X_host) in enumerate(layers):
            stream.submit(i, W_host, X_host)
            if i:
                consume(stream.collect(i - 1))
        consume(stream.collect(len(layers) - 1))

    ``collect(i)`` waits for layer i and returns pinned host tensors (pair_table, signed_table, result,
    codes, words) that stay valid until ``submit(i + 2)``."""

    OUT = ("pair_table", "signed_table", "result", "codes", "words")

    def __init__(self, sweep: LayerSweep):
        self.sw = sweep
        d = sweep.dev
        self.s_in, self.s_run, self.s_out = torch.cuda.Stream(d), torch.cuda.Stream(d), torch.cuda.Stream(d)
        self.W = [torch.empty((sweep.M, sweep.K), dtype=torch.bfloat16, device=d) for _ in range(2)]
        self.X = [torch.empty((sweep.T, sweep.K), dtype=torch.float32, device=d) for _ in range(2)]
        self.dev_out = [{k: torch.empty_like(getattr(sweep, k)) for k in self.OUT} for _ in range(2)]
        self.host_out = [{k: torch.empty(getattr(sweep, k).shape, dtype=getattr(sweep, k).dtype).pin_memory() for k in self.OUT}
                         for _ in range(2)]
        ev = lambda: [torch.cuda.Event() for _ in range(2)]
        self.in_ready, self.in_free, self.out_ready, self.out_done = ev(), ev(), ev(), ev()
        self.h2d_bytes = self.W[0].numel() * 2 + self.X[0].numel() * 4
        self.d2h_bytes = sum(t.numel() * t.element_size() for t in self.dev_out[0].values())
        self.before_run = None       # optional callable run on the compute stream before every sweep

    def submit(self, i: int, W_host: torch.Tensor, X_host: torch.Tensor) -> None:
        slot = i & 1
        sw = self.sw
        with torch.cuda.stream(self.s_in):
            if i >= 2:
                self.s_in.wait_event(self.in_free[slot])      # the sweep of layer i - 2 has read this slot
            self.W[slot].copy_(W_host, non_blocking=True)
            self.X[slot].copy_(X_host, non_blocking=True)
            self.in_ready[slot].record(self.s_in)
        with torch.cuda.stream(self.s_run):
            self.s_run.wait_event(self.in_ready[slot])
            if i >= 2:
                self.s_run.wait_event(self.out_done[slot])    # the results of layer i - 2 have left this slot
            if self.before_run is not None:
                self.before_run()
            sw.run(self.W[slot], self.X[slot], self.s_run)
            self.in_free[slot].record(self.s_run)
            for k in self.OUT:
                self.dev_out[slot][k].copy_(getattr(sw, k), non_blocking=True)
            self.out_ready[slot].record(self.s_run)
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.out_ready[slot])
            for k in self.OUT:
                self.host_out[slot][k].copy_(self.dev_out[slot][k], non_blocking=True)
            self.out_done[slot].record(self.s_out)

    def collect(self, i: int) -> dict:
        slot = i & 1
        self.out_done[slot].synchronize()
        return self.host_out[slot]
