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
from typing import List, Optional, Sequence

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
    is followed by its negation; ``fp`` are FP singles; ``lloyd_iters`` = 0 disables the DD atom.
    ``share`` names another sweep of the same shape and alphabet (typically the same layer at another scale
    format): the large scratch buffers -- workspaces, the per-block arrays, the channel norms, the packed
    codes and scale words -- are then that sweep's, and only the small results (tables, result blocks, the DD
    table, counts) are this sweep's own.  Sweeps that share buffers must run one after the other on one stream,
    and the packed output of one is overwritten by the next.  ``grid_dp`` builds the DD atom by the grid-constrained
    dynamic programme instead of Lloyd iterations with a snap (``lloyd_iters`` > 0 then only says that there is a DD
    atom).  ``opq_q`` (a quantile in (0, 1), the paper's default 0.92) takes the outliers out of the weights before
    anything else and keeps them as a sparse stream; the search, the DD atom and the packer then work on the weights
    with the outliers zeroed.  ``wr_sigma`` (a fraction of the layer's elements, the paper's default 0.001) adds the
    sparse correction of the packed layer's residual after the packer."""

    def __init__(self, M: int, K: int, T: int, fmt: I.ScaleFormat, rom: Sequence[str], fp: Sequence[str] = (),
                 lloyd_iters: int = 8, pool_percent: float = 50.0, device="cuda", want_blocks: bool = False,
                 share: Optional["LayerSweep"] = None, grid_dp: bool = False, opq_q: Optional[float] = None,
                 wr_sigma: Optional[float] = None, opq_capacity: Optional[int] = None):
        self.M, self.K, self.T, self.fmt = M, K, T, fmt
        self.dev = torch.device(device)
        self.iters = lloyd_iters
        self.grid_dp = bool(grid_dp) and lloyd_iters > 0
        self.dd_iters = 0 if self.grid_dp else lloyd_iters        # iterations handed to sop_dd4_lloyd; its status entry
        self.rom_atoms = I.alphabet(rom, with_negations=True)
        if not self.rom_atoms:
            # element formats only (a promotion-profile comparison): singles, no pair, no DD atom; the first one is packed
            if lloyd_iters > 0 or not fp:
                raise ValueError("without ROM atoms there is no DD atom to refine: need fp candidates and lloyd_iters = 0")
            n_bits = I.fp_atom(fp[0]).n_bits
        else:
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
        if share is not None:
            if (share.M, share.K, share.T, len(share.full_atoms), share.full_atoms[0].n_bits) != (M, K, T, nF, n_bits):
                raise ValueError("a sweep shares buffers only with a sweep of the same shape and alphabet size")
            self.c, self.ws_norm, self.ws_search, self.ws_lloyd = share.c, share.ws_norm, share.ws_search, share.ws_lloyd
        else:
            self.c = torch.empty(K, dtype=torch.float32, device=d)
            self.ws_norm = B.alloc_workspace(B.channel_norms_workspace(T, K), d)
            self.ws_search = B.alloc_workspace(B.pair_search_workspace(M, K, nF), d)
            self.ws_lloyd = B.alloc_workspace(B.dd4_lloyd_workspace(M, K), d)
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
        self.single = not self.rom_atoms                      # one element format packed alone: no sign choice, no selector
        if self.single:
            self.use_sign = 0
        self.container = scale_word_container(fmt, bool(self.use_sign), not self.single)
        self.counts = torch.zeros(2, dtype=torch.int64, device=d)
        if share is not None:
            self.codes, self.full_cos, self.full_sse = share.codes, share.full_cos, share.full_sse
            self.words = share._words_store[:B.words_nbytes(self.NB, self.container)]
        else:
            self.codes = torch.empty(self.NB * 2 * n_bits, dtype=torch.uint8, device=d)
            self._words_store = torch.empty(B.words_nbytes(self.NB, 16), dtype=torch.uint8, device=d)   # room for any container
            self.words = self._words_store[:B.words_nbytes(self.NB, self.container)]
            self.full_cos = torch.empty((nF, self.NB), dtype=torch.float32, device=d)
            self.full_sse = torch.empty((nF, self.NB), dtype=torch.float32, device=d)
        # the two sparse side streams (both off unless asked for)
        self.opq_m = B.opq_threshold(opq_q, 16) if opq_q is not None else None
        self.wr_keep = int(math.ceil(wr_sigma * M * K)) if wr_sigma is not None else 0
        if self.opq_m is not None and share is not None and getattr(share, "opq_m", None) == self.opq_m:
            # the outlier stream does not depend on the scale format: the sharing sweep's is this sweep's too
            self.W_opq, self.opq_row_start, self.opq_records = share.W_opq, share.opq_row_start, share.opq_records
            self.opq_count, self.ws_opq = share.opq_count, share.ws_opq
        elif self.opq_m is not None:
            cap = opq_capacity if opq_capacity is not None else max(1024, M * K // 32)    # 3 % of the elements: six times the Gaussian rate at q = 0.92
            self.W_opq = torch.empty((M, K), dtype=torch.bfloat16, device=d)
            self.opq_row_start = torch.zeros(M + 1, dtype=torch.int32, device=d)
            self.opq_records = torch.zeros(cap, dtype=torch.int32, device=d)
            self.opq_count = torch.zeros(1, dtype=torch.int64, device=d)
            self.ws_opq = B.opq_workspace(M, K, d)
        if self.wr_keep:
            self.wr_row_start = torch.zeros(M + 1, dtype=torch.int32, device=d)
            self.wr_records = torch.zeros(2 * self.wr_keep + 1024, dtype=torch.int32, device=d)     # ties at the threshold all enter
            self.wr_count = torch.zeros(1, dtype=torch.int64, device=d)
            self.wr_exp = torch.zeros(1, dtype=torch.int32, device=d)
            self.wr_tau = torch.zeros(1, dtype=torch.float32, device=d)
            self.ws_wr = B.wr_workspace(M, K, d)
        self.kernel_launches_per_step = 0
        self.lloyd_launches = 0
        if lloyd_iters > 0:      # (the query takes the table size in place of the iterations for the dynamic programme)
            self.lloyd_launches = (B.dd4_lloyd_launches(M, K, 1 << n_bits, B.LLOYD_GRID_DP) if self.grid_dp
                                   else B.dd4_lloyd_launches(M, K, lloyd_iters))

    def run(self, W: torch.Tensor, X: torch.Tensor, stream=None, norms: bool = True, reuse_prepass: bool = False,
            codes: Optional[torch.Tensor] = None, words: Optional[torch.Tensor] = None) -> None:
        """One pass of the whole hot path over device-resident W [M, K] bf16 and X [T, K] fp32.  ``norms`` =
        False skips the channel norms (and the outlier extraction, if any): they do not depend on the scale format, so
        a sweep that shares the buffers of another one (same layer, other format) uses what that one has just computed.
        ``reuse_prepass``: the same holds for the exponent histogram of the block scales behind the per-layer
        shift: the search takes it from the shared workspace as the sweep of this layer at the previous format
        left it, and only derives this format's shifts.  ``codes`` / ``words``: buffers of the sizes of ``self.codes`` /
        ``self.words`` that receive the packed layer instead of them (a stream hands in the slot the result leaves from)."""
        codes = self.codes if codes is None else codes
        words = self.words if words is None else words
        n = 0
        if norms:
            B.sop_channel_norms(X, self.c, self.ws_norm, stream)
            n += 2
        if self.opq_m is not None:
            if norms:          # like the norms, the outlier stream of a layer is extracted once for all its scale formats
                B.sop_opq_extract(W, self.opq_m, self.W_opq, self.opq_row_start, self.opq_records, self.opq_count, self.ws_opq, stream)
                n += 3
            W = self.W_opq
        if self.iters > 0:
            # every fixed candidate and every table entry among them; the best single of the result is FMTa
            B.sop_pair_search(W, self.c, self.fmt_c, self.atoms_c, self.pair_table, self.signed_table, self.rom_result,
                              self.ws_search, block_cos=self.full_cos, block_sse=self.full_sse, eval_mask=self.fixed_mask,
                              stream=stream, reuse_prepass=reuse_prepass)
            n += 3
            B.sop_dd4_lloyd(W, self.c, self.fmt_c, self.atoms_c, self.full_cos, self.pool_rank, self.dd_iters, self.dd_lut,
                            self.distortion, self.pool_count, self.ws_lloyd, search_result=self.rom_result, stream=stream,
                            grid_dp=self.grid_dp)
            n += self.lloyd_launches
            B.sop_pair_search(W, self.c, self.fmt_c, self.atoms_c, self.pair_table, self.signed_table, self.result,
                              self.ws_search, dd_lut=self.dd_lut, dd_mask=self.dd_mask, block_cos=self.full_cos,
                              block_sse=self.full_sse, eval_mask=self.dd_mask, load_mask=self.fixed_mask,
                              k_mode=B.K_FROM_RESULT, prev_result=self.rom_result, keep_loaded=True, stream=stream)
        else:
            B.sop_pair_search(W, self.c, self.fmt_c, self.atoms_c, self.pair_table, self.signed_table, self.result,
                              self.ws_search, block_cos=self.full_cos, block_sse=self.full_sse, stream=stream,
                              reuse_prepass=reuse_prepass)
            n += 1
        n += 2
        B.sop_pack(W, self.c, self.fmt_c, self.atoms_c, codes, words, search_result=self.result,
                   index_a=0 if self.single else B.PAIR_FROM_RESULT, index_b=B.NO_ATOM if self.single else B.PAIR_FROM_RESULT,
                   use_sign=self.use_sign, container_bits=self.container, word_sign_bits=self.use_sign,
                   counts=self.counts, dd_lut=self.dd_lut if self.dd_mask else None, dd_mask=self.dd_mask,
                   block_cos=self.full_cos, stream=stream)
        n += 1
        if self.wr_keep:
            B.sop_wr_extract(W, self.c, self.fmt_c, self.atoms_c, codes, words, self.wr_keep, self.wr_row_start,
                             self.wr_records, self.wr_count, self.wr_exp, self.ws_wr, tau=self.wr_tau,
                             index_a=0 if self.single else B.PAIR_FROM_RESULT, index_b=B.NO_ATOM if self.single else B.PAIR_FROM_RESULT,
                             search_result=self.result, use_sign=self.use_sign, container_bits=self.container,
                             word_sign_bits=self.use_sign, dd_lut=self.dd_lut if self.dd_mask else None, dd_mask=self.dd_mask,
                             stream=stream)
            n += 18
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

    def sparse_outputs(self) -> dict:
        """The two sparse streams of the last pass: per stream the row starts, the records that fit the buffer and
        the count; for Wr also the layer exponent and the threshold."""
        torch.cuda.synchronize(self.dev)
        out = {}
        if self.opq_m is not None:
            n = int(self.opq_count.item())
            out["opq"] = dict(count=n, row_start=self.opq_row_start.cpu().numpy().view(np.uint32),
                              records=self.opq_records[:min(n, self.opq_records.numel())].cpu().numpy().view(np.uint32),
                              W_out=self.W_opq.cpu(), m=self.opq_m)
        if self.wr_keep:
            n = int(self.wr_count.item())
            out["wr"] = dict(count=n, row_start=self.wr_row_start.cpu().numpy().view(np.uint32),
                             records=self.wr_records[:max(0, min(n, self.wr_records.numel()))].cpu().numpy().view(np.uint32),
                             scale_exp=int(self.wr_exp.item()), tau=float(self.wr_tau.item()), n_keep=self.wr_keep)
        return out

    def outputs(self) -> SweepOutputs:
        torch.cuda.synchronize(self.dev)
        if self.iters > 0:
            B.check_lloyd_status(self.distortion, self.dd_iters)  # a codebook from an unfinished call is not handed out
        nF, nR = len(self.full_atoms), len(self.rom_atoms)
        return SweepOutputs(
            c=self.c.cpu(), pair_table=B.read_pair_table(self.pair_table, nF),
            signed_table=B.read_pair_table(self.signed_table, nF), result=B.read_result(self.result),
            rom_result=B.read_result(self.rom_result) if self.iters > 0 else {},
            dd_lut=self.dd_lut.cpu().numpy(), distortion=self.distortion.cpu().numpy(),
            pool_count=int(self.pool_count.item()), codes=self.codes.cpu(), words=self.words.cpu(),
            counts=self.counts.cpu().numpy(), atoms=self.full_atoms)


class LayerStream:
    """Streams host-resident layers of one shape through a ``LayerSweep`` -- or through several sweeps that
    share their buffers (the same layer at several scale formats).  While layer i is swept, the weights and
    activations of layer i + 1 travel host -> device and the results of layer i - 1 travel device -> host: two
    input slots, two output slots per sweep, three CUDA streams ordered by events.  The host tensors must be
    pinned for the copies to overlap.

        stream = LayerStream(sweep)
        for i, (W_host, X_host) in enumerate(layers):
            stream.submit(i, W_host, X_host)
            if i:
                consume(stream.collect(i - 1))
        consume(stream.collect(len(layers) - 1))

    ``collect(i)`` waits for layer i and returns pinned host tensors (pair_table, signed_table, result,
    codes, words, distortion) that stay valid until ``submit(i + 2)`` -- one dict for a single sweep, a list
    of dicts (one per sweep) otherwise; it raises ``binding.LloydNotFinished`` when a Lloyd call of the layer
    reports that it did not run to its end.  ``streams`` hands in the three CUDA streams (copy in, compute,
    copy out) so that several LayerStream objects, one per layer shape, work as one ordered pipeline.  The packer
    writes codes and scale words straight into the slot they leave the device from.  ``graphs`` = True records
    the calls of every (slot, format) into a CUDA graph once (on zero-filled slots) and replays it per layer: no
    gaps between the dozen launches of a pass."""

    OUT = ("pair_table", "signed_table", "result", "codes", "words", "distortion")

    SMALL = ("pair_table", "signed_table", "result", "distortion")      # copied aside; codes and words are packed in place

    def __init__(self, sweep, streams=None, graphs: bool = False):
        self.single = isinstance(sweep, LayerSweep)
        self.sweeps = [sweep] if self.single else list(sweep)
        sw = self.sw = self.sweeps[0]
        d = sw.dev
        self.s_in, self.s_run, self.s_out = streams if streams is not None else (torch.cuda.Stream(d), torch.cuda.Stream(d), torch.cuda.Stream(d))
        self.W = [torch.zeros((sw.M, sw.K), dtype=torch.bfloat16, device=d) for _ in range(2)]
        self.X = [torch.zeros((sw.T, sw.K), dtype=torch.float32, device=d) for _ in range(2)]
        self.dev_out = [[{k: torch.empty_like(getattr(q, k)) for k in self.OUT} for q in self.sweeps] for _ in range(2)]
        self.host_out = [[{k: torch.empty(getattr(q, k).shape, dtype=getattr(q, k).dtype).pin_memory() for k in self.OUT}
                          for q in self.sweeps] for _ in range(2)]
        ev = lambda: [torch.cuda.Event() for _ in range(2)]
        self.in_ready, self.in_free, self.out_done = ev(), ev(), ev()
        self.out_ready = [[torch.cuda.Event() for _ in self.sweeps] for _ in range(2)]
        self.h2d_bytes = self.W[0].numel() * 2 + self.X[0].numel() * 4
        self.d2h_bytes = sum(t.numel() * t.element_size() for o in self.dev_out[0] for t in o.values())
        self.before_run = None       # optional callable run on the compute stream before every layer
        self.n_submitted = 0
        self.graphs = None
        if graphs:
            torch.cuda.synchronize(d)
            for slot in range(2):                 # the library's one-time set-ups happen outside the captures
                self._run_slot(slot, self.s_run)
            torch.cuda.synchronize(d)
            self.graphs = [[None] * len(self.sweeps) for _ in range(2)]
            side = torch.cuda.Stream(d)
            for slot in range(2):
                for f in range(len(self.sweeps)):
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=side):
                        self._run_format(slot, f, side)
                    self.graphs[slot][f] = g
            torch.cuda.synchronize(d)

    def _run_format(self, slot: int, f: int, stream) -> None:
        """The calls of one format on the layer in ``slot``, on ``stream``: the pass (packed output straight into the
        slot's buffers), then the small results set aside before the next format overwrites them."""
        q = self.sweeps[f]
        out = self.dev_out[slot][f]
        q.run(self.W[slot], self.X[slot], stream, norms=(f == 0), reuse_prepass=(f > 0), codes=out["codes"], words=out["words"])
        with torch.cuda.stream(stream):
            for k in self.SMALL:
                out[k].copy_(getattr(q, k), non_blocking=True)

    def _run_slot(self, slot: int, stream) -> None:
        for f in range(len(self.sweeps)):
            self._run_format(slot, f, stream)

    def submit(self, i: int, W_host: torch.Tensor, X_host: torch.Tensor) -> None:
        slot = i & 1
        with torch.cuda.stream(self.s_in):
            if i >= 2:
                self.s_in.wait_event(self.in_free[slot])      # the sweeps of layer i - 2 have read this slot
            self.W[slot].copy_(W_host, non_blocking=True)
            self.X[slot].copy_(X_host, non_blocking=True)
            self.in_ready[slot].record(self.s_in)
        with torch.cuda.stream(self.s_run):
            self.s_run.wait_event(self.in_ready[slot])
            if i >= 2:
                self.s_run.wait_event(self.out_done[slot])    # the results of layer i - 2 have left this slot
            if self.before_run is not None:
                self.before_run()
            for f in range(len(self.sweeps)):
                if self.graphs is not None:
                    self.graphs[slot][f].replay()
                else:
                    self._run_format(slot, f, self.s_run)
                self.out_ready[slot][f].record(self.s_run)
            self.in_free[slot].record(self.s_run)
        with torch.cuda.stream(self.s_out):
            for f in range(len(self.sweeps)):
                self.s_out.wait_event(self.out_ready[slot][f])     # a format's results leave while the next one is swept
                for k in self.OUT:
                    self.host_out[slot][f][k].copy_(self.dev_out[slot][f][k], non_blocking=True)
            self.out_done[slot].record(self.s_out)
        self.n_submitted = max(self.n_submitted, i + 1)

    def collect(self, i: int):
        slot = i & 1
        self.out_done[slot].synchronize()
        for f, q in enumerate(self.sweeps):
            if q.iters > 0:
                B.check_lloyd_status(self.host_out[slot][f]["distortion"], q.dd_iters)
        return self.host_out[slot][0] if self.single else self.host_out[slot]


class LayerSetSweep:
    """A set of layers (one transformer block, say), each swept at several scale formats: the unit of a model
    sweep that is streamed layer by layer.  Layers of one shape share their large buffers, and so do the formats
    of one layer; every (layer, format) keeps its own tables, result blocks and DD table.  ``run`` makes one
    pass: per layer the channel norms once, then per format the candidate sweep, the Lloyd refinement, the sweep
    of the new columns and the pack."""

    def __init__(self, shapes: Sequence[tuple], fmts: Sequence[I.ScaleFormat], rom: Sequence[str], fp: Sequence[str] = (),
                 lloyd_iters: int = 8, device="cuda", opq_q: Optional[float] = None, wr_sigma: Optional[float] = None):
        self.shapes, self.fmts = [tuple(s) for s in shapes], list(fmts)
        self.dev = torch.device(device)
        owner = {}
        self.sweeps: List[List[LayerSweep]] = []
        for shape in self.shapes:
            row = []
            for fmt in self.fmts:
                sw = LayerSweep(*shape, fmt, rom, fp, lloyd_iters, device=device, share=owner.get(shape), opq_q=opq_q, wr_sigma=wr_sigma)
                owner.setdefault(shape, sw)
                row.append(sw)
            self.sweeps.append(row)
        self.elements = sum(M * K for M, K, _ in self.shapes)
        self._graph = None

    def run(self, layers: Sequence[tuple], stream=None) -> None:
        """``layers``: one (W, X) pair of device tensors per shape given to the constructor, in that order."""
        for row, (W, X) in zip(self.sweeps, layers):
            for f, sw in enumerate(row):
                sw.run(W, X, stream, norms=(f == 0), reuse_prepass=(f > 0))

    @property
    def kernel_launches_per_step(self) -> int:
        return sum(sw.kernel_launches_per_step for row in self.sweeps for sw in row)

    def capture(self, layers: Sequence[tuple]) -> None:
        """Record one pass over these device tensors into a CUDA graph (see ``LayerSweep.capture``)."""
        self.run(layers)
        torch.cuda.synchronize(self.dev)
        side = torch.cuda.Stream(self.dev)
        side.wait_stream(torch.cuda.current_stream(self.dev))
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            self.run(layers, side)
        torch.cuda.current_stream(self.dev).wait_stream(side)
        self._graph, self._graph_inputs = graph, list(layers)

    def replay(self) -> None:
        self._graph.replay()

    def check(self) -> None:
        """After a synchronise: raises when a Lloyd call of the pass did not run to its end."""
        for row in self.sweeps:
            for sw in row:
                if sw.iters > 0:
                    B.check_lloyd_status(sw.distortion, sw.dd_iters)
