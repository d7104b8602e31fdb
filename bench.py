#!/usr/bin/env python
"""Benchmark of the SOP per-layer candidate sweep on B200.

Workload at every N: the 70B-shaped layer set (the largest single-GPU configuration): the five layers of one
transformer block (8192 x 8192, 1024 x 8192 twice, 28672 x 8192, 8192 x 28672, bf16, Student-t(5) * 0.02 with
lognormal(0, 1.2) input-channel scales, X 1024 x K), generated on the device from the seed, each swept at the
eight scale formats of the paper's scale-format table with the full n = 4 alphabet (NF4, SH4, BOF4, Split87,
DD4 by 8 Lloyd iterations, and their negations; every pair).  The model has 80 such blocks with layers that are
independent and identically distributed by seed; one block is the streamed unit and the timed subset.

One step = one pass of the whole hot path over that block: per layer the channel norms, then per scale format
the sweep of every fixed candidate (finds FMTa), the DD4 Lloyd refinement, the sweep of the two DD4 columns
(every pair), and the pack of the chosen pair.  The metric counts a weight element once per scale format.
With N > 1 every rank sweeps its own transformer block (layers are independent: no data-path collective).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload block|layer]

Prints ONE JSON line (rank 0).  ``--impl reference`` times the CPU oracle on a bounded sample.
``--workload layer`` runs a smaller case of the same kernels -- the block's first layer (8192 x 8192) at one scale
format (E5M6) -- sized for profiler captures (1.5 GB on the device, W larger than L2); its line says so in ``config``.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "G weight-elems/s through full alphabet pair sweep"
UNIT = "G weight-elems/s"
ROM4 = ["NF4", "SH4", "BOF4", "Split87"]
SCALE_FORMATS = ["UE4M4", "E4M3", "UE4M6", "E4M5", "UE5M7", "E5M6", "E4M7", "E8M7"]
WORKLOAD = dict(
    workload="config5: 70B-shaped layer set, transformer block b of 80 (layers are iid by seed: one block is the timed subset): "
             "8192x8192, 1024x8192 x2, 28672x8192, 8192x28672 bf16, Student-t(5)*0.02, lognormal(0,1.2) channel scales, "
             "X 1024xK, generated on device; NF4/SH4/BOF4/Split87/DD4(8 Lloyd iters) + negations, all pairs, at the "
             "eight scale formats UE4M4 E4M3 UE4M6 E4M5 UE5M7 E5M6 E4M7 E8M7",
    layers=["8192x8192", "1024x8192", "1024x8192", "28672x8192", "8192x28672"], T=1024, scale_formats=SCALE_FORMATS,
    rom=ROM4, fp=[], lloyd_iters=8, g=16)
# config 2 (the attention projection), kept for the per-config table and the full-size parity test
CONFIG2 = dict(M=4096, K=4096, T=512, scale_format="E5M6", rom=ROM4, fp=["E2M3", "E4M3"], lloyd_iters=8)
SM_COUNT, SCHEDULERS, LANES = 148, 4, 32

# DRAM traffic of the sweep kernel per weight element and launch, from the ncu capture summarised in the named
# file (dram__bytes_read.sum + dram__bytes_write.sum of one launch on the 8192x8192 layer at E5M6 divided by its
# elements; traffic grows in proportion to the elements, so a launch of the block is scaled by its elements).
# None: no capture of the kernel as it is now.
NCU_SWEEP_TRAFFIC = dict(source="profiles/kernels_config5_layer_8192x8192_E5M6.md", bytes_per_element_fixed_candidates=5.1796,
                         bytes_per_element_dd_columns=2.5803)
# the same for the reduction kernel (first call: the fixed candidates' entries; second call: the DD columns' entries)
NCU_REDUCE_TRAFFIC = dict(source="profiles/kernels_config5_layer_8192x8192_E5M6.md", bytes_per_element_fixed_candidates=4.0759,
                          bytes_per_element_dd_columns=5.0753)


# ---------------------------------------------------------------------------------------------------------
# operation and byte models of the search (both sweep launches together), per weight element
# ---------------------------------------------------------------------------------------------------------
def search_ops_n_step(n_lut: int, n_bits: int, n_fp: int) -> float:
    """The operation count of an n-step nearest-entry search: 6 shared (unpack, absmax, c w, norm, u), 2n + 5 per
    LUT candidate (n compare-select steps, fetch, four multiply-adds), 12 per FP candidate; per block 2 per pair of
    LUT candidates (diagonal included) and 6 per candidate."""
    pairs = n_lut * (n_lut + 1) // 2
    return 6 + n_lut * (2 * n_bits + 5) + n_fp * 12 + (2 * pairs + 6 * (n_lut + n_fp)) / 16.0


def search_ops_cell_lookup(n_lut: int, n_bits: int, n_fp: int, n_dd: int, signed: bool) -> float:
    """The operation count of the search as this library does it: W is unpacked in both launches (6 each); a LUT
    candidate costs 4 for the cell lookup (fetch, compare, select, unpack) and 5 packed multiply-adds on element
    pairs (2.5 per element) whatever n is; an FP candidate 12; per block 6 per evaluated candidate, 2 per
    candidate loaded by the second launch, 2 per pair entry (diagonal included), and with a signed scale 4 per
    base atom (the better of the atom and its negation) plus 2 per four-way entry."""
    pairs = n_lut * (n_lut + 1) // 2
    n_base = n_lut // 2 if signed else 0
    four = n_base * (n_base + 1) // 2
    per_block = 6 * (n_lut + n_fp) + 2 * (n_lut + n_fp - n_dd) + 2 * (pairs + n_fp) + 4 * n_base + 2 * four
    return 12 + n_lut * 6.5 + n_fp * 12 + per_block / 16.0


def sweep_kernel_ops_n_step(n_eval_lut: int, n_bits: int, n_eval_fp: int) -> float:
    """The part of ``search_ops_n_step`` that one launch of the evaluation kernel does: the shared 6, 2n + 5 per LUT
    candidate it evaluates, 12 per FP candidate, and per block 6 per evaluated candidate (its cosine)."""
    return 6 + n_eval_lut * (2 * n_bits + 5) + n_eval_fp * 12 + 6 * (n_eval_lut + n_eval_fp) / 16.0


def search_bytes(n_cand: int, n_dd: int) -> float:
    """Algorithmic DRAM bytes per element of the search as the call plan has it: W (2 bytes) read by each of the two
    evaluation launches, 8 bytes per block for every candidate's column written (per-block cosine and error: the
    reduction, the Lloyd pool and the pack read them), the fixed candidates' columns read by the first reduction and
    every column by the second."""
    return 2 * 2.0 + (8.0 * n_cand + 8.0 * (n_cand - n_dd) + 8.0 * n_cand) / 16.0


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={q}", "--format=csv,noheader,nounits",
                                          "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
                pw.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for nm, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        # "under load": the samples taken while the GPU drew more than half of the largest power seen
        load = [s for s, p in zip(sm, pw) if pw and p >= 0.5 * max(pw)]
        return dict(sm_mhz=statistics.median(load or sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm), samples_under_load=len(load),
                    power_w_max=max(pw) if pw else None)


def make_layer(seed: int):
    """The attention-projection layer of configuration 2 (host tensors)."""
    from paper_2605_14929_b200 import inputs as I
    return I.config2(seed, CONFIG2["M"], CONFIG2["K"], CONFIG2["T"])


# ---------------------------------------------------------------------------------------------------------
# the CPU oracle as a baseline: a bounded sample of the same workload
# ---------------------------------------------------------------------------------------------------------
def cpu_oracle_time(rows: int, fmt_name: str = "E5M6"):
    """Times the oracle pipeline, as it stands, on the first ``rows`` rows of the workload's 8192 x 8192 layer at one
    scale format (channel norms over the whole X, both searches, Lloyd, pack), single thread."""
    from paper_2605_14929_b200 import inputs as I
    from tests import oracle_pipeline
    L = I.config5_layer(0, 0, 0, rows=rows)
    t0 = time.perf_counter()
    oracle_pipeline.run(L, I.scale_format(fmt_name), WORKLOAD["rom"], WORKLOAD["fp"], WORKLOAD["lloyd_iters"])
    dt = time.perf_counter() - t0
    return rows * 8192 / dt / 1e9, dt


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows = 64
    for _ in range(min(args.warmup, 2)):
        cpu_oracle_time(16)
    times = []
    for _ in range(args.steps):
        _, dt = cpu_oracle_time(rows)
        times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = rows * 8192 / (ms * 1e-3) / 1e9
    sample = (f"per step the first {rows} of 8192 rows of the 8192x8192 layer at E5M6 (1 of 5 layers, 1 of 8 scale formats), "
              "full alphabet and pipeline, single thread")
    print(json.dumps(dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                          warmup=args.warmup, ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None,
                          dtype="f32", data="synthetic", config=WORKLOAD,
                          cpu_baseline=dict(value=value, unit=UNIT, cores=1, kind="oracle", sample=sample),
                          e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))))


# ---------------------------------------------------------------------------------------------------------
# the other configurations: short timings for the per-config table (rank 0, N = 1)
# ---------------------------------------------------------------------------------------------------------
def time_sweeps(sweeps, reps, flush):
    """Whole-path and sweep-only time (ms, medians) of a list of (sweep, W, X, norms) passes launched call by call;
    ``flush`` is a buffer larger than L2 that is rewritten before every pass, or None."""
    import torch
    from paper_2605_14929_b200 import binding as B
    st = torch.cuda.current_stream()

    def one():
        for sw, W, X, norms in sweeps:
            sw.run(W, X, st, norms=norms, reuse_prepass=not norms)
    for _ in range(3):
        one()
    torch.cuda.synchronize()
    whole, sweep = [], []
    B.profile_enable(True)
    for _ in range(reps):
        if flush is not None:
            flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        t_sw = 0.0
        for sw, W, X, norms in sweeps:
            sw.run(W, X, st, norms=norms, reuse_prepass=not norms)
            for back in range(2 if sw.iters > 0 else 1):           # with a DD atom the search is two calls
                t_sw += B.profile_ms(B.PROFILE_SWEEP, back) + B.profile_ms(B.PROFILE_REDUCE, back)
        e1.record(st)
        torch.cuda.synchronize()
        whole.append(e0.elapsed_time(e1))
        sweep.append(t_sw)
    B.profile_enable(False)
    return statistics.median(whole), statistics.median(sweep)


def per_config_table(dev, alu_peak, flush):
    """Configurations 1 to 4 at full size: G elements/s through the whole hot path and through the sweep launches
    alone, with the operation count per element and the fraction of the issue peak it amounts to."""
    import torch
    from paper_2605_14929_b200 import binding as B, inputs as I
    from paper_2605_14929_b200.pipeline import LayerSweep
    out = {}

    def entry(name, sweeps, elements, ops, note, fl, baseline=None):
        whole, sweep = time_sweeps(sweeps, 5, fl)
        out[name] = dict(elements_times_formats=elements, whole_path=dict(value=elements / whole / 1e6, unit=UNIT, ms=whole),
                         sweep_only=dict(value=elements / sweep / 1e6, unit=UNIT, ms=sweep), ops_per_element_n_step=ops,
                         frac_of_alu_peak=ops * elements / (sweep * 1e-3) / 1e12 / alu_peak, note=note)
        if baseline is not None:          # the oracle, as it stands, on a small sample of this configuration (one host core)
            n_el, sample, fn = baseline
            t0 = time.perf_counter()
            fn()
            dt = time.perf_counter() - t0
            out[name]["oracle_baseline"] = dict(value=n_el / dt / 1e9, unit=UNIT, cores=1, sample=sample, seconds=dt)

    # 1: single small layer, signed UE4M4, three ROM atoms
    from tests import oracle_pipeline
    import oracle
    L = I.config1(0)
    sw = LayerSweep(256, 1024, 128, I.scale_format("S1E4M4"), ["NF4", "SH4", "BOF4"], [], 0, device=dev)
    L1 = L
    entry("config1", [(sw, L.W.to(dev), L.X.to(dev), True)], 256 * 1024, search_ops_n_step(6, 4, 0),
          "256x1024, S1E4M4, NF4/SH4/BOF4 + negations, no DD atom; launch-latency sized (one wave of 32 CTAs)", flush,
          baseline=(256 * 1024, "the whole layer, whole pipeline",
                    lambda: oracle_pipeline.run(L1, I.scale_format("S1E4M4"), ["NF4", "SH4", "BOF4"], [], 0)))
    # 2: attention projection
    L = make_layer(0)
    sw = LayerSweep(CONFIG2["M"], CONFIG2["K"], CONFIG2["T"], I.scale_format("E5M6"), CONFIG2["rom"], CONFIG2["fp"], 8, device=dev)
    L2 = I.Layer(L.W[:128].contiguous(), L.X)
    entry("config2", [(sw, L.W.to(dev), L.X.to(dev), True)], CONFIG2["M"] * CONFIG2["K"], search_ops_n_step(10, 4, 2),
          "4096x4096, E5M6, 10 LUT candidates + E2M3/E4M3, all pairs; L2 flushed between passes", flush,
          baseline=(128 * CONFIG2["K"], "the first 128 of 4096 rows, whole pipeline",
                    lambda: oracle_pipeline.run(L2, I.scale_format("E5M6"), CONFIG2["rom"], CONFIG2["fp"], 8)))
    del sw
    # 3: the seven layers of one 7B-shaped transformer block, FP6 per block against FP8 per layer (singles only)
    fmt = I.scale_format("UE4M4")
    fp = ["E2M3", "E4M3^0"]
    sweeps, elements, own = [], 0, {}
    for which, (_, M, K) in enumerate(I.SHAPES_7B):
        Lw = I.config3_layer(0, 0, which, device=str(dev))
        sw = own.get((M, K))
        if sw is None:
            sw = own[(M, K)] = LayerSweep(M, K, 512, fmt, [], fp, 0, device=dev)
        sweeps.append((sw, Lw.W, Lw.X, True))
        elements += M * K
    L3 = I.config3_layer(0, 0, 4, rows=128)

    def oracle3():
        c = oracle.channel_norms(L3.X.numpy())
        oracle.pair_search(L3.W, c, fmt, [I.fp_atom(f) for f in fp])
    entry("config3", sweeps, elements, search_ops_n_step(0, 4, 2),
          "block 0 of 32 (seven layers, 218 M elements > L2), E2M3sUE4M4 vs E4M3^0: two FP singles, no pairs, no DD atom, pack of the FP6 single", None,
          baseline=(128 * L3.W.shape[1], "the first 128 rows of the 14336x4096 layer, channel norms and the search of both candidates", oracle3))
    del sweeps, own
    torch.cuda.empty_cache()
    # 4: the n = 5 MLP pair at both scale formats
    sweeps, elements = [], 0
    for which in (0, 1):
        Lw = I.config4_layer(0, which, device=str(dev))
        M, K = Lw.W.shape
        first = None
        for f in ("UE4M4", "E5M6"):
            sw = LayerSweep(M, K, 2048, I.scale_format(f), ["NF5", "SH5", "BOF5", "E2M2"], [], 16, device=dev, share=first)
            first = first or sw
            sweeps.append((sw, Lw.W, Lw.X, f == "UE4M4"))
            elements += M * K
    L4 = I.config4_layer(0, 0, rows=128)
    entry("config4", sweeps, elements, search_ops_n_step(10, 5, 0),
          "14336x4096 and 4096x14336 at UE4M4 and E5M6, 32-entry atoms, DD5 by 16 Lloyd iterations, all pairs", None,
          baseline=(128 * L4.W.shape[1], "the first 128 rows of the 14336x4096 layer at UE4M4, whole pipeline",
                    lambda: oracle_pipeline.run(L4, I.scale_format("UE4M4"), ["NF5", "SH5", "BOF5", "E2M2"], [], 16)))
    del sweeps
    torch.cuda.empty_cache()
    return out


def sparse_streams_table(dev, hbm_peak, of, flush):
    """The two sparse side streams (outlier extraction before the search, correction of the packed residual after it)
    on the 8192x8192 layer at E5M6: time of each by the library's events, record counts, algorithmic bytes and the
    fraction of the HBM peak they amount to.  They are off in the headline workload."""
    import torch
    from paper_2605_14929_b200 import binding as B, inputs as I
    from paper_2605_14929_b200.pipeline import LayerSweep
    L = I.config5_layer(0, 0, 0, device=str(dev))
    M, K = L.W.shape
    sw = LayerSweep(M, K, L.X.shape[0], I.scale_format("E5M6"), ROM4, [], 8, device=dev, opq_q=0.92, wr_sigma=0.001)
    for _ in range(2):
        sw.run(L.W, L.X)
    torch.cuda.synchronize(dev)
    B.profile_enable(True)
    t_opq, t_wr, t_all = [], [], []
    for _ in range(5):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        sw.run(L.W, L.X)
        e1.record()
        torch.cuda.synchronize(dev)
        t_opq.append(B.profile_ms(B.PROFILE_OPQ, 0)); t_wr.append(B.profile_ms(B.PROFILE_WR, 0)); t_all.append(e0.elapsed_time(e1))
    B.profile_enable(False)
    sp = sw.sparse_outputs()
    sw.outputs()                                   # raises if the Lloyd call of the pass did not finish
    E = M * K
    opq_ms, wr_ms, all_ms = sorted(t_opq)[2], sorted(t_wr)[2], sorted(t_all)[2]
    opq_bytes = (2.0 + 2.0 + 2 * 2.0 / 16.0) * E + 4.0 * sp["opq"]["count"]
    wr_bytes = 2 * (2.0 + 0.5 + sw.container / 8.0 / 16.0) * E + 4.0 * sp["wr"]["count"]

    def hbm(b, ms):
        return dict(achieved=b / (ms * 1e-3) / 1e9, peak=hbm_peak, unit="GB/s", frac=b / (ms * 1e-3) / 1e9 / hbm_peak, of=of)
    return dict(workload="8192x8192 at E5M6, ROM4 + DD4, outlier quantile 0.92, correction sparsity 0.001", elements=E,
                opq=dict(ms=opq_ms, records=sp["opq"]["count"], rate=sp["opq"]["count"] / E, threshold_m=sp["opq"]["m"],
                         bpw=32.0 * sp["opq"]["count"] / E, algorithmic_bytes=opq_bytes, hbm=hbm(opq_bytes, opq_ms),
                         note="three launches: mask + zeroed copy (W read once, written once), scan of the tile counts, records"),
                wr=dict(ms=wr_ms, records=sp["wr"]["count"], n_keep=sp["wr"]["n_keep"], scale_exp=sp["wr"]["scale_exp"],
                        bpw=32.0 * sp["wr"]["count"] / E, algorithmic_bytes=wr_bytes, hbm=hbm(wr_bytes, wr_ms),
                        note="two passes decode W, codes and scale words (2.6 bytes per element) into the residual: block maxima, then the "
                             "candidates above the bound they give; threshold, kept set and counts come from the candidate list, the "
                             "write pass decodes only blocks with a kept entry (eighteen launches, seven of them the unused "
                             "full-decode path that returns at once)"),
                whole_path_ms=all_ms, whole_path_value=E / all_ms / 1e6)


# ---------------------------------------------------------------------------------------------------------
# N > 1 bookkeeping (no data-path collective: the ranks only agree on the slowest time)
# ---------------------------------------------------------------------------------------------------------
def block_for_rank(rank: int) -> int:
    """Layer-parallel sharding of the model sweep: rank r takes transformer block r (all blocks come from seed 0)."""
    return rank


def reduce_times(named: dict, device, world: int) -> dict:
    """The largest value of every named time over the ranks (every rank gets the result)."""
    import torch
    import torch.distributed as dist
    keys = sorted(named)
    t = torch.tensor([float(named[k]) for k in keys], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return dict(zip(keys, (float(x) for x in t.cpu())))


def run_gpu(args) -> None:
    import torch
    import torch.distributed as dist
    from paper_2605_14929_b200 import binding as B, inputs as I, pipeline
    from paper_2605_14929_b200.pipeline import LayerSetSweep, LayerStream

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        if world == 1 and args.gpus > 1:
            raise SystemExit("--gpus N > 1 must be launched with torch.distributed.run (one rank per GPU)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    # the library is built in-tree beforehand; where it is missing (a fresh checkout) local rank 0 builds it with nvcc and
    # the other ranks wait for the file -- there is no other path: without it B.lib() raises
    from paper_2605_14929_b200 import build as libbuild
    if not os.path.exists(libbuild.LIB):
        if local == 0:
            libbuild.build()
        else:
            for _ in range(600):
                if os.path.exists(libbuild.LIB):
                    break
                time.sleep(1.0)
            time.sleep(2.0)
    B.lib()

    small = args.workload == "layer"                              # the profiling case: one layer, one format
    fmt_names = ["E5M6"] if small else WORKLOAD["scale_formats"]
    fmts = [I.scale_format(f) for f in fmt_names]
    S = len(fmts)
    block = block_for_rank(rank)                                  # every rank sweeps its own transformer block
    layers = [I.config5_layer(0, block, which, device=str(dev)) for which in range(1 if small else len(I.SHAPES_70B))]
    layer_names = WORKLOAD["layers"][:len(layers)]
    dev_layers = [(L.W, L.X) for L in layers]
    shapes = [(L.W.shape[0], L.W.shape[1], L.X.shape[0]) for L in layers]
    sset = LayerSetSweep(shapes, fmts, WORKLOAD["rom"], WORKLOAD["fp"], WORKLOAD["lloyd_iters"], device=dev)
    E = sset.elements                                             # weight elements of the block
    units = float(E * S)                                          # the metric counts an element once per scale format
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def one_step(launch):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        launch()
        e1.record(stream)
        return e0, e1

    # The timed steps replay the block's calls as one CUDA graph (what a job that sweeps 80 such blocks does).  A
    # replayed graph gives no per-kernel events, so one more pass is run call by call with the library's events
    # around its main kernels: those times feed the roofline object.
    launch_kind = "one CUDA graph replay per step"
    step_launch = sset.replay
    try:
        sset.capture(dev_layers)
    except RuntimeError as exc:                           # no graph capture here: time the calls themselves
        sys.stderr.write(f"graph capture failed ({exc}); timing call by call\n")
        torch.cuda.synchronize()
        launch_kind = "call by call (graph capture failed)"
        step_launch = lambda: sset.run(dev_layers, stream)
    for _ in range(max(3, args.warmup)):
        one_step(step_launch)
    barrier()
    sset.check()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    t_wall = time.perf_counter()
    evs = [one_step(step_launch) for _ in range(args.steps)]
    barrier()
    t_wall = time.perf_counter() - t_wall
    step_ms = [a.elapsed_time(b) for a, b in evs]
    clocks = sampler.stop() if rank == 0 else {}

    # ---- one pass call by call: per (layer, format) the library's events around its main kernels ----
    B.profile_enable(True)
    kern = dict(prepass=0.0, sweep1=0.0, sweep2=0.0, reduce1=0.0, reduce2=0.0, pool=0.0, lloyd=0.0, pack=0.0, norms=0.0)
    per_layer_sweep_ms = []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for row, (W, X) in zip(sset.sweeps, dev_layers):
        t_layer = 0.0
        for f, sw in enumerate(row):
            sw.run(W, X, stream, norms=(f == 0), reuse_prepass=(f > 0))
            s2, s1 = B.profile_ms(B.PROFILE_SWEEP, 0), B.profile_ms(B.PROFILE_SWEEP, 1)
            r2, r1 = B.profile_ms(B.PROFILE_REDUCE, 0), B.profile_ms(B.PROFILE_REDUCE, 1)
            kern["sweep2"] += s2
            kern["sweep1"] += s1
            kern["reduce2"] += r2
            kern["reduce1"] += r1
            kern["prepass"] += B.profile_ms(B.PROFILE_PREPASS, 1)
            kern["pool"] += B.profile_ms(B.PROFILE_POOL, 0)
            kern["lloyd"] += B.profile_ms(B.PROFILE_LLOYD, 0)
            kern["pack"] += B.profile_ms(B.PROFILE_PACK, 0)
            if f == 0:
                kern["norms"] += B.profile_ms(B.PROFILE_NORMS, 0)
            t_layer += s1 + s2 + r1 + r2
        per_layer_sweep_ms.append(t_layer)
    e1.record(stream)
    barrier()
    call_ms = e0.elapsed_time(e1)
    B.profile_enable(False)

    # ---- end to end through the streaming API with host buffers: every step copies the block's W and X from
    #      pinned host memory and reads every (layer, format)'s results (tables, result block, codes, scale
    #      words, distortion trace) back; the copies overlap the sweeps of the neighbouring layers ----
    host_layers = [(L.W.cpu().pin_memory(), L.X.cpu().pin_memory()) for L in layers]
    streams = (torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev))
    ls_of, order = {}, []
    for row, shape in zip(sset.sweeps, shapes):
        if shape not in ls_of:
            ls_of[shape] = LayerStream(row, streams, graphs=True)
        order.append(ls_of[shape])
    h2d = sum(ls.h2d_bytes for ls in order)
    d2h = sum(ls.d2h_bytes for ls in order)
    count = {id(ls): 0 for ls in order}

    def e2e_step():
        for ls, (Wh, Xh) in zip(order, host_layers):
            i = count[id(ls)]
            ls.submit(i, Wh, Xh)
            if i:
                ls.collect(i - 1)
            count[id(ls)] = i + 1
    for _ in range(2):
        e2e_step()
    for ls in set(order):
        ls.collect(count[id(ls)] - 1)
    barrier()
    e2e_steps = max(2, min(args.steps, 10))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(streams[0])
    for _ in range(e2e_steps):
        e2e_step()
    for ls in set(order):
        ls.collect(count[id(ls)] - 1)
    e1.record(streams[2])
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    del order, ls_of, host_layers

    ms = sum(step_ms) / len(step_ms)
    job_value = pipeline.job_throughput(units, ms * 1e-3) / 1e9   # all ranks' element-formats / slowest rank's time
    red = reduce_times(dict(kern, _ms=ms, _e2e_ms=e2e_ms, _call_ms=call_ms), dev, world)      # the slowest rank's, each
    ms, e2e_ms, call_ms = red.pop("_ms"), red.pop("_e2e_ms"), red.pop("_call_ms")
    kern = red
    if rank == 0:
        peaks = {}
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except OSError:
            pass
        sm_max = peaks.get("sm_max_mhz", 1965.0)
        alu_peak = SM_COUNT * SCHEDULERS * LANES * sm_max * 1e6 / 1e12          # T thread-instructions/s
        hbm_peak = peaks.get("hbm_gbs", 6650.0)
        of = "measured" if peaks else "fallback"
        n_lut, nb = len(sset.sweeps[0][0].full_atoms), 4
        n_dd = 2
        signed = [bool(f.sign_bits) for f in fmts]
        ops_n_step = search_ops_n_step(n_lut, nb, 0)
        ops_cell = sum(search_ops_cell_lookup(n_lut, nb, 0, n_dd, s) for s in signed) / S
        n_pass = len(shapes) * S                                        # (layer, format) passes of a step
        sweep_t = (kern["sweep1"] + kern["sweep2"]) * 1e-3              # the 2 n_pass launches of the evaluation kernel
        reduce_t = (kern["reduce1"] + kern["reduce2"]) * 1e-3           # the 2 n_pass launches of the reduction kernel
        search_t = sweep_t + reduce_t
        # the evaluation kernel by itself: its own share of the operation count
        ops_sweep = sweep_kernel_ops_n_step(n_lut - n_dd, nb, 0) + sweep_kernel_ops_n_step(n_dd, nb, 0)
        ach_sweep = ops_sweep * units / sweep_t / 1e12
        ach = ops_n_step * units / search_t / 1e12
        ach_cell = ops_cell * units / search_t / 1e12
        alg_bytes = search_bytes(n_lut, n_dd)
        sweep_bytes = 2 * 2.0 + 8.0 * n_lut / 16.0                       # W by each launch, every column written once
        bpe = [NCU_SWEEP_TRAFFIC["bytes_per_element_fixed_candidates"], NCU_SWEEP_TRAFFIC["bytes_per_element_dd_columns"]]
        traffic = None if None in bpe else (bpe[0] + bpe[1]) / 2.0 * units / n_pass
        rbpe = [NCU_REDUCE_TRAFFIC["bytes_per_element_fixed_candidates"], NCU_REDUCE_TRAFFIC["bytes_per_element_dd_columns"]]
        roofline = dict(
            kernel="sweep_kernel", launches_per_step=2 * n_pass, bound="alu", achieved=ach_sweep, peak=alu_peak, unit="T thread-instr/s",
            frac=ach_sweep / alu_peak, traffic=traffic, traffic_source=NCU_SWEEP_TRAFFIC["source"],
            peak_source=f"{SM_COUNT} SMs x {SCHEDULERS} schedulers x {LANES} lanes x {sm_max:.0f} MHz (clocks.max.sm, {of})",
            avg_launch_ms=sweep_t * 1e3 / (2 * n_pass),
            ops_per_element=dict(fixed_candidates=sweep_kernel_ops_n_step(n_lut - n_dd, nb, 0), dd_columns=sweep_kernel_ops_n_step(n_dd, nb, 0)),
            algorithmic_bytes_per_launch=sweep_bytes / 2.0 * units / n_pass,
            note="the dominant kernel of the step: the evaluation of every candidate on every block (two launches per layer and "
                 "format: the fixed candidates, then the DD columns), against its own share of the n-step operation count; "
                 "`search` below is the whole search (evaluation + reduction of the table entries) against the whole count",
            search=dict(
                kernels=["sweep_kernel", "reduce_kernel"], launches_per_step=4 * n_pass, ms_per_step=search_t * 1e3,
                n_step_search=dict(ops_per_element=ops_n_step, achieved=ach, frac=ach / alu_peak,
                                   note="operation count of an n-step nearest-entry search: 6 shared, 2n + 5 per LUT candidate and "
                                        "element, per block 6 per candidate and 2 per pair of candidates (diagonal included)"),
                cell_lookup=dict(ops_per_element=ops_cell, achieved=ach_cell, frac=ach_cell / alu_peak,
                                 note="operation count of this library's own scheme: one-step cell lookup (4) and packed multiply-adds "
                                      "(2.5) per LUT candidate and element, W unpacked in both launches, loaded columns, signed entries"),
                reduce_kernel=dict(ms_per_step=reduce_t * 1e3, avg_launch_ms=reduce_t * 1e3 / (2 * n_pass),
                                   traffic=None if None in rbpe else (rbpe[0] + rbpe[1]) / 2.0 * units / n_pass,
                                   traffic_source=NCU_REDUCE_TRAFFIC["source"],
                                   algorithmic_bytes_per_launch=(8.0 * (n_lut - n_dd) + 8.0 * n_lut) / 16.0 / 2.0 * units / n_pass,
                                   hbm=dict(achieved=(8.0 * (n_lut - n_dd) + 8.0 * n_lut) / 16.0 * units / reduce_t / 1e9, peak=hbm_peak,
                                            unit="GB/s", frac=(8.0 * (n_lut - n_dd) + 8.0 * n_lut) / 16.0 * units / reduce_t / 1e9 / hbm_peak, of=of)),
                bytes_per_element=dict(algorithmic=alg_bytes, w_twice=4.0, over_w_twice=alg_bytes / 4.0),
                hbm=dict(achieved=alg_bytes * units / search_t / 1e9, peak=hbm_peak, unit="GB/s",
                         frac=alg_bytes * units / search_t / 1e9 / hbm_peak, of=of,
                         note="algorithmic bytes of the search (W twice, every column written once and read by the reductions) over "
                              "its time: the search is far from the HBM roofline")))
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        try:
            per_config = per_config_table(dev, alu_peak, flush) if world == 1 and not small else None
        except Exception as exc:                               # the headline line does not depend on the side table
            per_config = dict(error=repr(exc))
        if per_config is not None and "error" not in per_config:
            per_config["config5"] = dict(elements_times_formats=units, whole_path=dict(value=units / ms / 1e6, unit=UNIT, ms=ms),
                                         sweep_only=dict(value=units / (search_t * 1e3) / 1e6, unit=UNIT, ms=search_t * 1e3),
                                         ops_per_element_n_step=ops_n_step, frac_of_alu_peak=ach / alu_peak,
                                         note="the headline workload: block 0, five layers, eight scale formats")
        try:
            sparse = sparse_streams_table(dev, hbm_peak, of, flush) if world == 1 else None
            if sparse is not None and not small:
                # the whole block with both streams on: the outlier stream once per layer, the correction per (layer, format)
                sset2 = LayerSetSweep(shapes, fmts, WORKLOAD["rom"], WORKLOAD["fp"], WORKLOAD["lloyd_iters"], device=dev,
                                      opq_q=0.92, wr_sigma=0.001)
                for _ in range(2):
                    sset2.run(dev_layers, stream)
                torch.cuda.synchronize(dev)
                ts = []
                for _ in range(3):
                    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a0.record(stream)
                    sset2.run(dev_layers, stream)
                    a1.record(stream)
                    torch.cuda.synchronize(dev)
                    ts.append(a0.elapsed_time(a1))
                sset2.check()
                sparse["block"] = dict(ms_per_step=sorted(ts)[1], value=units / sorted(ts)[1] / 1e6, unit=UNIT,
                                       note="the headline workload with both streams on (outlier quantile 0.92, correction sparsity "
                                            "0.001), launched call by call; compare with kernels_ms.ms_per_step_call_by_call")
                del sset2
        except Exception as exc:
            sparse = dict(error=repr(exc))
        cpu_rows = 1536
        cpu_val, cpu_dt = cpu_oracle_time(cpu_rows)
        line = dict(
            metric=METRIC, value=job_value, unit=UNIT, n_gpus=world, steps=args.steps,
            warmup=max(3, args.warmup), ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None,
            dtype="f32", data="synthetic",
            config=dict(WORKLOAD if not small else dict(WORKLOAD, workload="profiling case of config5: its first layer (8192x8192) at E5M6 only",
                                                        layers=layer_names, scale_formats=fmt_names),
                        block=f"rank r sweeps block r (seed 0)", elements_per_step=E, element_formats_per_step=units,
                        l2=("inputs larger than L2: 1.1 GB of W per step, every layer above 126 MB except the two 1024x8192 ones; "
                            "a layer's eight formats run back to back, as in a real sweep, so its W may be served from L2 there")
                        if not small else "W (134 MB) and the per-block columns (335 MB) are larger than L2",
                        launch=launch_kind, parallelism=f"layer-parallel x{world}, no collective"),
            kernels_ms=dict(kern, ms_per_step_call_by_call=call_ms, search_ms_per_layer=dict(zip(layer_names, per_layer_sweep_ms)),
                            note="sums over the (layer, format) passes of one step launched call by call, CUDA events recorded by the "
                                 "library around its main kernels; sweep1 / reduce1 = the fixed candidates' columns and the table "
                                 "entries among them (finds FMTa), sweep2 / reduce2 = the DD columns and their entries, lloyd = the "
                                 "iteration launches only, norms once per layer"),
            sweep_only=dict(value=world * units / search_t / 1e9, unit=UNIT,
                            note="element-formats / time of the search launches of a step (every candidate, every pair: evaluation "
                                 "and reduction kernels)"),
            roofline=roofline, per_config=per_config, sparse_streams=sparse,
            cpu_baseline=dict(value=cpu_val, unit=UNIT, cores=1, kind="oracle",
                              sample=f"first {cpu_rows} of 8192 rows of the 8192x8192 layer at E5M6 (one layer, one format), whole "
                                     f"pipeline, {cpu_dt:.1f} s"),
            e2e=dict(value=world * units / (e2e_ms * 1e-3) / 1e9, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                     ms_per_step=e2e_ms, steps=e2e_steps),
            gpu_launches=sset.kernel_launches_per_step * args.steps, clocks=clocks, wall_s=t_wall)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="block", choices=["block", "layer"],
                    help="block: the benchmark (one transformer block, eight scale formats); layer: its first layer at one format, for profiler captures")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
