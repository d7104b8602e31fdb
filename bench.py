#!/usr/bin/env python
"""Benchmark of the SOP per-layer candidate sweep on B200.

One step = one pass of the whole hot path over one synthetic layer: channel norms, sweep of every fixed
candidate (single-candidate reduction: finds FMTa), DD4 Lloyd refinement, sweep of the two DD4 columns
with the fixed candidates' per-block values loaded (all pairs), pack of the chosen pair.
Workload at every N: the attention-projection configuration (W 4096 x 4096 bf16 with 1 % outlier
channels, X 512 x 4096, E5M6 scale, NF4/SH4/BOF4/Split87/DD4 and negations plus E2M3/E4M3 singles).
With N > 1 every rank sweeps its own layer (layers are independent: no data-path collective).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

Prints ONE JSON line (rank 0).  ``--impl reference`` times the CPU oracle on a bounded sample.
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
WORKLOAD = dict(workload="config2: attention projection 4096x4096 bf16, 1% outlier channels x20, X 512x4096, "
                         "E5M6 scale, NF4/SH4/BOF4/Split87/DD4(8 Lloyd iters) + negations + E2M3/E4M3, all pairs",
                M=4096, K=4096, T=512, scale_format="E5M6", rom=["NF4", "SH4", "BOF4", "Split87"], fp=["E2M3", "E4M3"],
                lloyd_iters=8, g=16)
SM_COUNT, SCHEDULERS, LANES = 148, 4, 32


def sweep_ops_per_element(n_lut: int, n_bits: int, n_fp: int, n_loaded: int, n_slots2: int, n_slots4: int) -> float:
    """Algorithmic thread-level operations per weight element of one sweep launch: 6 shared (unpack,
    absmax, c w, norm, u), 2n + 5 per evaluated LUT candidate (n-step search + reconstruct + 4 fused
    multiply-adds), 12 per evaluated FP candidate, and per block: 6 per evaluated candidate (sqrt,
    divide, products), 2 per loaded candidate, 2 per two-way table entry and 6 per four-way entry."""
    n_eval = n_lut + n_fp
    return 6 + n_lut * (2 * n_bits + 5) + n_fp * 12 + (6 * n_eval + 2 * n_loaded + 2 * n_slots2 + 6 * n_slots4) / 16.0


# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture of the sweep kernel on this
# workload (cold cache; see the summary under profiles/); average over the two launches of one step
NCU_TRAFFIC_BYTES = dict(sweep_kernel=93.1e6)


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
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for nm, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def make_layer(seed: int):
    from paper_2605_14929_b200 import inputs as I
    return I.config2(seed, WORKLOAD["M"], WORKLOAD["K"], WORKLOAD["T"])


def cpu_oracle_time(rows: int, seed: int = 0):
    """Times the oracle pipeline, as it stands, on the first ``rows`` rows of the workload's layer."""
    from paper_2605_14929_b200 import inputs as I
    from tests import oracle_pipeline
    L = make_layer(seed)
    sub = I.Layer(L.W[:rows].contiguous(), L.X)
    t0 = time.perf_counter()
    oracle_pipeline.run(sub, I.scale_format(WORKLOAD["scale_format"]), WORKLOAD["rom"], WORKLOAD["fp"], WORKLOAD["lloyd_iters"])
    dt = time.perf_counter() - t0
    return rows * WORKLOAD["K"] / dt / 1e9, dt


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows = 128
    for _ in range(args.warmup):
        cpu_oracle_time(64)
    times = []
    for _ in range(args.steps):
        _, dt = cpu_oracle_time(rows)
        times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = rows * WORKLOAD["K"] / (ms * 1e-3) / 1e9
    sample = f"first {rows} of {WORKLOAD['M']} rows per step, full alphabet and pipeline, single thread"
    print(json.dumps(dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                          warmup=args.warmup, ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None,
                          dtype="f32", data="synthetic", config=WORKLOAD,
                          cpu_baseline=dict(value=value, unit=UNIT, cores=1, kind="oracle", sample=sample),
                          e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))))


def run_gpu(args) -> None:
    import torch
    import torch.distributed as dist
    from paper_2605_14929_b200 import binding as B, inputs as I
    from paper_2605_14929_b200.pipeline import LayerSweep

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
    B.lib()

    M, K, T = WORKLOAD["M"], WORKLOAD["K"], WORKLOAD["T"]
    fmt = I.scale_format(WORKLOAD["scale_format"])
    L = make_layer(rank)                                  # every rank sweeps its own layer
    Wh, Xh = L.W.pin_memory(), L.X.pin_memory()
    Wd, Xd = Wh.to(dev), Xh.to(dev)
    sw = LayerSweep(M, K, T, fmt, WORKLOAD["rom"], WORKLOAD["fp"], WORKLOAD["lloyd_iters"], device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # > L2 (126 MB)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def one_step(launch):
        flush.fill_(1)                                    # evict W / X from L2 between timed steps
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        launch()
        e1.record(stream)
        return e0, e1

    # The timed steps replay the layer's calls as one CUDA graph (what a job that sweeps many layers of one shape
    # does).  A replayed graph gives no per-kernel events, so the same number of steps is then run call by call
    # with the library's events around its main kernels: those times feed the roofline object.
    launch_kind = "one CUDA graph replay per step"
    step_launch = sw.replay
    try:
        sw.capture(Wd, Xd)
    except RuntimeError as exc:                           # no graph capture here: time the calls themselves
        sys.stderr.write(f"graph capture failed ({exc}); timing call by call\n")
        torch.cuda.synchronize()
        launch_kind = "call by call (graph capture failed)"
        step_launch = lambda: sw.run(Wd, Xd, stream)
    for _ in range(max(3, args.warmup)):
        one_step(step_launch)
    barrier()
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

    B.profile_enable(True)
    kern = dict(sweep1=[], sweep2=[], lloyd=[], pack=[], norms=[])
    evs2 = []
    for _ in range(args.steps):
        evs2.append(one_step(lambda: sw.run(Wd, Xd, stream)))
        # the library's own events around its main kernels, on the launching stream (waits for this step)
        kern["sweep2"].append(B.profile_ms(B.PROFILE_SWEEP, 0))
        kern["sweep1"].append(B.profile_ms(B.PROFILE_SWEEP, 1))
        kern["lloyd"].append(B.profile_ms(B.PROFILE_LLOYD, 0))
        kern["pack"].append(B.profile_ms(B.PROFILE_PACK, 0))
        kern["norms"].append(B.profile_ms(B.PROFILE_NORMS, 0))
    barrier()
    call_ms = sum(a.elapsed_time(b) for a, b in evs2) / len(evs2)
    clocks = sampler.stop() if rank == 0 else {}
    B.profile_enable(False)

    # ---- end to end through the public API with host buffers: H2D of W and X, the path, D2H of the results ----
    # end to end through the streaming API: every step copies its W and X from pinned host memory and reads its
    # results (tables, result block, codes, scale words) back; copies of neighbouring steps overlap the sweep
    from paper_2605_14929_b200.pipeline import LayerStream
    ls = LayerStream(sw)
    ls.before_run = lambda: flush.fill_(1)          # same L2 eviction as the device-resident timing
    h2d, d2h = ls.h2d_bytes, ls.d2h_bytes
    for i in range(3):
        ls.submit(i, Wh, Xh)
    ls.collect(2)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(ls.s_in)
    for i in range(args.steps):
        ls.submit(i, Wh, Xh)
        if i:
            ls.collect(i - 1)
    ls.collect(args.steps - 1)
    e1.record(ls.s_out)
    barrier()
    e2e_ms = e0.elapsed_time(e1) / args.steps

    ms = sum(step_ms) / len(step_ms)
    from paper_2605_14929_b200 import pipeline
    job_value = pipeline.job_throughput(float(M * K), ms * 1e-3) / 1e9   # all ranks' elements / slowest rank's time
    kavg = {k: sum(v) / len(v) for k, v in kern.items()}
    knames = sorted(kavg)
    t = torch.tensor([ms, e2e_ms] + [kavg[k] for k in knames], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    vals = [float(x) for x in t.cpu()]
    ms, e2e_ms = vals[0], vals[1]
    kavg = dict(zip(knames, vals[2:]))
    E = M * K
    if rank == 0:
        peaks = {}
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except OSError:
            pass
        full = sw.full_atoms
        nb = full[0].n_bits
        n_lut = sum(a.kind == I.KIND_LUT for a in full)
        n_fp = len(full) - n_lut
        n_dd = bin(sw.dd_mask).count("1")
        n_base = (n_lut // 2) if fmt.sign_bits else 0
        slots2 = len(full) + n_lut * (n_lut - 1) // 2
        slots4 = n_base * (n_base + 1) // 2
        ops1 = sweep_ops_per_element(n_lut - n_dd, nb, n_fp, 0, len(full) - n_dd, 0)      # fixed candidates, singles only
        ops2 = sweep_ops_per_element(n_dd, nb, 0, len(full) - n_dd, slots2, slots4)       # DD columns, every pair
        sm_max = peaks.get("sm_max_mhz", 1965.0)
        alu_peak = SM_COUNT * SCHEDULERS * LANES * sm_max * 1e6 / 1e12          # T thread-instructions/s
        hbm_peak = peaks.get("hbm_gbs", 6650.0)
        of = "measured" if peaks else "fallback"
        # sweep kernel: two launches per step; achieved = algorithmic ops of both / time of both
        sweep_t = (kavg["sweep1"] + kavg["sweep2"]) * 1e-3
        sweep_ach = (ops1 + ops2) * E / sweep_t / 1e12
        sweep_roof = dict(kernel="sweep_kernel", launches_per_step=2, bound="alu", achieved=sweep_ach, peak=alu_peak,
                          unit="T thread-instr/s", frac=sweep_ach / alu_peak,
                          traffic=NCU_TRAFFIC_BYTES["sweep_kernel"] if (M, K) == (4096, 4096) else None,
                          peak_source=f"{SM_COUNT} SMs x {SCHEDULERS} schedulers x {LANES} lanes x {sm_max:.0f} MHz (clocks.max.sm, {of})",
                          ops_per_element=dict(fixed_candidates_singles=ops1, dd_columns_all_pairs=ops2),
                          avg_launch_ms=sweep_t * 1e3 / 2,
                          hbm=dict(achieved=2 * 2.0 * E / sweep_t / 1e9, peak=hbm_peak, unit="GB/s",
                                   frac=2 * 2.0 * E / sweep_t / 1e9 / hbm_peak, of=of,
                                   note="W read once per launch; the kernel is far from the HBM roofline"))
        # the Lloyd iterations walk only the pool elements in cells that hold a decision threshold (a few per
        # cent of the pool), so their launches are bound by launch and dependency latency, not by a roofline
        dominant = sweep_roof
        cpu_rows = 1024
        cpu_val, cpu_dt = cpu_oracle_time(cpu_rows)
        line = dict(
            metric=METRIC, value=job_value, unit=UNIT, n_gpus=world, steps=args.steps,
            warmup=max(3, args.warmup), ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None,
            dtype="f32", data="synthetic", config=dict(WORKLOAD, l2="flushed between timed steps (256 MB write)", launch=launch_kind,
                                                       parallelism=f"layer-parallel x{world}, no collective"),
            kernels_ms=dict(kavg, ms_per_step_call_by_call=call_ms,
                            note="per step of a second pass of the same number of steps launched call by call (a replayed graph "
                                 "gives no per-kernel events), CUDA events recorded by the library around its main kernels; "
                                       "sweep1 = fixed candidates (singles), sweep2 = DD columns (all pairs), "
                                       "lloyd = all Lloyd iterations (one cooperative launch where the grid fits)"),
            sweep_only=dict(value=world * E / sweep_t / 1e9, unit=UNIT,
                            note="elements / time of the two sweep launches of a step (every candidate, every pair)"),
            roofline=dominant,
            cpu_baseline=dict(value=cpu_val, unit=UNIT, cores=1, kind="oracle",
                              sample=f"first {cpu_rows} of {M} rows, whole pipeline, {cpu_dt:.1f} s"),
            e2e=dict(value=world * E / (e2e_ms * 1e-3) / 1e9, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                     ms_per_step=e2e_ms),
            gpu_launches=sw.kernel_launches_per_step * args.steps, clocks=clocks, wall_s=t_wall)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
