#!/usr/bin/env python
"""Benchmark of the tANS decode + dequantise path on B200.

One step = one pass of the whole hot path (stage tables, read compressed streams, decode,
dequantise, store) over one synthetic workload, as ONE batched kernel launch.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload large|resnet50|resnet18|conv3x3|sweep]
                  [--layout private|interleaved|quads|strips] [--lanes 32|64|128|256] [--impl ours|reference]
                  [--no-settled | --no-idle] [--no-variants] [--no-fused] [--fused-only]

Prints one JSON line (rank 0).  With --impl reference the CPU oracle is timed instead.

The timed launches are queued back to back and rotate over at least two full sets of buffers; the
layer descriptors say that the inputs were settled before the timing began and that a launch does not
touch the output set of the launch before it (ANS_DESC_INPUTS_SETTLED | ANS_DESC_OUTPUT_IDLE), so
consecutive launches may overlap at their ends and the per-launch time is the rate of a stream of
decode calls.  --no-idle keeps the first flag only (a launch waits for the one before it before its
first write), --no-settled neither (it waits before it reads anything); the line also carries the
headline workload timed without the flags, and a launch bracketed alone by its own pair of events.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synthgen as sg  # noqa: E402

METRIC = "decoded weights/sec and achieved HBM GB/s (fraction of B200 peak), 1 GPU"
NOMINAL_PEAK_GBS = 8000.0
FALLBACK_PEAK_GBS = 6650.0


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the 8 matrices, from the 2-matrix capture in
# profiles/ans_decode_kernel_quads_large.md: reads scale with the matrices (4 x 25.20 MB); writes are the
# output (1073.74 MB) less what is still in L2 when the kernel ends, which the capture shows as
# 268.44 - 217.17 = 51.27 MB (40-51 MB from capture to capture, whatever the size)
NCU_TRAFFIC = {("large", "quads", 32, 8, 8192, 0, 0): 4 * 25.20e6 + 1073.74e6 - 51.27e6}      # 256-state table (the default)


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_PEAK_GBS, "fallback"


def make_specs(args):
    if args.workload == "sweep":
        return sg.workload_sweep(table_log=args.table_log or 12, chunk=args.chunk or 16384, n=args.symbols)
    if args.workload == "large":
        return sg.workload_large(n_mats=args.mats, dim=args.dim, chunk=args.chunk or 32768,
                                 table_log=args.table_log or 8)
    if args.workload in ("resnet18", "resnet50"):
        return sg.WORKLOADS[args.workload](table_log=args.table_log or 8, chunk=args.chunk or 16384)
    return sg.workload_conv3x3()


WORKLOAD_TEXT = {
    "conv3x3": "single 3x3 conv 64->64 (36,864 weights), 4-bit zero-point, 12-bit table, 4096-symbol chunks, fp32",
    "resnet18": "ResNet-18 conv weights (20 layers, 11.2M), bitwidth {2,3,4,6}, 0.8-1.5 bit/weight, 16K chunks, bf16 "
                "(256-state tables unless --table-log says otherwise)",
    "resnet50": "ResNet-50 conv weights (53 layers, 23.5M), 1-8 bit mixed precision, P(zp) 0.85-0.95, 16K chunks, bf16 "
                "(256-state tables unless --table-log says otherwise)",
    "sweep": "256M 8-bit symbols, two-sided geometric (2.5 bit), decode-only to uint8",
    "large": "large dense layers: 8 matrices of 8192x8192 (537M weights), 3-bit zero-point, P(zp)=0.7, 32K chunks, bf16 "
             "(256-state table, the paper's coder size, unless --table-log says otherwise)",
}


# the container and lanes per chunk each workload is timed on unless --layout / --lanes say otherwise: the
# fastest measured (quads: one symbol per look-up, lanes in step; strips: a look-up may stand for a run of the
# dominant symbol, which pays when one symbol owns most of the states, as in the ResNet-50 workload)
DEFAULTS = {"large": ("quads", 32), "resnet18": ("strips", 64), "resnet50": ("strips", 32), "sweep": ("quads", 32),
            "conv3x3": ("quads", 32)}


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None
        self.first, self.last = 0, None                       # rows taken while the timed rounds ran

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "20"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
            t_end = time.perf_counter() + 5.0               # be sampling before the warm-up starts
            while not self.rows and time.perf_counter() < t_end:
                time.sleep(0.01)
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass

    def summary(self):
        """Median SM clock and the throttle reasons seen in rows [first, last): the samples taken
        while the timed rounds ran."""
        rows = self.rows[self.first:self.last]
        sm = [float(r[1]) for r in rows if len(r) >= 9 and r[1].replace(".", "").isdigit()]
        mx = [float(r[2]) for r in rows if len(r) >= 9 and r[2].replace(".", "").isdigit()]
        reasons = set()
        for r in rows:
            if len(r) < 9:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples_in_timed_region": len(sm)}


def cpu_baseline(specs, syms, layout_name, args_lanes=32):
    """The CPU oracle, as it stands, decoding + dequantising a bounded sample of the same
    workload on this host's cores: single thread and all cores."""
    import oracle
    layout = {"private": oracle.PRIVATE, "interleaved": oracle.INTERLEAVED, "quads": oracle.QUADS,
              "strips": oracle.STRIPS}[layout_name]
    cores = os.cpu_count() or 1
    target = 48_000_000                         # symbols in the sample (about 10-30 s of CPU work in all)
    sample, total = [], 0
    for spec, sym in zip(specs, syms):
        take = min(sym.size, max(0, target - total))
        take -= take % spec.chunk_symbols if take > spec.chunk_symbols else 0
        if take <= 0:
            break
        s = sym[:take]
        f = oracle.normalize_freqs(oracle.histogram(s), spec.alphabet, spec.table_log)
        T = oracle.Table(f, spec.table_log)
        sample.append((spec, T, oracle.pack(T, s, spec.chunk_symbols, args_lanes // 32, layout)))
        total += take

    def run(threads):
        best = float("inf")
        for _ in range(3):
            t0 = time.perf_counter()
            for spec, T, P in sample:
                out, rc = oracle.unpack(T, P, threads=threads)
                assert rc == 0
                oracle.dequant(out, spec.zero_point, spec.scale, spec.out_dtype, threads=threads)
            best = min(best, time.perf_counter() - t0)
        return total / best

    one = run(1)
    many = run(cores) if cores > 1 else one
    return {"value": many, "unit": "weights/s", "cores": cores, "kind": "oracle",
            "single_thread_value": one,
            "sample": f"first {total} weights of the workload ({len(sample)} layer(s)), {layout_name} container, "
                      f"decode + dequant, best of 3"}


def run_reference(args):
    """--impl reference: the CPU oracle timed on the host cores, bounded sample per step."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    specs = make_specs(args)
    layout = {"private": oracle.PRIVATE, "interleaved": oracle.INTERLEAVED, "quads": oracle.QUADS,
              "strips": oracle.STRIPS}[args.layout]
    cores = os.cpu_count() or 1
    args_lanes = args.lanes
    target = 24_000_000
    sample, total = [], 0
    for spec in specs:
        take = min(spec.n, max(0, target - total))
        if take <= 0:
            break
        sub = sg.LayerSpec(spec.name, (take,), spec.bitwidth, spec.alphabet, spec.zero_point, spec.theta, spec.scale,
                           spec.table_log, spec.chunk_symbols, spec.out_dtype, spec.key)
        s = sg.draw_symbols(sub)
        T = oracle.Table(oracle.normalize_freqs(oracle.histogram(s), spec.alphabet, spec.table_log), spec.table_log)
        sample.append((spec, T, oracle.pack(T, s, spec.chunk_symbols, args_lanes // 32, layout)))
        total += take

    def step():
        for spec, T, P in sample:
            out, rc = oracle.unpack(T, P, threads=cores)
            assert rc == 0
            oracle.dequant(out, spec.zero_point, spec.scale, spec.out_dtype, threads=cores)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    value = total / dt
    sample_txt = f"first {total} weights of the workload per step, {args.layout} container, all {cores} cores"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "weights/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": specs[0].out_dtype if len({sp.out_dtype for sp in specs}) == 1 else "mixed", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[args.workload], "layout": args.layout, "sample": sample_txt},
        "cpu_baseline": {"value": value, "unit": "weights/s", "cores": cores, "kind": "oracle", "sample": sample_txt},
        "e2e": {"value": value, "unit": "weights/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def reduce_max(x: float, world: int) -> float:
    """Max over ranks (identity for one rank)."""
    if world <= 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device="cuda" if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


MIN_REGION_S = 0.5          # device time the timed rounds of a workload add up to, at least
LATER_ROUND = 100           # launches of every timed round after the first, at least


def time_workload(db, steps, warmup, n_sets, world, min_region_s=MIN_REGION_S, max_rounds=2000):
    """Rounds of K back-to-back launches, each round bracketed by CUDA events on the launching
    stream.  The host must not be what is timed, so every round goes behind a device-side spin of
    a few milliseconds (outside the brackets): by the time the device reaches the first launch all
    K are queued.  The first round is the K steps the command line asked for; further rounds (of
    at least LATER_ROUND launches each, so that a round's first and last launch, which overlap
    nothing, weigh little) repeat until the rounds add up to min_region_s of device time, so that
    clock samples fall inside the timed region.  A last round brackets every launch by itself.
    Returns (per-round milliseconds per step, per-launch milliseconds of the last round); the
    launches made are counted in time_workload.launches."""
    import torch
    import torch.distributed as dist
    st = torch.cuda.current_stream()
    time_workload.launches = warmup * db.launches_per_decode()
    for i in range(warmup):
        db.decode(i % n_sets)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    spin = int(2e7)                                       # cycles: about 10 ms

    def one_round(per_launch=False, n=steps):
        evs = []
        torch.cuda._sleep(spin)
        time_workload.launches += n * db.launches_per_decode()
        if per_launch:
            for i in range(steps):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(st)
                db.decode(i % n_sets)
                b.record(st)
                evs.append((a, b))
        else:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(st)
            for i in range(n):
                db.decode(i % n_sets)
            b.record(st)
            evs.append((a, b))
        return evs

    rounds, total_ms = [], 0.0
    while True:
        n = steps if not rounds else max(steps, LATER_ROUND)
        ev = one_round(n=n)
        torch.cuda.synchronize()
        ms = ev[0][0].elapsed_time(ev[0][1])
        rounds.append(ms / n)
        total_ms += ms
        if total_ms >= min_region_s * 1e3 or len(rounds) >= max_rounds:
            break
    pairs = one_round(per_launch=True)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    each = [a.elapsed_time(b) for a, b in pairs]
    assert db.read_status() == 0, "decoder flagged a stream"
    return rounds, each


LAYOUT_IDS = {"private": "ANS_LAYOUT_PRIVATE", "interleaved": "ANS_LAYOUT_INTERLEAVED", "quads": "ANS_LAYOUT_QUADS",
              "strips": "ANS_LAYOUT_STRIPS"}


def build_case(ans, args, workload, layout_name, lanes, table_log=0, chunk=0, local=0, by_channel=False, flags=3):
    """Draw the workload's symbols, pack them with the library's host packer, put everything on
    the device.  Returns (specs, syms, layers, db, n_sets, working-set text)."""
    import copy
    from concurrent.futures import ThreadPoolExecutor
    from paper_2406_06237_b200.runtime import DeviceBatch, pack_layer
    a2 = copy.copy(args)
    a2.workload, a2.table_log, a2.chunk = workload, table_log, chunk
    specs = make_specs(a2)
    layout = getattr(ans, LAYOUT_IDS[layout_name])
    cores = os.cpu_count() or 1
    if by_channel:
        # the paper's own grouping (Section III-B): one chunk per layer, one lane per input channel of the
        # tensor as stored (O x I x H x W), pieces of H * W symbols; layers whose input channels are no
        # multiple of 32 (the first conv, which the paper leaves uncompressed) are left out
        import dataclasses
        specs = [dataclasses.replace(sp, chunk_symbols=sp.n) for sp in specs
                 if len(sp.shape) == 4 and sp.shape[1] % 32 == 0 and sp.shape[1] <= 2048]
        layout = ans.ANS_LAYOUT_CHANNELS

    def prep(spec):
        sym = sg.draw_symbols(spec, threads=max(1, cores // 4))
        ln, piece = lanes, 1
        if by_channel:
            ln, piece = spec.shape[1], spec.shape[2] * spec.shape[3]
        pl = pack_layer(sym, spec.alphabet, spec.table_log, spec.chunk_symbols, ln, layout, spec.bitwidth,
                        spec.zero_point, spec.scale, ans.DTYPES[spec.out_dtype], n_threads=max(1, cores // 2),
                        piece_symbols=piece)
        return sym, pl

    with ThreadPoolExecutor(4) as ex:
        prepared = list(ex.map(prep, specs))
    syms = [p[0] for p in prepared]
    layers = [p[1] for p in prepared]
    out_bytes = sum(L.n_symbols * ans.ELEM_SIZE[L.out_dtype] for L in layers)
    # keep the working set out of L2 (126 MB): a big workload is larger than L2 by itself; a small
    # one exists in several full copies (compressed bytes, tables, outputs) and the timed launches
    # rotate over them, so that between two uses of a copy at least 3 x L2 bytes have gone by
    ws = out_bytes + sum(L.compressed_bytes() for L in layers)
    small = ws < (512 << 20)
    # (a big one in two, so that a launch never writes the buffers the launch before it writes)
    n_sets = min(64, max(2, -(-(512 << 20) // max(ws, 1)))) if small else 2
    # the tables and the compressed bytes are on the device before the first timed launch and never
    # change: the descriptors say so (ANS_DESC_INPUTS_SETTLED), which lets a strips launch fetch them
    # and begin while the launch before it drains; where the launches rotate over several output
    # sets, a launch writes a set that the launch before it does not touch (ANS_DESC_OUTPUT_IDLE)
    settled = bool(flags & 1) and not args.no_settled
    db = DeviceBatch(layers, f"cuda:{local}", n_out_sets=n_sets, inputs_settled=settled,
                     output_idle=bool(flags & 2) and n_sets >= 2 and settled and not args.no_idle)
    policy = (f"inputs larger than L2: launches rotate over {n_sets} full copies of the workload "
              f"({n_sets * ws / 2**20:.0f} MB in all)" if small
              else f"working set (compressed + output) is larger than L2; launches alternate between {n_sets} full copies")
    return specs, syms, layers, db, n_sets, policy


def figures(ans, layers, db, rounds, each, peak):
    """Throughput and roofline figures of one measured case."""
    n_w = db.n_symbols()
    out_bytes = sum(L.n_symbols * ans.ELEM_SIZE[L.out_dtype] for L in layers)
    # algorithmic bytes of one launch: everything compressed read once, each layer's table
    # once, every decoded element written once
    table_read = sum(4 << L.table_log for L in layers)
    comp_bytes = db.compressed_bytes()
    algo_bytes = comp_bytes + table_read + out_bytes
    kernel_ms = statistics.mean(rounds)                   # average launch duration over all timed rounds
    achieved = algo_bytes / (kernel_ms * 1e-3) / 1e9
    return {"n_w": n_w, "out_bytes": out_bytes, "comp_bytes": comp_bytes, "algo_bytes": algo_bytes,
            "kernel_ms": kernel_ms, "achieved": achieved, "frac": achieved / peak,
            "frac_nominal": achieved / NOMINAL_PEAK_GBS,
            "coded_bits": 8.0 * comp_bytes / max(1, n_w)}


def entropy_bits(specs, syms):
    ent = 0.0
    for spec, sym in zip(specs, syms):
        c = np.bincount(sym, minlength=256).astype(np.float64)
        p = c[c > 0] / max(1, sym.size)
        ent += float(-(p * np.log2(p)).sum()) * sym.size
    return ent


# (workload, container, lanes, table_log, chunk) measured beside the headline: the other table size
# quoted for the large layers, the two ResNets, one cell of the granularity sweep
# last field: the descriptor flags (3: ANS_DESC_INPUTS_SETTLED | ANS_DESC_OUTPUT_IDLE, 1: the first only,
# 0: none: every launch waits for the one before it); resnet50 is measured all three ways
VARIANTS = [("large", "quads", 32, 12, 0, 3), ("resnet50", "strips", 32, 0, 0, 3),
            ("resnet50", "strips", 64, 0, 0, 3), ("resnet50", "strips", 64, 0, 0, 1), ("resnet50", "strips", 64, 0, 0, 0),
            ("resnet50", "strips", 32, 0, 0, 0), ("resnet50", "quads", 32, 0, 0, 3),
            ("resnet50", "strips", 32, 12, 0, 3), ("resnet18", "strips", 64, 0, 0, 3),
            ("resnet18", "quads", 32, 0, 0, 3), ("sweep", "quads", 32, 12, 16384, 3)]


FUSED_COPIES = 12           # device copies of the compressed matrix the fused launches rotate over (> L2 in all)


def run_fused(ans, args, local, sampler=None, M=128, min_region_s=0.3):
    """Decode fused into its consumer (paper Section I, Section III-C): Y = X W^T for one matrix of
    the `large` workload (dim x dim, 256-state table, strips container in blocks of 64 x 64), M rows
    of X, against the same product taken in two steps (ans_decode_dequant to bf16, then
    torch.matmul).  Rounds of back-to-back calls behind a device-side spin, as for the decode
    workloads; the calls rotate over FUSED_COPIES copies of the compressed matrix so that it comes
    from DRAM."""
    import torch
    from paper_2406_06237_b200.runtime import DeviceBatch, gemm_block_order, pack_gemm_layer
    spec = sg.workload_large(n_mats=1, dim=args.dim, chunk=4096, table_log=8)[0]
    N = K = args.dim
    cores = os.cpu_count() or 1
    sym = sg.draw_symbols(spec, threads=max(1, cores // 4))
    pl = pack_gemm_layer(sym.reshape(N, K), spec.alphabet, 8, spec.bitwidth, spec.zero_point, spec.scale,
                         n_threads=max(1, cores // 2))
    db = DeviceBatch([pl] * FUSED_COPIES, f"cuda:{local}")
    x_full = torch.randn(M, K, device=f"cuda:{local}").to(torch.bfloat16)
    x = x_full
    y = torch.empty(M, N, dtype=torch.float32, device=f"cuda:{local}")
    st = torch.cuda.current_stream()
    descs = db.h_descs[0]
    outs = [db.output(i).view(N, K) for i in range(FUSED_COPIES)]

    def fused(i):
        ans.ans_decode_gemm_bf16(descs[i], x.data_ptr(), x.shape[0], N, K, y.data_ptr(), db.status.data_ptr(), st.cuda_stream)

    def two_steps(i):
        ans.ans_decode_dequant(descs[i], db.status.data_ptr(), st.cuda_stream)
        return torch.matmul(x, outs[i].t())

    def timed(fn, steps):
        for i in range(5):
            fn(i % FUSED_COPIES)
        torch.cuda.synchronize()
        rounds, total = [], 0.0
        while total < min_region_s * 1e3 and len(rounds) < 500:
            torch.cuda._sleep(int(2e7))
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(st)
            for i in range(steps):
                fn(i % FUSED_COPIES)
            b.record(st)
            torch.cuda.synchronize()
            ms = a.elapsed_time(b)
            rounds.append(ms / steps)
            total += ms
        return rounds

    if sampler:
        sampler.first = len(sampler.rows)
    steps = 4 * FUSED_COPIES
    rf = timed(fused, steps)
    rt = timed(two_steps, steps)
    if sampler:
        sampler.last = len(sampler.rows)
    assert db.read_status() == 0, "decoder flagged a stream"
    # agreement of the two routes on the last copy (W's blocks put back in row-major order)
    order = torch.from_numpy(gemm_block_order().ravel()).to(x.device)
    last = FUSED_COPIES - 1
    fused(last)
    w = db.output(last).view(N // 64, K // 64, 4096)[:, :, order].view(N // 64, K // 64, 64, 64).permute(0, 2, 1, 3)
    ref = x.float() @ w.reshape(N, K).float().t()
    err = float((y - ref).abs().max() / ref.abs().max())
    f_ms, t_ms = sum(rf) / len(rf), sum(rt) / len(rt)
    comp = pl.compressed_bytes()
    res = {"workload": f"Y = X W^T, X {M} x {K} bf16, W {N} x {K} compressed ({comp * 8 / (N * K):.3f} bit/weight, 256-state table)",
           "kernel": "ans_decode_gemm_wide_kernel (tcgen05.mma, fp32 accumulator in tensor memory)",
           "fused_ms_mean": f_ms, "decode_then_matmul_ms_mean": t_ms, "speedup_over_two_steps": t_ms / f_ms,
           "weights_per_s": N * K / (f_ms * 1e-3), "tensor_tflops": 2.0 * M * N * K / (f_ms * 1e-3) / 1e12,
           "dram_bytes_fused_algorithmic": comp + M * K * 2 + M * N * 4,
           "dram_bytes_two_steps_algorithmic": comp + 2 * (N * K * 2) + M * K * 2 + M * N * 2,
           "timed_rounds": [len(rf), len(rt)], "launches_per_round": steps,
           "max_rel_difference_between_the_routes": err,
           "l2_policy": f"calls rotate over {FUSED_COPIES} device copies of the compressed matrix "
                        f"({FUSED_COPIES * comp / 2**20:.0f} MB in all)",
           "bound": "the decode's instruction issue, as for the decode kernels (see profiles/); not the tensor cores",
           "clocks": sampler.summary() if sampler else None}
    launches = (len(rf) + len(rt)) * steps + 11
    # the same with 16 rows of X (the kernel then takes its form with the operands exchanged)
    x = x_full[:16].contiguous()
    r16f = timed(fused, steps)
    r16t = timed(two_steps, steps)
    assert db.read_status() == 0, "decoder flagged a stream"
    res["rows_16"] = {"fused_ms_mean": sum(r16f) / len(r16f), "decode_then_matmul_ms_mean": sum(r16t) / len(r16t),
                      "speedup_over_two_steps": (sum(r16t) / len(r16t)) / (sum(r16f) / len(r16f))}
    launches += (len(r16f) + len(r16t)) * steps + 10
    del db
    torch.cuda.empty_cache()
    return res, launches


def run_ours(args):
    import torch
    import paper_2406_06237_b200 as ans

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    ans.lib()                                           # fail loudly if the library is missing

    t_setup = time.perf_counter()
    by_channel = args.grouping == "channel"
    if by_channel:
        args.no_cpu_baseline = args.no_e2e = True
    specs, syms, layers, db, n_sets, policy = build_case(ans, args, args.workload, args.layout, args.lanes,
                                                         args.table_log, args.chunk, local, by_channel)
    setup_s = time.perf_counter() - t_setup

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    peak, peak_kind = measured_peak()
    sampler.first = len(sampler.rows)
    rounds, each = time_workload(db, args.steps, args.warmup, n_sets, world)
    launches = time_workload.launches
    sampler.last = len(sampler.rows)
    db_flags = db.h_descs[0][0].flags if layers else 0
    clocks = sampler.summary() if rank == 0 else None
    # the same launches with the descriptor flags cleared: every launch waits for the one before it
    waiting_ms = None
    if db_flags and world == 1:
        db.set_flags(0)
        wr, _ = time_workload(db, args.steps, 3, n_sets, world, min_region_s=0.15)
        launches += time_workload.launches + 3
        waiting_ms = sum(wr) / len(wr)
        db.set_flags(int(db_flags))
    ms_per_step = reduce_max(rounds[0], world)          # the K steps asked for: the first round
    fg = figures(ans, layers, db, rounds, each, peak)
    n_w = fg["n_w"]
    value = world * n_w / (ms_per_step * 1e-3)

    kname = "ans_decode_strips_kernel" if args.layout == "strips" else f"ans_decode_kernel<{args.layout}>"
    # DRAM bytes per launch from an ncu capture of this kernel (see profiles/), only for the
    # configuration that capture covers; None otherwise
    traffic = NCU_TRAFFIC.get((args.workload, args.layout, args.lanes, args.mats, args.dim, args.chunk, args.table_log))
    roofline = {"bound": "hbm", "achieved": fg["achieved"], "peak": peak, "unit": "GB/s", "frac": fg["frac"],
                "traffic": traffic, "kernel": kname, "peak_kind": f"of {peak_kind}",
                "algorithmic_bytes_per_launch": fg["algo_bytes"], "kernel_ms_mean": fg["kernel_ms"],
                "timed_rounds": len(rounds), "launches_per_round": [args.steps, max(args.steps, LATER_ROUND)],
                "round_ms_per_launch_min": min(rounds), "round_ms_per_launch_max": max(rounds),
                "launch_bracketed_alone_ms_median": statistics.median(each), "launch_bracketed_alone_ms_min": min(each),
                "frac_of_nominal_8TBs": fg["frac_nominal"],
                "kernel_ms_mean_launches_waiting": waiting_ms,
                "frac_launches_waiting": (fg["frac"] * fg["kernel_ms"] / waiting_ms) if waiting_ms else None,
                "note": "kernel_ms_mean: CUDA events around rounds of back-to-back launches, divided by the launches "
                        "(gaps between launches included; the descriptors carry the flags in config.desc_flags, so a launch may "
                        "begin while the one before it drains; *_launches_waiting: the same with the flags cleared); HBM is the metric's roofline, the kernels themselves are "
                        "held by instruction issue and shared-memory wavefronts (see profiles/)"}

    # end to end through the host-buffer entry point: pinned host buffers in, pinned out
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(ans, db, layers, args, world)
    ent_bits = entropy_bits(specs, syms)
    cpu = cpu_baseline(specs, syms, args.layout, args.lanes) if world == 1 and rank == 0 and not args.no_cpu_baseline else None
    head_specs = specs

    # the other workloads and table sizes, each measured the same way (shorter regions)
    variants = []
    if args.workload == "large" and not args.table_log and not args.chunk and world == 1 and not args.no_variants \
            and args.mats == 8 and args.dim == 8192:
        del db
        torch.cuda.empty_cache()
        for wl, lay, ln, tl, ck, vflag in VARIANTS:
            vs, vy, vl, vdb, vsets, vpol = build_case(ans, args, wl, lay, ln, tl, ck, local, flags=vflag)
            sampler.first = len(sampler.rows)
            vr, ve = time_workload(vdb, min(args.steps, 200) if wl in ("large", "sweep") else max(args.steps, 100), 5, vsets, 1,
                                   min_region_s=0.3)
            sampler.last = len(sampler.rows)
            vf = figures(ans, vl, vdb, vr, ve, peak)
            variants.append({"workload": wl, "layout": lay, "lanes": ln, "table_log": vl[0].table_log,
                             "chunk_symbols": vl[0].chunk_symbols, "weights": vf["n_w"], "out_dtype": vs[0].out_dtype,
                             "kernel_ms_mean": vf["kernel_ms"], "timed_rounds": len(vr),
                             "launch_bracketed_alone_ms_median": statistics.median(ve),
                             "value": vf["n_w"] / (vf["kernel_ms"] * 1e-3), "unit": "weights/s",
                             "achieved_gbs": vf["achieved"], "frac": vf["frac"], "frac_of_nominal_8TBs": vf["frac_nominal"],
                             "coded_bits_per_weight": vf["coded_bits"],
                             "entropy_bits_per_weight": entropy_bits(vs, vy) / max(1, vf["n_w"]),
                             "desc_flags": int(vdb.h_descs[0][0].flags),
                             "l2_policy": vpol, "clocks": sampler.summary()})
            launches += time_workload.launches
            del vdb
            torch.cuda.empty_cache()
    fused = None
    if world == 1 and not args.no_fused and args.workload == "large" and args.dim % 256 == 0:
        try:
            del db
        except NameError:
            pass
        torch.cuda.empty_cache()
        fused, fl = run_fused(ans, args, local, sampler)
        launches += fl
    # the two workloads of the target (at least 60 % of 8 TB/s on each), at the paper's table size
    # (256 states) and at 4096 states, side by side
    targets = None
    if variants:
        def best(wl, tl):
            fr = [v["frac_of_nominal_8TBs"] for v in variants if v["workload"] == wl and v["table_log"] == tl]
            return max(fr) if fr else None
        targets = {"bar_frac_of_8TBs": 0.60,
                   "large_256_states": fg["frac_nominal"], "large_4096_states": best("large", 12),
                   "resnet50_256_states": best("resnet50", 8), "resnet50_4096_states": best("resnet50", 12)}
    if rank == 0:
        sampler.stop()
    if rank != 0:
        return
    dts = sorted({sp.out_dtype for sp in head_specs})
    out = {
        "metric": METRIC, "value": value, "unit": "weights/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": dts[0] if len(dts) == 1 else "mixed", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[args.workload], "name": args.workload, "layout": args.layout,
                   "lanes": "one per input channel (channels container)" if by_channel else args.lanes,
                   "grouping": args.grouping, "table_log": layers[0].table_log, "chunk_symbols": layers[0].chunk_symbols,
                   "layers": len(layers), "weights": n_w, "out_dtype": head_specs[0].out_dtype,
                   "arithmetic": "integer decode, one fp32 multiply per weight, round-to-nearest-even to the output type",
                   "l2_policy": policy, "desc_flags": int(db_flags),
                   "per_gpu": "every rank decodes its own replica of the workload; no collective on the data path"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline, "cpu_baseline": cpu,
        "targets": targets, "variants": variants, "fused": fused,
        "compression": {"coded_bits_per_weight": fg["coded_bits"], "entropy_bits_per_weight": ent_bits / max(1, n_w),
                        "gap_bits_per_weight": fg["coded_bits"] - ent_bits / max(1, n_w),
                        "compressed_bytes": fg["comp_bytes"], "output_bytes": fg["out_bytes"]},
        "setup_s": setup_s,
    }
    print(json.dumps(out))


def run_e2e(ans, db, layers, args, world):
    """Same metric through ans_decode_dequant_host: per layer, compressed bytes go host -> device,
    the layer is decoded, the weights come back device -> host, all inside the timed region."""
    import torch
    n_w = sum(L.n_symbols for L in layers)
    st = torch.cuda.current_stream().cuda_stream
    pinned_in, pinned_out, need = [], [], 0
    for i, L in enumerate(layers):
        bufs = []
        for a in (L.stream, L.sub_offsets, L.lane_meta):
            t = torch.empty(max(a.nbytes, 1), dtype=torch.uint8, pin_memory=True)
            t.numpy()[:a.nbytes] = a.reshape(-1).view(np.uint8)
            bufs.append(t)
        pinned_in.append(bufs)
        pinned_out.append(torch.empty(max(L.n_symbols * ans.ELEM_SIZE[L.out_dtype], 1), dtype=torch.uint8, pin_memory=True))
        need = max(need, ans.ans_host_scratch_bytes(db.h_descs[0][i], L.stream.nbytes))
    scratch = torch.empty(need, dtype=torch.uint8, device="cuda")
    lib = ans.lib()
    import ctypes

    def step():
        for i, L in enumerate(layers):
            if L.n_symbols == 0:
                continue
            s, o, m = pinned_in[i]
            rc = lib.ans_decode_dequant_host(ctypes.byref(db.h_descs[0][i]), s.data_ptr(), L.stream.nbytes,
                                             o.data_ptr(), m.data_ptr(), pinned_out[i].data_ptr(),
                                             scratch.data_ptr(), need, st)
            assert rc == 0, rc

    steps = max(1, min(args.steps, 5))
    step()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    torch.cuda.synchronize()
    dt = reduce_max((time.perf_counter() - t0) / steps, world)
    h2d = sum(L.compressed_bytes() for L in layers)
    d2h = sum(L.n_symbols * ans.ELEM_SIZE[L.out_dtype] for L in layers)
    return {"value": world * n_w / dt, "unit": "weights/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "ms_per_step": dt * 1e3, "steps": steps, "api": "ans_decode_dequant_host (pinned host buffers)"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", choices=list(WORKLOAD_TEXT))
    ap.add_argument("--layout", default=None, choices=["private", "interleaved", "quads", "strips"],
                    help="container; default: the fastest measured for the workload")
    ap.add_argument("--lanes", type=int, default=0, help="lanes per chunk (a multiple of 32); default: per workload")
    ap.add_argument("--grouping", default="chunks", choices=["chunks", "channel"],
                    help="channel (ResNet workloads): one stream per input channel of every conv, as in the paper")
    ap.add_argument("--chunk", type=int, default=0)
    ap.add_argument("--table-log", type=int, default=0)
    ap.add_argument("--mats", type=int, default=8, help="large workload: number of matrices (8 = full size)")
    ap.add_argument("--dim", type=int, default=8192, help="large workload: matrix dimension (8192 = full size)")
    ap.add_argument("--symbols", type=int, default=1 << 28, help="sweep workload: number of symbols (2^28 = full size)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-variants", action="store_true")
    ap.add_argument("--no-fused", action="store_true", help="skip the fused decode + matrix product measurement")
    ap.add_argument("--no-settled", action="store_true",
                    help="set neither ANS_DESC_INPUTS_SETTLED nor ANS_DESC_OUTPUT_IDLE: every launch waits for the one "
                         "before it before it reads anything")
    ap.add_argument("--no-idle", action="store_true",
                    help="set ANS_DESC_INPUTS_SETTLED only: a launch waits for the one before it before its first write")
    ap.add_argument("--fused-only", action="store_true",
                    help="only the fused decode + matrix product measurement (one short region), as one JSON line")
    args = ap.parse_args()
    if args.layout is None:
        args.layout = DEFAULTS[args.workload][0]
    if not args.lanes:
        args.lanes = DEFAULTS[args.workload][1] if args.layout == DEFAULTS[args.workload][0] else 32
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args.gpus, run_impl, args)              # not under torchrun: start the N ranks here
    else:
        run_impl(args)


def run_impl(args):
    if args.impl == "reference":
        run_reference(args)
    elif args.fused_only:
        import torch
        import paper_2406_06237_b200 as ans
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
        ans.lib()
        res, launches = run_fused(ans, args, 0, None, min_region_s=0.02)
        print(json.dumps({"fused": res, "gpu_launches": launches}))
    else:
        run_ours(args)


def _rank_entry(rank, n, port, target, targs):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    target(*targs)


def spawn_ranks(n, target, *targs):
    """Start n local ranks, one process per GPU, with the environment torchrun would give them
    (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR = 127.0.0.1, a free MASTER_PORT), and wait for them."""
    import socket
    import torch.multiprocessing as mp
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    mp.spawn(_rank_entry, args=(n, port, target, targs), nprocs=n, join=True)


if __name__ == "__main__":
    main()
