#!/usr/bin/env python
"""Benchmark of the tANS decode + dequantise path on B200.

One step = one pass of the whole hot path (stage tables, read compressed streams, decode,
dequantise, store) over one synthetic workload, as ONE batched kernel launch.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload large|resnet50|resnet18|conv3x3|sweep]
                  [--layout private|interleaved|quads] [--lanes 32|64|128|256] [--impl ours|reference]

Prints one JSON line (rank 0).  With --impl reference the CPU oracle is timed instead.
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


# dram__bytes_read.sum + dram__bytes_write.sum per launch, scaled from the 2-matrix capture in
# profiles/ans_decode_kernel_quads_large.md to the 8 matrices of a full launch
NCU_TRAFFIC = {("large", "quads", 32, 8, 8192, 0, 0): 1021.9e6}      # 256-state table (the default)


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


# the container each workload is timed on unless --layout says otherwise: the fastest measured
DEFAULT_LAYOUT = {"large": "quads", "resnet18": "quads", "resnet50": "quads", "sweep": "quads", "conv3x3": "quads"}


class ClockSampler:
    """nvidia-smi clocks and throttle reasons, sampled while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None
        self.first, self.last, self.in_timed = 0, None, None     # rows taken under the timed load

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
        out = {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
               "reasons": sorted(reasons), "samples": len(sm)}
        if self.in_timed is not None and self.in_timed < len(sm):
            out["samples_in_timed_region"] = self.in_timed
            out["note"] = ("the timed region is shorter than a few sampling periods (20 ms): the same launches "
                           "were kept running right after it until 5 samples were in")
        return out


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
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
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


def time_workload(db, steps, warmup, flush, n_sets, world, sampler=None):
    """K timed steps, each bracketed by CUDA events on the launching stream; the L2 flush (if
    any) sits outside the brackets.  Returns per-step milliseconds (max over ranks of the sum)."""
    import torch
    import torch.distributed as dist
    st = torch.cuda.current_stream()
    for i in range(warmup):
        if flush is not None:
            flush.add_(1)
        db.decode(i % n_sets)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    if sampler is not None:
        sampler.first = len(sampler.rows)
    # The host must not be what is timed: a spin of a few milliseconds goes first (outside every
    # bracket), so that the K launches and their events are all queued by the time the device
    # reaches them and run back to back.
    torch.cuda._sleep(int(2e7))
    for i in range(steps):
        if flush is not None:
            flush.add_(1)
        ev[i][0].record(st)
        db.decode(i % n_sets)
        ev[i][1].record(st)
    torch.cuda.synchronize()
    if sampler is not None and sampler.proc is not None:
        # a clock reading needs a few sampling periods of load: keep the same launches going
        # (outside every timing bracket) until they are in
        sampler.in_timed = len(sampler.rows) - sampler.first
        t_end = time.perf_counter() + 2.0
        while len(sampler.rows) - sampler.first < 5 and time.perf_counter() < t_end:
            for i in range(steps):
                db.decode(i % n_sets)
            torch.cuda.synchronize()
        sampler.last = len(sampler.rows)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ms = [a.elapsed_time(b) for a, b in ev]               # each launch by itself
    span = ev[0][0].elapsed_time(ev[-1][1])               # the K steps as one region, gaps included
    assert db.read_status() == 0, "decoder flagged a stream"
    return ms, span


def run_ours(args):
    import torch
    import paper_2406_06237_b200 as ans
    from paper_2406_06237_b200.runtime import DeviceBatch, pack_layer

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

    layout = {"private": ans.ANS_LAYOUT_PRIVATE, "interleaved": ans.ANS_LAYOUT_INTERLEAVED,
              "quads": ans.ANS_LAYOUT_QUADS, "strips": ans.ANS_LAYOUT_STRIPS}[args.layout]
    specs = make_specs(args)
    t_setup = time.perf_counter()
    from concurrent.futures import ThreadPoolExecutor
    cores = os.cpu_count() or 1

    by_channel = args.grouping == "channel"
    if by_channel:
        # the paper's own grouping (Section III-B): one chunk per layer, one lane per input channel,
        # weights stored channels-last so that lane c carries input channel c; layers whose input
        # channels are no multiple of 32 (the first conv, which the paper leaves uncompressed) are left out
        import dataclasses
        specs = [dataclasses.replace(sp, chunk_symbols=sp.n) for sp in specs
                 if len(sp.shape) == 4 and sp.shape[1] % 32 == 0 and sp.shape[1] <= 2048]
        args.no_cpu_baseline = args.no_e2e = True

    def prep(spec):
        sym = sg.draw_symbols(spec, threads=max(1, cores // 4))
        lanes = args.lanes
        if by_channel:
            sym = np.ascontiguousarray(sym.reshape(spec.shape).transpose(0, 2, 3, 1)).ravel()
            lanes = spec.shape[1]
        pl = pack_layer(sym, spec.alphabet, spec.table_log, spec.chunk_symbols, lanes, layout, spec.bitwidth,
                        spec.zero_point, spec.scale, ans.DTYPES[spec.out_dtype], n_threads=max(1, cores // 2))
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
    n_sets = min(64, max(2, -(-(512 << 20) // max(ws, 1)))) if small else 1
    db = DeviceBatch(layers, f"cuda:{local}", n_out_sets=n_sets)
    flush = None
    setup_s = time.perf_counter() - t_setup

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms, span = time_workload(db, args.steps, args.warmup, flush, n_sets, world, sampler if rank == 0 else None)
    clocks = sampler.stop() if rank == 0 else None
    total_ms = reduce_max(span, world)
    ms_per_step = total_ms / args.steps
    n_w = db.n_symbols()
    value = world * n_w / (ms_per_step * 1e-3)

    # algorithmic bytes of one launch: everything compressed read once, each layer's table
    # once, every decoded element written once
    table_read = sum(4 << L.table_log for L in layers)
    comp_bytes = db.compressed_bytes()
    algo_bytes = comp_bytes + table_read + out_bytes
    peak, peak_kind = measured_peak()
    kernel_ms = statistics.mean(ms)
    achieved = algo_bytes / (kernel_ms * 1e-3) / 1e9
    kname = f"ans_decode_kernel<{args.layout}>"
    # DRAM bytes per launch from an ncu capture of this kernel (see profiles/), only for the
    # configuration that capture covers; None otherwise
    traffic = NCU_TRAFFIC.get((args.workload, args.layout, args.lanes, args.mats, args.dim, args.chunk, args.table_log))
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "kernel": kname, "peak_kind": f"of {peak_kind}",
                "algorithmic_bytes_per_launch": algo_bytes, "kernel_ms_mean": kernel_ms,
                "kernel_ms_median": statistics.median(ms), "kernel_ms_min": min(ms),
                "frac_of_nominal_8TBs": achieved / NOMINAL_PEAK_GBS,
                "note": "HBM is the metric's roofline; ncu shows the kernel held by instruction issue, the integer "
                        "pipe and shared-memory wavefronts together (see profiles/)"}

    # end to end through the host-buffer entry point: pinned host buffers in, pinned out
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(ans, db, layers, args, world)

    # the same workload with the other table size the design notes quote (2^12 states)
    variants = []
    if args.workload == "large" and not args.table_log and world == 1 and not args.no_variants:
        db = None
        torch.cuda.empty_cache()
        with ThreadPoolExecutor(4) as ex:
            layers12 = list(ex.map(lambda sp_sy: pack_layer(sp_sy[1], sp_sy[0].alphabet, 12, sp_sy[0].chunk_symbols,
                                                            args.lanes, layout, sp_sy[0].bitwidth, sp_sy[0].zero_point,
                                                            sp_sy[0].scale, ans.DTYPES[sp_sy[0].out_dtype],
                                                            n_threads=max(1, cores // 2)), zip(specs, syms)))
        db12 = DeviceBatch(layers12, f"cuda:{local}", n_out_sets=1)
        ms12, _ = time_workload(db12, min(args.steps, 50), 5, None, 1, 1)
        bytes12 = db12.compressed_bytes() + sum(4 << 12 for _ in layers12) + out_bytes
        k12 = statistics.mean(ms12)
        variants.append({"table_log": 12, "layout": args.layout, "kernel_ms_mean": k12, "value": n_w / (k12 * 1e-3), "unit": "weights/s",
                         "achieved_gbs": bytes12 / (k12 * 1e-3) / 1e9, "frac": bytes12 / (k12 * 1e-3) / 1e9 / peak,
                         "coded_bits_per_weight": 8.0 * db12.compressed_bytes() / n_w})
        del db12

    if rank != 0:
        return
    hist = np.zeros(256, dtype=np.float64)
    ent_bits = 0.0
    for spec, sym in zip(specs, syms):
        c = np.bincount(sym, minlength=256).astype(np.float64)
        p = c[c > 0] / max(1, sym.size)
        ent_bits += float(-(p * np.log2(p)).sum()) * sym.size
    coded_bits = 8.0 * comp_bytes
    cpu = cpu_baseline(specs, syms, args.layout, args.lanes) if world == 1 and not args.no_cpu_baseline else None
    out = {
        "metric": METRIC, "value": value, "unit": "weights/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[args.workload], "name": args.workload, "layout": args.layout,
                   "lanes": "one per input channel" if args.grouping == "channel" else args.lanes,
                   "grouping": args.grouping, "table_log": layers[0].table_log, "chunk_symbols": layers[0].chunk_symbols,
                   "layers": len(layers), "weights": n_w, "out_dtype": specs[0].out_dtype,
                   "l2_policy": (f"inputs larger than L2: launches rotate over {n_sets} full copies of the workload "
                                 f"({n_sets * ws / 2**20:.0f} MB in all)"
                                 if small else "working set (compressed + output) is larger than L2"),
                   "per_gpu": "every rank decodes its own replica of the workload; no collective on the data path"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": args.steps, "roofline": roofline, "cpu_baseline": cpu,
        "variants": variants,
        "compression": {"coded_bits_per_weight": coded_bits / max(1, n_w), "entropy_bits_per_weight": ent_bits / max(1, n_w),
                        "gap_bits_per_weight": (coded_bits - ent_bits) / max(1, n_w),
                        "compressed_bytes": comp_bytes, "output_bytes": out_bytes},
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
    ap.add_argument("--lanes", type=int, default=32)
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
    args = ap.parse_args()
    if args.layout is None:
        args.layout = DEFAULT_LAYOUT[args.workload]
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
