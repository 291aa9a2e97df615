#!/usr/bin/env python
"""Benchmark of the FastSGD compress + decompress-accumulate hot path on B200.

One step = one pass of the whole path over one batch of synthetic gradients: every simulated
worker's gradient is compressed (one fused kernel: abs-sum pass, grid barrier, encode pass), then every stream is
decompress-accumulated into one dense vector.  The metric is input GB/s = 4 n W / t.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--impl reference]

Under torchrun (N > 1) every rank runs an independent replica (the path has no exchange step
on one node: "replicas only"); value = units of all ranks / max-over-ranks time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "compress+decompress input GB/s (fp32 gradient)"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


WORKLOADS = {
    # name: (description, default workers, default keep)
    "c1": "n=1,048,576 N(0,1e-3^2), 1% kept, 1 worker",
    "c2": "n=25,557,032 Student-t(3) x per-layer log-uniform scale over 161 blocks, 0.5% kept, 4 workers",
    "c3": "n=50,000,000 clustered-sparse Laplace, 80% of nonzeros kept, 1 worker",
    "c4": "n=335,141,888 per-block normal, 8 workers",
    "c5": "n=2^k N(0,1e-3^2) with 1% outliers x100",
}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period: float = 0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def sample_once(self):
        if not self.ok:
            return
        nv = self.nv
        try:
            self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
            r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
            names = {
                "hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40,
                "sw_thermal_slowdown": 0x20, "hw_power_brake_slowdown": 0x80, "sync_boost": 0x10,
            }
            for k, bit in names.items():
                if r & bit:
                    self.reasons.add(k)
        except Exception:
            pass

    def run(self):
        while not self._stop.is_set():
            self.sample_once()
            time.sleep(self.period)

    def stop(self):
        self._stop.set()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0}
        return {"sm_mhz": float(statistics.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "sm_mhz_p10": float(np.percentile(self.samples, 10)),
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def run_reference(args, rank):
    """The oracle, as it stands, on the host cores: the reference arm of this tier."""
    if rank != 0:
        return
    import oracle
    from paper_2112_04291_b200 import workloads
    wl = workloads.make(args.workload, n=args.n, workers=1, keep=args.keep)
    v, n = wl.grads[0], wl.n
    po = oracle.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
    # size the per-step sample so that the whole run stays near a minute
    probe = v[: min(n, 1 << 20)]
    t0 = time.perf_counter()
    oracle.compress(probe, po)
    per_elem = (time.perf_counter() - t0) / probe.size * 1.3
    budget = 60.0 / max(1, args.steps + args.warmup)
    ns = int(max(1 << 16, min(n, budget / per_elem)))
    sample = np.ascontiguousarray(v[:ns])
    dense = np.zeros(ns, np.float32)

    def step():
        rc, s = oracle.compress(sample, po)
        assert rc == 0
        assert oracle.decompress_accumulate(s, ns, po, dense) == 0

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = 4.0 * ns * args.steps / dt / 1e9
    desc = f"first {ns} entries of worker 0 of {args.workload}, compress + decompress-accumulate, 1 thread"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {WORKLOADS[args.workload]}", "n": n, "sample_n": ns},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_sweep(args):
    """Config 5: n = 2^10 .. 2^30 in powers of 4, keep in {0.01, 0.1, 1, 10} %, one worker; compress-only,
    decompress-only and combined, each as the median of single eager calls timed with CUDA events,
    with a 256 MiB write between calls (every size up to 2^24 would otherwise sit in L2).  Writes a
    markdown table to args.sweep and prints one JSON line about the largest point."""
    import torch
    from paper_2112_04291_b200 import binding, workloads

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    dev = torch.device("cuda", 0)
    peak, peak_kind = measured_peak()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    iters = max(5, min(args.steps, 20))
    rows, last = [], None
    max_log2 = args.sweep_max_log2
    for log2n in range(10, max_log2 + 1, 2):
        n = 1 << log2n
        v = workloads.normal_outliers(n, seed=0)
        grad = torch.from_numpy(v).to(dev)
        for keep in (1e-4, 1e-3, 1e-2, 1e-1):
            base = workloads.base_for_keep(v, max(1, int(round(keep * n))))
            pg = binding.params(base)
            binding.ensure_workspace(n, pg, dev)
            cap = (min(binding.compress_bound(n, pg), max(4 * n, 1 << 20)) + 255) & ~255
            out = torch.zeros(cap, dtype=torch.uint8, device=dev)
            dense = torch.zeros(n, dtype=torch.float32, device=dev)

            def comp():
                rc = binding.compress(grad, pg, out)
                assert rc == 0, rc

            def dec():
                rc = binding.decompress_accumulate(out, cap, n, pg, dense)
                assert rc == 0, rc

            def both():
                comp()
                dec()

            def med(fn):
                ts = []
                for it in range(iters + 3):
                    flush.fill_(it & 0xFF)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    fn()
                    e1.record()
                    torch.cuda.synchronize()
                    if it >= 3:
                        ts.append(e0.elapsed_time(e1))
                return statistics.median(ts)

            both()
            total, d, status = binding.stream_info(out)
            assert status == 0 and binding.decode_status() == 0
            listed = binding.listed_tiles(1)
            ms_c, ms_d, ms_b = med(comp), med(dec), med(both)
            alg_c, alg_d = 8.0 * n + total, total + 8.0 * d
            tr_c, tr_d = traffic_model(n, [total], [d], listed)
            row = {"log2n": log2n, "keep": keep, "kept": d, "stream_bytes": total,
                   "compress_ms": ms_c, "decompress_ms": ms_d, "combined_ms": ms_b,
                   "compress_in_gbs": 4.0 * n / ms_c / 1e6, "decompress_in_gbs": 4.0 * n / ms_d / 1e6,
                   "combined_in_gbs": 4.0 * n / ms_b / 1e6,
                   "compress_frac": alg_c / ms_c / 1e6 / peak, "decompress_frac": alg_d / ms_d / 1e6 / peak,
                   "combined_frac": (alg_c + alg_d) / ms_b / 1e6 / peak,
                   "compress_dram_frac": tr_c / ms_c / 1e6 / peak, "combined_dram_frac": (tr_c + tr_d) / ms_b / 1e6 / peak}
            rows.append(row)
            last = row
            del out, dense
        del grad, v
    with open(args.sweep, "w") as f:
        f.write("| n | keep | kept | stream bytes | compress us | GB/s in | frac | dram frac | decompress us | GB/s in | frac | combined us | GB/s in | frac | dram frac |\n")
        f.write("|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|\n")
        for r in rows:
            f.write("| 2^%d | %g | %d | %d | %.1f | %.0f | %.3f | %.3f | %.1f | %.0f | %.3f | %.1f | %.0f | %.3f | %.3f |\n" % (
                r["log2n"], r["keep"], r["kept"], r["stream_bytes"], r["compress_ms"] * 1e3, r["compress_in_gbs"],
                r["compress_frac"], r["compress_dram_frac"], r["decompress_ms"] * 1e3, r["decompress_in_gbs"], r["decompress_frac"],
                r["combined_ms"] * 1e3, r["combined_in_gbs"], r["combined_frac"], r["combined_dram_frac"]))
    line = {"metric": METRIC, "value": last["combined_in_gbs"], "unit": UNIT, "n_gpus": 1, "steps": iters, "warmup": 3,
            "ms_per_step": last["combined_ms"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": "c5 sweep, largest point: n=2^%d, keep %g" % (last["log2n"], last["keep"]),
                       "points": len(rows), "table": args.sweep, "l2": "256 MiB written between timed calls",
                       "launch": "eager, one call per timed region"},
            "roofline": {"bound": "hbm", "peak": peak, "peak_kind": "of " + peak_kind, "unit": "GB/s",
                         "achieved": last["combined_frac"] * peak, "frac": last["combined_frac"], "traffic": None}}
    print(json.dumps(line), flush=True)


def run_keys_table(args):
    """Size per gradient key (the paper's two tables on the space cost of the gradient key, restated on
    synthetic keys): Algorithm 2 as printed (one chain, one M; written by fastsgd_key_encode_paper) for
    l = 1..5, the product stream's key part (groups of 2^14, flags and deltas as planes) for the same l,
    and a byte-granular delta baseline (every delta in whole bytes plus a 2-bit byte count).  The key sets
    are the kept keys of the benchmark gradients, obtained through the product path (compress, decode
    into a zero vector, positions of the non-zeros).  Writes a markdown table to args.keys_table."""
    import torch
    from paper_2112_04291_b200 import binding, workloads

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    dev = torch.device("cuda", 0)
    rows = []
    sets = [("c2 worker 0 (25.6 M, 0.5 %, layered)", "c2", {}), ("c3 (50 M, clustered runs)", "c3", {}),
            ("c5 2^24, 1 % (uniform)", "c5", {"n": 1 << 24, "keep": 1e-2}), ("c5 2^26, 0.1 % (uniform)", "c5", {"n": 1 << 26, "keep": 1e-3})]
    for label, name, kw in sets:
        wl = workloads.make(name, workers=1, **kw)
        n = wl.n
        grad = torch.from_numpy(wl.grads[0]).to(dev)
        row = {"set": label, "n": n}
        keys = None
        for l in (1, 2, 3, 4, 5):
            pg = binding.params(wl.base, wl.tau, l, wl.group_log2)
            binding.ensure_workspace(n, pg, dev)
            cap = (min(binding.compress_bound(n, pg), max(4 * n, 1 << 20)) + 255) & ~255
            out = torch.zeros(cap, dtype=torch.uint8, device=dev)
            assert binding.compress(grad, pg, out) == 0
            total, d, status = binding.stream_info(out)
            assert status == 0 and d > 0
            G = (n + (1 << wl.group_log2) - 1) >> wl.group_log2
            row["grouped_l%d" % l] = (8.0 * (total - 64 - 8 * G) - 8.0 * d) / d      # blobs minus the code bytes (incl. padding)
            row["grouped_dir_l%d" % l] = (8.0 * (total - 64) - 8.0 * d) / d          # ... plus the directory
            if keys is None:
                dense = torch.zeros(n, dtype=torch.float32, device=dev)
                assert binding.decompress_accumulate(out, cap, n, pg, dense) == 0 and binding.decode_status() == 0
                keys = torch.nonzero(dense).flatten().to(torch.int32).contiguous()
                assert keys.numel() == d
                del dense
            buf = torch.empty(binding.key_encode_paper_bound(keys.numel(), l), dtype=torch.uint8, device=dev)
            ts = []
            for it in range(8):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                assert binding.key_encode_paper(keys, l, buf) == 0
                e1.record()
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1))
            hdr = buf[:16].cpu().numpy()
            nbits = int(hdr[8:16].view(np.uint64)[0])
            row["paper_l%d" % l] = nbits / keys.numel()
            row["paper_M"] = int(hdr[0:4].view(np.uint32)[0])
            row["paper_us_l%d" % l] = statistics.median(ts[2:]) * 1e3
            del out, buf
        # the group size trades the directory (8 bytes per group) against shorter deltas: l = 2, groups of 2^12, 2^14, 2^16
        for glog in (12, 14, 16):
            pg = binding.params(wl.base, wl.tau, 2, glog)
            binding.ensure_workspace(n, pg, dev)
            cap = (min(binding.compress_bound(n, pg), max(4 * n, 1 << 20)) + 255) & ~255
            out = torch.zeros(cap, dtype=torch.uint8, device=dev)
            assert binding.compress(grad, pg, out) == 0
            total, d, status = binding.stream_info(out)
            assert status == 0 and d == keys.numel()
            Gg = (n + (1 << glog) - 1) >> glog
            row["glog%d_blobs" % glog] = (8.0 * (total - 64 - 8 * Gg) - 8.0 * d) / d
            row["glog%d_with_dir" % glog] = (8.0 * (total - 64) - 8.0 * d) / d
            del out
        k = keys.cpu().numpy().astype(np.int64)
        delta = np.diff(np.concatenate([[0], k]))
        nbytes = np.maximum(1, (np.floor(np.log2(np.maximum(delta, 1))).astype(np.int64) + 8) // 8)
        row["byte_granular"] = float((8 * nbytes + 2).sum()) / k.size
        row["d"] = int(k.size)
        rows.append(row)
        del grad, keys
    with open(args.keys_table, "w") as f:
        f.write("| key set | kept keys | format | l=1 | l=2 | l=3 | l=4 | l=5 |\n|---|---|---|---|---|---|---|---|\n")
        for r in rows:
            f.write("| %s | %d | Algorithm 2 as printed (one chain, M = %d), bits per key | %s |\n" % (
                r["set"], r["d"], r["paper_M"], " | ".join("%.2f" % r["paper_l%d" % l] for l in range(1, 6))))
            f.write("| | | product stream, key part of the blobs | %s |\n" % " | ".join("%.2f" % r["grouped_l%d" % l] for l in range(1, 6)))
            f.write("| | | product stream, key part + directory | %s |\n" % " | ".join("%.2f" % r["grouped_dir_l%d" % l] for l in range(1, 6)))
            f.write("| | | byte-granular deltas + 2-bit byte count: %.2f; plain 32-bit keys: 32.00 | | | | | |\n" % r["byte_granular"])
            f.write("| | | fastsgd_key_encode_paper, us per call | %s |\n" % " | ".join("%.1f" % r["paper_us_l%d" % l] for l in range(1, 6)))
            f.write("| | | product stream at l = 2 by group size, key part / + directory: 2^12: %.2f / %.2f; 2^14: %.2f / %.2f; 2^16: %.2f / %.2f | | | | | |\n" % (
                r["glog12_blobs"], r["glog12_with_dir"], r["glog14_blobs"], r["glog14_with_dir"], r["glog16_blobs"], r["glog16_with_dir"]))
    best = rows[0]
    print(json.dumps({"metric": "bits per gradient key", "value": best["paper_l2"], "unit": "bits", "n_gpus": 1,
                      "higher_is_better": False, "data": "synthetic", "config": {"workload": "key sets of c2, c3, c5", "table": args.keys_table},
                      "rows": rows}), flush=True)



TILE = 1 << 14            # entries per tile of the encoder = per group of the stream
L2_BYTES = 126e6


def ncu_traffic_of(profile_md: str):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch as recorded in a summary under profiles/
    (a line `dram_bytes_per_launch = N`, written there from the capture it describes); None if absent."""
    try:
        import re
        txt = open(os.path.join(ROOT, "profiles", profile_md)).read()
        m = re.search(r"dram_bytes_per_launch\s*=\s*([0-9.eE+]+)", txt)
        c = re.search(r"captured_at_commit\s*=\s*([0-9a-f]+)", txt)
        return {"bytes": float(m.group(1)), "source": "profiles/" + profile_md, "commit": c.group(1) if c else None} if m else None
    except Exception:
        return None


def traffic_model(n, stream_bytes, kept, listed):
    """DRAM bytes the two kernels have to move, counted rather than assumed: the sum pass reads every gradient
    once (4 n each); the encode pass reads again only the tiles the kernel listed (it leaves their number per
    gradient in the workspace), 64 KiB each; the streams are written once and read once; every kept entry is a
    read-modify-write of one 32-byte sector of the accumulator (never more than the whole accumulator)."""
    W = len(stream_bytes)
    comp = sum(4.0 * n + min(4.0 * n, 4.0 * TILE * listed[w]) + stream_bytes[w] for w in range(W))
    dec = float(sum(stream_bytes)) + min(64.0 * float(sum(kept)), 8.0 * n)
    return comp, dec


def series_stats(ts):
    return {"median": statistics.median(ts), "min": min(ts)}


def measure_config(torch, binding, dev, wl, grads, peak, reps, flush, outs=None, dense=None, use_graph=True):
    """One compact entry of the `configs` table: compress-only, decompress-only and combined; median and min.
    Two timing protocols.  `*_flushed`: every repetition timed by its own pair of CUDA events after 256 MiB were
    written.  That leaves L2 full of dirty lines, and their write-back (126 MB) competes with the first 40-50 us
    of whatever runs next.  So where one launch's input is at least 1.5 x L2 and a step takes less than 1 ms the entry's own figures come from
    launches that follow one another with no flush, alternating between two copies of the input at different
    addresses (nothing of a launch's input is left in L2 for the next launch but one to find): means of 10
    launches per pair of events.  Smaller inputs have only the flushed protocol."""
    n, W = wl.n, wl.workers
    pg = binding.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
    binding.ensure_workspace(n, pg, dev)
    cap = (min(binding.compress_bound(n, pg), max(4 * n, 1 << 20)) + 255) & ~255
    if outs is None:
        outs = [torch.zeros(cap, dtype=torch.uint8, device=dev) for _ in range(W)]
    if dense is None:
        dense = torch.zeros(n, dtype=torch.float32, device=dev)
    else:
        dense.zero_()

    def comp():
        rc = binding.compress_batch(grads, pg, outs)
        if rc:
            raise binding.FastSGDError(rc, "fastsgd_compress_batch")

    def dec():
        rc = binding.decompress_accumulate_batch(outs, [cap] * W, n, pg, dense)
        if rc:
            raise binding.FastSGDError(rc, "fastsgd_decompress_accumulate_batch")

    def both():
        comp()
        dec()

    both()
    infos = [binding.stream_info(o) for o in outs]
    assert all(st == 0 for _, _, st in infos) and binding.decode_status() == 0, infos
    stream_bytes = [tb for tb, _, _ in infos]
    kept = [d for _, d, _ in infos]
    listed = binding.listed_tiles(W)

    # the same C-ABI calls replayed from CUDA graphs, as the headline step is (eager calls if capture fails)
    def graph_of(fn):
        if not use_graph:
            return fn
        try:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn()
            g.replay()
            torch.cuda.synchronize()
            return g.replay
        except Exception as exc:
            print(f"[bench] CUDA graph capture failed, launching eagerly: {exc}", file=sys.stderr)
            return fn

    comp_run, dec_run, both_run = graph_of(comp), graph_of(dec), graph_of(both)

    def series(fn, cold):
        ts = []
        for it in range(reps + 3):
            if cold:
                flush.fill_(it & 0xFF)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            if it >= 3:
                ts.append(e0.elapsed_time(e1))
        return ts

    tc, td, tb = series(comp_run, True), series(dec_run, True), series(both_run, True)
    in_bytes = 4.0 * n * W
    # (for launches of a millisecond and more the write-back is below 3 % and the flushed protocol stays)
    rotate = in_bytes >= 1.5 * L2_BYTES and statistics.median(tb) < 1.0
    tc_flushed, tb_flushed = tc, tb
    if rotate:
        grads2 = [g.clone() for g in grads]

        def comp2():
            rc = binding.compress_batch(grads2, pg, outs)
            if rc:
                raise binding.FastSGDError(rc, "fastsgd_compress_batch")

        def both2():
            comp2()
            dec()

        comp_run2, both_run2 = graph_of(comp2), graph_of(both2)

        def series_rot(f1, f2, pairs=5):
            ts = []
            for it in range(max(4, reps // 4) + 1):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(pairs):
                    f1()
                    f2()
                e1.record()
                torch.cuda.synchronize()
                if it >= 1:
                    ts.append(e0.elapsed_time(e1) / (2 * pairs))
            return ts

        tc, tb = series_rot(comp_run, comp_run2), series_rot(both_run, both_run2)
        del grads2
    alg_c = 8.0 * n * W + float(sum(stream_bytes))
    alg_d = float(sum(stream_bytes)) + 8.0 * float(sum(kept))
    tr_c, tr_d = traffic_model(n, stream_bytes, kept, listed)
    mc, md, mb = statistics.median(tc), statistics.median(td), statistics.median(tb)
    entry = {
        "n": n, "workers": W, "keep": wl.keep_fraction, "kept": int(sum(kept)), "stream_bytes": int(sum(stream_bytes)),
        "listed_tiles": int(sum(listed)), "tiles": W * ((n + TILE - 1) // TILE),
        "compress_ms": series_stats(tc), "decompress_ms": series_stats(td), "combined_ms": series_stats(tb),
        "input_gbs": in_bytes / mb / 1e6,
        "frac": (alg_c + alg_d) / mb / 1e6 / peak, "frac_nominal_8000": (alg_c + alg_d) / mb / 1e6 / 8000.0,
        "dram_frac": (tr_c + tr_d) / mb / 1e6 / peak,
        "compress_frac": alg_c / mc / 1e6 / peak, "compress_dram_frac": tr_c / mc / 1e6 / peak,
        "decompress_frac": alg_d / md / 1e6 / peak, "decompress_sector_frac": tr_d / md / 1e6 / peak,
    }
    if rotate:
        entry["protocol"] = ("compress and combined: launches back to back on two alternating copies of the input, no flush "
                             "(input per launch >= 1.5 x L2, step < 1 ms), mean of 10 per event pair; decompress and *_flushed: 256 MiB written "
                             "before every launch")
        entry["compress_ms_flushed"] = series_stats(tc_flushed)
        entry["combined_ms_flushed"] = series_stats(tb_flushed)
        entry["frac_flushed"] = (alg_c + alg_d) / statistics.median(tb_flushed) / 1e6 / peak
    else:
        entry["protocol"] = "256 MiB written before every launch"
    if entry["frac"] > 1.2:
        entry["note"] = "frac counts two full reads of every gradient; the kernel skipped most tiles: dram_frac is the hardware figure"
    if in_bytes < L2_BYTES:
        tw = series(both_run, False)
        entry["combined_ms_l2_warm"] = series_stats(tw)
    assert all(binding.stream_info(o)[2] == 0 for o in outs) and binding.decode_status() == 0
    return entry


def configs_table(torch, binding, workloads, dev, peak, reps, c2_entry, use_graph=True):
    """Every benchmark configuration besides the headline: c1, c3, c4 at three keep ratios with its 8 workers, c5 at
    n = 2^26, 2^28, 2^30 at four keep ratios.  Inputs are drawn on the host (the same seeded generators as the
    parity tests), the next workload while the current one is being timed."""
    from concurrent.futures import ThreadPoolExecutor
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    plan = [
        ("c1", lambda: [workloads.make("c1")]),
        ("c3", lambda: [workloads.make("c3")]),
        ("c5_2^26", lambda: workloads.with_keeps(workloads.make("c5", n=1 << 26), (1e-4, 1e-3, 1e-2, 1e-1))),
        ("c4", lambda: workloads.with_keeps(workloads.make("c4", threads=8), (1e-4, 1e-3, 1e-2))),
        ("c5_2^28", lambda: workloads.with_keeps(workloads.make("c5", n=1 << 28), (1e-4, 1e-3, 1e-2, 1e-1))),
        ("c5_2^30", lambda: workloads.with_keeps(workloads.make("c5", n=1 << 30), (1e-4, 1e-3, 1e-2, 1e-1))),
    ]
    table = {"c2": c2_entry}
    with ThreadPoolExecutor(max_workers=1) as pool:
        fut = pool.submit(plan[0][1])
        for i, (name, _) in enumerate(plan):
            wls = fut.result()
            if i + 1 < len(plan):
                fut = pool.submit(plan[i + 1][1])
            n, W = wls[0].n, wls[0].workers
            grads = [torch.from_numpy(g).to(dev) for g in wls[0].grads]
            pg0 = binding.params(wls[0].base, wls[0].tau, wls[0].flag_bits, wls[0].group_log2)
            cap = (min(binding.compress_bound(n, pg0), max(4 * n, 1 << 20)) + 255) & ~255
            outs = [torch.zeros(cap, dtype=torch.uint8, device=dev) for _ in range(W)]
            dense = torch.zeros(n, dtype=torch.float32, device=dev)
            for wl in wls:
                key = name if len(wls) == 1 else "%s_keep_%g" % (name, wl.keep_fraction)
                table[key] = measure_config(torch, binding, dev, wl, grads, peak, reps, flush, outs, dense, use_graph)
            del grads, outs, dense, wls
            torch.cuda.empty_cache()
    return table


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2", choices=sorted(WORKLOADS))
    ap.add_argument("--n", type=int, default=None)
    ap.add_argument("--workers", type=int, default=None)
    ap.add_argument("--keep", type=float, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="headline workload only: skip the table of the other configurations")
    ap.add_argument("--no-sustained", action="store_true", help="skip the 2 s replay that follows the timed steps")
    ap.add_argument("--no-graph", action="store_true", help="launch every call eagerly instead of replaying a CUDA graph of the step")
    ap.add_argument("--sweep", default=None, metavar="FILE", help="config 5: size x keep-ratio sweep, markdown table written to FILE")
    ap.add_argument("--sweep-max-log2", type=int, default=30)
    ap.add_argument("--keys-table", default=None, metavar="FILE", help="size per gradient key for l = 1..5 on the benchmark key sets, markdown table written to FILE")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2112_04291_b200 import multirank
    rank, world, local_rank = multirank.env_rank()

    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.sweep:
        if rank == 0:
            run_sweep(args)
        return
    if args.keys_table:
        if rank == 0:
            run_keys_table(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2112_04291_b200 import binding, workloads

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        multirank.init("nccl", dev)

    # ---- inputs: generated on the host with fixed seeds (each rank its own), resident in HBM
    wl = workloads.make(args.workload, n=args.n, workers=args.workers, keep=args.keep, seed=multirank.rank_seed(rank))
    n, W = wl.n, wl.workers
    pg = binding.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
    binding.ensure_workspace(n, pg, dev)
    host_grads = [torch.from_numpy(g).pin_memory() for g in wl.grads]
    grads = [g.to(dev, non_blocking=True) for g in host_grads]
    cap = min(binding.compress_bound(n, pg), max(4 * n, 1 << 20))
    cap = (cap + 255) & ~255
    outs = [torch.zeros(cap, dtype=torch.uint8, device=dev) for _ in range(W)]
    dense = torch.zeros(n, dtype=torch.float32, device=dev)
    torch.cuda.synchronize()

    def compress_all():
        # all workers' gradients in one launch (per 8 gradients); same streams as one call per gradient
        rc = binding.compress_batch(grads, pg, outs)
        if rc:
            raise binding.FastSGDError(rc, "fastsgd_compress_batch")

    def decompress_all():
        # all workers' streams in one launch (per 8 streams); same result as one call per stream
        rc = binding.decompress_accumulate_batch(outs, [cap] * W, n, pg, dense)
        if rc:
            raise binding.FastSGDError(rc, "fastsgd_decompress_accumulate_batch")

    def step():
        compress_all()
        decompress_all()

    # one checked step before anything is timed
    step()
    infos = [binding.stream_info(o) for o in outs]
    assert all(st == 0 for _, _, st in infos), infos
    assert binding.decode_status() == 0
    stream_bytes = [tb for tb, _, _ in infos]
    kept = [d for _, d, _ in infos]

    def barrier():
        multirank.barrier(world, cuda=True)

    def timed(fn, steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        return multirank.max_over_ranks(e0.elapsed_time(e1), world, dev)

    flush_buf = None

    def timed_flushed(fn, steps):
        """Like timed(), for work whose inputs fit in L2: 256 MiB are written before every call (untimed),
        each call is bracketed by its own pair of events, the durations are added up."""
        nonlocal flush_buf
        if flush_buf is None:
            flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        barrier()
        total = 0.0
        for it in range(steps):
            flush_buf.fill_(it & 0xFF)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            total += e0.elapsed_time(e1)
        barrier()
        return multirank.max_over_ranks(total, world, dev)

    l0 = binding.launch_count()
    step()
    launches_per_step = binding.launch_count() - l0

    def make_graph(fn):
        """The same C-ABI calls, captured once into a CUDA graph and replayed (cuts launch gaps)."""
        if args.no_graph:
            return None
        try:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                fn()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn()
            g.replay()
            torch.cuda.synchronize()
            return g
        except Exception as exc:      # capture not possible: stay eager
            print(f"[bench] CUDA graph capture failed, launching eagerly: {exc}", file=sys.stderr)
            return None

    g_step, g_comp, g_dec = make_graph(step), make_graph(compress_all), make_graph(decompress_all)
    run_step = g_step.replay if g_step else step
    run_comp = g_comp.replay if g_comp else compress_all
    run_dec = g_dec.replay if g_dec else decompress_all

    for _ in range(args.warmup):
        run_step()
    sampler = ClockSampler(local_rank)
    sampler.start()
    step_exceeds_l2 = 4.0 * n * W > 1.5 * 126e6
    ms_total = timed(run_step, args.steps) if step_exceeds_l2 else timed_flushed(run_step, args.steps)
    launches = launches_per_step * args.steps
    sampler.sample_once()
    sampler.stop()
    ms_step = ms_total / args.steps

    # the same step, every repetition bracketed by its own pair of events (median and min beside the mean above)
    def timed_each(fn, steps, cold):
        nonlocal flush_buf
        if cold and flush_buf is None:
            flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        ts = []
        for it in range(steps):
            if cold:
                flush_buf.fill_(it & 0xFF)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        return ts

    each = timed_each(run_step, max(20, args.steps), True)

    # sustained: the same graph replayed back to back for at least 2 s, clocks sampled every 10 ms
    sustained = None
    if not args.no_sustained:
        sus = ClockSampler(local_rank)
        sus.start()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_end, reps_s = time.perf_counter() + 2.0, 0
        e0.record()
        while time.perf_counter() < t_end:
            for _ in range(200):
                run_step()
            reps_s += 200
            torch.cuda.synchronize()
        e1.record()
        torch.cuda.synchronize()
        sus.stop()
        ms_sus = multirank.max_over_ranks(e0.elapsed_time(e1), world, dev) / reps_s
        sustained = {"ms_per_step": ms_sus, "steps": reps_s}
        sustained.update(sus.summary())

    # separate phases (same protocol, fewer steps)
    sub = max(3, min(args.steps, 50))
    ms_comp = (timed(run_comp, sub) if step_exceeds_l2 else timed_flushed(run_comp, sub)) / sub
    ms_dec = timed_flushed(run_dec, sub) / sub      # (streams and touched lines of dense_out would otherwise stay in L2)

    # the caller's set-up of the accumulator (4n bytes written), timed apart and not part of the step
    ms_zero = timed_flushed(lambda: dense.zero_(), sub) / sub
    decompress_all()        # (the accumulator holds one step's result again)

    # the step that follows the path: decode + Adam on the decoded coordinates only (same streams; eager, flushed)
    theta = torch.zeros(n, dtype=torch.float32, device=dev)
    adam_m, adam_v, adam_g = torch.zeros_like(theta), torch.zeros_like(theta), torch.zeros_like(theta)
    hyper = binding.Adam(1e-3, 0.9, 0.999, 1e-8)

    def adam_all():
        rc = binding.sparse_adam_update_batch(outs, [cap] * W, n, pg, hyper, adam_g, theta, adam_m, adam_v)
        if rc:
            raise binding.FastSGDError(rc, "fastsgd_sparse_adam_update_batch")

    adam_all()
    ms_adam = timed_flushed(adam_all, sub) / sub
    # the same step on the state kept as (theta, m, v, g) per coordinate
    adam_state = torch.zeros(4 * n, dtype=torch.float32, device=dev)

    def adam_packed():
        rc = binding.sparse_adam_update_packed_batch(outs, [cap] * W, n, pg, hyper, adam_state)
        if rc:
            raise binding.FastSGDError(rc, "fastsgd_sparse_adam_update_packed_batch")

    adam_packed()
    ms_adam_packed = timed_flushed(adam_packed, sub) / sub
    del adam_state
    assert binding.decode_status() == 0
    del theta, adam_m, adam_v, adam_g

    # config 3 is sparse before it is compressed: worker 0 as key-value pairs (eager, flushed)
    kv_info = None
    nz = np.flatnonzero(wl.grads[0]) if args.workload == "c3" else np.zeros(0, np.int64)      # (decided by the workload, the same on every rank)
    if nz.size:
        kv_keys = torch.from_numpy(nz.astype(np.uint32).view(np.int32)).to(dev)
        kv_vals = torch.from_numpy(wl.grads[0][nz]).to(dev)
        kv_out = torch.zeros(cap, dtype=torch.uint8, device=dev)

        def kv_one():
            rc = binding.compress_kv(kv_keys, kv_vals, n, pg, kv_out)
            if rc:
                raise binding.FastSGDError(rc, "fastsgd_compress_kv")

        def dense_one():
            rc = binding.compress(grads[0], pg, kv_out)
            if rc:
                raise binding.FastSGDError(rc, "fastsgd_compress")

        kv_one()
        assert binding.stream_info(kv_out) == binding.stream_info(outs[0])
        kv_info = {"pairs": int(nz.size), "ms": timed_flushed(kv_one, sub) / sub, "dense_call_ms": timed_flushed(dense_one, sub) / sub,
                   "note": "fastsgd_compress_kv on worker 0's non-zero entries against fastsgd_compress on its dense vector; "
                           "same stream; 256 MiB written before every call; not part of value / ms_per_step"}
        del kv_keys, kv_vals, kv_out
    assert all(binding.stream_info(o)[2] == 0 for o in outs) and binding.decode_status() == 0

    # per-kernel durations from CUDA events recorded on the launching stream
    binding.kernel_timing_enable(True)
    barrier()
    for _ in range(sub):
        step()
    torch.cuda.synchronize()
    ktimes = binding.kernel_timing_read()
    binding.kernel_timing_enable(False)

    # tiles the encode pass read a second time, as the kernel counted them (one launch per 8 gradients: the
    # counters hold the last launch's)
    compress_all()
    listed = binding.listed_tiles(min(W, 8))
    if W > 8:
        listed = None

    peak, peak_kind = measured_peak()
    in_bytes = 4.0 * n * W
    alg_comp = 8.0 * n * W + float(sum(stream_bytes))              # two reads of the gradient + stream written
    alg_dec = float(sum(stream_bytes)) + 8.0 * float(sum(kept))    # stream read + read-modify-write of kept entries
    value = in_bytes * world / (ms_step * 1e-3) / 1e9

    per_launch_bytes = {
        "k_abs_sum": 4.0 * n + 8.0 * ((n + 16383) // 16384),
        "k_compress": (8.0 * n * W + float(sum(stream_bytes))) / max(1, (W + 7) // 8),
        "k_decode_accumulate": (float(sum(stream_bytes)) + 8.0 * float(sum(kept))) / max(1, (W + 7) // 8),
    }
    kernels = {}
    for k, (ms, cnt) in ktimes.items():
        if cnt:
            avg = ms / cnt
            kernels[k] = {"launches": cnt, "avg_us": avg * 1e3, "share": None,
                          "achieved_gbs": per_launch_bytes[k] / (avg * 1e-3) / 1e9}
    tot = sum(ms for ms, cnt in ktimes.values()) or 1.0
    for k in kernels:
        kernels[k]["share"] = ktimes[k][0] / tot
    dom = max(kernels, key=lambda k: kernels[k]["share"]) if kernels else None
    # DRAM traffic per launch: counted from what the kernel did (tiles it listed for a second read), and, for the
    # default workload, the dram__bytes_read.sum + dram__bytes_write.sum of the ncu capture summarised under profiles/
    tr_c = tr_d = None
    if listed is not None:
        tr_c, tr_d = traffic_model(n, stream_bytes, kept, listed)
    default_c2 = args.workload == "c2" and args.n is None and args.workers is None and args.keep is None
    per_launch_traffic = {"k_compress": tr_c, "k_decode_accumulate": tr_d, "k_abs_sum": None}
    roofline = None
    if dom:
        traffic = per_launch_traffic.get(dom)
        dur = kernels[dom]["avg_us"] * 1e-6
        roofline = {"bound": "hbm", "kernel": dom, "achieved": kernels[dom]["achieved_gbs"], "peak": peak,
                    "unit": "GB/s", "frac": kernels[dom]["achieved_gbs"] / peak, "peak_kind": f"of {peak_kind}",
                    "traffic": traffic, "traffic_kind": "counted by the kernel: 4nW + 64 KiB per tile it read a second time + streams",
                    "dram_frac": (traffic / dur / 1e9 / peak) if traffic else None,
                    "traffic_ncu": ncu_traffic_of("k_compress_c2_4workers.md") if (default_c2 and dom == "k_compress") else None,
                    "algorithmic_bytes_per_launch": per_launch_bytes[dom]}
        if roofline["frac"] > 1.2:
            roofline["note"] = "frac counts two full reads of every gradient; the kernel skipped most tiles: dram_frac is the hardware figure"

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{args.workload}: {WORKLOADS[args.workload]}", "n": n, "workers": W,
                   "keep_fraction": wl.keep_fraction, "base": wl.base, "tau": wl.tau, "flag_bits": wl.flag_bits,
                   "group_log2": wl.group_log2, "parallelism": "replicas only" if world > 1 else "single GPU",
                   "launch": "cuda graph replay of the step's C-ABI calls" if g_step else "eager C-ABI calls",
                   "l2": ("inputs of one step (W x 4n bytes) exceed 1.5 x the L2 size; no explicit flush" if step_exceeds_l2
                          else "256 MiB written before every timed step (its inputs would fit in L2)")
                         + "; decompress-only leg and the per-step median/min: 256 MiB written before every call",
                   "dense_zero_fill": "the caller's zeroing of the accumulator (4n bytes) is not part of value; see dense_zero_fill_ms"},
        "clocks": sampler.summary(),
        "ms_per_step_each": series_stats(each),
        "gpu_launches": launches,
        "elements_per_s": n * W * world / (ms_step * 1e-3),
        "combined": {"algorithmic_gbs": (alg_comp + alg_dec) * world / (ms_step * 1e-3) / 1e9,
                     "frac_of_hbm_peak": (alg_comp + alg_dec) / (ms_step * 1e-3) / 1e9 / peak,
                     "frac_of_nominal_8000": (alg_comp + alg_dec) / (ms_step * 1e-3) / 1e9 / 8000.0},
        "compress": {"ms": ms_comp, "input_gbs": in_bytes / (ms_comp * 1e-3) / 1e9,
                     "algorithmic_gbs": alg_comp / (ms_comp * 1e-3) / 1e9,
                     "frac_of_hbm_peak": alg_comp / (ms_comp * 1e-3) / 1e9 / peak,
                     "frac_of_nominal_8000": alg_comp / (ms_comp * 1e-3) / 1e9 / 8000.0},
        "decompress": {"ms": ms_dec, "input_gbs": in_bytes / (ms_dec * 1e-3) / 1e9,
                       "algorithmic_gbs": alg_dec / (ms_dec * 1e-3) / 1e9,
                       "frac_of_hbm_peak": alg_dec / (ms_dec * 1e-3) / 1e9 / peak,
                       "frac_of_nominal_8000": alg_dec / (ms_dec * 1e-3) / 1e9 / 8000.0,
                       "sector_bytes": float(sum(stream_bytes)) + 64.0 * float(sum(kept)),
                       "sector_gbs": (float(sum(stream_bytes)) + 64.0 * float(sum(kept))) / (ms_dec * 1e-3) / 1e9},
        "dense_zero_fill_ms": ms_zero,
        "sparse_adam_update": {"ms": ms_adam, "packed_state_ms": ms_adam_packed,
                               "touched_bytes": float(sum(stream_bytes)) + 40.0 * float(sum(kept)),
                               "note": "decode + Adam step on decoded coordinates only; one launch (up to 8 streams); "
                                       "256 MiB written before every call; not part of value / ms_per_step"},
        "compress_kv": kv_info,
        "stream": {"bytes_per_worker": float(sum(stream_bytes)) / W, "kept_per_worker": float(sum(kept)) / W,
                   "bits_per_kept_entry": 8.0 * sum(stream_bytes) / max(1, sum(kept)),
                   "ratio_vs_dense_fp32": in_bytes / max(1.0, float(sum(stream_bytes)))},
        "kernels": kernels,
        "roofline": roofline,
    }
    if tr_c is not None:
        line["combined"]["dram_frac"] = (tr_c + tr_d) / (ms_step * 1e-3) / 1e9 / peak
        line["combined"]["dram_frac_of_nominal_8000"] = (tr_c + tr_d) / (ms_step * 1e-3) / 1e9 / 8000.0
        line["compress"]["dram_frac"] = tr_c / (ms_comp * 1e-3) / 1e9 / peak
        line["listed_tiles"] = {"per_worker": listed, "of": (n + TILE - 1) // TILE}
    if sustained:
        mhz_b, mhz_s = line["clocks"].get("sm_mhz"), sustained.get("sm_mhz")
        sustained["value"] = in_bytes * world / (sustained["ms_per_step"] * 1e-3) / 1e9
        sustained["frac"] = (alg_comp + alg_dec) / (sustained["ms_per_step"] * 1e-3) / 1e9 / peak
        sustained["frac_of_nominal_8000"] = (alg_comp + alg_dec) / (sustained["ms_per_step"] * 1e-3) / 1e9 / 8000.0
        if tr_c is not None:
            sustained["dram_frac"] = (tr_c + tr_d) / (sustained["ms_per_step"] * 1e-3) / 1e9 / peak
        sustained["ms_x_mhz"] = sustained["ms_per_step"] * mhz_s if mhz_s else None
        sustained["burst_ms_x_mhz"] = ms_step * mhz_b if mhz_b else None
        line["sustained"] = sustained

    # ---- end to end through the host-buffer C-ABI calls (pinned host memory)
    if not args.no_e2e:
        scratch = torch.empty(binding.host_scratch_bytes(n, pg), dtype=torch.uint8, device=dev)
        host_outs = [torch.zeros(cap, dtype=torch.uint8).pin_memory() for _ in range(W)]
        host_dense = torch.zeros(n, dtype=torch.float32).pin_memory()
        produced = [0] * W

        def e2e_step():
            for w in range(W):
                rc, produced[w], st = binding.compress_host(host_grads[w], pg, host_outs[w], scratch)
                assert rc == 0 and st == 0, (rc, st)
            rc, st = binding.decompress_accumulate_host(host_outs, produced, n, pg, host_dense, scratch)
            assert rc == 0 and st == 0, (rc, st)

        e2e_steps = max(2, min(args.steps, 5))
        e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        torch.cuda.synchronize()
        dt = multirank.max_over_ranks(time.perf_counter() - t0, world, dev)
        line["e2e"] = {"value": in_bytes * world * e2e_steps / dt / 1e9, "unit": UNIT, "steps": e2e_steps,
                       "h2d_bytes_per_step": int(4 * n * W + sum(produced)),
                       "d2h_bytes_per_step": int(sum(produced) + 64 * W + 4 * n + 8)}
        del scratch

    # ---- the oracle on this machine's host cores (reported baseline, not the target)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        po = oracle.params(wl.base, wl.tau, wl.flag_bits, wl.group_log2)
        reps, t_cpu = 0, 0.0
        odense = np.zeros(n, np.float32)
        while t_cpu < 10.0 and reps < 64:       # a bounded sample: about 10 s of single-thread work
            t0 = time.perf_counter()
            streams = []
            for g in wl.grads:
                rc, s = oracle.compress(g, po)
                assert rc == 0
                streams.append(s)
            for s in streams:
                assert oracle.decompress_accumulate(s, n, po, odense) == 0
            t_cpu += time.perf_counter() - t0
            reps += 1
        line["cpu_baseline"] = {"value": in_bytes * reps / t_cpu / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
                                "host_cores_present": os.cpu_count(),
                                "sample": f"{reps} full step(s) of {args.workload} ({W} workers, n={n}), single thread"}

    # ---- the other configurations (one GPU, default workload only)
    if rank == 0 and world == 1 and default_c2 and not args.no_configs:
        c2_entry = {
            "n": n, "workers": W, "keep": wl.keep_fraction, "kept": int(sum(kept)), "stream_bytes": int(sum(stream_bytes)),
            "listed_tiles": int(sum(listed)) if listed else None, "tiles": W * ((n + TILE - 1) // TILE),
            "combined_ms": series_stats(each), "compress_ms": {"mean": ms_comp}, "decompress_ms": {"mean": ms_dec},
            "input_gbs": value, "frac": line["combined"]["frac_of_hbm_peak"],
            "frac_nominal_8000": line["combined"]["frac_of_nominal_8000"], "dram_frac": line["combined"].get("dram_frac"),
            "note": "the headline: value and ms_per_step are the mean of a CUDA-graph replay of --steps steps"}
        del grads, outs, dense, host_grads, wl
        torch.cuda.empty_cache()
        try:
            line["configs"] = configs_table(torch, binding, workloads, dev, peak, 20, c2_entry, use_graph=not args.no_graph)
            line["configs_launch"] = "every leg a CUDA graph replay of its C-ABI calls, each repetition timed by its own pair of events after 256 MiB were written" if not args.no_graph else "eager C-ABI calls"
        except Exception as exc:          # the headline stands by itself
            line["configs"] = {"c2": c2_entry}
            line["configs_error"] = repr(exc)

    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
