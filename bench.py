#!/usr/bin/env python
"""Benchmark of the segmented scan / sum / SpMV library on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = one pass of the segmented-scan hot path (tile load, tensor-core block
prefix, flag pass, revert, carries, look-back, store) over the headline workload:
the density-sweep configuration (n = 2^30 fp16 values uniform in [-1,1), fp32
output) with Bernoulli(1e-3) start flags.  The line printed at the end also
carries, under "configs", short measurements of all five benchmark
configurations (N = 1 only).  Inputs are seeded and synthetic (mmv_inputs); they
are generated on the host and uploaded before the timed region.  Every working
set here is larger than the 126 MB L2 except configuration 1, for which a
buffer larger than L2 is rewritten between timed launches.

With --impl reference the same metric is produced by the CPU oracle on the
box's host cores (a deliberately plain sequential program).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

import mmv_inputs as gen  # noqa: E402

METRIC = "segmented scan throughput (input elements per second)"
UNIT = "Gelem/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0

# DRAM traffic of the headline kernel from the ncu capture of its n = 2^26 case
# (the summary of that capture is kept with the other profiles): reads 3.003 B/element, writes 4 B/element minus
# the ~58 MB of output that are still in L2 when a launch ends; both scale with n.
NCU_READ_BYTES_PER_ELEM = 3.003
NCU_WRITE_BYTES_PER_ELEM = 4.0
NCU_WRITE_L2_RESIDUE_BYTES = 57.7e6


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--log2n", type=int, default=30, help="headline size (default 2^30)")
    ap.add_argument("--case", default="p1e-3", help="flag pattern of the headline workload")
    ap.add_argument("--no-configs", action="store_true", help="skip the per-configuration table")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU baseline")
    ap.add_argument("--scan-shape", type=int, default=-1, choices=[-1, 0, 2],
                    help="with --profile-case: force the wide (0) or narrow (2) tiles of the floating-point scan (-1: the library chooses)")
    ap.add_argument("--profile-case", default=None, choices=["scan_f16", "scan_i8", "seg_sum", "seg_sum_short", "seg_sum_mid", "spmv", "minmax", "wide", "compress"],
                    help="run one small case a few times and exit (the command profiled with ncu)")
    return ap.parse_args()


def measured_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs.

    Every sample is stamped when it arrives; summary(t0, t1) keeps the ones taken inside the
    window, i.e. while the GPU was under the benchmark's load.
    """
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), line.strip()))

    def __exit__(self, *a):
        if self.proc is not None:
            self.proc.kill()
            self.proc.wait()
            self.thread.join(timeout=1.0)

    def count_between(self, t0, t1):
        return sum(1 for t, _ in list(self.rows) if t0 <= t <= t1)

    def summary(self, t0=float("-inf"), t1=float("inf")):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for t, r in list(self.rows):
            if not (t0 <= t <= t1):
                continue
            parts = [p.strip() for p in r.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


# ---------------------------------------------------------------------------
# the reference arm: the CPU oracle, as it stands
# ---------------------------------------------------------------------------
def time_oracle_scan(x, f, reps=2, got=()):
    """Times the oracle's fp16 scan on (x, f).  The baseline leg has the oracle's result for the whole
    workload in hand, so it also reports how far each result in `got` (CUDA or host tensors: the device
    scan and the chunked scan of the host vectors) is from it, as the largest |error| / bound over all
    elements."""
    import oracle
    oracle.build()
    best, z, a = float("inf"), None, None
    for _ in range(reps):
        t0 = time.perf_counter()
        z, a = oracle.seg_scan_f16(x, f)
        best = min(best, time.perf_counter() - t0)
    worst = []
    for g in got:
        w, step = 0.0, 1 << 26
        for o in range(0, x.shape[0], step):
            _, ratio, _ = oracle.check_fp(g[o:o + step].cpu().numpy(), z[o:o + step], a[o:o + step])
            w = max(w, ratio)
        worst.append(w)
    return best, worst


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    n = 1 << min(args.log2n, 27)          # bounded sample of the headline workload
    x = gen.f16_uniform(5, n)
    f = gen.config5_flags(n, args.case)
    for _ in range(max(1, min(args.warmup, 2))):
        oracle.seg_scan_f16(x, f)
    steps = max(1, args.steps)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.seg_scan_f16(x, f)
    dt = (time.perf_counter() - t0) / steps
    val = n / dt / 1e9
    sample = f"first 2^{int(np.log2(n))} elements of the headline workload per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"C5 seg-scan n=2^{args.log2n} fp16 U[-1,1) -> fp32, uint8 flags {args.case}",
                   "sample_per_step": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ---------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------
def shard_plan(world: int, rank: int, log2n: int):
    """Work of one rank.  N = 1: the whole vector.  N > 1: ONE vector of world * 2^log2n elements cut into
    contiguous shards, rank r holding elements [r * 2^log2n, (r + 1) * 2^log2n) (weak scaling: the shard size
    is fixed).  Every shard is scanned by itself; the one exchange of the path is an all-gather of the
    16-byte shard records, after which every rank folds the records in front of it into its carry."""
    n = 1 << log2n
    if n % gen.CHUNK and world > 1:
        raise SystemExit("bench: shards are whole generator chunks (log2n >= 24) when --gpus > 1")
    return {"rank": rank, "world": world, "n": n, "global_n": world * n,
            "first_chunk": rank * (n // gen.CHUNK) if world > 1 else 0,
            "collectives_on_data_path": 1 if world > 1 else 0}


def shard_record(last_value_bits: int, first_start: int, n: int):
    """The 16-byte record of a shard as two int64 words, laid out as mmv_seg_scan_shard writes it:
    word 0 = value bits | has_start << 32, word 1 = index of the first start (n if none)."""
    has = 1 if first_start < n else 0
    return np.array([(int(last_value_bits) & 0xffffffff) | (has << 32), int(first_start)], dtype=np.int64)


def fold_records(records, rank: int, is_float: bool = True):
    """Carry into shard `rank`: the fold of the records in front of it with the operator of the segmented
    scan on pairs, (v1, f1) + (v2, f2) = (f2 ? v2 : v1 + v2, f1 | f2) (Section 4.2, steps 3-5, applied to the
    shards' last values and flags).  `records`: world x 2 int64 as gathered.  Written for the CPU test of the
    shard plan and for the benchmark's own cross-check; the library folds on the device."""
    rec = np.asarray(records, dtype=np.int64).reshape(-1, 2)
    carry = np.float32(0.0) if is_float else 0
    for r in range(rank):
        bits = int(rec[r, 0]) & 0xffffffff
        has = (int(rec[r, 0]) >> 32) & 1
        if is_float:
            v = np.array([bits], dtype=np.uint32).view(np.float32)[0]
            carry = v if has else np.float32(carry + v)
        else:
            v = bits - (1 << 32) if bits >= (1 << 31) else bits
            carry = v if has else ((carry + v + (1 << 31)) % (1 << 32)) - (1 << 31)
    return carry


def reduce_max_over_ranks(torch, dist, values, device):
    """Max over ranks of a list of floats (identity when the process group is not initialised)."""
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if dist is not None and dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_value(world: int, n_per_rank: int, ms: float) -> float:
    """Gelem/s of the whole job: all ranks' elements over the slowest rank's time."""
    return world * n_per_rank / ms / 1e6

def event_time_ms(torch, fn, steps, flush=None):
    """Average device time of fn() over `steps` launches, CUDA events on the current stream."""
    if flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1) / steps
    total = 0.0
    for _ in range(steps):
        flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        e1.synchronize()
        total += e0.elapsed_time(e1)
    return total / steps


def graph_time_ms(torch, fn, steps, flush=None):
    """The same measurement with the call captured once in a CUDA graph and replayed: the device time of
    the call's memset and kernels without the host's per-call work (tensor-map encoding, ctypes)."""
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    torch.cuda.synchronize()
    return event_time_ms(torch, g.replay, steps, flush)


def bench_configs(torch, mmv, peak, steps, warmup, l2_flush, cpu_leg):
    """Short measurements of the five configurations (device-resident inputs).  With cpu_leg the
    oracle is timed on one host core over the whole input of every configuration (the baseline leg)
    and, its result being in hand, the device result is compared with it.  Parity at these sizes is
    also a test: tests/test_gpu_full_size.py makes the same calls."""
    res = []

    def baseline(units, run_oracle, compare):
        """One run of the oracle over the whole configuration -> the record's cpu_baseline entry."""
        if not cpu_leg:
            return {}
        import oracle
        t0 = time.perf_counter()
        want = run_oracle(oracle)
        sec = time.perf_counter() - t0
        d = {"value": units / sec / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
             "sample": f"the whole configuration, one run, {sec:.2f} s"}
        d.update(compare(oracle, want))
        return {"cpu_baseline": d}

    def fp_compare(got):
        def cmp(oracle, want):
            ok, ratio, i = oracle.check_fp(got, want[0], want[1])
            if not ok:
                raise SystemExit(f"bench: device result outside the bound (ratio {ratio} at {i})")
            return {"device_result_worst_err_over_bound": ratio}
        return cmp

    def rec(name, units, bytes_, ms, extra=None):
        d = {"config": name, "units": int(units), "ms": ms, "gelem_s": units / ms / 1e6,
             "gb_s": bytes_ / ms / 1e6, "frac_of_measured_peak": bytes_ / ms / 1e6 / peak,
             "frac_of_8tbs": bytes_ / ms / 1e6 / NOMINAL_HBM_GBS}
        if extra:
            d.update(extra)
        res.append(d)

    def run_scan(name, x, f, flush=None):
        n = x.shape[0]
        dt = mmv.F16_TO_F32 if x.dtype == np.float16 else mmv.I8_TO_I32
        xd, fd = torch.from_numpy(x).cuda(), torch.from_numpy(f).cuda()
        out = torch.empty(n, dtype=torch.float32 if dt == mmv.F16_TO_F32 else torch.int32, device="cuda")
        ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, dt, mmv.SEG_FLAGS_U8, n)
        fn = lambda: mmv.seg_scan(xd, fd, out=out, workspace=ws)  # noqa: E731
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        ms = event_time_ms(torch, fn, steps, flush)
        ms_graph = graph_time_ms(torch, fn, steps, flush) if n <= (1 << 26) else None
        assert mmv.last_async_status(ws) == 0
        bpe = (2 if dt == mmv.F16_TO_F32 else 1) + 1 + 4
        if dt == mmv.F16_TO_F32:
            extra = baseline(n, lambda o: o.seg_scan_f16(x, f), fp_compare(out.cpu().numpy()))
        else:
            def cmp_int(oracle, want):
                bad = int(np.count_nonzero(out.cpu().numpy() != want))
                if bad:
                    raise SystemExit(f"bench: {bad} mismatches in {name}")
                return {"device_result_mismatches": 0}
            extra = baseline(n, lambda o: o.seg_scan_i8(x, f), cmp_int)
        if ms_graph is not None:
            extra = {**extra, "ms_replayed_from_cuda_graph": ms_graph}
        rec(name, n, n * bpe, ms, extra)
        del xd, fd, out, ws

    x, f = gen.config1()
    run_scan("C1 seg-scan n=2^20 fp16 flags 1/64 (L2 flushed between launches)", x, f, l2_flush)

    x, off = gen.config2()
    n, nseg = x.shape[0], off.shape[0] - 1
    xd, od = torch.from_numpy(x).cuda(), torch.from_numpy(off).cuda()
    out = torch.empty(nseg, dtype=torch.float32, device="cuda")
    ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, n, nseg)
    fn = lambda: mmv.seg_sum(xd, od, out=out, workspace=ws)  # noqa: E731
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ms = event_time_ms(torch, fn, steps)
    ms_graph = graph_time_ms(torch, fn, steps)
    assert mmv.last_async_status(ws) == 0
    rec("C2 seg-sum n=2^26 fp16 N(0,1), CSR offsets len U{1..4096}", n, 2 * n + 4 * (nseg + 1) + 4 * nseg, ms,
        {"segments": nseg, "ms_replayed_from_cuda_graph": ms_graph, **baseline(n, lambda o: o.seg_sum_csr_f16(x, off), fp_compare(out.cpu().numpy()))})
    del xd, od, out, ws

    # the same recipe four times larger (the n >= 2^28 point of the target), and the flag-encoded
    # form of the segmented sum over the same segments (start flags instead of offsets)
    x, off = gen.config2(1 << 28)
    n, nseg = x.shape[0], off.shape[0] - 1
    xd, od = torch.from_numpy(x).cuda(), torch.from_numpy(off).cuda()
    out = torch.empty(nseg, dtype=torch.float32, device="cuda")
    ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, n, nseg)
    fn = lambda: mmv.seg_sum(xd, od, out=out, workspace=ws)  # noqa: E731
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ms = event_time_ms(torch, fn, steps)
    assert mmv.last_async_status(ws) == 0
    rec("C2x4 seg-sum n=2^28 fp16 N(0,1), CSR offsets len U{1..4096}", n, 2 * n + 4 * (nseg + 1) + 4 * nseg, ms,
        {"segments": nseg, **baseline(n, lambda o: o.seg_sum_csr_f16(x, off), fp_compare(out.cpu().numpy()))})
    del od, ws
    f = gen.start_flags_of_offsets(off, n)
    fd = torch.from_numpy(f).cuda()
    outf = torch.empty(n, dtype=torch.float32, device="cuda")
    kd = torch.zeros(1, dtype=torch.int64, device="cuda")
    ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.F16_TO_F32, mmv.SEG_FLAGS_U8, n)
    fn = lambda: mmv.seg_sum(xd, fd, out=outf, num_segments=kd, workspace=ws)  # noqa: E731
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ms = event_time_ms(torch, fn, steps)
    assert mmv.last_async_status(ws) == 0
    k = int(kd.item())
    if k != nseg - int(np.count_nonzero(np.diff(off.astype(np.int64)) == 0)):
        raise SystemExit(f"bench: flag-form seg-sum found {k} segments")
    rec("N1 seg-sum (start flags) n=2^28 fp16 N(0,1), same segments as C2x4", n, 2 * n + n + 4 * k, ms,
        {"segments": k, **baseline(n, lambda o: o.seg_sum_flags_f16(x, f), fp_compare(outf[:k].cpu().numpy()))})
    del xd, fd, out, outf, ws

    # and sixteen times larger: the fixed cost of a call (launch, set-up, the partition of the offsets and the
    # grid-wide barrier behind it, the first loads: about 10 us) is a tenth of the call at n = 2^28 and a
    # fortieth here, so this line shows the rate the kernel sustains
    x, off = gen.config2(1 << 30)
    n, nseg = x.shape[0], off.shape[0] - 1
    xd, od = torch.from_numpy(x).cuda(), torch.from_numpy(off).cuda()
    out = torch.empty(nseg, dtype=torch.float32, device="cuda")
    ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, n, nseg)
    fn = lambda: mmv.seg_sum(xd, od, out=out, workspace=ws)  # noqa: E731
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ms = event_time_ms(torch, fn, steps)
    assert mmv.last_async_status(ws) == 0
    rec("C2x16 seg-sum n=2^30 fp16 N(0,1), CSR offsets len U{1..4096}", n, 2 * n + 4 * (nseg + 1) + 4 * nseg, ms,
        {"segments": nseg, **baseline(n, lambda o: o.seg_sum_csr_f16(x, off), fp_compare(out.cpu().numpy()))})
    del xd, od, out, ws

    x, f = gen.config3()
    run_scan("C3 seg-scan n=2^28 int8 flags 1e-3", x, f)

    # configuration 4, and the same with 10 % of the rows empty (the paper's corner case of empty rows)
    for name, empty in (("C4 CSR SpMV 2^20 rows, nnz/row Zipf(1.5) cap 1e4", 0.0),
                        ("C4e the same with 10 % of the rows empty", 0.1)):
        rowptr, col, val, xv = gen.config4(empty_fraction=empty)
        rows, nnz = rowptr.shape[0] - 1, val.shape[0]
        rd, cd, vd, xd = (torch.from_numpy(t).cuda() for t in (rowptr, col, val, xv))
        y = torch.empty(rows, dtype=torch.float32, device="cuda")
        ws = mmv.alloc_workspace(mmv.OP_SPMV_CSR, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, nnz, rows)
        fn = lambda: mmv.spmv_csr(rd, cd, vd, xd, y=y, workspace=ws)  # noqa: E731
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        ms = event_time_ms(torch, fn, steps)
        assert mmv.last_async_status(ws) == 0
        rec(name, nnz, 6 * nnz + 4 * (rows + 1) + 4 * xv.shape[0] + 4 * rows, ms,
            {"nnz": nnz, **baseline(nnz, lambda o: o.spmv_csr(rowptr, col, val, xv), fp_compare(y.cpu().numpy()))})
        del rd, cd, vd, xd, y, ws
    # The paper's other segmented-sum shapes: segment lengths with the minimum / average / maximum of the
    # matrices of its Table 5.1, about 2^26 fp16 values each (the dense-boundary regime of the kernel).
    for kind in gen.ROW_LENGTH_MIXES:
        x, off = gen.seg_sum_row_mix(kind, 1 << 26)
        n, nseg = x.shape[0], off.shape[0] - 1
        xd, od = torch.from_numpy(x).cuda(), torch.from_numpy(off).cuda()
        out = torch.empty(nseg, dtype=torch.float32, device="cuda")
        ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, n, nseg)
        fn = lambda: mmv.seg_sum(xd, od, out=out, workspace=ws)  # noqa: E731
        for _ in range(warmup):
            fn()
        torch.cuda.synchronize()
        ms = event_time_ms(torch, fn, steps)
        assert mmv.last_async_status(ws) == 0
        lens = np.diff(off.astype(np.int64))
        rec(f"T5.1 seg-sum fp16, segment lengths min/avg/max {int(lens.min())}/{lens.mean():.0f}/{int(lens.max())} ({kind})",
            n, 2 * n + 4 * (nseg + 1) + 4 * nseg, ms, {"segments": nseg})
        del xd, od, out, ws

    # The blocked sparse-attention matrices of the paper's SpMV experiment: 65,536 rows and columns,
    # 2 global and 3 window blocks, block sizes 2..64, 2..8 random blocks ("b-X_r-Y").  One record for all
    # twelve; bytes as for C4.  The vector (256 KB) stays in cache, unlike C4's.
    bsa = []
    for block in gen.BSA_BLOCKS:
        for rb in gen.BSA_RANDOM:
            rowptr, col, val, xv = gen.block_sparse_attention_csr(block, rb)
            rows, nnz = rowptr.shape[0] - 1, val.shape[0]
            rd, cd, vd, xd = (torch.from_numpy(t).cuda() for t in (rowptr, col, val, xv))
            y = torch.empty(rows, dtype=torch.float32, device="cuda")
            ws = mmv.alloc_workspace(mmv.OP_SPMV_CSR, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, nnz, rows)
            fn = lambda: mmv.spmv_csr(rd, cd, vd, xd, y=y, workspace=ws)  # noqa: E731
            for _ in range(warmup):
                fn()
            torch.cuda.synchronize()
            ms = event_time_ms(torch, fn, steps, l2_flush if 6 * nnz < (256 << 20) else None)
            assert mmv.last_async_status(ws) == 0
            bytes_ = 6 * nnz + 4 * (rows + 1) + 4 * xv.shape[0] + 4 * rows
            bsa.append({"matrix": f"b-{block}_r-{rb}", "nnz": nnz, "us": ms * 1e3, "gnnz_s": nnz / ms / 1e6,
                        "gb_s": bytes_ / ms / 1e6})
            del rd, cd, vd, xd, y, ws
    res.append({"config": "BSA CSR SpMV, blocked sparse attention 65,536 x 65,536 (L2 flushed between launches of the small ones)",
                "matrices": bsa})
    torch.cuda.empty_cache()
    return res


def run_ours(args):
    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        # (a bounded time-out: a rank that dies leaves the others with an error, not with an endless wait)
        import datetime
        dist.init_process_group("nccl", device_id=torch.device("cuda", local), timeout=datetime.timedelta(seconds=300))

    import paper_2506_23906_b200 as mmv

    plan = shard_plan(world, rank, args.log2n)
    n = plan["n"]
    x = gen.config5_values(n, first_chunk=plan["first_chunk"])
    f = gen.config5_flags(n, args.case, first_chunk=plan["first_chunk"])
    peak, peak_kind = measured_peak()

    # pinned host buffers (end-to-end leg) and device-resident copies (kernel leg)
    xh = torch.from_numpy(x).pin_memory()
    fh = torch.from_numpy(f).pin_memory()
    oh = torch.empty(n, dtype=torch.float32).pin_memory()
    xd = torch.empty(n, dtype=torch.float16, device="cuda")
    fd = torch.empty(n, dtype=torch.uint8, device="cuda")
    od = torch.empty(n, dtype=torch.float32, device="cuda")
    ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.F16_TO_F32, mmv.SEG_FLAGS_U8, n)
    xd.copy_(xh)
    fd.copy_(fh)
    l2_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    # N > 1: this rank's 16-byte shard record and the gathered records of all ranks
    my_record = torch.zeros(2, dtype=torch.int64, device="cuda")
    records = torch.zeros(2 * world, dtype=torch.int64, device="cuda")

    if world == 1:
        def step():
            mmv.seg_scan(xd, fd, out=od, workspace=ws)
        load_step = step
    else:
        def step():
            # shard scan -> one all-gather of the records (NCCL, the path's only exchange) -> local fold + carry
            mmv.seg_scan_shard(xd, fd, rank == 0, od, my_record, ws)
            dist.all_gather_into_tensor(records, my_record)
            mmv.seg_scan_shard_finish(records, rank, world, od, torch.float16)

        def load_step():
            # the same kernels without the exchange: what keeps the GPU busy while the clocks are sampled (every
            # rank makes its own number of these, so they must not contain a collective)
            mmv.seg_scan_shard(xd, fd, rank == 0, od, my_record, ws)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clk:
        for _ in range(max(3, args.warmup)):
            step()
        barrier()
        launches0 = mmv.kernel_launch_count()
        t_load0 = time.perf_counter()
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        barrier()
        launches = mmv.kernel_launch_count() - launches0
        # The timed region can be shorter than the sampler's period: keep the GPU under the very same
        # load (untimed) until a handful of clock samples have been taken inside the window.
        t_extra0 = time.perf_counter()
        while clk.count_between(t_load0, time.perf_counter()) < 6 and time.perf_counter() - t_extra0 < 1.5:
            for _ in range(16):
                load_step()
            torch.cuda.synchronize()
        t_load1 = time.perf_counter()
    clocks = clk.summary(t_load0, t_load1)
    clocks["window"] = "timed steps followed by identical untimed steps until >= 6 samples"
    ms = e0.elapsed_time(e1) / args.steps
    if mmv.last_async_status(ws) != 0:
        raise SystemExit("bench: device-side error status")

    # end to end: the library's call for HOST vectors (pinned): every step copies the 3 n input bytes
    # to the device, scans, and brings the 4 n result bytes back, chunk by chunk on three streams.
    # N > 1: the shard's inputs are copied in, the shard path above runs, the result is copied out.
    e2e_steps = max(1, min(args.steps, 5))
    e2e_chunk = min(1 << 25, n)
    if world == 1:
        scratch = mmv.host_scan_scratch(mmv.F16_TO_F32, e2e_chunk)

        def e2e_step():
            mmv.seg_scan_host(xh, fh, out=oh, chunk=e2e_chunk, scratch=scratch)
    else:
        scratch = ws

        def e2e_step():
            xd.copy_(xh, non_blocking=True)
            fd.copy_(fh, non_blocking=True)
            step()
            oh.copy_(od, non_blocking=True)
    e2e_step()
    barrier()
    if mmv.last_async_status(scratch) != 0:
        raise SystemExit("bench: device-side error status (host scan)")
    # (the baseline leg below compares every element of this result with the oracle's; without that leg the
    #  end of the vector is at least compared with the device scan)
    if (args.no_cpu or world > 1) and not torch.allclose(oh[-(1 << 20):], od[-(1 << 20):].cpu(), rtol=1e-4, atol=1e-3):
        raise SystemExit("bench: the scan of the host vectors and the device scan disagree")
    if world > 1:
        # cross-check of the exchange: the carry this rank added must be the fold of the gathered records as
        # the definition gives it, and element 0 must continue the shard in front (or start a segment)
        carry = float(fold_records(records.cpu().numpy(), rank))
        first = int(my_record.cpu()[1])
        want0 = float(x[0]) + (0.0 if (rank == 0 or first == 0) else carry)
        if abs(float(od[0].cpu()) - want0) > 2e-3 * (abs(carry) + 1.0) + 1e-6:
            raise SystemExit(f"bench: rank {rank}: element 0 is {float(od[0].cpu())}, expected {want0}")
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps

    ms, e2e_ms = reduce_max_over_ranks(torch, dist if world > 1 else None, [ms, e2e_ms], "cuda")

    if rank == 0:
        bytes_per_launch = 7 * n
        achieved = bytes_per_launch / ms / 1e6
        line = {
            "metric": METRIC, "value": whole_job_value(world, n, ms), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"C5 seg-scan n=2^{args.log2n} fp16 U[-1,1) -> fp32, uint8 flags {args.case}",
                       "n_per_gpu": n, "timing": "inputs (7 B/elem working set) larger than L2; no flush needed",
                       "parallelism": ("one GPU" if world == 1 else
                                       f"one vector of {world} x 2^{args.log2n} elements in {world} contiguous shards; per step one "
                                       f"all-gather of {world} 16-byte shard records (NCCL), carries folded locally")},
            "clocks": clocks,
            "e2e": {"value": whole_job_value(world, n, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": 3 * n,
                    "d2h_bytes_per_step": 4 * n, "ms_per_step": e2e_ms, "steps": e2e_steps,
                    "call": (f"mmv_seg_scan_host, pinned host vectors, chunks of 2^{int(np.log2(e2e_chunk))} elements" if world == 1
                             else "copy in, mmv_seg_scan_shard, all-gather, mmv_seg_scan_shard_finish, copy out (pinned host vectors)")},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": achieved / peak, "peak_kind": peak_kind,
                         "frac_of_8tbs_nominal": achieved / NOMINAL_HBM_GBS,
                         "algorithmic_bytes_per_elem": 7,
                         "algorithmic_bytes": bytes_per_launch,
                         "traffic": (NCU_READ_BYTES_PER_ELEM + NCU_WRITE_BYTES_PER_ELEM) * n - NCU_WRITE_L2_RESIDUE_BYTES,
                         "traffic_kind": "constant from an ncu capture of this kernel at n=2^26, scaled by n (not a counter of this run)"},
        }
        del xh, fh
        if not args.no_cpu and world == 1:
            mmv.seg_scan(xd, fd, out=od, workspace=ws)
            sec, (worst, worst_host) = time_oracle_scan(x, f, reps=2, got=(od, oh))
            line["cpu_baseline"] = {"value": n / sec / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": f"the whole headline workload (n=2^{args.log2n}), best of 2, {sec:.2f} s",
                                    "device_result_worst_err_over_bound": worst,
                                    "host_vector_result_worst_err_over_bound": worst_host}
            if not (worst <= 1.0 and worst_host <= 1.0):
                raise SystemExit(f"bench: a result is outside the bound (device {worst}, host vectors {worst_host})")
            # the same definition chunk-parallel over all cores this process may use (sequential carry hand-over)
            import oracle
            best_all, used = float("inf"), 0
            for _ in range(2):
                t0 = time.perf_counter()
                _, _, used = oracle.seg_scan_f16_all_cores(x, f)
                best_all = min(best_all, time.perf_counter() - t0)
            line["cpu_baseline_all_cores"] = {"value": n / best_all / 1e9, "unit": UNIT, "cores": used, "kind": "oracle, chunk-parallel",
                                              "sample": f"the whole headline workload (n=2^{args.log2n}), best of 2, {best_all:.2f} s"}
        del oh
        del xd, fd, od
        torch.cuda.empty_cache()
        if world == 1 and not args.no_configs:
            def l2_flush():
                l2_buf.zero_()
            cfgs = bench_configs(torch, mmv, peak, min(args.steps, 20), max(3, args.warmup), l2_flush, not args.no_cpu)
            # the seven flag patterns of configuration 5 on the headline values
            xd = torch.from_numpy(x).cuda()
            od = torch.empty(n, dtype=torch.float32, device="cuda")
            sweep = []
            for case, _ in gen.C5_CASES:
                fc = gen.config5_flags(n, case)
                fd = torch.from_numpy(fc).cuda()
                fn = lambda: mmv.seg_scan(xd, fd, out=od, workspace=ws)  # noqa: E731
                for _ in range(3):
                    fn()
                torch.cuda.synchronize()
                cms = event_time_ms(torch, fn, min(args.steps, 10))
                assert mmv.last_async_status(ws) == 0
                sweep.append({"tag": case, "case": case, "ms": cms, "gelem_s": n / cms / 1e6, "gb_s": 7 * n / cms / 1e6,
                              "frac_of_measured_peak": 7 * n / cms / 1e6 / peak,
                              "frac_of_8tbs": 7 * n / cms / 1e6 / NOMINAL_HBM_GBS})
                del fd
            # the plain scan: no flag vector at all (6 B per element)
            fn = lambda: mmv.seg_scan(xd, None, out=od, workspace=ws)  # noqa: E731
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            cms = event_time_ms(torch, fn, min(args.steps, 10))
            assert mmv.last_async_status(ws) == 0
            sweep.append({"tag": "plain", "case": "no flag vector (plain scan, 6 B/elem)", "ms": cms, "gelem_s": n / cms / 1e6,
                          "gb_s": 6 * n / cms / 1e6, "frac_of_measured_peak": 6 * n / cms / 1e6 / peak,
                          "frac_of_8tbs": 6 * n / cms / 1e6 / NOMINAL_HBM_GBS})
            # the exclusive variant on the headline flags (same traffic)
            fd = torch.from_numpy(f).cuda()
            fn = lambda: mmv.seg_scan(xd, fd, out=od, workspace=ws, exclusive=True)  # noqa: E731
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            cms = event_time_ms(torch, fn, min(args.steps, 10))
            assert mmv.last_async_status(ws) == 0
            sweep.append({"tag": "excl", "case": f"exclusive scan, {args.case}", "ms": cms, "gelem_s": n / cms / 1e6,
                          "gb_s": 7 * n / cms / 1e6, "frac_of_measured_peak": 7 * n / cms / 1e6 / peak,
                          "frac_of_8tbs": 7 * n / cms / 1e6 / NOMINAL_HBM_GBS})
            # bfloat16 input values (the headline values converted on the device), same flags and traffic
            xb = xd.to(torch.bfloat16)
            fn = lambda: mmv.seg_scan(xb, fd, out=od, workspace=ws)  # noqa: E731
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            cms = event_time_ms(torch, fn, min(args.steps, 10))
            assert mmv.last_async_status(ws) == 0
            sweep.append({"tag": "bf16", "case": f"bf16 values, {args.case}", "ms": cms, "gelem_s": n / cms / 1e6,
                          "gb_s": 7 * n / cms / 1e6, "frac_of_measured_peak": 7 * n / cms / 1e6 / peak,
                          "frac_of_8tbs": 7 * n / cms / 1e6 / NOMINAL_HBM_GBS})
            # segmented running maximum and the plain running maximum (CUDA cores: the operator has no inverse)
            wsm = mmv.alloc_workspace(mmv.OP_SEG_SCAN_MINMAX, mmv.F16_TO_F32, mmv.SEG_FLAGS_U8, n)
            for label, fl, per in ((f"running maximum, {args.case}", fd, 7), ("running maximum, no flag vector", None, 6)):
                fn = lambda: mmv.seg_scan_minmax(xd, fl, out=od, workspace=wsm)  # noqa: E731,B023
                for _ in range(3):
                    fn()
                torch.cuda.synchronize()
                cms = event_time_ms(torch, fn, min(args.steps, 10))
                assert mmv.last_async_status(wsm) == 0
                sweep.append({"tag": "max" if fl is not None else "max-plain", "case": label, "ms": cms, "gelem_s": n / cms / 1e6, "gb_s": per * n / cms / 1e6,
                              "frac_of_measured_peak": per * n / cms / 1e6 / peak,
                              "frac_of_8tbs": per * n / cms / 1e6 / NOMINAL_HBM_GBS})
            del wsm
            # int8 values with int64 results (10 B/elem): the headline flags over int8 values made on the device
            xi8 = (xd * 127).to(torch.int8)
            od64 = torch.empty(n, dtype=torch.int64, device="cuda")
            wsw = mmv.alloc_workspace(mmv.OP_SEG_SCAN_WIDE, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
            fn = lambda: mmv.seg_scan_wide(xi8, fd, out=od64, workspace=wsw)  # noqa: E731
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            cms = event_time_ms(torch, fn, min(args.steps, 10))
            assert mmv.last_async_status(wsw) == 0
            sweep.append({"tag": "i8->i64", "case": f"int8 -> int64 scan, {args.case} (10 B/elem)", "ms": cms, "gelem_s": n / cms / 1e6,
                          "gb_s": 10 * n / cms / 1e6, "frac_of_measured_peak": 10 * n / cms / 1e6 / peak,
                          "frac_of_8tbs": 10 * n / cms / 1e6 / NOMINAL_HBM_GBS})
            del xi8, od64, wsw
            # COMPRESS of the headline values under the headline flags (flags are read twice: count, scatter)
            outc = torch.empty(n, dtype=torch.float16, device="cuda")
            kc = torch.zeros(1, dtype=torch.int64, device="cuda")
            wsc = mmv.alloc_workspace(mmv.OP_COMPRESS, mmv.F16_TO_F32, mmv.SEG_FLAGS_U8, n)
            fn = lambda: mmv.compress(xd, fd, out=outc, count=kc, workspace=wsc)  # noqa: E731
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            cms = event_time_ms(torch, fn, min(args.steps, 10))
            kept = int(kc.item())
            cbytes = n + 4 * kept
            sweep.append({"tag": "compress", "case": f"COMPRESS, {args.case} ({kept} kept)", "ms": cms, "gelem_s": n / cms / 1e6,
                          "gb_s": cbytes / cms / 1e6, "frac_of_measured_peak": cbytes / cms / 1e6 / peak,
                          "frac_of_8tbs": cbytes / cms / 1e6 / NOMINAL_HBM_GBS})
            del fd, xb, outc, wsc
            line["configs"] = cfgs
            line["c5_density_sweep"] = sweep
            # a compact digest as the LAST key, so that the end of the line alone shows every case:
            # [name, time in us, GB/s of algorithmic bytes, fraction of the nominal 8 TB/s]
            digest = [[c["config"].split(" ")[0] + (("/" + c["config"].split("(")[-1].rstrip(")")) if c["config"].startswith("T5.1") else ""),
                       round(c["ms"] * 1e3, 1), round(c["gb_s"]), round(c["frac_of_8tbs"], 3)] for c in cfgs if "ms" in c]
            digest += [["C5/" + c["tag"], round(c["ms"] * 1e3, 1), round(c["gb_s"]), round(c["frac_of_8tbs"], 3)] for c in sweep]
            line["digest_name_us_gbs_fracof8tbs"] = digest
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_profile_case(args):
    """One small case, `steps` launches, no timing: the target of the ncu captures under profiles/."""
    import torch
    import paper_2506_23906_b200 as mmv
    torch.cuda.set_device(0)
    mmv.debug_force_scan_shape(args.scan_shape)
    n = 1 << min(args.log2n, 27)
    if args.profile_case in ("scan_f16", "scan_i8"):
        f16 = args.profile_case == "scan_f16"
        x = gen.f16_uniform(5, n) if f16 else gen.i8_uniform(3, n)
        f = gen.config5_flags(n, args.case)
        xd, fd = torch.from_numpy(x).cuda(), torch.from_numpy(f).cuda()
        out = torch.empty(n, dtype=torch.float32 if f16 else torch.int32, device="cuda")
        ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN, mmv.F16_TO_F32 if f16 else mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
        fn = lambda: mmv.seg_scan(xd, fd, out=out, workspace=ws)  # noqa: E731
    elif args.profile_case == "minmax":
        # the segmented running maximum on the flag pattern --case names (p0: no start at all)
        x = gen.f16_uniform(5, n)
        f = gen.config5_flags(n, args.case)
        xd, fd = torch.from_numpy(x).cuda(), torch.from_numpy(f).cuda()
        out = torch.empty(n, dtype=torch.float32, device="cuda")
        ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN_MINMAX, mmv.F16_TO_F32, mmv.SEG_FLAGS_U8, n)
        fn = lambda: mmv.seg_scan_minmax(xd, fd, out=out, workspace=ws)  # noqa: E731
    elif args.profile_case == "wide":
        # int8 values with int64 results on the flag pattern --case names
        x = gen.i8_uniform(3, n)
        f = gen.config5_flags(n, args.case)
        xd, fd = torch.from_numpy(x).cuda(), torch.from_numpy(f).cuda()
        out = torch.empty(n, dtype=torch.int64, device="cuda")
        ws = mmv.alloc_workspace(mmv.OP_SEG_SCAN_WIDE, mmv.I8_TO_I32, mmv.SEG_FLAGS_U8, n)
        fn = lambda: mmv.seg_scan_wide(xd, fd, out=out, workspace=ws)  # noqa: E731
    elif args.profile_case == "compress":
        # COMPRESS of fp16 values under the flag pattern --case names (p0.5: the staged route of warps with many kept elements)
        x = gen.f16_uniform(5, n)
        f = gen.config5_flags(n, args.case)
        xd, fd = torch.from_numpy(x).cuda(), torch.from_numpy(f).cuda()
        out = torch.empty(n, dtype=torch.float16, device="cuda")
        kc = torch.zeros(1, dtype=torch.int64, device="cuda")
        ws = mmv.alloc_workspace(mmv.OP_COMPRESS, mmv.F16_TO_F32, mmv.SEG_FLAGS_U8, n)
        fn = lambda: mmv.compress(xd, fd, out=out, count=kc, workspace=ws)  # noqa: E731
    elif args.profile_case in ("seg_sum", "seg_sum_short", "seg_sum_mid"):
        # configuration 2, or the Table 5.1 mixes with segment lengths 1/6/44 and 18/119/204 (dense boundaries)
        x, off = gen.config2(n) if args.profile_case == "seg_sum" else gen.seg_sum_row_mix(args.profile_case[8:], n)
        n = x.shape[0]
        xd, od = torch.from_numpy(x).cuda(), torch.from_numpy(off).cuda()
        out = torch.empty(off.shape[0] - 1, dtype=torch.float32, device="cuda")
        ws = mmv.alloc_workspace(mmv.OP_SEG_SUM, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, n, off.shape[0] - 1)
        fn = lambda: mmv.seg_sum(xd, od, out=out, workspace=ws)  # noqa: E731
    else:
        rowptr, col, val, xv = gen.config4(rows=1 << 18)
        rd, cd, vd, xd = (torch.from_numpy(t).cuda() for t in (rowptr, col, val, xv))
        y = torch.empty(rowptr.shape[0] - 1, dtype=torch.float32, device="cuda")
        ws = mmv.alloc_workspace(mmv.OP_SPMV_CSR, mmv.F16_TO_F32, mmv.SEG_OFFSETS_I32, val.shape[0], rowptr.shape[0] - 1)
        fn = lambda: mmv.spmv_csr(rd, cd, vd, xd, y=y, workspace=ws)  # noqa: E731
    for _ in range(max(1, args.steps)):
        fn()
    torch.cuda.synchronize()
    print(json.dumps({"profile_case": args.profile_case, "n": n, "status": mmv.last_async_status(ws)}))


def main():
    args = parse_args()
    if args.profile_case:
        run_profile_case(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
