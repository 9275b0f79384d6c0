#!/usr/bin/env python
"""Benchmark of the sparse-embedding train step (pooled lookup forward + backward with fused
row-wise Adagrad) on seeded synthetic input.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl native|reference] [--workload cfg3]

One step = one pass of the whole path over one batch.  Prints ONE JSON line on rank 0.
`value` is whole-job throughput with inputs resident in HBM; `e2e` is the same metric through
the C ABI with inputs in pinned host memory (host->device copies and the device->host read of
the pooled output inside the timed region).  The default line is on configuration 3, the largest
configuration whose tables fit in HBM; on one GPU the same line carries a `workloads` list with
configuration 2, configuration 4 (cached, in steady state) and the centre point of configuration 5,
each measured the same way with its own clocks.  `--workload X` measures X alone.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2305_01515_b200 import workload as wl  # noqa: E402

METRIC = "train_step_embedding_lookups_per_sec"
UNIT = "lookups/s"


NOMINAL_HBM_GBS = 8000.0        # HBM3e of a B200, nominal; fractions are printed against it and the measured copy rate
REPEATS = 5                     # the K-step region is timed this many times; median and min are printed


def make_spec(name: str, rank: int, args=None):
    tables = getattr(args, "tables", 0) if args is not None else 0
    if name == "cfg1":
        return wl.config1(seed=rank)
    if name == "cfg2":
        return wl.config2(seed=rank, tables=tables) if tables else wl.config2(seed=rank)
    if name == "cfg3":
        return wl.config3(seed=rank, tables=tables) if tables else wl.config3(seed=rank)
    if name == "cfg4":
        return wl.config4(seed=rank, hbm_budget_gb=getattr(args, "budget_gb", wl.BENCH_CFG4_BUDGET_GB),
                          n_batches=getattr(args, "warmup", 12) + getattr(args, "steps", 8))
    if name == "cfg5":
        spec = wl.config5(seed=rank, rows=getattr(args, "rows", 50_000_000), batch=getattr(args, "batch", 16384),
                          pooling=getattr(args, "pooling", 50), alpha=getattr(args, "alpha", 1.0),
                          cache_fraction=getattr(args, "cache_fraction", 0.10))
        spec.reuse_prob, spec.reuse_window = 0.0, 0
        return spec
    raise SystemExit(f"unknown workload {name}")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def fractions(gbs: float, peak: float):
    return {"gbs": gbs, "frac_of_measured": gbs / peak, "frac_of_nominal": gbs / NOMINAL_HBM_GBS}


TRAFFIC_FILE = os.path.join(ROOT, "profiles", "ncu_dram_traffic.json")


def kernel_source_hash(files) -> str:
    """sha256 over the kernel sources a profiler capture depends on."""
    import hashlib

    h = hashlib.sha256()
    for f in files:
        with open(os.path.join(ROOT, "paper_2305_01515_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def ncu_traffic_per_lookup(kernel: str, workload: str):
    """DRAM bytes (read + write) per lookup of `kernel` on `workload` from the profiler captures recorded in
    profiles/ncu_dram_traffic.json ({kernel: {workload: record}}), or None when there is no capture for this
    workload or the kernel sources have changed since it was taken (the record carries their hash)."""
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f).get(kernel, {}).get(workload)
    except (OSError, ValueError):
        return None, "no capture file"
    if not rec:
        return None, "no capture of this kernel on this workload"
    if rec.get("source_sha256") != kernel_source_hash(rec.get("source_files", [])):
        return None, "kernel sources changed since the capture"
    return float(rec["dram_bytes_per_lookup"]), rec.get("capture", "")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.idx = gpu_index
        self.t0 = self.t1 = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50", "-i",
                 str(self.idx)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def mark(self, begin: bool):
        if begin:
            self.t0 = time.time()
        else:
            self.t1 = time.time()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        for ts, line in self.rows:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            inside = self.t0 is not None and self.t0 - 0.05 <= ts <= (self.t1 or ts) + 0.15
            try:
                if inside:
                    sm.append(float(f[1]))
                mx = float(f[2])
            except ValueError:
                continue
            if inside:
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
        if not sm:       # region shorter than one sample: use every sample taken
            for ts, line in self.rows:
                f = [x.strip() for x in line.split(",")]
                try:
                    sm.append(float(f[1]))
                except (ValueError, IndexError):
                    pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_sample(spec, idx, off, grad, tables):
    """Compact sub-problem for the CPU oracle: the lookups of `tables` over the whole batch, the
    table shrunk to the rows those lookups touch (initial weights from the counter-based
    generator)."""
    B = spec.batch
    dims, woff, roff, ooff, widx, soff, sgrad, Ws = [], [0], [0], [0], [], [0], [], []
    for t in tables:
        seg = idx[off[t * B]:off[(t + 1) * B]]
        rows = np.unique(seg)
        Ws.append(wl.weights_numpy(spec, t, rows).reshape(-1))
        widx.append(np.searchsorted(rows, seg))
        lens = np.diff(off[t * B:(t + 1) * B + 1])
        soff.extend((soff[-1] + np.cumsum(lens)).tolist())
        D = int(spec.dims[t])
        dims.append(D)
        woff.append(woff[-1] + len(rows) * D)
        roff.append(roff[-1] + len(rows))
        ooff.append(ooff[-1] + D)
        sgrad.append(grad[:, spec.out_offset[t]:spec.out_offset[t + 1]])
    return dict(dtype=spec.dtype, dim=np.array(dims, np.int32), out_offset=np.array(ooff[:-1], np.int32),
                weight_offset=np.array(woff[:-1], np.int64), row_offset=np.array(roff, np.int64),
                W=np.concatenate(Ws), idx=np.concatenate(widx).astype(np.int64), off=np.array(soff, np.int64),
                grad=np.ascontiguousarray(np.concatenate(sgrad, axis=1)), B=B, lr=spec.lr, eps=spec.eps)


def time_oracle(sample, steps: int, warmup: int):
    """Oracle forward + backward on the sample, `steps` times; returns (lookups/s, threads)."""
    import oracle

    threads = oracle.max_threads()
    oracle.set_threads(threads)
    n = len(sample["idx"])
    W = sample["W"].copy()
    m = np.zeros(int(sample["row_offset"][-1]), np.float32)
    args = (sample["dtype"], sample["dim"], sample["out_offset"], sample["weight_offset"])

    def step():
        oracle.tbe_forward(*args, W, sample["B"], sample["idx"], sample["off"])
        oracle.tbe_backward_rowwise_adagrad(*args, sample["row_offset"], W, m, sample["B"], sample["idx"],
                                            sample["off"], sample["grad"], sample["lr"], sample["eps"])

    for _ in range(warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = time.perf_counter() - t0
    return n * steps / dt, threads, dt / steps


def run_reference(args, rank: int, world: int):
    if rank != 0:
        return
    spec = make_spec(args.workload, 0, args)
    idx, off = wl.BatchStream(spec).next()
    grad = wl.gen_grad(spec, 0)
    tables = list(range(min(8, spec.T)))
    sample = oracle_sample(spec, idx, off, grad, tables)
    value, threads, sec = time_oracle(sample, args.steps, args.warmup)
    desc = (f"tables {tables} of batch 0 ({len(sample['idx'])} of {len(idx)} lookups), tables compacted to the rows "
            f"touched; forward + backward per step")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": spec.name, "sample": desc},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def reduce_over_ranks(times_ms, counts, world: int, device):
    """Whole-job figures from per-rank ones: MAX over ranks of every time, SUM of every count."""
    import torch
    import torch.distributed as dist

    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    c = torch.tensor(list(counts), dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return [float(x) for x in t], [float(x) for x in c]


def measure_uncached(args, spec, dev, rank: int, world: int, steps: int, warmup: int, with_e2e: bool, with_cpu: bool):
    """Configurations 1-3 (all tables in HBM): the train step timed REPEATS times over `steps` steps, the
    per-kernel pass, the end-to-end pass and (on request) the CPU oracle.  Returns the record of the workload."""
    import torch
    import torch.distributed as dist

    from paper_2305_01515_b200 import binding as mb
    from paper_2305_01515_b200.harness import DeviceModel

    local_rank = dev.index
    model = DeviceModel(spec, device=dev)
    R = args.rotate
    io_t = torch.float16 if args.io_dtype == "f16" else torch.float32     # pooled output and its gradient
    io_b = 2 if args.io_dtype == "f16" else 4
    host, devb = [], []
    for k in range(R):
        idx, off = wl.gen_batch(spec, k)
        grad = wl.gen_grad(spec, k)
        h = (torch.from_numpy(idx).pin_memory(), torch.from_numpy(off).pin_memory(),
             torch.from_numpy(grad).to(io_t).pin_memory())
        host.append(h)
        devb.append(tuple(x.to(dev) for x in h))
    n_max = max(len(h[0]) for h in host)
    model.reserve(n_max)
    B, TD, eb = spec.batch, spec.total_dim, spec.elem_bytes
    out = torch.empty((B, TD), dtype=io_t, device=dev)
    stream = torch.cuda.current_stream(dev)

    # One training step.  The index-only half of the backward (ordering the lookups by row) does not
    # need the gradient, so it runs on a second stream beside the forward pass; the gradient half
    # follows the forward pass on the main stream.
    side = torch.cuda.Stream(dev, priority=-1)   # its small grids get SM slots at once, beside the forward's blocks
    ev_fork, ev_sorted = torch.cuda.Event(), torch.cuda.Event()

    def train_step(i, o, g, out_t, mid=None, sequential=args.sequential):
        n = i.numel()
        if sequential:
            model.forward(i, o, n, out=out_t, stream=stream)
            if mid is not None:
                mid.record(stream)
            model.backward(i, o, n, g, stream=stream)
            return
        ev_fork.record(stream)                 # after the previous step's use of the workspace
        side.wait_event(ev_fork)
        model.backward_sort(i, o, n, stream=side)
        ev_sorted.record(side)
        model.forward(i, o, n, out=out_t, stream=stream)
        if mid is not None:
            mid.record(stream)
        stream.wait_event(ev_sorted)
        model.backward_apply(o, n, g, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()

    # distinct rows per table of every rotating batch (for the compulsory byte count), from the library's own
    # distinct-row output on a scratch copy of the state
    uniq_bytes = []
    row_off = torch.from_numpy(spec.row_offset).to(dev)
    dims_t = torch.from_numpy(spec.dims.astype(np.int64)).to(dev)
    for k in range(R):
        i, o, g = devb[k]
        uq = torch.empty(i.numel(), dtype=torch.int64, device=dev)
        nu = torch.zeros(1, dtype=torch.int64, device=dev)
        model.backward_sort(i, o, i.numel(), uniq_rows_out=uq, n_unique_out=nu, stream=stream)
        torch.cuda.synchronize(dev)
        U = int(nu.item())
        tab = torch.bucketize(uq[:U], row_off[1:], right=True)
        uniq_bytes.append((U, float((dims_t[tab] * eb).sum().item())))
        del uq

    for k in range(warmup):
        i, o, g = devb[k % R]
        train_step(i, o, g, out)
    torch.cuda.synchronize(dev)

    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    lookups = sum(host[k % R][0].numel() for k in range(steps))
    launches0 = mb.launch_count()
    region_ms, fwd_ms, bwd_ms = [], [], []
    sampler.mark(True)
    for rep in range(REPEATS):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * steps + 1)]
        barrier()
        torch.cuda.synchronize(dev)
        ev[0].record(stream)
        for k in range(steps):
            i, o, g = devb[k % R]
            train_step(i, o, g, out, mid=ev[2 * k + 1])
            ev[2 * k + 2].record(stream)
        torch.cuda.synchronize(dev)
        barrier()
        region_ms.append(ev[0].elapsed_time(ev[-1]))
        fwd_ms.append(sum(ev[2 * k].elapsed_time(ev[2 * k + 1]) for k in range(steps)) / steps)
        bwd_ms.append(sum(ev[2 * k + 1].elapsed_time(ev[2 * k + 2]) for k in range(steps)) / steps)
    sampler.mark(False)
    launches = (mb.launch_count() - launches0) // REPEATS
    clocks = sampler.stop()

    # per-kernel device times over the same K steps, bracketed by CUDA events on the launch stream;
    # one stream here, so that no kernel's time includes another stream's kernels running beside it
    mb.trace_enable(True)
    for k in range(steps):
        i, o, g = devb[k % R]
        train_step(i, o, g, out, sequential=True)
    trace = mb.trace_report()
    mb.trace_enable(False)

    e2e = None
    if with_e2e:
        # end to end: every step copies its inputs from pinned host memory to the device and reads the
        # pooled output back to pinned host memory.  Copies run on their own streams (input copy of
        # step k+1 and output copy of step k-1 overlap the kernels of step k; two buffers each way).
        s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        h_out = [torch.empty((B, TD), dtype=io_t).pin_memory() for _ in range(2)]
        d_in = [(torch.empty(n_max, dtype=torch.int64, device=dev), torch.empty(spec.T * B + 1, dtype=torch.int64, device=dev),
                 torch.empty((B, TD), dtype=io_t, device=dev)) for _ in range(2)]
        d_out = [torch.empty((B, TD), dtype=io_t, device=dev) for _ in range(2)]

        def e2e_run(n_steps):
            ev_in = [torch.cuda.Event() for _ in range(n_steps)]
            ev_cmp = [torch.cuda.Event() for _ in range(n_steps)]
            ev_out = [torch.cuda.Event() for _ in range(n_steps)]
            h2d_b = d2h_b = 0
            for k in range(n_steps):
                hi, ho, hg = host[k % R]
                n = hi.numel()
                di, do_, dg = d_in[k & 1]
                with torch.cuda.stream(s_in):
                    if k >= 2:
                        s_in.wait_event(ev_cmp[k - 2])          # the kernels that read this buffer are done
                    di[:n].copy_(hi, non_blocking=True)
                    do_.copy_(ho, non_blocking=True)
                    dg.copy_(hg, non_blocking=True)
                    ev_in[k].record(s_in)
                stream.wait_event(ev_in[k])
                if k >= 2:
                    stream.wait_event(ev_out[k - 2])            # the output buffer has been read back
                train_step(di[:n], do_, dg, d_out[k & 1])
                ev_cmp[k].record(stream)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_cmp[k])
                    h_out[k & 1].copy_(d_out[k & 1], non_blocking=True)
                    ev_out[k].record(s_out)
                h2d_b += n * 8 + ho.numel() * 8 + hg.numel() * io_b
                d2h_b += h_out[0].numel() * io_b
            stream.wait_stream(s_out)
            stream.wait_stream(s_in)
            return h2d_b, d2h_b

        e2e_run(min(2, warmup))
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        s_in.wait_event(e0)
        h2d, d2h = e2e_run(steps)
        e1.record(stream)
        torch.cuda.synchronize(dev)
        barrier()
        e2e = (e0.elapsed_time(e1), h2d, d2h)

    ms_med = float(np.median(region_ms))
    times, (all_lookups,) = reduce_over_ranks([ms_med, min(region_ms), e2e[0] if e2e else 0.0], [float(lookups)], world, dev)
    ms_med, ms_min, e2e_ms = times
    rec = None
    if rank == 0:
        peak, peak_src = measured_peaks()
        n_avg = lookups / steps
        # Eq. 3: one row of D*p bytes per lookup and pass
        per_lookup = sum(float(spec.tables[t].dim) * eb * spec.tables[t].pooling for t in range(spec.T)) / \
            sum(spec.tables[t].pooling for t in range(spec.T))
        row_bytes_exact = 0.0
        for k in range(steps):
            off = host[k % R][1].numpy()
            row_bytes_exact += sum(float(off[(t + 1) * B] - off[t * B]) * float(spec.dims[t]) * eb for t in range(spec.T))
        row_bytes_exact /= steps
        u_avg = sum(uniq_bytes[k % R][0] for k in range(steps)) / steps
        ub_avg = sum(uniq_bytes[k % R][1] for k in range(steps)) / steps
        idx_bytes = 8.0 * n_avg + 8.0 * (spec.T * B + 1)
        # compulsory DRAM bytes: every distinct row once per pass (read in the forward, read and written in the
        # backward), its state read and written, the output written and its gradient read once, the indices
        # read by the forward and by the key pass; the sort's scratch traffic is not counted
        comp_fwd = ub_avg + idx_bytes + float(io_b) * B * TD
        comp_bwd = 2.0 * ub_avg + 8.0 * u_avg + float(io_b) * B * TD + idx_bytes
        comp_reduce = 2.0 * ub_avg + 8.0 * u_avg + float(io_b) * B * TD + 8.0 * n_avg
        alg = {
            "tbe_forward_kernel": (n_avg * (per_lookup + 8) + 8 * (spec.T * B + 1) + float(io_b) * B * TD, comp_fwd),
            "reduce_chunks": (n_avg * (per_lookup + 8), comp_reduce),      # row-equivalent + sorted key and bag id
        }
        top = max(trace.items(), key=lambda kv: kv[1][0]) if trace else (None, (0.0, 0))
        kernels = {k: {"ms_per_step": v[0] / steps, "launches_per_step": v[1] / steps} for k, v in trace.items()}
        roof = None
        if top[0] in alg:
            avg_ms = top[1][0] / top[1][1]
            ach = alg[top[0]][0] / (avg_ms * 1e-3) / 1e9
            per_lk, traffic_note = ncu_traffic_per_lookup(top[0], spec.name) if args.io_dtype == "f32" else (None, "fp16 i/o")
            traffic = per_lk * n_avg if per_lk is not None else None
            roof = {"kernel": top[0], "bound": "hbm", "achieved": ach, "peak": peak, "unit": "GB/s",
                    "frac": ach / peak, "frac_of_nominal": ach / NOMINAL_HBM_GBS,
                    "traffic": traffic, "traffic_source": traffic_note,
                    "dram_traffic_rate": fractions(traffic / (avg_ms * 1e-3) / 1e9, peak) if traffic else None,
                    # the share of the DRAM peak the kernel really uses (profiler bytes), beside the Eq. 3 figure above
                    "frac_by_dram_traffic": (traffic / (avg_ms * 1e-3) / 1e9 / peak) if traffic else None,
                    "compulsory_bytes_per_launch": alg[top[0]][1],
                    "compulsory_rate": fractions(alg[top[0]][1] / (avg_ms * 1e-3) / 1e9, peak),
                    "peak_source": peak_src, "nominal_peak": NOMINAL_HBM_GBS,
                    "algorithmic_bytes_per_launch": alg[top[0]][0], "avg_launch_ms": avg_ms,
                    "note": "achieved / frac = Eq. 3 bytes (a row per lookup, rows served by L2 included, so it can pass 1 of a DRAM peak) / time; "
                            "frac_by_dram_traffic = profiler DRAM bytes / time / peak; compulsory = distinct rows only",
                    "timing": "CUDA events around every launch, separate single-stream pass of the same K steps"}
        step_bytes = 2.0 * row_bytes_exact
        ms_step = ms_med / steps
        rec = {
            "value": all_lookups / (ms_med * 1e-3), "ms_per_step": ms_step, "ms_per_step_min": ms_min / steps,
            "ms_per_step_repeats": [m / steps for m in region_ms], "repeats": REPEATS,
            "config": {"workload": spec.name, "tables": spec.T, "rows_total": int(spec.row_offset[-1]),
                       "dims": sorted(set(int(d) for d in spec.dims)), "storage": "fp16" if spec.dtype == wl.FP16 else "fp32",
                       "weight_gb": spec.weight_bytes / 1e9, "batch": B, "lookups_per_step": n_avg,
                       "distinct_rows_per_step": u_avg, "parallelism": f"{world} replica(s), own batches",
                       "io_dtype": args.io_dtype,
                       "schedule": "sequential" if args.sequential else "backward's sort on a second stream beside the forward",
                       "l2": f"inputs larger than L2: {spec.weight_bytes / 1e9:.2f} GB of weights, {R} batches rotate"},
            "samples_per_sec": world * B / (ms_step * 1e-3),
            "forward_ms": float(np.median(fwd_ms)), "backward_ms": float(np.median(bwd_ms)),
            "forward_lookups_per_sec": n_avg / (float(np.median(fwd_ms)) * 1e-3),
            "step_eq3": fractions(step_bytes / (ms_step * 1e-3) / 1e9, peak),
            "step_compulsory": dict(fractions((comp_fwd + comp_bwd) / (ms_step * 1e-3) / 1e9, peak),
                                    bytes_per_step=comp_fwd + comp_bwd),
            "clocks": clocks, "gpu_launches": int(launches), "kernels": kernels, "roofline": roof,
        }
        if e2e:
            rec["e2e"] = {"value": all_lookups / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": e2e[1] // steps,
                          "d2h_bytes_per_step": e2e[2] // steps, "ms_per_step": e2e_ms / steps,
                          "schedule": "input and output copies on their own streams, double-buffered"}
        if with_cpu and world == 1:
            idx0, off0, g0 = (x.numpy() for x in host[0])
            tables = list(range(min(8, spec.T)))
            sample = oracle_sample(spec, idx0, off0, g0.astype(np.float32), tables)
            v, threads, sec = time_oracle(sample, 3, 1)
            rec["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
                                   "sample": f"tables {tables} of batch 0 ({len(sample['idx'])} lookups), tables "
                                             f"compacted to the rows touched, 3 steps of forward + backward"}
    model.close()
    del model, devb, out
    torch.cuda.empty_cache()
    return rec


def host_link_bandwidth(dev, nbytes: int = 1 << 30):
    """Measured pinned host<->device copy bandwidth (GB/s), one direction at a time."""
    import torch

    h = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
    d = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    res = []
    for src, dst in ((h, d), (d, h)):
        dst.copy_(src, non_blocking=True)
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(3):
            dst.copy_(src, non_blocking=True)
        e1.record()
        torch.cuda.synchronize(dev)
        res.append(3 * nbytes / (e0.elapsed_time(e1) * 1e-3) / 1e9)
    return res[0], res[1]


def host_gather_rates(model, n_rows: int = 200_000):
    """GB/s of mts_host_gather_rows on random rows of every cache's table group (host threads only)."""
    import torch

    from paper_2305_01515_b200 import binding as mb

    rng = np.random.default_rng(0)
    rates = {}
    for g, c in enumerate(model.caches):
        _, t0, t1 = model.groups[g]
        rows_g = int(model.spec.row_offset[t1] - model.spec.row_offset[t0])
        rb = c.dim * model.spec.elem_bytes
        n = min(n_rows, model.fetch_rows[g])
        keys = torch.from_numpy(rng.integers(0, rows_g, n).astype(np.int64))
        best = 1e9
        for _ in range(3):
            t0_ = time.perf_counter()
            mb.host_gather_rows(model.host_rows_ptr(g), keys.numpy(), n, rb, model.fetch_host[0][g], model.gather_threads)
            best = min(best, time.perf_counter() - t0_)
        rates[str(c.dim)] = n * rb / best / 1e9
    return rates


def measure_cached(args, spec, dev, steps: int, warmup: int):
    """Configurations 4 and 5: rows in pinned host memory behind HBM caches, pipelined train step.  `warmup`
    batches bring the caches to their steady state, the next `steps` batches are timed.  Returns the record."""
    import torch

    from paper_2305_01515_b200 import binding as mb
    from paper_2305_01515_b200.harness import DeviceModel
    from paper_2305_01515_b200.pipeline import CachedTrainer

    t_setup = time.time()
    policy = mb.POLICY_LFU if args.policy == "lfu" else mb.POLICY_LRU
    two_level = args.l2_fraction > 0.0
    if two_level:        # two cache levels run the sequential schedule with kernel data movement
        args.sequential, args.fetch, args.lock_depth = True, "sm", 0
    model = DeviceModel(spec, device=dev, lock_depth=args.lock_depth, policy=policy, l2_fraction=args.l2_fraction)
    h2d_gbs, d2h_gbs = host_link_bandwidth(dev)
    stream = wl.BatchStream(spec)
    # the tag step and the data movement run up to COOLDOWN batches ahead of the training: that many batches
    # follow the timed ones, so that every timed step carries the side work of a steady state
    COOLDOWN = 3
    K = warmup + steps
    host = [stream.next() for _ in range(K + COOLDOWN)]
    n_max = max(len(b[0]) for b in host)
    model.reserve(n_max)
    batches = [(torch.from_numpy(i).to(dev), torch.from_numpy(o).to(dev), o) for i, o in host]
    R = min(4, K)
    grads = [torch.from_numpy(wl.gen_grad(spec, k)).to(dev) for k in range(R)]
    glist = [grads[k % R] for k in range(K + COOLDOWN)]
    setup_s = time.time() - t_setup
    trainer = CachedTrainer(model, pipelined=not args.sequential, host_gather=args.fetch == "host",
                            tag_on_main=args.tag_on_main)
    trainer.record_timeline = args.timeline
    gather_gbs = host_gather_rates(model) if args.fetch == "host" else None
    main = torch.cuda.current_stream(dev)
    marks = {}
    traced = []

    def on_step(t):
        if warmup - 1 <= t < K:
            e = torch.cuda.Event(enable_timing=True)
            e.record(main)
            marks[t] = e
        if t == warmup - 1 and args.trace:
            mb.trace_enable(True)          # per-kernel times of the launches from here on
        if t == K - 1 and args.trace:
            traced.append(mb.trace_report())
            mb.trace_enable(False)

    sampler = ClockSampler(dev.index)
    sampler.start()
    time.sleep(0.3)
    launches0 = mb.launch_count()
    sampler.mark(True)
    trainer.run(batches, glist, on_step=on_step)
    torch.cuda.synchronize(dev)
    sampler.mark(False)
    kernels = None
    if args.trace and traced:
        kernels = {k: {"ms_per_step": v[0] / steps, "launches_per_step": v[1] / steps} for k, v in traced[0].items()}
    # diagnostics on the last batch, GPU otherwise idle: lookups that bypass the cache, forward and backward alone
    K_all = K + COOLDOWN
    last_ctx = (K_all - 1) % DeviceModel.N_CTX
    n_last = batches[K_all - 1][0].numel()
    bypass = int((model.ctx[last_ctx]["slot"][:n_last] < 0).sum().item())
    out_d = torch.empty((spec.batch, spec.total_dim), dtype=torch.float32, device=dev)
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    model.forward(batches[K_all - 1][0], batches[K_all - 1][1], n_last, out=out_d, stream=main, ctx=last_ctx)
    f0.record(main)
    for _ in range(3):
        model.forward(batches[K_all - 1][0], batches[K_all - 1][1], n_last, out=out_d, stream=main, ctx=last_ctx)
    f1.record(main)
    torch.cuda.synchronize(dev)
    fwd_alone_ms = f0.elapsed_time(f1) / 3
    clocks = sampler.stop()
    launches = mb.launch_count() - launches0
    ms = marks[warmup - 1].elapsed_time(marks[K - 1])
    per_step = sorted(marks[t - 1].elapsed_time(marks[t]) for t in range(warmup, K))
    hist = np.stack(trainer.history)[warmup:K]                     # [steps, caches, counters]
    lookups = float(hist[:, :, 0].sum())
    hit = float(hist[:, :, 2].sum()) / max(lookups, 1.0)
    eb = spec.elem_bytes
    dims = [d for d, _, _ in model.groups]
    miss_bytes = sum(float(hist[:, g, 6].sum()) * dims[g] * eb for g in range(len(dims)))
    dirty_bytes = sum(float(hist[:, g, 8].sum()) * dims[g] * eb for g in range(len(dims)))
    B = spec.batch
    eq3 = 0.0
    for k in range(warmup, K):
        off = host[k][1]
        for t in range(spec.T):
            eq3 += 2.0 * float(off[(t + 1) * B] - off[t * B]) * float(spec.dims[t]) * eb
    peak, peak_src = measured_peaks()
    t_meas = ms * 1e-3

    def roof_vs(hbm_gbs):
        t_hbm = eq3 / (hbm_gbs * 1e9)
        t_h2d = miss_bytes / (h2d_gbs * 1e9)
        t_d2h = dirty_bytes / (d2h_gbs * 1e9)
        t_roof = max(t_hbm, t_h2d, t_d2h)
        return t_roof, t_hbm, t_h2d, t_d2h

    t_roof, t_hbm, t_h2d, t_d2h = roof_vs(peak)
    rec = {
        "value": lookups / t_meas, "ms_per_step": ms / steps, "ms_per_step_median": per_step[len(per_step) // 2],
        "ms_per_step_min": per_step[0],
        "config": {"workload": spec.name, "note": spec.note, "tables": spec.T, "rows_total": int(spec.row_offset[-1]),
                   "host_weight_gb": spec.weight_bytes / 1e9, "cache_fraction": spec.cache_fraction, "batch": B,
                   "policy": args.policy, "lookups_per_step": lookups / steps, "warmup_batches": warmup,
                   "timed_batches": steps, "schedule": "sequential" if args.sequential else "pipelined",
                   "lock_depth": args.lock_depth,
                   "missed_rows": "gathered by host threads, copy engine" if args.fetch == "host" else "read by a kernel over the host link",
                   "l2": "inputs larger than L2 (host tier and caches are GBs)", "setup_seconds": setup_s},
        "samples_per_sec": B * steps / t_meas, "hit_rate_per_lookup": hit,
        "unique_hit_rate": float(hist[:, :, 4].sum()) / max(float(hist[:, :, 1].sum()), 1.0),
        "overflow_rows": float(hist[:, :, 9].sum()), "lookups_bypassing_cache_last_step": bypass,
        "forward_alone_ms_last_step": fwd_alone_ms,
        "host_link": {"h2d_gbs": h2d_gbs, "d2h_gbs": d2h_gbs, "miss_gb_per_step": miss_bytes / steps / 1e9,
                      "dirty_evict_gb_per_step": dirty_bytes / steps / 1e9,
                      "achieved_h2d_gbs": miss_bytes / t_meas / 1e9},
        "roofline": {"bound": "host-link" if t_roof != t_hbm else "hbm", "t_hbm_ms": t_hbm * 1e3 / steps,
                     "t_h2d_ms": t_h2d * 1e3 / steps, "t_d2h_ms": t_d2h * 1e3 / steps,
                     "achieved": t_roof / t_meas, "peak": 1.0, "unit": "fraction of the slower of HBM and host-link time",
                     "frac": t_roof / t_meas, "frac_with_nominal_hbm": roof_vs(NOMINAL_HBM_GBS)[0] / t_meas,
                     "traffic": None, "peak_source": peak_src},
        "clocks": clocks, "gpu_launches": int(launches), "kernels": kernels,
    }
    if gather_gbs is not None:
        rec["host_link"]["host_gather_gbs_by_dim"] = gather_gbs
        # what the host threads did over the whole run (warm-up and cooldown batches included), per batch:
        # the caches take turns at the cores, so the sum of the two times is a floor of the step time
        st = model.host_copy_stats
        nb = float(K + COOLDOWN)
        g_s, s_s = sum(x["gather_s"] for x in st), sum(x["scatter_s"] for x in st)
        g_b, s_b = sum(x["gather_bytes"] for x in st), sum(x["scatter_bytes"] for x in st)
        rec["host_threads"] = {"threads": model.gather_threads,
                               "workers": "python threads" if args.timeline else "threads of the library (mts_mover); their gather / "
                                          "scatter times include waiting for the other caches' turn at the cores",
                               "gather_ms_per_batch": g_s * 1e3 / nb,
                               "scatter_ms_per_batch": s_s * 1e3 / nb,
                               "gather_gbs": g_b / max(g_s, 1e-9) / 1e9, "scatter_gbs": s_b / max(s_s, 1e-9) / 1e9,
                               "wait_for_turn_ms_per_batch": sum(x["wait_s"] for x in st) * 1e3 / nb}
    if args.timeline:
        # device time of every phase of the last batches, ms since the first mark (perturbs the run a little)
        by_batch = {}
        for name, t, ms_at in trainer.timeline():
            by_batch.setdefault(t, {})[name] = round(ms_at, 2)
        rec["worker_phases_ms"] = trainer.host_phases()
        rec["timeline_ms"] = {str(t): dict(sorted(by_batch[t].items(), key=lambda kv: kv[1]))
                              for t in sorted(by_batch) if K - 4 <= t < K}
    if two_level:
        l2_hits = float(hist[:, :, 10].sum())
        rec["two_level"] = {"l2_fraction": args.l2_fraction, "l1_hit_rate_per_lookup": hit,
                            "l2_hit_rate_per_lookup": l2_hits / max(lookups, 1.0),
                            "store_rate_per_lookup": 1.0 - hit - l2_hits / max(lookups, 1.0),
                            "promoted_rows_per_step": float(hist[:, :, 12].sum()) / steps,
                            "demoted_rows_per_step": float(hist[:, :, 13].sum()) / steps,
                            "l2_evicted_rows_per_step": float(hist[:, :, 14].sum()) / steps,
                            "l2_bypass_rows_per_step": float(hist[:, :, 16].sum()) / steps,
                            "l2_dropped_rows_per_step": float(hist[:, :, 18].sum()) / steps,
                            "schedule": "sequential, rows moved by kernels"}
    trainer.close()
    model.close()
    del model, trainer, batches, grads, glist
    torch.cuda.empty_cache()
    return rec


def finish_line(rec, world: int, steps: int, warmup: int):
    line = {"metric": METRIC, "value": rec.pop("value"), "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": rec.pop("ms_per_step"), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic"}
    line.update(rec)
    line.setdefault("e2e", None)
    return line


def sub_record(rec, steps: int, warmup: int):
    """A workload measured beside the headline one: the same figures, without the per-kernel table."""
    keep = {k: v for k, v in rec.items() if k not in ("kernels", "ms_per_step_repeats")}
    keep.update(unit=UNIT, steps=steps, warmup=warmup, workload=rec["config"]["workload"])
    return keep


def run_sweep(args, dev):
    """Configuration 5: one-factor sweeps around the centre point (batch 16K, pooling 50, Zipf 1.0,
    cache 10%) plus the four extreme corners.  Prints one JSON line per point (hit rate, lookups/s,
    roofline fraction); not the default bench line."""
    import copy

    centre = dict(batch=16384, pooling=50, alpha=1.0, cache_fraction=0.10)
    points = [dict(centre)]
    for b in (1024, 4096, 65536):
        points.append(dict(centre, batch=b))
    for L in (1, 10, 200):
        points.append(dict(centre, pooling=L))
    for a in (0.6, 0.8, 1.2, 1.4):
        points.append(dict(centre, alpha=a))
    for c in (0.01, 0.05, 0.25, 0.50):
        points.append(dict(centre, cache_fraction=c))
    points += [dict(batch=1024, pooling=1, alpha=0.6, cache_fraction=0.01),
               dict(batch=65536, pooling=200, alpha=1.4, cache_fraction=0.50),
               dict(batch=1024, pooling=200, alpha=1.4, cache_fraction=0.01),
               dict(batch=65536, pooling=1, alpha=0.6, cache_fraction=0.50)]
    for p in points:
        a = copy.copy(args)
        a.batch, a.pooling, a.alpha, a.cache_fraction = p["batch"], p["pooling"], p["alpha"], p["cache_fraction"]
        j = measure_cached(a, make_spec("cfg5", 0, a), dev, args.steps, args.warmup)
        print(json.dumps({"point": p, "lookups_per_sec": j["value"], "ms_per_step": j["ms_per_step"],
                          "hit_rate_per_lookup": j["hit_rate_per_lookup"], "unique_hit_rate": j["unique_hit_rate"],
                          "overflow_rows": j["overflow_rows"], "roofline_frac": j["roofline"]["frac"],
                          "bound": j["roofline"]["bound"], "miss_gb_per_step": j["host_link"]["miss_gb_per_step"],
                          "achieved_h2d_gbs": j["host_link"]["achieved_h2d_gbs"]}), flush=True)


DEFAULT_STEPS = {"cfg1": (100, 10), "cfg2": (100, 10), "cfg3": (8, 4), "cfg4": (24, 16), "cfg5": (20, 30)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default per workload: 100 for cfg1/cfg2, 8-10 otherwise)")
    ap.add_argument("--warmup", type=int, default=None, help="warm-up steps (default per workload; cached ones need 12-30 to reach steady state)")
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default=None,
                    help="cfg1 ... cfg5 or cfg5-sweep; default: cfg3 as the headline and, on one GPU, cfg2 / cfg4 / cfg5 beside it")
    ap.add_argument("--rotate", type=int, default=4, help="distinct batches that take turns")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--budget-gb", type=float, default=wl.BENCH_CFG4_BUDGET_GB, help="cfg4: HBM budget; host weights are 4x this")
    ap.add_argument("--rows", type=int, default=50_000_000, help="cfg5: rows of the single table")
    ap.add_argument("--batch", type=int, default=16384, help="cfg5: batch size")
    ap.add_argument("--pooling", type=int, default=50, help="cfg5: lookups per bag")
    ap.add_argument("--alpha", type=float, default=1.0, help="cfg5: Zipf exponent")
    ap.add_argument("--cache-fraction", type=float, default=0.10, help="cfg5: cache slots / rows")
    ap.add_argument("--l2-fraction", type=float, default=0.0,
                    help="cached workloads: share of the rows a second, exclusive cache level in pinned host memory holds "
                         "(Section 5.3.2); 0 = one level")
    ap.add_argument("--policy", default="lru", choices=["lru", "lfu"], help="cached workloads: replacement policy (Section 5.5.2)")
    ap.add_argument("--io-dtype", default="f32", choices=["f32", "f16"],
                    help="type of the pooled output and of its gradient (uncached workloads); the headline metric is f32")
    ap.add_argument("--fetch", default="host", choices=["sm", "host"],
                    help="cached workloads: missed rows gathered by host threads into a pinned buffer and moved by the copy "
                         "engine (host), or read over the host link by a kernel (sm)")
    ap.add_argument("--sequential", action="store_true", help="one stream only (no sort beside the forward, no cache pipeline)")
    ap.add_argument("--lock-depth", type=int, default=2,
                    help="cached workloads: batches a stamped way stays unevictable (Section 5.7 invariant)")
    ap.add_argument("--timeline", action="store_true",
                    help="cached workloads: add the device timeline of the last batches (events on every stream) to the line")
    ap.add_argument("--tag-on-main", action="store_true",
                    help="cached workloads: the tag step between the training steps on their stream, instead of two "
                         "batches ahead on a stream of its own")
    ap.add_argument("--trace", action="store_true",
                    help="cached workloads: CUDA events around every launch of the run (perturbs the timing)")
    ap.add_argument("--tables", type=int, default=0,
                    help="cfg2 / cfg3: fewer tables (a small case for profiler captures; not a bench line)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    headline = args.workload or "cfg3"
    beside = [] if (args.workload or world > 1) else ["cfg2", "cfg5", "cfg4"]

    def counts(name):
        k, w = DEFAULT_STEPS.get(name, (8, 8))
        k = args.steps if args.steps is not None else k
        w = args.warmup if args.warmup is not None else w
        return k, max(w, 3)

    if args.impl == "reference":
        args.steps = args.steps if args.steps is not None else 3
        args.warmup = args.warmup if args.warmup is not None else 1
        args.workload = headline
        run_reference(args, rank, world)
        return
    if world == 1 and args.gpus > 1:
        raise SystemExit("launch with torch.distributed.run for --gpus > 1")

    import torch
    import torch.distributed as dist

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if headline == "cfg5-sweep":
        args.steps, args.warmup = counts("cfg5")
        run_sweep(args, dev)
        return
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def measure(name, is_headline):
        k, w = counts(name) if (is_headline or args.steps is None) else DEFAULT_STEPS[name]
        if not is_headline:
            k, w = DEFAULT_STEPS[name]
        a = argparse.Namespace(**vars(args))
        a.steps, a.warmup = k, w
        if name in ("cfg4", "cfg5"):
            if world > 1:
                raise SystemExit("cached workloads are single-GPU bench lines")
            return measure_cached(a, make_spec(name, rank, a), dev, k, w), k, w
        return measure_uncached(a, make_spec(name, rank, a), dev, rank, world, k, w, with_e2e=is_headline,
                                with_cpu=is_headline and not args.no_cpu_baseline), k, w

    rec, k, w = measure(headline, True)
    subs = []
    for name in beside:
        r, sk, sw = measure(name, False)
        if rank == 0:
            subs.append(sub_record(r, sk, sw))
    if rank == 0:
        line = finish_line(rec, world, k, w)
        if subs:
            line["workloads"] = subs
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
