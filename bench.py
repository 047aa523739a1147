#!/usr/bin/env python
"""Benchmark of the hot path: corrected INT2/INT4-KV chunk attention + quantize-append.

One "step" is one pass of the whole path over one chunk: kvq_attn_corrected of the BF16 current
chunk over [packed cache ; current chunk] with the correction on, followed by
kvq_quantize_append of that chunk's K/V (the cache length is rewound after every step so that
all steps do identical work).  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

The headline (`value`, `roofline`, `e2e`, `cpu_baseline`) is measured on --workload (default: `long`, the
largest single-GPU configuration).  At one GPU the same line also carries `per_workload`: every other
configuration timed call by call (attention with the correction on and off, quantize-append), each over a
timed region of at least 100 ms with its own clock samples.

Multi-GPU (torchrun, one rank per GPU): (batch, head) units are independent, so every rank runs
its own instance of the workload (weak scaling, no data-path collective); the value is the sum
over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import concurrent.futures
import json
import math
import os
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "corrected INT2-KV chunk-attention TFLOP/s"
L2_FLUSH_BYTES = 512 << 20
MIN_REGION_MS = 120.0          # every leg's timed region is at least this long (the clock sampler polls every 50 ms)

# dram__bytes_read.sum + dram__bytes_write.sum per launch of attn_tcgen05_kernel, from the ncu captures
# summarised under profiles/ (launches_bench_long.md gives the commands; the figures go stale when the kernel changes)
NCU_TRAFFIC_BYTES = {}
try:
    with open(os.path.join(ROOT, "profiles", "traffic.json")) as _f:
        NCU_TRAFFIC_BYTES = json.load(_f)
except OSError:
    pass


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "tf_burst": p["bf16_tflops"], "tf_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "tf_burst": 1590.0, "tf_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        import tempfile
        self.index, self.proc, self.lines = index, None, []
        self.path = os.path.join(tempfile.gettempdir(), f"kvq_clocks_{os.getpid()}_{index}.csv")

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-i", str(self.index),
                 "-lms", "50", "-f", self.path], stdout=subprocess.DEVNULL, stderr=subprocess.DEVNULL)
            time.sleep(0.3)
        except OSError:
            self.proc = None

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        try:
            with open(self.path) as f:
                self.lines = [ln.strip() for ln in f]
            os.remove(self.path)
        except OSError:
            self.lines = []
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def chunk_stream(w, n_chunks, need_q_last=True):
    """Yields (q, k, v) BF16 bit arrays of chunks 0 .. n_chunks-1, drawn ahead on a few host threads (one
    generator per tensor and chunk, so the order of drawing does not change the bits).  Only the last chunk
    comes with its queries."""
    from paper_2605_26266_b200 import inputs
    workers = max(1, min(8, len(os.sched_getaffinity(0)) - 1))
    with concurrent.futures.ThreadPoolExecutor(max_workers=workers) as pool:
        pending = []
        nxt = 0
        while nxt < n_chunks or pending:
            while nxt < n_chunks and len(pending) < 2 * workers:
                pending.append(pool.submit(inputs.make_chunk, w, nxt, None, need_q_last and nxt == n_chunks - 1))
                nxt += 1
            yield pending.pop(0).result()


def oracle_sample(w, steps, warm=0, kv_of_units=None, cur_of_units=None):
    """Times the CPU oracle (as it stands) on a bounded sample of the workload: `heads_s` heads,
    `rows_s` query rows over the full key length, plus the quantize-append of those heads' chunk.
    kv_of_units / cur_of_units: the sample heads' chunks if the caller has drawn them already.
    Returns (seconds per step list, flops per step, sample description, threads)."""
    from oracle import kvq_oracle as O
    from paper_2605_26266_b200 import inputs
    heads_s = min(w.heads, 2)
    rows_s = min(w.chunk, max(64, int(1.0e10 / (4.0 * (w.n_cached + w.chunk) * w.head_dim * heads_s))))
    units = [(0, h) for h in range(heads_s)]
    sel = lambda a: np.stack([a[b, h] for (b, h) in units])[None]
    cache = O.Cache(1, heads_s, w.head_dim, w.bits, w.group, w.capacity)
    n = 0
    if kv_of_units is None:
        kv_of_units, cur_of_units = [], None
        for c, (q, k, v) in enumerate(chunk_stream(w, w.cached_chunks + 1)):
            if c < w.cached_chunks:
                kv_of_units.append((sel(k), sel(v)))
            else:
                cur_of_units = (sel(q), sel(k), sel(v))
    for k, v in kv_of_units:
        n = O.quantize_append(cache, n, k, v)
    q, k, v = cur_of_units
    rows = np.linspace(0, w.chunk - 1, rows_s).astype(np.int64)
    sigma = 1.0 / math.sqrt(w.head_dim)
    times = []
    for i in range(warm + steps):
        t0 = time.perf_counter()
        O.attn_corrected(cache, 0, n, q, k, v, sigma, correction=True, rows=rows)
        O.quantize_append(cache, n, k, v)
        dt = time.perf_counter() - t0
        if i >= warm:
            times.append(dt)
    flops = 4.0 * heads_s * rows_s * (w.n_cached + w.chunk) * w.head_dim
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = len(os.sched_getaffinity(0))
    sample = (f"{heads_s} of {w.batch * w.heads} (batch,head) units, {rows_s} of {w.chunk} query rows over all "
              f"{w.n_cached + w.chunk} keys, plus quantize-append of those units' chunk; numpy FP64")
    return times, flops, sample, threads


def describe(w, n_cached=None):
    ns = w.n_cached if n_cached is None else n_cached
    return (f"{w.name}: batch {w.batch}, heads {w.heads}, head_dim {w.head_dim}, chunk {w.chunk}, "
            f"cache {ns} tokens, INT{w.bits} g={w.group}, Hadamard-{w.head_dim}, correction on")


def roofline_of(w, n_cached, attn_ms, peaks):
    """The two limits the benchmark spec names for one attention call and which of them binds: dense BF16 tensor
    throughput (burst peak: the calls are timed one by one) and packed-cache bytes over HBM bandwidth."""
    flops, nbytes = w.flops(n_cached), w.attn_bytes(n_cached)
    t_tensor = flops / (peaks["tf_burst"] * 1e12)
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    sec = attn_ms * 1e-3
    tf, gbs = flops / sec / 1e12, nbytes / sec / 1e9
    tensor_bound = t_tensor >= t_hbm
    return {"bound": "tensor" if tensor_bound else "hbm",
            "achieved": tf if tensor_bound else gbs, "peak": peaks["tf_burst"] if tensor_bound else peaks["hbm_gbs"],
            "unit": "TFLOP/s" if tensor_bound else "GB/s", "frac": max(t_tensor, t_hbm) / sec,
            "tflops": tf, "hbm_gbs": gbs, "frac_of_burst": tf / peaks["tf_burst"],
            "frac_of_sustained": tf / peaks["tf_sustained"], "frac_of_hbm": gbs / peaks["hbm_gbs"]}


class Problem:
    """One workload resident in HBM: the cache built chunk by chunk by the append kernel, the current chunk's
    Q/K/V, an output buffer, a status word.  Host copies are kept only where asked for."""

    def __init__(self, B, w, dev, keep_host=False, sample_units=0):
        import torch
        self.B, self.w, self.dev = B, w, dev
        self.cache = B.Cache(w.batch, w.heads, w.head_dim, w.bits, w.group, w.capacity, device=dev)
        to_dev = lambda bits: torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)
        self.sample_kv, self.sample_cur, self.host = [], None, None
        sel = lambda a: np.ascontiguousarray(a[:1, :sample_units])
        for c, (q, k, v) in enumerate(chunk_stream(w, w.cached_chunks + 1)):
            if c < w.cached_chunks:
                B.kvq_quantize_append(self.cache, to_dev(k), to_dev(v))
                if sample_units:
                    self.sample_kv.append((sel(k), sel(v)))
            else:
                self.q, self.k, self.v = to_dev(q), to_dev(k), to_dev(v)
                if sample_units:
                    self.sample_cur = (sel(q), sel(k), sel(v))
                if keep_host:
                    self.host = (q, k, v)
        self.n_cached = self.cache.length
        self.out = torch.empty_like(self.q)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.sigma = 1.0 / math.sqrt(w.head_dim)

    def attn(self, flags, n_cached=None, q=None, k=None, v=None, out=None):
        self.B.kvq_attn_corrected(self.cache, self.q if q is None else q, self.k if k is None else k,
                                  self.v if v is None else v, self.sigma, flags,
                                  cache_len=self.n_cached if n_cached is None else n_cached,
                                  out=self.out if out is None else out, status_word=self.status)

    def append(self, n_cached=None, k=None, v=None):
        self.B.kvq_quantize_append(self.cache, self.k if k is None else k, self.v if v is None else v,
                                   cache_len=self.n_cached if n_cached is None else n_cached)

    def check_status(self):
        s = int(self.status.item())
        if s != 0:
            raise SystemExit(f"device-side wait timed out, status {s}")


def time_calls(fn, n, flush, warm=3):
    """Mean milliseconds of fn() over n calls, each bracketed by CUDA events on the current stream, an L2 flush
    before every call."""
    import torch
    recs = []
    for i in range(warm + n):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        if i >= warm:
            recs.append((e0, e1))
    torch.cuda.synchronize()
    return float(np.mean([a.elapsed_time(b) for a, b in recs]))


def time_alternately(fa, fb, n, flush, warm=3):
    """Mean milliseconds of fa() and of fb(), n calls each, taken in turn (a, b, a, b, ...) so that both see the
    same clocks and the same power state: what a ratio of the two is made from."""
    import torch
    recs = ([], [])
    for i in range(warm + n):
        for j, fn in enumerate((fa, fb)):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            if i >= warm:
                recs[j].append((e0, e1))
    torch.cuda.synchronize()
    return tuple(float(np.mean([a.elapsed_time(b) for a, b in r])) for r in recs)


def repeats_for(fn, flush, floor):
    """How many timed calls make a region of at least MIN_REGION_MS (estimated from three calls)."""
    est = max(time_calls(fn, 3, flush, warm=2), 1e-3)
    return max(floor, int(math.ceil(MIN_REGION_MS / est)))


def leg(B, prob, n_cached, flush, peaks, dev_index, floor=10):
    """One row of per_workload: attention with the correction on and off, quantize-append, each timed call by
    call over a region of at least MIN_REGION_MS, with the clocks sampled meanwhile."""
    w = prob.w
    on = lambda: prob.attn(B.KVQ_CORRECTION_ON, n_cached)
    off = lambda: prob.attn(B.KVQ_CORRECTION_OFF, n_cached)
    app = lambda: prob.append(n_cached)
    n_on, n_app = repeats_for(on, flush, floor), repeats_for(app, flush, floor)
    sampler = ClockSampler(dev_index)
    sampler.start()
    on_ms, off_ms = time_alternately(on, off, n_on, flush)
    app_ms = time_calls(app, n_app, flush)
    clocks = sampler.stop()
    prob.check_status()
    r = roofline_of(w, n_cached, on_ms, peaks)
    app_gbs = w.append_bytes() / (app_ms * 1e-3) / 1e9
    return {"workload": describe(w, n_cached), "attn_us": on_ms * 1e3, "attn_uncorrected_us": off_ms * 1e3,
            "correction_overhead": on_ms / off_ms - 1.0, "append_us": app_ms * 1e3,
            "tflops": r["tflops"], "hbm_gbs": r["hbm_gbs"], "bound": r["bound"], "frac": r["frac"],
            "frac_of_burst": r["frac_of_burst"], "frac_of_sustained": r["frac_of_sustained"],
            "append_gbs": app_gbs, "append_frac_of_hbm": app_gbs / peaks["hbm_gbs"],
            "timed_calls": {"attn": n_on, "append": n_app}, "clocks": clocks}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="long")
    ap.add_argument("--impl", default="kvq", choices=["kvq", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-workload", action="store_true")
    ap.add_argument("--profile", action="store_true",
                    help="only warm-up and timed steps of --workload (no correction-off, end-to-end, CPU or "
                         "per-workload legs): the command to run under ncu")
    args = ap.parse_args()

    from paper_2605_26266_b200 import inputs
    w = inputs.WORKLOADS[args.workload]
    if args.profile:
        args.no_e2e = args.no_cpu_baseline = args.no_per_workload = True
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    config = {"workload": describe(w), "l2": f"flushed between steps ({L2_FLUSH_BYTES >> 20} MiB write)",
              "parallelism": f"replicas x{world}"}

    if args.impl == "reference":
        # the oracle on the host cores; rank 0 only
        if rank != 0:
            return
        steps = max(1, min(args.steps, 5))
        times, flops, sample, threads = oracle_sample(w, steps, warm=min(args.warmup, 1))
        sec = float(np.mean(times))
        val = flops / sec / 1e12
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus, "gpus_used": 0, "steps": steps,
            "warmup": min(args.warmup, 1), "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    from paper_2605_26266_b200 import build
    build.build_library()
    from paper_2605_26266_b200 import binding as B

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()

    # ---- set-up (untimed): inputs resident in HBM, cache built chunk by chunk by the append kernel ----
    from paper_2605_26266_b200 import replicas
    wr = replicas.replica_workload(w, rank)
    want_cpu = world == 1 and not args.no_cpu_baseline
    prob = Problem(B, wr, dev, keep_host=not args.no_e2e, sample_units=min(w.heads, 2) if want_cpu else 0)
    n_cached = prob.n_cached
    q, k, v, out = prob.q, prob.k, prob.v, prob.out
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    flags = B.KVQ_CORRECTION_ON

    def step(record=None):
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record()
        prob.attn(flags)
        e1.record()
        prob.append()
        e2.record()
        if record is not None:
            record.append((e0, e1, e2))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        flush.zero_()
        step()
    barrier()

    sampler = ClockSampler(local_rank)
    sampler.start()
    recs = []
    barrier()
    for _ in range(args.steps):
        flush.zero_()
        step(recs)
    barrier()
    attn_ms = np.array([a.elapsed_time(b_) for a, b_, _ in recs])
    app_ms = np.array([b_.elapsed_time(c) for _, b_, c in recs])
    step_ms = float((attn_ms + app_ms).mean())
    prob.check_status()
    eager_step_ms = step_ms

    # The step's kernels replayed from a CUDA graph (the calls only enqueue on the caller's stream, so they
    # capture as they are): the same work without the gaps between launches.  `value` is taken from this run,
    # the per-kernel times above from the eager one.
    if not args.profile:
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                prob.attn(flags)
                prob.append()
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(3):
            flush.zero_()
            graph.replay()
        grecs = []
        barrier()
        for _ in range(args.steps):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay()
            e1.record()
            grecs.append((e0, e1))
        barrier()
        step_ms = float(np.mean([a.elapsed_time(b_) for a, b_ in grecs]))
        prob.check_status()
    clocks = sampler.stop()

    # correction off, same kernel: cost of the correction
    attn_off_ms = attn_on_again_ms = float("nan")
    if not args.profile:
        attn_on_again_ms, attn_off_ms = time_alternately(lambda: prob.attn(B.KVQ_CORRECTION_ON), lambda: prob.attn(B.KVQ_CORRECTION_OFF),
                                                          max(3, min(args.steps, 20)), flush)

    # ---- end to end through the public call with HOST buffers ----
    e2e_ms = e2e_serial_ms = 0.0
    if not args.no_e2e:
        qh, kh, vh = prob.host
        hq, hk, hv = (torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).pin_memory() for a in (qh, kh, vh))
        hout = torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        n_e2e = max(3, min(args.steps, 20))
        # (a) one step at a time: copy in, attend, append, copy out, all on one stream
        e2e_recs = []
        barrier()
        for i in range(n_e2e + 3):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            dq.copy_(hq, non_blocking=True); dk.copy_(hk, non_blocking=True); dv.copy_(hv, non_blocking=True)
            prob.attn(flags, q=dq, k=dk, v=dv)
            prob.append(k=dk, v=dv)
            hout.copy_(out, non_blocking=True)
            e1.record()
            if i >= 3:
                e2e_recs.append((e0, e1))
        barrier()
        e2e_serial_ms = float(np.mean([a.elapsed_time(b_) for a, b_ in e2e_recs]))
        # (b) the way a caller streams chunks: the next step's host-to-device copies and the previous step's
        # device-to-host copy run on their own streams beside this step's kernels (two sets of device buffers);
        # the L2 flush sits on the compute stream inside the timed region
        s_in, s_out, s_cmp = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
        bufs = [(dq, dk, dv, out), (torch.empty_like(q), torch.empty_like(k), torch.empty_like(v), torch.empty_like(out))]
        houts = [hout, torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()]

        def pipelined(n):
            ev_in = [torch.cuda.Event() for _ in range(n)]
            ev_cmp = [torch.cuda.Event() for _ in range(n)]
            ev_out = [torch.cuda.Event() for _ in range(n)]
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record(s_cmp)
            s_in.wait_event(t0); s_out.wait_event(t0)
            for i in range(n):
                bq, bk, bv, bo = bufs[i & 1]
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(ev_cmp[i - 2])          # the kernels that read this input set are done
                    bq.copy_(hq, non_blocking=True); bk.copy_(hk, non_blocking=True); bv.copy_(hv, non_blocking=True)
                    ev_in[i].record(s_in)
                s_cmp.wait_event(ev_in[i])
                if i >= 2:
                    s_cmp.wait_event(ev_out[i - 2])             # this output buffer has been copied out
                flush.zero_()
                prob.attn(flags, q=bq, k=bk, v=bv, out=bo)
                prob.append(k=bk, v=bv)
                ev_cmp[i].record(s_cmp)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_cmp[i])
                    houts[i & 1].copy_(bo, non_blocking=True)
                    ev_out[i].record(s_out)
            s_cmp.wait_event(ev_out[n - 1]); s_cmp.wait_event(ev_in[n - 1])
            t1.record(s_cmp)
            torch.cuda.synchronize()
            return t0.elapsed_time(t1) / n

        pipelined(4)
        barrier()
        e2e_ms = pipelined(n_e2e)
        barrier()
        prob.check_status()
    # ---- reduce over ranks: slowest rank's time ----
    step_ms, attn_mean, app_mean, attn_off_ms, attn_on_again_ms, e2e_ms, eager_step_ms = replicas.max_over_ranks(
        [step_ms, float(attn_ms.mean()), float(app_ms.mean()), attn_off_ms, attn_on_again_ms, e2e_ms, eager_step_ms], device=dev)

    # ---- the other configurations, call by call (one GPU only: a multi-GPU run holds every GPU meanwhile) ----
    per_workload = None
    if world == 1 and not args.no_per_workload:
        per_workload = {}
        for name in ("tiny", "sweep_int4", "sweep_int2", "dit", "long", "pipeline", "prefix"):
            wl = inputs.WORKLOADS[name]
            if wl.head_dim != 128 and name != "tiny":
                continue
            pr = prob if name == w.name else Problem(B, wl, dev)
            if name == "pipeline":
                # steps 0, 7 and 15 of the 16-chunk pipeline: the same cache attended over its first t chunks
                # (longest window first: a step's append overwrites the chunk behind its window)
                rows = {t: leg(B, pr, t * wl.chunk, flush, peaks, local_rank) for t in (15, 7, 0)}
                for t in (0, 7, 15):
                    per_workload[f"pipeline_step{t}"] = rows[t]
            else:
                per_workload[name] = leg(B, pr, pr.n_cached, flush, peaks, local_rank)
            if pr is not prob:
                del pr
                torch.cuda.empty_cache()

    if rank == 0:
        flops = w.flops()
        value = replicas.aggregate_value(flops, world, step_ms)
        roof = roofline_of(w, n_cached, attn_mean, peaks)
        app_gbs = w.append_bytes() / (app_mean * 1e-3) / 1e9
        res = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config,
            "launch": "eager calls (--profile)" if args.profile else "step replayed from a CUDA graph",
            "ms_per_step_eager": eager_step_ms,
            "us_per_call": {"attn_corrected": attn_mean * 1e3, "attn_uncorrected": attn_off_ms * 1e3,
                            "quantize_append": app_mean * 1e3,
                            # corrected and uncorrected calls taken in turn: the ratio is free of clock drift
                            "correction_overhead": attn_on_again_ms / attn_off_ms - 1.0},
            "hbm_gbs": {"attn": roof["hbm_gbs"], "attn_frac_of_peak": roof["frac_of_hbm"],
                        "quantize_append": app_gbs, "quantize_append_frac_of_peak": app_gbs / peaks["hbm_gbs"]},
            # the dominant kernel against the slower of its two limits; the duration is the whole
            # kvq_attn_corrected call (query pre-pass, attention kernel, merge of split units), CUDA events
            "roofline": {"kernel": "attn_tcgen05_kernel", "bound": roof["bound"], "achieved": roof["achieved"],
                         "peak": roof["peak"], "unit": roof["unit"], "frac": roof["frac"],
                         "peak_kind": ("burst bf16" if roof["bound"] == "tensor" else "hbm copy") + ", " + peaks["source"],
                         "frac_of_sustained": roof["frac_of_sustained"],
                         "traffic": NCU_TRAFFIC_BYTES.get(w.name)},
            # kernels of this library launched inside the timed region: per step the attention call's
            # (pre-pass, attention, merge as the problem needs them) plus one quantize-append
            "gpu_launches": (B.kvq_attn_kernel_launches(prob.cache, n_cached, q.shape[2], k.shape[2], flags) + 1) * args.steps,
            "clocks": clocks,
        }
        if not args.no_e2e:
            res["e2e"] = {"value": world * flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                          "mode": "host copies on their own streams beside the kernels (two buffer sets), L2 flush inside",
                          "serial_ms_per_step": e2e_serial_ms,
                          "h2d_bytes_per_step": int(3 * q.numel() * 2), "d2h_bytes_per_step": int(out.numel() * 2),
                          "ms_per_step": e2e_ms}
        if per_workload is not None:
            res["per_workload"] = per_workload
        if want_cpu:
            times, oflops, sample, threads = oracle_sample(w, 2, warm=0, kv_of_units=prob.sample_kv,
                                                           cur_of_units=prob.sample_cur)
            res["cpu_baseline"] = {"value": oflops / float(np.mean(times)) / 1e12, "unit": "TFLOP/s", "cores": threads,
                                   "kind": "oracle", "sample": sample}
        print(json.dumps(res))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
