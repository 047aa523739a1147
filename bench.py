#!/usr/bin/env python
"""Benchmark of the hot path: corrected INT2/INT4-KV chunk attention + quantize-append.

One "step" is one pass of the whole path over one chunk: kvq_attn_corrected of the BF16 current
chunk over [packed cache ; current chunk] with the correction on, followed by
kvq_quantize_append of that chunk's K/V (the cache length is rewound after every step so that
all steps do identical work).  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Multi-GPU (torchrun, one rank per GPU): (batch, head) units are independent, so every rank runs
its own instance of the workload (weak scaling, no data-path collective); the value is the sum
over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
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


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "tf_burst": p["bf16_tflops"], "tf_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "tf_burst": 1590.0, "tf_sustained": 1400.0, "source": "fallback"}


# ncu dram__bytes_read.sum + dram__bytes_write.sum per launch of the attention kernel (profiles/)
NCU_TRAFFIC_BYTES = {
    "sweep_int2": 33.10e6,    # profiles/attn_tcgen05_sweep_int2.md, capture 4
    "dit": 209.3e6,           # profiles/attn_tcgen05_dit.md
}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

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


def oracle_sample(w, steps, warm=0):
    """Times the CPU oracle (as it stands) on a bounded sample of the workload: `heads_s` heads,
    `rows_s` query rows over the full key length, plus the quantize-append of those heads' chunk.
    Returns (seconds per step list, flops per step, sample description, threads)."""
    from oracle import kvq_oracle as O
    from paper_2605_26266_b200 import inputs
    heads_s = min(w.heads, 2)
    rows_s = min(w.chunk, max(64, int(2.0e9 / (4.0 * (w.n_cached + w.chunk) * w.head_dim * heads_s))))
    units = [(0, h) for h in range(heads_s)]
    sel = lambda a: np.stack([a[b, h] for (b, h) in units])[None]
    cache = O.Cache(1, heads_s, w.head_dim, w.bits, w.group, w.capacity)
    n = 0
    for c in range(w.cached_chunks):
        _, k, v = inputs.make_chunk(w, c)
        n = O.quantize_append(cache, n, sel(k), sel(v))
    q, k, v = inputs.make_chunk(w, w.cached_chunks)
    q, k, v = sel(q), sel(k), sel(v)
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="sweep_int2")
    ap.add_argument("--impl", default="kvq", choices=["kvq", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--profile", action="store_true",
                    help="only warm-up and timed steps (no correction-off, end-to-end or CPU legs): the command to run under ncu")
    args = ap.parse_args()

    from paper_2605_26266_b200 import inputs
    w = inputs.WORKLOADS[args.workload]
    if args.profile:
        args.no_e2e = args.no_cpu_baseline = True
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    config = {"workload": f"{w.name}: batch {w.batch}, heads {w.heads}, head_dim {w.head_dim}, chunk {w.chunk}, "
                          f"cache {w.n_cached} tokens, INT{w.bits} g={w.group}, Hadamard-{w.head_dim}, correction on",
              "l2": f"flushed between steps ({L2_FLUSH_BYTES >> 20} MiB write)", "parallelism": f"replicas x{world}"}

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

    def to_dev(bits):
        return torch.from_numpy(bits.view(np.int16)).to(dev).view(torch.bfloat16)

    cache = B.Cache(w.batch, w.heads, w.head_dim, w.bits, w.group, w.capacity, device=dev)
    for c in range(w.cached_chunks):
        _, k, v = inputs.make_chunk(wr, c)
        B.kvq_quantize_append(cache, to_dev(k), to_dev(v))
    n_cached = cache.length
    qh, kh, vh = inputs.make_chunk(wr, w.cached_chunks)
    q, k, v = to_dev(qh), to_dev(kh), to_dev(vh)
    out = torch.empty_like(q)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    sigma = 1.0 / math.sqrt(w.head_dim)
    flags = B.KVQ_CORRECTION_ON

    def step(record=None):
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        e0.record()
        B.kvq_attn_corrected(cache, q, k, v, sigma, flags, cache_len=n_cached, out=out, status_word=status)
        e1.record()
        B.kvq_quantize_append(cache, k, v, cache_len=n_cached)
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
    clocks = sampler.stop()
    attn_ms = np.array([a.elapsed_time(b_) for a, b_, _ in recs])
    app_ms = np.array([b_.elapsed_time(c) for _, b_, c in recs])
    step_ms = float((attn_ms + app_ms).mean())
    if int(status.item()) != 0:
        raise SystemExit(f"device-side wait timed out, status {int(status.item())}")
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
                B.kvq_attn_corrected(cache, q, k, v, sigma, flags, cache_len=n_cached, out=out, status_word=status)
                B.kvq_quantize_append(cache, k, v, cache_len=n_cached)
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
        if int(status.item()) != 0:
            raise SystemExit(f"device-side wait timed out, status {int(status.item())}")

    # correction off, same kernel: cost of the correction
    recs_off = []
    for i in range(0 if args.profile else max(3, min(args.steps, 20)) + 3):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.kvq_attn_corrected(cache, q, k, v, sigma, B.KVQ_CORRECTION_OFF, cache_len=n_cached, out=out, status_word=status)
        e1.record()
        if i >= 3:
            recs_off.append((e0, e1))
    torch.cuda.synchronize()
    attn_off_ms = float(np.mean([a.elapsed_time(b_) for a, b_ in recs_off])) if recs_off else float("nan")

    # ---- end to end through the public call with HOST buffers ----
    if not args.no_e2e:
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
            B.kvq_attn_corrected(cache, dq, dk, dv, sigma, flags, cache_len=n_cached, out=out, status_word=status)
            B.kvq_quantize_append(cache, dk, dv, cache_len=n_cached)
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
                B.kvq_attn_corrected(cache, bq, bk, bv, sigma, flags, cache_len=n_cached, out=bo, status_word=status)
                B.kvq_quantize_append(cache, bk, bv, cache_len=n_cached)
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
    # ---- reduce over ranks: slowest rank's time ----
    step_ms, attn_mean, app_mean, attn_off_ms, e2e_ms, eager_step_ms = replicas.max_over_ranks(
        [step_ms, float(attn_ms.mean()), float(app_ms.mean()), attn_off_ms, 0.0 if args.no_e2e else e2e_ms,
         eager_step_ms], device=dev)

    if rank == 0:
        flops = w.flops()
        value = replicas.aggregate_value(flops, world, step_ms)
        attn_tf = flops / (attn_mean * 1e-3) / 1e12
        bursty = attn_mean < 1.0
        peak = peaks["tf_burst"] if bursty else peaks["tf_sustained"]
        res = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config,
            "launch": "eager calls (--profile)" if args.profile else "step replayed from a CUDA graph",
            "ms_per_step_eager": eager_step_ms,
            "us_per_call": {"attn_corrected": attn_mean * 1e3, "attn_uncorrected": attn_off_ms * 1e3,
                            "quantize_append": app_mean * 1e3,
                            "correction_overhead": attn_mean / attn_off_ms - 1.0},
            "hbm_gbs": {"attn": w.attn_bytes() / (attn_mean * 1e-3) / 1e9,
                        "quantize_append": w.append_bytes() / (app_mean * 1e-3) / 1e9,
                        "quantize_append_frac_of_peak": w.append_bytes() / (app_mean * 1e-3) / 1e9 / peaks["hbm_gbs"]},
            "roofline": {"kernel": "attn_tcgen05_kernel", "bound": "tensor", "achieved": attn_tf, "peak": peak,
                         "unit": "TFLOP/s", "frac": attn_tf / peak,
                         "peak_kind": ("burst" if bursty else "sustained") + " bf16, " + peaks["source"],
                         "frac_of_sustained": attn_tf / peaks["tf_sustained"],
                         "traffic": NCU_TRAFFIC_BYTES.get(w.name)},
            # kernels of this library launched inside the timed region: per step the attention call's
            # (pre-pass, attention, merge as the problem needs them) plus one quantize-append
            "gpu_launches": (B.kvq_attn_kernel_launches(cache, n_cached, q.shape[2], k.shape[2], flags) + 1) * args.steps,
            "clocks": clocks,
        }
        if not args.no_e2e:
            res["e2e"] = {"value": world * flops / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                          "mode": "host copies on their own streams beside the kernels (two buffer sets), L2 flush inside",
                          "serial_ms_per_step": e2e_serial_ms,
                          "h2d_bytes_per_step": int(3 * q.numel() * 2), "d2h_bytes_per_step": int(out.numel() * 2),
                          "ms_per_step": e2e_ms}
        if world == 1 and not args.no_cpu_baseline:
            times, oflops, sample, threads = oracle_sample(w, 2, warm=0)
            res["cpu_baseline"] = {"value": oflops / float(np.mean(times)) / 1e12, "unit": "TFLOP/s", "cores": threads,
                                   "kind": "oracle", "sample": sample}
        print(json.dumps(res))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
