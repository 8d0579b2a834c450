#!/usr/bin/env python
"""Benchmark of the quantize-and-attend hot path.

One step = one pass of the whole path over one batch of seeded synthetic input:
prefill compression of every layer, then `decode_steps` x (append + decode attention)
across all layers, including the re-compression of the tail after 100 tokens.

Workload: the LLaMA3-8B-shaped configuration (batch 8, 32 query / 8 KV heads, context
4096, bf16, 40 % salient at 4-bit / 60 % at 2-bit, 128 decode steps), instantiated as
`--layers` independent layers so that consecutive decode launches read different caches
(the set cycled through is several times larger than L2, as it is in a real model).

  value      decode-attention throughput: algorithmic bytes the decode calls must read
             (packed codes + per-token scale/zero + tail + channel factors + q/out)
             divided by the device time of the decode phase, inputs resident in HBM.
  e2e        the same metric through the C ABI with host buffers: every decode step copies
             q, k, v from pinned host memory and reads the output back; the prefill copies
             Q, K, V from pinned host memory.
  roofline   for the dominant kernel (decode attention): achieved = algorithmic bytes per
             decode call / average device time per decode call in the timed region.
  cpu_baseline  the NumPy oracle timed on the host cores on a bounded sample of units.

`--impl reference` times the oracle alone (there is no other reference program).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

METRIC = "mixed_bit_kv_decode_attention_hbm_gbs"
UNIT = "GB/s"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# DRAM bytes of one k_decode launch (= one decode-attention call) measured with ncu
# (dram__bytes_read.sum + dram__bytes_write.sum), keyed by workload id; the captures and their
# conditions are in profiles/k_decode_config2.md and profiles/k_decode_config4.md (the first
# decode steps after a prefill, when the tail holds a few tokens).
PROFILED_DRAM_BYTES_PER_DECODE_CALL = {2: 28.26e6, 4: 449.6e6 + 19.0e6}


def algorithmic_decode_bytes(w, n_windows: int, n_tail: int) -> int:
    """Bytes one decode-attention call must read for ALL units of one layer: packed K and V
    codes, one (scale, zero) fp32 pair per token per tensor, the full-precision tail, the
    channel factors of every (segment, class), q and the output."""
    import math
    per_unit = 0
    n_s0 = int(math.floor(w.saliency_ratio * w.context))
    n_sw = int(math.floor(w.saliency_ratio * w.window))
    for bits, n0, nw in ((w.bits_hi, n_s0, n_sw), (w.bits_lo, w.context - n_s0, w.window - n_sw)):
        per_unit += (n0 + n_windows * nw) * (32 * bits + 16)
        per_unit += ((1 if n0 > 0 else 0) + (n_windows if nw > 0 else 0)) * 2 * 128 * 4
    per_unit += n_tail * 2 * 128 * 2
    per_unit += w.group * 128 * 2 * 2
    return per_unit * w.units_per_layer


def oracle_sample(w, n_units: int, n_steps: int, layer: int = 0):
    """Times the oracle on `n_units` units of the workload: prefill compression and
    `n_steps` decode steps.  Returns (decode GB/s, prefill tokens/s, seconds, threads)."""
    from oracle import zipcache_oracle as zo
    from workloads import make_prefill, make_decode_step, decode_probe_flags
    Q, K, V = make_prefill(w, layer, "cpu")
    every = [(b, kv) for b in range(w.batch) for kv in range(w.n_kv_heads)]
    order = np.random.RandomState(1234).permutation(len(every))
    units = [every[j] for j in order[: min(n_units, len(every))]]
    f64 = lambda t: t.to(torch.float64).numpy()
    Qh, Kh, Vh = f64(Q), f64(K), f64(V)
    P = zo.probe_positions(w.context, w.rho_recent, w.rho_random, w.seed(layer))
    oc = zo.ZipCacheOracle(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.saliency_ratio,
                           w.bits_hi, w.bits_lo, w.window, units=units)
    t0 = time.perf_counter()
    oc.prefill_compress(Qh, Kh, Vh, P)
    t_pre = time.perf_counter() - t0
    flags = decode_probe_flags(w, layer, n_steps)
    steps = [tuple(f64(t) for t in make_decode_step(w, layer, s, "cpu")) for s in range(n_steps)]
    t0 = time.perf_counter()
    nbytes = 0
    for s, (q, k, v) in enumerate(steps):
        oc.append(k, v)
        oc.decode_attention(q, flags[s])
        nbytes += algorithmic_decode_bytes(w, 0, s + 1) // w.units_per_layer * len(units)
    t_dec = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    return (nbytes / t_dec / 1e9, len(units) * w.context / t_pre, t_pre + t_dec, threads,
            f"{len(units)} of {w.units_per_layer} units of one layer: prefill compression + "
            f"{n_steps} decode steps")


def rank_layers(rank: int, layers_per_rank: int):
    """Layers (independent units of work) owned by one rank: the path shards over units with
    no exchange step, so ranks never share a layer."""
    return [rank * layers_per_rank + i for i in range(layers_per_rank)]


def max_over_ranks(values, dist, device):
    """Element-wise maximum of per-rank timings (the slowest rank sets the job's time)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def aggregate_throughput(bytes_per_rank: int, world: int, ms: float) -> float:
    """Whole-job GB/s: every rank moves `bytes_per_rank` in the slowest rank's time."""
    return world * bytes_per_rank / (ms * 1e-3) / 1e9


def run_reference(args):
    """The oracle as the reference arm: same metric, same workload, bounded sample."""
    from workloads import get_config
    w = get_config(2)
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals, times = [], []
    sample = ""
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        gbs, tps, secs, threads, sample = oracle_sample(w, 16, 32)
        if i >= args.warmup:
            vals.append(gbs)
            times.append(time.perf_counter() - t0)
    v = float(np.mean(vals))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(times)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": f"{w.name} (oracle on a sample per step: {sample})"},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--decode-steps", type=int, default=0,
                    help="profiling only: fewer decode steps than the workload's own")
    ap.add_argument("--items", default="overlap", choices=["overlap", "single"],
                    help="overlap: ZC_FLAG_OVERLAP_CALLS (the layers' calls share the GPU: few large "
                         "work items); single: items sized for a call that has the GPU to itself")
    ap.add_argument("--append", default="deferred", choices=["deferred", "kernel"],
                    help="deferred: zc_append hands the new row to the next zc_decode_attention "
                         "(ZC_FLAG_DEFER_APPEND); kernel: zc_append copies with its own launch")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
        return

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist = dist_
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"

    import paper_2405_14256_b200 as zc
    from workloads import get_config, make_prefill, make_decode_step, decode_probe_flags
    zc.load_library()
    w = get_config(args.config)
    R = args.layers
    n_dec = args.decode_steps or w.decode_steps
    # rank r owns layers r*R .. r*R+R-1 (independent units: no collective on the data path)
    layer_ids = rank_layers(rank, R)
    probes = [zc.zc_default_probes(w.context, w.rho_recent, w.rho_random, w.seed(ly))
              for ly in layer_ids]
    inputs = [make_prefill(w, ly, dev) for ly in layer_ids]
    cfg = zc.ZcConfig.make(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context, n_dec,
                           w.saliency_ratio, w.bits_hi, w.bits_lo, w.window)
    _, ws_bytes = zc.zc_cache_bytes(cfg)
    workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)   # shared by all layers
    caches = [zc.ZipCache(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context, n_dec,
                          w.saliency_ratio, w.bits_hi, w.bits_lo, w.window, device=dev,
                          workspace=workspace, defer_append=args.append == "deferred",
                          overlap_calls=args.items == "overlap")
              for _ in range(R)]
    flags = [decode_probe_flags(w, ly, n_dec) for ly in layer_ids]
    # decode inputs: 4 distinct seeded sets per step, cycled over layers (fresh N(0,1) each)
    dec_in = [[make_decode_step(w, v, s, dev) for v in range(4)] for s in range(n_dec)]
    outs = [torch.empty_like(dec_in[0][0][0]) for _ in range(R)]
    stream = torch.cuda.Stream()

    def prefill_all():
        for i, c in enumerate(caches):
            Q, K, V = inputs[i]
            c.prefill_compress(Q, K, V, probes[i])

    def decode_all():
        nbytes = 0
        for s in range(n_dec):
            for i, c in enumerate(caches):
                q, k, v = dec_in[s][i % 4]
                c.append(k, v)
                nbytes += zc.zc_decode_bytes(c.handle)
                c.decode_attention(q, flags[i][s], out=outs[i])
        return nbytes

    with torch.cuda.stream(stream):
        prefill_all()
        l0 = sum(zc.zc_launch_count(c.handle) for c in caches)
        stream.synchronize()
        # capture the decode phase once: replaying it re-runs the same device work on the
        # state a prefill leaves behind (the handles' host-side counters stay at capture end)
        graph = torch.cuda.CUDAGraph()
        l1 = sum(zc.zc_launch_count(c.handle) for c in caches)
        with torch.cuda.graph(graph, stream=stream):
            dec_bytes = decode_all()
        l2 = sum(zc.zc_launch_count(c.handle) for c in caches)
    launches_prefill, launches_decode = l0, l2 - l1
    n_decode_calls = n_dec * R

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def one_step(ev):
        with torch.cuda.stream(stream):
            ev[0].record(stream)
            prefill_all()
            ev[1].record(stream)
            graph.replay()
            ev[2].record(stream)

    mk = lambda: [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    for _ in range(args.warmup):
        one_step(mk())
    sync_all()
    sampler = ClockSampler(local_rank)
    sampler.start()
    evs = [mk() for _ in range(args.steps)]
    t_wall0 = time.perf_counter()
    for ev in evs:
        one_step(ev)
    sync_all()
    t_wall = time.perf_counter() - t_wall0
    clocks = sampler.stop()
    t_pre = sum(ev[0].elapsed_time(ev[1]) for ev in evs) / args.steps      # ms per step
    t_dec = sum(ev[1].elapsed_time(ev[2]) for ev in evs) / args.steps
    t_step = evs[0][0].elapsed_time(evs[-1][2]) / args.steps
    t_step, t_pre, t_dec = max_over_ranks([t_step, t_pre, t_dec], dist, dev)

    # ---- end to end through the C ABI with host buffers ----
    e2e = None
    if not args.no_e2e:
        pin = lambda t: t.cpu().pin_memory()
        host_in = [tuple(pin(t) for t in inputs[i]) for i in range(min(4, R))]
        # The inputs of one decode step (q, k_new, v_new of every layer) travel as one pinned
        # buffer and the step's results come back as one: one copy each way per decode step,
        # the layers' calls back to back between them.
        per_layer = [torch.cat([t.reshape(-1) for t in dec_in[s][v]]) for s in range(n_dec) for v in range(4)]
        host_step = [pin(torch.stack([per_layer[4 * s + (i % 4)] for i in range(R)])) for s in range(n_dec)]
        del per_layer
        dq = [torch.empty_like(t) for t in inputs[0]]
        dd_step = torch.empty_like(host_step[0], device=dev)
        dd = []
        for i in range(R):
            views, at = [], 0
            for t in dec_in[0][0]:
                views.append(dd_step[i, at:at + t.numel()].view(t.shape))
                at += t.numel()
            dd.append(views)
        outs_e = torch.empty((R,) + tuple(outs[0].shape), dtype=outs[0].dtype, device=dev)
        host_out = torch.empty_like(outs_e, device="cpu").pin_memory()
        caches_e = [zc.ZipCache(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context, n_dec,
                                w.saliency_ratio, w.bits_hi, w.bits_lo, w.window, device=dev,
                                workspace=workspace, defer_append=args.append == "deferred",
                                overlap_calls=args.items == "overlap")
                    for _ in range(R)]
        h2d = d2h = 0
        sync_all()
        e0, e1, e2_ = mk()
        with torch.cuda.stream(stream):
            e0.record(stream)
            for i, c in enumerate(caches_e):
                for dst, src in zip(dq, host_in[i % len(host_in)]):
                    dst.copy_(src, non_blocking=True)
                    h2d += src.numel() * src.element_size()
                c.prefill_compress(dq[0], dq[1], dq[2], probes[i])
            e1.record(stream)
            eb = 0
            for s in range(n_dec):
                dd_step.copy_(host_step[s], non_blocking=True)
                h2d += host_step[s].numel() * host_step[s].element_size()
                for i, c in enumerate(caches_e):
                    c.append(dd[i][1], dd[i][2])
                    eb += zc.zc_decode_bytes(c.handle)
                    c.decode_attention(dd[i][0], flags[i][s], out=outs_e[i])
                host_out.copy_(outs_e, non_blocking=True)
                d2h += outs_e.numel() * outs_e.element_size()
            e2_.record(stream)
        sync_all()
        te_dec, te_pre = max_over_ranks([e1.elapsed_time(e2_), e0.elapsed_time(e1)], dist, dev)
        e2e = {"value": aggregate_throughput(eb, world, te_dec), "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
               "prefill_tokens_per_s": world * R * w.batch * w.context / (te_pre * 1e-3),
               "note": "eager C-ABI calls, pinned host buffers, copies inside the timed region: per "
                       "layer one copy of the prompt's Q, K, V; per decode step one copy of all "
                       "layers' q, k_new, v_new to the device and one of all results back"}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    peak, peak_kind = _peaks()
    value = aggregate_throughput(dec_bytes, world, t_dec)
    per_call_us = t_dec * 1e3 / n_decode_calls
    achieved = dec_bytes / (t_dec * 1e-3) / 1e9          # per GPU
    traffic = PROFILED_DRAM_BYTES_PER_DECODE_CALL.get(w.cfg_id)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{w.name} x {R} independent layers per GPU",
                   "l2": f"inputs larger than L2: {R} caches "
                         f"({R * dec_bytes / n_decode_calls / 1e6:.0f} MB) cycled every decode step",
                   "batch": w.batch, "context": w.context, "n_q_heads": w.n_q_heads,
                   "n_kv_heads": w.n_kv_heads, "decode_steps": n_dec, "bits": "4/2",
                   "saliency_ratio": w.saliency_ratio, "decode_phase": "CUDA graph replay",
                   "items": ("ZC_FLAG_OVERLAP_CALLS: consecutive layers' calls run side by side"
                             if args.items == "overlap" else "sized for one call at a time"),
                   "append": ("zc_append defers the copy into the next zc_decode_attention "
                              "(ZC_FLAG_DEFER_APPEND)" if args.append == "deferred"
                              else "zc_append launches its own copy kernel")},
        "prefill_tokens_per_s": world * R * w.batch * w.context / (t_pre * 1e-3),
        "prefill_ms": t_pre, "decode_ms": t_dec, "decode_us_per_call": per_call_us,
        "pct_of_hbm_peak": 100.0 * achieved / peak,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_kind": f"of {peak_kind}",
                     "kernel": "k_decode (one launch per call: decode phase time / decode calls; "
                               "consecutive calls run side by side)",
                     "bytes_per_launch": dec_bytes / n_decode_calls,
                     "us_per_launch": per_call_us},
        "clocks": clocks,
        "gpu_launches": int(launches_prefill + launches_decode),
        "wall_s_timed": t_wall,
    }
    if e2e is not None:
        line["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1:
        gbs, tps, secs, threads, sample = oracle_sample(w, 64, 96)
        line["cpu_baseline"] = {"value": gbs, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": sample, "prefill_tokens_per_s": tps, "seconds": secs}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
