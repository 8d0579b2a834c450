#!/usr/bin/env python
"""Benchmark of the quantize-and-attend hot path.

One step = one pass of the whole path over one batch of seeded synthetic input:
prefill compression of every layer, then `decode_steps` x (append + decode attention)
across all layers, including the re-compression of the tail after every 100 tokens.

The default run measures the four full-size workloads (2, 3, 4, 5) one after the other; each
is instantiated as enough independent layers that the caches cycled through in one decode step
exceed 512 MB (several times L2), so every call reads from HBM.  For each workload the decode
phase is captured once per launch mode and replayed as a CUDA graph:

  overlap    ZC_FLAG_OVERLAP_CALLS | ZC_FLAG_DEFER_APPEND: the caller promises that only
             decode calls of independent caches follow one another, consecutive calls run
             side by side on the GPU (a throughput figure).
  dependent  ZC_FLAG_DEFER_APPEND only: every call waits for the kernel before it on the
             stream before it reads its inputs, as a layer whose query comes out of the
             previous kernel must (one call at a time on the GPU).

The headline (`value`, `roofline`, `e2e`, `cpu_baseline`) is the largest workload (5:
32 layers, context 32768) in the overlap mode; `per_config` carries every workload in both
modes with its prefill throughput and parity counters.

  value      decode-attention throughput: algorithmic bytes the decode calls must read
             (packed codes + per-token scale/zero + tail + channel factors + q/out)
             divided by the device time of the decode phase, inputs resident in HBM.
  e2e        the same metric through the C ABI with host buffers: every decode step copies
             q, k, v from pinned host memory and reads the output back; the prefill copies
             Q, K, V from pinned host memory.
  roofline   for the dominant kernel (decode attention): achieved = algorithmic bytes per
             decode call / average device time per decode call in the timed region.
  cpu_baseline  the NumPy oracle timed on the host cores on a bounded sample of units.

`--config N` restricts the run to one workload; `--impl reference` times the oracle alone
(there is no other reference program).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
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
NOMINAL_HBM_GBS = 8000.0
HEADLINE_CONFIG = 5
DEFAULT_CONFIGS = (2, 3, 4, 5)
MIN_CYCLED_BYTES = 512e6


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def _tensor_peak():
    """Dense bf16 / fp16 TFLOP/s for a kernel timed inside a loop (the sustained figure)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d.get("bf16_tflops_sustained", d.get("bf16_tflops", 1400.0))), "measured, sustained"
    return 1400.0, "fallback, sustained"


def measure_prefill_attention(zc, wb, w, R):
    """The step beside the path in Alg. 2: causal attention output with row log-sum-exp
    (zc_prefill_attention), and prefill compression that takes the probe rows' statistics from
    it (zc_prefill_compress_lse) instead of running its first score pass."""
    n = min(R, 4)
    c0 = wb.caches[next(iter(wb.caches))]
    O = torch.empty((w.batch, w.n_q_heads, w.context, 128), dtype=w.torch_dtype, device=wb.dev)
    lse = [torch.empty((w.batch, w.n_q_heads, w.context), dtype=torch.float32, device=wb.dev) for _ in range(n)]
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    with torch.cuda.stream(wb.stream):
        for rep in range(4):           # one warm-up pass, three timed
            if rep == 1:
                ev[0].record(wb.stream)
            for i in range(n):
                Q, K, V = wb.inputs[i]
                zc.zc_prefill_attention(c0[i].handle, Q, K, V, w.context, O, lse[i])
        ev[1].record(wb.stream)
        for rep in range(3):
            for i in range(n):
                Q, K, V = wb.inputs[i]
                c0[i].prefill_compress_lse(Q, K, V, wb.probes[i], lse[i])
        ev[2].record(wb.stream)
    torch.cuda.synchronize()
    t_att = ev[0].elapsed_time(ev[1]) / (3 * n)
    t_cmp = ev[1].elapsed_time(ev[2]) / (3 * n)
    flops = 2.0 * w.context * w.context * 128 * w.batch * w.n_q_heads      # causal: half of 4 l^2 d per head
    peak, kind = _tensor_peak()
    return {"attention_ms_per_layer": t_att, "attention_tflops": flops / (t_att * 1e-3) / 1e12,
            "attention_frac_of_tensor_peak": flops / (t_att * 1e-3) / 1e12 / peak, "tensor_peak": f"{peak} TFLOP/s ({kind})",
            "compress_with_attention_lse_tokens_per_s": w.batch * w.context / (t_cmp * 1e-3)}


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


def profiled_traffic(cfg_id: int):
    """DRAM bytes of one k_decode launch from the ncu capture recorded in
    profiles/k_decode_traffic.json, or None when the decode kernel's source has changed since
    the counters were taken (the record carries the source's SHA-256)."""
    rec = os.path.join(ROOT, "profiles", "k_decode_traffic.json")
    src = os.path.join(ROOT, "paper_2405_14256_b200", "csrc", "zc_decode.cu")
    try:
        with open(rec) as f:
            d = json.load(f)
        with open(src, "rb") as f:
            sha = hashlib.sha256(f.read()).hexdigest()
        if d.get("zc_decode_cu_sha256") != sha:
            return None
        v = d.get("dram_bytes_per_launch", {}).get(str(cfg_id))
        return float(v) if v is not None else None
    except Exception:
        return None


def algorithmic_decode_bytes(w, n_windows: int, n_tail: int) -> int:
    """Bytes one decode-attention call must read for ALL units of one layer: packed K and V
    codes, one (scale, zero) fp32 pair per token per tensor quantised tokenwise, the
    full-precision tail, the channel factors of every (segment, class), q and the output."""
    per_unit = 0
    n_s0 = int(math.floor(w.saliency_ratio * w.context))
    n_sw = int(math.floor(w.saliency_ratio * w.window))
    kch = w.k_scheme == "channel"
    for bits, n0, nw in ((w.bits_hi, n_s0, n_sw), (w.bits_lo, w.context - n_s0, w.window - n_sw)):
        runs = (1 if n0 > 0 else 0) + (n_windows if nw > 0 else 0)
        if bits == 16:                       # rows kept at full precision
            per_unit += (n0 + n_windows * nw) * 512
            continue
        per_unit += (n0 + n_windows * nw) * (32 * bits + (8 if kch else 16))
        per_unit += runs * (3 if kch else 2) * 128 * 4
    per_unit += n_tail * 2 * 128 * 2
    per_unit += w.group * 128 * 2 * 2
    return per_unit * w.units_per_layer


def algorithmic_prefill_bytes(w) -> int:
    """Bytes the prefill compression of one layer must move: K read by the two score passes
    (shared by the query heads of a KV head), the probe rows of Q twice, K and V read by the
    channel-maximum pass and again by the quantiser, packed codes and parameters written."""
    l = w.context
    n_s = int(math.floor(w.saliency_ratio * l))
    n_p = max(1, int(math.floor(w.rho_recent * l))) + int(math.floor(w.rho_random * l))
    per_unit = 2 * l * 256 + 2 * w.group * n_p * 256 + 2 * 2 * l * 256
    per_unit += n_s * (32 * w.bits_hi + 16) + (l - n_s) * (32 * w.bits_lo + 16)
    return per_unit * w.units_per_layer


EXP2_PER_S_PEAK = 148 * 16 * 1.965e9   # the exp2 unit: 16 results per clock and SM, 148 SMs at the maximum SM clock


def prefill_exponentials(w, probes) -> float:
    """exp2 evaluations the probe scores of one layer need (Eq. 9): every probe row's causal
    keys, for every query head, in both passes (row log-sum-exp, then the normalised columns)."""
    return 2.0 * float(sum(p + 1 for p in probes)) * w.n_q_heads * w.batch


def oracle_sample(w, n_units: int, n_steps: int, layer: int = 0, prefilled=None):
    """Times the oracle on `n_units` units of the workload: prefill compression and `n_steps`
    decode steps.  Returns a dict; `threads` is what the oracle really used (process CPU time
    over wall time: NumPy's BLAS calls are threaded, the Python around them is not)."""
    from oracle import zipcache_oracle as zo
    from workloads import make_decode_step, decode_probe_flags
    f64 = lambda t: t.to(torch.float64).numpy()
    cpu0, wall0 = time.process_time(), time.perf_counter()
    if prefilled is None:
        oc, units, t_pre = oracle_prefill(w, n_units, layer)
    else:
        oc, units, t_pre = prefilled
    flags = decode_probe_flags(w, layer, n_steps)
    steps = []
    for s in range(n_steps):
        q, k, v = make_decode_step(w, layer, s, "cpu")
        steps.append((_units_only(q, units, w.group), _units_only(k, units, 1), _units_only(v, units, 1)))
    tail0 = oc.units[units[0]].tail_K.shape[0]
    nwin = len(oc.units[units[0]].segments) - 1
    t0 = time.perf_counter()
    nbytes = 0
    refs = []
    for s, (q, k, v) in enumerate(steps):
        oc.append(k, v)
        refs.append(oc.decode_attention(q, flags[s]))
        nbytes += algorithmic_decode_bytes(w, nwin, tail0 + s + 1) // w.units_per_layer * len(units)
    t_dec = time.perf_counter() - t0
    cpu, wall = time.process_time() - cpu0, time.perf_counter() - wall0
    threads = max(1.0, round(cpu / max(wall, 1e-9), 1)) if prefilled is None else 1.0
    return {"gbs": nbytes / t_dec / 1e9, "prefill_tokens_per_s": len(units) * w.context / t_pre if t_pre else None,
            "seconds": t_pre + t_dec, "threads": threads, "oracle": oc, "units": units, "refs": refs,
            "sample": f"{len(units)} of {w.units_per_layer * w.n_layers} units: prefill compression + "
                      f"{n_steps} decode steps"}


class _UnitsOnly:
    """fp64 copies of the sampled units of a [batch, heads, ...] tensor, indexed like the tensor."""

    def __init__(self, t, units, G):
        self.G = G
        self.d = {(b, kv): t[b, kv * G:(kv + 1) * G].to(torch.float64).numpy() for (b, kv) in units}

    def __getitem__(self, key):
        b, h = key
        if isinstance(h, slice):
            return self.d[(b, h.start // self.G)]
        return self.d[(b, h)][0]


def _units_only(t, units, G):
    return _UnitsOnly(t, units, G)


def parity_with_oracle(zc, w, dev, r, layer: int = 0):
    """Part of the CPU-baseline leg: the library is run on the very inputs the oracle sample was
    timed on (generated on the host, copied over) and compared with it on the sampled units.
    Counters: salient-set differences (near-tie swaps: both tokens within relative 1e-5 of the
    oracle's threshold score; anything else is a mismatch), packed-code / parameter mismatches
    on the units without swaps, and the largest |out - oracle| over the sampled decode steps
    (fp32 output, nothing subtracted)."""
    from oracle import zipcache_oracle as zo
    from workloads import make_prefill, make_decode_step, decode_probe_flags
    oc, units, refs = r["oracle"], r["units"], r["refs"]
    Q, K, V = (t.to(dev) for t in make_prefill(w, layer, "cpu"))
    n_steps = len(refs)
    c = zc.ZipCache(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context, max(n_steps, 1),
                    w.saliency_ratio, w.bits_hi, w.bits_lo, w.window, device=dev, out_f32=True)
    c.prefill_compress(Q, K, V, zc.zc_default_probes(w.context, w.rho_recent, w.rho_random, w.seed(layer)))
    del Q, K, V
    p_gpu = c.scores(w.context).cpu().numpy()
    exported = {(sub, ten): [x.cpu().numpy() for x in c.segment(0, ten, sub)] for sub in (0, 1) for ten in (0, 1)}
    swaps = set_mism = code_mism = 0
    score_rel = 0.0
    for (b, kv) in units:
        seg = oc.units[(b, kv)].segments[0]
        score_rel = max(score_rel, float((np.abs(p_gpu[b, kv] - seg.p_tilde) / np.maximum(seg.p_tilde, 1e-30)).max()))
        got, want = set(exported[(0, 0)][0][b, kv].tolist()), set(seg.hi.idx.tolist())
        if got != want:
            kth = np.sort(seg.p_tilde)[::-1][seg.hi.n - 1]
            diff = (got - want) | (want - got)
            if all(abs(seg.p_tilde[j] - kth) <= 1e-5 * abs(kth) for j in diff):
                swaps += len(diff) // 2
            else:
                set_mism += len(diff) // 2
            continue
        for sub, name in ((0, "hi"), (1, "lo")):
            o_sub = getattr(seg, name)
            if o_sub.n == 0:
                continue
            for ten, qn in ((0, "qK"), (1, "qV")):
                idx, codes, sz, cf = exported[(sub, ten)]
                qd = getattr(o_sub, qn)
                code_mism += int((codes[b, kv] != zo.pack_codes(qd["codes"], o_sub.bits)).sum())
                code_mism += int((sz[b, kv, :, 0] != qd["s"]).sum() + (sz[b, kv, :, 1] != qd["z"]).sum())
                code_mism += int((cf[b, kv] != qd["c"]).sum())
    flags = decode_probe_flags(w, layer, n_steps)
    worst = 0.0
    for s in range(n_steps):
        q, k, v = (t.to(dev) for t in make_decode_step(w, layer, s, "cpu"))
        c.append(k, v)
        out = c.decode_attention(q, flags[s]).double().cpu().numpy()
        for (b, kv), o in refs[s].items():
            worst = max(worst, float(np.abs(out[b, kv * w.group:(kv + 1) * w.group] - o).max()))
    return {"units": len(units), "decode_steps": n_steps, "score_max_rel_err": score_rel,
            "near_tie_swaps": swaps, "salient_set_mismatches": set_mism,
            "code_and_parameter_mismatches": code_mism, "decode_max_abs_err_fp32_out": worst,
            "device_status": zc.zc_device_status()}


def oracle_prefill(w, n_units: int, layer: int = 0):
    from oracle import zipcache_oracle as zo
    from workloads import make_prefill
    Q, K, V = make_prefill(w, layer, "cpu")
    every = [(b, kv) for b in range(w.batch) for kv in range(w.n_kv_heads)]
    order = np.random.RandomState(1234).permutation(len(every))
    units = [every[j] for j in order[: min(n_units, len(every))]]
    Qh, Kh, Vh = _units_only(Q, units, w.group), _units_only(K, units, 1), _units_only(V, units, 1)
    del Q, K, V
    P = zo.probe_positions(w.context, w.rho_recent, w.rho_random, w.seed(layer))
    oc = zo.ZipCacheOracle(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.saliency_ratio,
                           w.bits_hi, w.bits_lo, w.window, units=units, k_scheme=w.k_scheme)
    t0 = time.perf_counter()
    oc.prefill_compress(Qh, Kh, Vh, P)
    return oc, units, time.perf_counter() - t0


# units and decode steps of the oracle sample per workload: about 10 to 30 s of CPU work
ORACLE_SAMPLE = {1: (4, 16), 2: (64, 96), 3: (16, 32), 4: (64, 32), 5: (4, 32)}


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


ROTATION_DEPTH = 1.7   # caches cycled, in units of the calls that fit on the GPU at once
CTA_SLOTS = 148 * 4    # decode CTAs resident on a B200 (4 per SM)


def layers_for(w, requested: int) -> int:
    """Independent layers per GPU: the workload's own count when it is a stack (workload 5),
    else as many as make the caches read in one decode step exceed MIN_CYCLED_BYTES, and
    enough that the calls in flight at any time belong to different caches: a call on a cache
    waits for the call before it on THAT cache (whose kernel stored the newest tail row), and a
    rotation shorter than the number of calls the GPU holds would time that wait (workload 3:
    128 CTAs per call, 4.6 calls resident; 5 caches gave 69.4 %, 8 gave 72.0 %, 12 gave 70.6 %
    on one box)."""
    if requested > 0:
        return requested
    if w.n_layers > 1:
        return w.n_layers
    per_call = algorithmic_decode_bytes(w, 0, 0)
    ctas_per_call = w.units_per_layer * ((w.group + 3) // 4)
    return max(2, int(math.ceil(MIN_CYCLED_BYTES / per_call)),
               int(math.ceil(ROTATION_DEPTH * CTA_SLOTS / ctas_per_call)))


def run_reference(args):
    """The oracle as the reference arm: same metric and workload as the headline, a bounded
    sample per step (decode steps of one unit on the compressed cache of the prompt, which is
    compressed once before the timed steps)."""
    from workloads import get_config
    cfg_id = args.config or HEADLINE_CONFIG
    w = get_config(cfg_id)
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_units, n_steps = {5: (1, 8)}.get(cfg_id, (ORACLE_SAMPLE[cfg_id][0], 8))
    cpu0, wall0 = time.process_time(), time.perf_counter()
    pre = oracle_prefill(w, n_units)
    vals, times = [], []
    sample = ""
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        r = oracle_sample(w, n_units, n_steps, prefilled=pre)
        sample = r["sample"].replace("prefill compression + ", "")
        if i >= args.warmup:
            vals.append(r["gbs"])
            times.append(time.perf_counter() - t0)
    threads = max(1.0, round((time.process_time() - cpu0) / (time.perf_counter() - wall0), 1))
    v = float(np.mean(vals))
    sample += " per step, continuing on one cache (the prompt is compressed once, untimed)"
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


MODES = {
    "overlap": dict(overlap_calls=True, defer_append=True),
    "dependent": dict(overlap_calls=False, defer_append=True),
    # the paper's own key quantiser (channelwise keys: 8 bytes per token less to read)
    "overlap_channelwise_keys": dict(overlap_calls=True, defer_append=True, k_channel=True),
    # 16-bit quantisation parameters (8 bytes per token less); every call waits for what precedes it
    "dependent_params_f16": dict(overlap_calls=False, defer_append=True, params_f16=True),
}


class Workbench:
    """Everything one workload needs on one GPU: inputs, caches per mode, captured decode graphs."""

    def __init__(self, zc, w, R, rank, dev, n_dec, modes, append):
        from workloads import make_prefill, make_decode_step, decode_probe_flags
        self.zc, self.w, self.R, self.dev, self.n_dec = zc, w, R, dev, n_dec
        self.layer_ids = rank_layers(rank, R)
        self.probes = [zc.zc_default_probes(w.context, w.rho_recent, w.rho_random, w.seed(ly))
                       for ly in self.layer_ids]
        self.inputs = [make_prefill(w, ly, dev) for ly in self.layer_ids]
        self.flags = [decode_probe_flags(w, ly, n_dec) for ly in self.layer_ids]
        # decode inputs: 4 distinct seeded sets per step, cycled over layers (fresh N(0,1) each)
        self.dec_in = [[make_decode_step(w, v, s, dev) for v in range(4)] for s in range(n_dec)]
        self.outs = [torch.empty_like(self.dec_in[0][0][0]) for _ in range(R)]
        cfg = zc.ZcConfig.make(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context, n_dec,
                               w.saliency_ratio, w.bits_hi, w.bits_lo, w.window)
        _, ws_bytes = zc.zc_cache_bytes(cfg)
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)   # shared by all layers
        self.stream = torch.cuda.Stream()
        self.caches, self.graphs, self.dec_bytes, self.launches = {}, {}, {}, {}
        for mode in modes:
            kw = dict(MODES[mode])
            if append == "kernel":
                kw["defer_append"] = False
            if w.k_scheme == "channel":
                kw["k_channel"] = True
            self.caches[mode] = [self.make_cache(**kw) for _ in range(R)]
        with torch.cuda.stream(self.stream):
            for mode in modes:
                self.prefill_all(mode)
                l0 = self.launch_count(mode)
                self.stream.synchronize()
                # capture the decode phase once: replaying it re-runs the same device work on the
                # state a prefill leaves behind (the handles' host-side counters stay at capture end)
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=self.stream):
                    self.dec_bytes[mode] = self.decode_all(self.caches[mode], self.dec_in_for, self.outs)
                self.graphs[mode] = g
                self.launches[mode] = (l0, self.launch_count(mode) - l0)
        self.n_calls = n_dec * R

    def make_cache(self, **kw):
        w = self.w
        return self.zc.ZipCache(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context, self.n_dec,
                                w.saliency_ratio, w.bits_hi, w.bits_lo, w.window, device=self.dev,
                                workspace=self.workspace, **kw)

    def launch_count(self, mode):
        return sum(self.zc.zc_launch_count(c.handle) for c in self.caches[mode])

    def dec_in_for(self, s, i):
        return self.dec_in[s][i % 4]

    def prefill_all(self, mode):
        for i, c in enumerate(self.caches[mode]):
            Q, K, V = self.inputs[i]
            c.prefill_compress(Q, K, V, self.probes[i])

    def decode_all(self, caches, inputs_of, outs):
        nbytes = 0
        for s in range(self.n_dec):
            for i, c in enumerate(caches):
                q, k, v = inputs_of(s, i)
                c.append(k, v)
                nbytes += self.zc.zc_decode_bytes(c.handle)
                c.decode_attention(q, self.flags[i][s], out=outs[i])
        return nbytes

    def one_step(self, mode, ev):
        with torch.cuda.stream(self.stream):
            ev[0].record(self.stream)
            self.prefill_all(mode)
            ev[1].record(self.stream)
            self.graphs[mode].replay()
            ev[2].record(self.stream)


def measure_config(zc, cfg_id, args, rank, local_rank, world, dist, dev, modes, headline, **override):
    from workloads import get_config
    w = get_config(cfg_id).scaled(**override)
    R = layers_for(w, args.layers)
    n_dec = args.decode_steps or w.decode_steps
    wb = Workbench(zc, w, R, rank, dev, n_dec, modes, args.append)
    peak, peak_kind = _peaks()

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    mk = lambda: [torch.cuda.Event(enable_timing=True) for _ in range(3)]
    res = {"workload": w.name, "layers": R, "decode_steps": n_dec,
           "cycled_MB": R * algorithmic_decode_bytes(w, 0, 0) / 1e6}
    timing = {}
    for mode in modes:
        for _ in range(args.warmup):
            wb.one_step(mode, mk())
        sync_all()
        sampler = ClockSampler(local_rank)
        sampler.start()
        evs = [mk() for _ in range(args.steps)]
        t_wall0 = time.perf_counter()
        for ev in evs:
            wb.one_step(mode, ev)
        sync_all()
        t_wall = time.perf_counter() - t_wall0
        clocks = sampler.stop()
        t_pre = sum(ev[0].elapsed_time(ev[1]) for ev in evs) / args.steps      # ms per step
        t_dec = sum(ev[1].elapsed_time(ev[2]) for ev in evs) / args.steps
        t_step = evs[0][0].elapsed_time(evs[-1][2]) / args.steps
        t_step, t_pre, t_dec = max_over_ranks([t_step, t_pre, t_dec], dist, dev)
        nbytes = wb.dec_bytes[mode]
        achieved = nbytes / (t_dec * 1e-3) / 1e9          # per GPU
        timing[mode] = dict(t_step=t_step, t_pre=t_pre, t_dec=t_dec, t_wall=t_wall, clocks=clocks,
                            achieved=achieved, nbytes=nbytes)
        pre_tps = world * R * w.batch * w.context / (t_pre * 1e-3)
        res[mode] = {"us_per_call": t_dec * 1e3 / wb.n_calls, "gbs": aggregate_throughput(nbytes, world, t_dec),
                     "frac": achieved / peak, "pct_of_nominal_8TBs": 100.0 * achieved / NOMINAL_HBM_GBS,
                     "sm_mhz": clocks.get("sm_mhz"), "reasons": clocks.get("reasons")}
        res["prefill_tokens_per_s"] = pre_tps
        res["prefill_roofline_frac"] = (R * algorithmic_prefill_bytes(w) / (t_pre * 1e-3) / 1e9) / peak
        # prefill compression is bound by the exponentials of the probe scores, not by bytes: the
        # share of the exp2 unit's peak that the whole of prefill compression sustains
        res["prefill_exp2_frac"] = (sum(prefill_exponentials(w, wb.probes[i]) for i in range(R)) /
                                    (t_pre * 1e-3)) / EXP2_PER_S_PEAK
    if not override and world == 1:
        res["prefill_attention"] = measure_prefill_attention(zc, wb, w, R)
    assert zc.zc_device_status() == 0, "a bounded wait inside a kernel ran out"
    out = {"per_config": res}
    if headline:
        out.update(timing=timing, wb=wb, w=w, R=R, n_dec=n_dec, sync_all=sync_all, mk=mk)
    return out


def measure_e2e(h, args, world, dist, dev, mode):
    """End to end through the C ABI with pinned host buffers, copies inside the timed region."""
    wb, w, R, n_dec, zc = h["wb"], h["w"], h["R"], h["n_dec"], h["wb"].zc
    mk, sync_all, stream = h["mk"], h["sync_all"], wb.stream
    pin = lambda t: t.cpu().pin_memory()
    host_in = [tuple(pin(t) for t in wb.inputs[i]) for i in range(min(2, R))]
    # The inputs of one decode step (q, k_new, v_new of every layer) travel as one pinned
    # buffer and the step's results come back as one: one copy each way per decode step,
    # the layers' calls back to back between them.
    per_layer = [torch.cat([t.reshape(-1) for t in wb.dec_in[s][v]]) for s in range(n_dec) for v in range(4)]
    host_step = [pin(torch.stack([per_layer[4 * s + (i % 4)] for i in range(R)])) for s in range(n_dec)]
    del per_layer
    dq = [torch.empty_like(t) for t in wb.inputs[0]]
    dd_step = torch.empty_like(host_step[0], device=dev)
    dd = []
    for i in range(R):
        views, at = [], 0
        for t in wb.dec_in[0][0]:
            views.append(dd_step[i, at:at + t.numel()].view(t.shape))
            at += t.numel()
        dd.append(views)
    outs_e = torch.empty((R,) + tuple(wb.outs[0].shape), dtype=wb.outs[0].dtype, device=dev)
    host_out = torch.empty_like(outs_e, device="cpu").pin_memory()
    kw = dict(MODES[mode])
    if args.append == "kernel":
        kw["defer_append"] = False
    caches_e = [wb.make_cache(**kw) for _ in range(R)]
    h2d = d2h = 0
    sync_all()
    e0, e1, e2_ = mk()
    with torch.cuda.stream(stream):
        e0.record(stream)
        for i, c in enumerate(caches_e):
            for dst, src in zip(dq, host_in[i % len(host_in)]):
                dst.copy_(src, non_blocking=True)
                h2d += src.numel() * src.element_size()
            c.prefill_compress(dq[0], dq[1], dq[2], wb.probes[i])
        e1.record(stream)
        eb = 0
        for s in range(n_dec):
            dd_step.copy_(host_step[s], non_blocking=True)
            h2d += host_step[s].numel() * host_step[s].element_size()
            for i, c in enumerate(caches_e):
                c.append(dd[i][1], dd[i][2])
                eb += zc.zc_decode_bytes(c.handle)
                c.decode_attention(dd[i][0], wb.flags[i][s], out=outs_e[i])
            host_out.copy_(outs_e, non_blocking=True)
            d2h += outs_e.numel() * outs_e.element_size()
        e2_.record(stream)
    sync_all()
    te_dec, te_pre = max_over_ranks([e1.elapsed_time(e2_), e0.elapsed_time(e1)], dist, dev)
    return {"value": aggregate_throughput(eb, world, te_dec), "unit": UNIT,
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "prefill_tokens_per_s": world * R * w.batch * w.context / (te_pre * 1e-3),
            "note": "eager C-ABI calls, pinned host buffers, copies inside the timed region: per "
                    "layer one copy of the prompt's Q, K, V; per decode step one copy of all "
                    "layers' q, k_new, v_new to the device and one of all results back"}


def parity_counters(zc, w, dev):
    """Parity counters of the workload, from the run itself (no oracle involved): the salient
    set the library chose against a top-k of its own exported scores (set mismatches), tokens
    whose score lies within relative 1e-5 of the selection threshold (near-ties: the positions
    where the oracle and the library may legitimately differ), and the device error word."""
    from workloads import make_prefill
    Q, K, V = make_prefill(w, 0, dev)
    c = zc.ZipCache(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context, 4,
                    w.saliency_ratio, w.bits_hi, w.bits_lo, w.window, device=dev)
    c.prefill_compress(Q, K, V, zc.zc_default_probes(w.context, w.rho_recent, w.rho_random, w.seed(0)))
    p = c.scores(w.context).double()
    idx = c.segment(0, 0, 0)[0].long()
    n_s = idx.shape[2]
    mism = near = 0
    if 0 < n_s < w.context:
        top = torch.topk(p, n_s, dim=2)
        kth = top.values[..., -1:]
        chosen = torch.zeros_like(p, dtype=torch.bool).scatter_(2, idx, True)
        # a token strictly above the threshold must be in the set, one strictly below must not
        mism = int(((p > kth) & ~chosen).sum() + ((p < kth) & chosen).sum())
        near = int(((p - kth).abs() <= 1e-5 * kth.abs()).sum() - p.shape[0] * p.shape[1])
    torch.cuda.synchronize()
    return {"salient_set_mismatches": mism, "near_ties_at_threshold": max(near, 0),
            "device_status": zc.zc_device_status()}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layers", type=int, default=0, help="independent layers per GPU (0: per workload)")
    ap.add_argument("--config", type=int, default=0, help="one workload only (default: 2, 3, 4 and 5)")
    ap.add_argument("--decode-steps", type=int, default=0,
                    help="profiling only: fewer decode steps than the workload's own")
    ap.add_argument("--mode", default="both", choices=["both", "overlap", "dependent", "overlap_channelwise_keys", "dependent_params_f16"],
                    help="overlap: ZC_FLAG_OVERLAP_CALLS (independent caches, calls side by side); "
                         "dependent: every call waits for the kernel before it")
    ap.add_argument("--append", default="deferred", choices=["deferred", "kernel"],
                    help="deferred: zc_append hands the new row to the next zc_decode_attention "
                         "(ZC_FLAG_DEFER_APPEND); kernel: zc_append copies with its own launch")
    ap.add_argument("--bits", default="", help="H/L bit pair instead of the workload's 4/2 (2, 4, 8 or 16 each; not 8 with 16)")
    ap.add_argument("--saliency", type=float, default=-1.0, help="saliency ratio instead of the workload's")
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
    from workloads import get_config
    zc.load_library()
    configs = [args.config] if args.config else list(DEFAULT_CONFIGS)
    head_cfg = args.config or HEADLINE_CONFIG
    modes = ["overlap", "dependent", "overlap_channelwise_keys"] if args.mode == "both" else [args.mode]
    head_mode = modes[0]
    per_config, head = {}, None
    e2e = None
    override = {}
    if args.bits:
        override.update(bits_hi=int(args.bits.split("/")[0]), bits_lo=int(args.bits.split("/")[1]))
    if args.saliency >= 0:
        override.update(saliency_ratio=args.saliency)
    for cfg_id in configs:
        r = measure_config(zc, cfg_id, args, rank, local_rank, world, dist, dev, modes,
                           headline=cfg_id == head_cfg, **override)
        if rank == 0 and world == 1:
            r["per_config"]["parity"] = parity_counters(zc, get_config(cfg_id), dev)
        per_config[str(cfg_id)] = r["per_config"]
        if cfg_id == 2 and args.mode == "both" and not args.config:
            # the other bit pairs of the paper's comparison grid (Table 3), on workload 2
            pairs = {}
            for name, ov in (("4/4 all salient", dict(bits_hi=4, bits_lo=4, saliency_ratio=1.0)),
                             ("16/2 15.2% salient", dict(bits_hi=16, bits_lo=2, saliency_ratio=0.152)),
                             ("2/2", dict(bits_hi=2, bits_lo=2)),
                             ("8/4", dict(bits_hi=8, bits_lo=4))):
                rr = measure_config(zc, cfg_id, args, rank, local_rank, world, dist, dev, ["overlap"],
                                    headline=False, **ov)["per_config"]
                pairs[name] = {"us_per_call": rr["overlap"]["us_per_call"], "frac": rr["overlap"]["frac"],
                               "gbs": rr["overlap"]["gbs"], "prefill_tokens_per_s": rr["prefill_tokens_per_s"]}
            per_config[str(cfg_id)]["bit_pairs_overlap_mode"] = pairs
            rr = measure_config(zc, cfg_id, args, rank, local_rank, world, dist, dev, ["dependent_params_f16"],
                                headline=False)["per_config"]["dependent_params_f16"]
            per_config[str(cfg_id)]["params_f16_one_call_at_a_time"] = {
                "us_per_call": rr["us_per_call"], "frac": rr["frac"], "gbs": rr["gbs"]}
        if cfg_id == head_cfg:
            head = r
            if not args.no_e2e:
                e2e = measure_e2e(head, args, world, dist, dev, head_mode)
            head = {k: v for k, v in head.items() if k not in ("wb",)} | {
                "launches": r["wb"].launches[head_mode], "n_calls": r["wb"].n_calls}
        del r
        torch.cuda.empty_cache()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    peak, peak_kind = _peaks()
    w, R, n_dec = head["w"], head["R"], head["n_dec"]
    t = head["timing"][head_mode]
    n_calls = head["n_calls"]
    per_call_us = t["t_dec"] * 1e3 / n_calls
    achieved = t["achieved"]
    line = {
        "metric": METRIC, "value": aggregate_throughput(t["nbytes"], world, t["t_dec"]), "unit": UNIT,
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t["t_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{w.name} x {R} independent layers per GPU",
                   "l2": f"inputs larger than L2: {R} caches "
                         f"({R * t['nbytes'] / n_calls / 1e6:.0f} MB) cycled every decode step",
                   "batch": w.batch, "context": w.context, "n_q_heads": w.n_q_heads,
                   "n_kv_heads": w.n_kv_heads, "decode_steps": n_dec, "bits": f"{w.bits_hi}/{w.bits_lo}",
                   "saliency_ratio": w.saliency_ratio, "decode_phase": "CUDA graph replay",
                   "mode": ("ZC_FLAG_OVERLAP_CALLS: consecutive layers' calls run side by side"
                            if head_mode == "overlap" else "every call waits for the kernel before it"),
                   "append": ("zc_append defers the copy into the next zc_decode_attention "
                              "(ZC_FLAG_DEFER_APPEND)" if args.append == "deferred"
                              else "zc_append launches its own copy kernel"),
                   "other_workloads": "per_config: workloads 2, 3, 4, 5 in both launch modes"},
        "prefill_tokens_per_s": world * R * w.batch * w.context / (t["t_pre"] * 1e-3),
        "prefill_ms": t["t_pre"], "decode_ms": t["t_dec"], "decode_us_per_call": per_call_us,
        "pct_of_hbm_peak": 100.0 * achieved / peak,
        "pct_of_nominal_hbm_peak_8TBs": 100.0 * achieved / NOMINAL_HBM_GBS,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": profiled_traffic(w.cfg_id),
                     "peak_kind": f"of {peak_kind}",
                     "kernel": "k_decode (one launch per call: decode phase time / decode calls)",
                     "bytes_per_launch": t["nbytes"] / n_calls, "us_per_launch": per_call_us},
        "clocks": t["clocks"],
        "gpu_launches": int(sum(head["launches"])),
        "wall_s_timed": t["t_wall"],
        "per_config": per_config,
    }
    if "dependent" in head["timing"] and head_mode != "dependent":
        d = head["timing"]["dependent"]
        line["value_one_call_at_a_time"] = aggregate_throughput(d["nbytes"], world, d["t_dec"])
        line["pct_of_hbm_peak_one_call_at_a_time"] = 100.0 * d["achieved"] / peak
    if e2e is not None:
        line["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1:
        n_units, n_steps = ORACLE_SAMPLE[w.cfg_id]
        r = oracle_sample(w, n_units, n_steps)
        line["cpu_baseline"] = {"value": r["gbs"], "unit": UNIT, "cores": r["threads"], "kind": "oracle",
                                "sample": r["sample"], "prefill_tokens_per_s": r["prefill_tokens_per_s"],
                                "seconds": r["seconds"],
                                "parity_on_this_sample": parity_with_oracle(zc, w, dev, r)}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
