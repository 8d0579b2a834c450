"""GPU parity of decode calls that are in flight together: consecutive zc_decode_attention
calls on one stream start without waiting for one another, so everything two calls may share
(workspace regions, arrival counters, buffers that alias) has to be kept apart or ordered by
the library.  Every call here is issued back to back with no host synchronisation; results
are compared with the oracle afterwards."""
import numpy as np
import pytest
import torch

from workloads import make_prefill, make_decode_step
import zc_testlib as tl

pytestmark = pytest.mark.gpu


def _prefilled(w, layers, shared_ws=True, **kw):
    import paper_2405_14256_b200 as zc
    caches, oracles = [], []
    ws = None
    for ly in range(layers):
        Q, K, V = make_prefill(w, ly, tl.DEV)
        P = tl.probes_for(w, ly)
        oc = tl.make_oracle(w)
        oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
        c = zc.ZipCache(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context, 256,
                        w.saliency_ratio, w.bits_hi, w.bits_lo, w.window, device=tl.DEV,
                        workspace=ws, **kw)
        if shared_ws:
            ws = c.workspace
        c.prefill_compress(Q, K, V, P.tolist())
        caches.append(c)
        oracles.append(oc)
    return caches, oracles


def _check(w, got, ref_units):
    """Worst excess over the bound of the edge-size tests (see zc_testlib.output_excess)."""
    G = w.group
    worst = -1.0
    g = tl.to64(got)
    for (bi, kv), o in ref_units.items():
        worst = max(worst, tl.output_excess(g[bi, kv * G:(kv + 1) * G], o, w.torch_dtype))
    return worst


@pytest.mark.parametrize("layers,steps,kw", [
    (4, 40, dict(context=300, batch=2, n_q_heads=8, n_kv_heads=2, window=16)),      # 160 calls, 2 flushes per layer
    (1, 90, dict(context=200, batch=1, n_q_heads=4, n_kv_heads=4, window=100)),     # one cache, call after call
    (2, 100, dict(context=150, batch=1, n_q_heads=4, n_kv_heads=2, window=16)),     # 6 windows: 14 items per unit
    (3, 30, dict(context=260, batch=2, n_q_heads=16, n_kv_heads=2, dtype="bf16")),  # two head groups per unit
])
@pytest.mark.parametrize("overlap_items", [False, True])
def test_calls_in_flight_together_match_the_oracle(layers, steps, kw, overlap_items):
    import paper_2405_14256_b200 as zc
    w = tl.small_workload(**kw)
    caches, oracles = _prefilled(w, layers, defer_append=True, overlap_calls=overlap_items)
    ins = [[make_decode_step(w, ly, s, tl.DEV) for ly in range(layers)] for s in range(steps)]
    # runs of probe steps: consecutive calls on one cache then add to the same window statistics
    flags = [[bool(f) or (s % 5 < 2) for s, f in enumerate(tl.decode_probe_flags(w, ly, steps))]
             for ly in range(layers)]
    outs = [[torch.empty_like(ins[0][0][0]) for _ in range(layers)] for _ in range(steps)]
    torch.cuda.synchronize()
    for s in range(steps):                      # more than 64 calls with nothing between them
        for ly, c in enumerate(caches):
            q, k, v = ins[s][ly]
            c.append(k, v)
            c.decode_attention(q, bool(flags[ly][s]), out=outs[s][ly])
    torch.cuda.synchronize()
    assert zc.zc_device_status() == 0
    worst = -1.0
    for s in range(steps):
        for ly, oc in enumerate(oracles):
            q, k, v = ins[s][ly]
            oc.append(tl.to64(k), tl.to64(v))
            ref = oc.decode_attention(tl.to64(q), bool(flags[ly][s]))
            worst = max(worst, _check(w, outs[s][ly], ref))
    assert worst <= 0.0, worst
    # the re-compressed windows depend on the statistics every probe step added, in order
    for ly, (c, oc) in enumerate(zip(caches, oracles)):
        n_seg = zc.zc_num_segments(c.handle)
        assert n_seg == len(oc.units[oc.unit_ids[0]].segments)
        for seg in range(1, n_seg):
            assert tl.compare_segment(c, oc, seg) == 0


def test_a_call_that_reads_the_previous_output_waits_for_it():
    """q of step s + 1 IS the output buffer of step s (distinct buffers per step, nothing
    between the calls): the library has to order each call behind the one that produces its
    input.  The oracle is fed the outputs the GPU produced."""
    import paper_2405_14256_b200 as zc
    w = tl.small_workload(context=400, batch=2, n_q_heads=8, n_kv_heads=2, window=100)
    steps = 80
    (c,), (oc,) = _prefilled(w, 1, defer_append=True, overlap_calls=True)
    kv = [make_decode_step(w, 0, s, tl.DEV) for s in range(steps)]
    bufs = [kv[0][0].clone()] + [torch.empty_like(kv[0][0]) for _ in range(steps)]
    torch.cuda.synchronize()
    for s in range(steps):
        c.append(kv[s][1], kv[s][2])
        c.decode_attention(bufs[s], False, out=bufs[s + 1])
    torch.cuda.synchronize()
    assert zc.zc_device_status() == 0
    worst = -1.0
    for s in range(steps):
        oc.append(tl.to64(kv[s][1]), tl.to64(kv[s][2]))
        ref = oc.decode_attention(tl.to64(bufs[s]), False)
        worst = max(worst, _check(w, bufs[s + 1], ref))
    assert worst <= 0.0, worst


def test_calls_that_write_the_same_output_land_in_order():
    """Two caches, every call writes the same output buffer, nothing between the calls: the
    buffer must end up holding the last call's result, and an input buffer that a later call
    overwrites must have been read by then."""
    import paper_2405_14256_b200 as zc
    w = tl.small_workload(context=300, batch=2, n_q_heads=8, n_kv_heads=2)
    caches, oracles = _prefilled(w, 2, defer_append=True, overlap_calls=True)
    steps = 10
    ins = [[make_decode_step(w, ly, s, tl.DEV) for ly in range(2)] for s in range(steps)]
    out = torch.empty_like(ins[0][0][0])
    torch.cuda.synchronize()
    for s in range(steps):
        for ly, c in enumerate(caches):
            q, k, v = ins[s][ly]
            c.append(k, v)
            c.decode_attention(q, False, out=out)
    torch.cuda.synchronize()
    assert zc.zc_device_status() == 0
    ref = None
    for s in range(steps):
        for ly, oc in enumerate(oracles):
            q, k, v = ins[s][ly]
            oc.append(tl.to64(k), tl.to64(v))
            ref = oc.decode_attention(tl.to64(q), False)
    assert _check(w, out, ref) <= 0.0


@pytest.mark.parametrize("window", [100, 16])   # 16: a window is re-compressed inside the graph
def test_captured_calls_replay_to_the_same_results(window):
    """A CUDA graph of back-to-back calls, replayed twice, then calls issued directly again:
    the replays and the direct calls must not disturb each other's ordering state."""
    import paper_2405_14256_b200 as zc
    w = tl.small_workload(context=300, batch=2, n_q_heads=8, n_kv_heads=2, window=window)
    layers, steps = 3, 30
    outs_all = []
    for mode in ("direct", "graph"):
        caches, _ = _prefilled(w, layers, defer_append=True, overlap_calls=True)
        ins = [[make_decode_step(w, ly, s, tl.DEV) for ly in range(layers)] for s in range(steps)]
        outs = [[torch.empty_like(ins[0][0][0]) for _ in range(layers)] for _ in range(steps)]

        def issue():
            for s in range(steps):
                for ly, c in enumerate(caches):
                    q, k, v = ins[s][ly]
                    c.append(k, v)
                    c.decode_attention(q, s % 7 == 0, out=outs[s][ly])
        torch.cuda.synchronize()
        if mode == "direct":
            issue()
        else:
            st = torch.cuda.Stream()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(st):
                with torch.cuda.graph(g, stream=st):
                    issue()
                g.replay()
                # a replay appends the same rows again at the same tail positions and reads
                # the same inputs: the outputs of the second replay equal those of the first
                first = [[o.clone() for o in row] for row in outs]
                if window < steps:
                    # a re-compressed window leaves statistics of the window after it behind:
                    # compress the prompts again first, as a benchmark loop over one graph does
                    for ly, c in enumerate(caches):
                        Q, K, V = make_prefill(w, ly, tl.DEV)
                        c.prefill_compress(Q, K, V, tl.probes_for(w, ly).tolist())
                g.replay()
            torch.cuda.synchronize()
            for a, b in zip(first, outs):
                for x, y in zip(a, b):
                    assert torch.equal(x, y)
        torch.cuda.synchronize()
        assert zc.zc_device_status() == 0
        outs_all.append(outs)
    for a, b in zip(outs_all[0], outs_all[1]):
        for x, y in zip(a, b):
            assert torch.equal(x, y)


@pytest.mark.parametrize("promise", [False])
def test_a_producer_that_lets_us_start_early_is_waited_for(promise):
    """q of the second call is written, between the two calls, by a kernel of "another library"
    that triggers programmatic launch completion at its very start and stores q 100 us later
    (tests/helpers/zc_test_kernels.cu).  Without ZC_FLAG_OVERLAP_CALLS the decode kernel must
    not read q before that kernel has completed."""
    import ctypes as C
    import os
    import sys
    sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), "helpers"))
    import build_helpers
    helper = C.CDLL(build_helpers.build())
    helper.zct_late_copy.restype = C.c_int
    helper.zct_late_copy.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_longlong, C.c_void_p]
    import paper_2405_14256_b200 as zc
    w = tl.small_workload(context=400, batch=2, n_q_heads=8, n_kv_heads=2)
    for defer in (False, True):
        (c,), (oc,) = _prefilled(w, 1, defer_append=defer, overlap_calls=promise)
        q0, k0, v0 = make_decode_step(w, 0, 0, tl.DEV)
        q1, k1, v1 = make_decode_step(w, 0, 1, tl.DEV)
        q_buf = torch.zeros_like(q1)             # stale contents: zeros
        k_buf, v_buf = torch.zeros_like(k1), torch.zeros_like(v1)
        st = torch.cuda.current_stream().cuda_stream
        torch.cuda.synchronize()
        c.append(k0, v0)
        o0 = c.decode_attention(q0, False)
        for dst, src in ((q_buf, q1), (k_buf, k1), (v_buf, v1)):
            rc = helper.zct_late_copy(dst.data_ptr(), src.data_ptr(), dst.numel() * dst.element_size(),
                                      200000, st)
            assert rc == 0
        c.append(k_buf, v_buf)
        o1 = c.decode_attention(q_buf, True)
        torch.cuda.synchronize()
        assert zc.zc_device_status() == 0
        assert torch.equal(q_buf, q1)
        for (q, k, v, o, fl) in ((q0, k0, v0, o0, False), (q1, k1, v1, o1, True)):
            oc.append(tl.to64(k), tl.to64(v))
            ref = oc.decode_attention(tl.to64(q), fl)
            assert _check(w, o, ref) <= 0.0
