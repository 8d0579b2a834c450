"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by
element, on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import zipcache_oracle as zo
from workloads import get_config, make_prefill
import zc_testlib as tl

pytestmark = pytest.mark.gpu


def _staged_quant_case(w, edit=None):
    Q, K, V = make_prefill(w, 0, tl.DEV)
    if edit is not None:
        edit(K, V)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w)
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    n_s = zo.salient_count(w.saliency_ratio, w.context)
    sal = np.zeros((w.batch, w.n_kv_heads, max(n_s, 1)), dtype=np.int32)
    for (bi, kv), u in oc.units.items():
        sal[bi, kv, :n_s] = u.segments[0].hi.idx
    cache = tl.make_cache(w)
    cache.prefill_compress(None, K, V, None, salient_idx=torch.tensor(sal, device=tl.DEV))
    torch.cuda.synchronize()
    assert tl.compare_segment(cache, oc, 0) == 0


@pytest.mark.parametrize("l", [1, 2, 17, 64, 100, 513])
@pytest.mark.parametrize("ratio", [0.0, 0.5, 1.0])
def test_quantize_pack_bit_exact_edge_lengths(l, ratio):
    _staged_quant_case(tl.small_workload(context=l, saliency_ratio=ratio, n_q_heads=2,
                                         n_kv_heads=2, rho_recent=0.2, rho_random=0.2))


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("bits", [(4, 2), (4, 4), (2, 2), (2, 4), (8, 8), (8, 4), (8, 2), (4, 8)])
def test_quantize_pack_bit_exact_bit_pairs(dtype, bits):
    _staged_quant_case(tl.small_workload(dtype=dtype, context=333, batch=2, n_q_heads=8,
                                         n_kv_heads=2, bits_hi=bits[0], bits_lo=bits[1],
                                         outlier_fixed=0))


def test_quantize_degenerate_rows():
    """All-zero token, constant channel, constant token: the rules for flat rows and zero
    channels must give the oracle's codes and parameters."""
    w = tl.small_workload(context=130, n_q_heads=1, n_kv_heads=1, saliency_ratio=0.5)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    K[0, 0, 5, :] = 0
    V[0, 0, 5, :] = 0
    K[0, 0, :, 7] = 0          # all-zero channel
    V[0, 0, :, 9] = 1.25       # constant channel
    V[0, 0, 11, :] = -0.5      # constant token
    P = tl.probes_for(w)
    oc = tl.make_oracle(w)
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    cache = tl.make_cache(w)
    cache.prefill_compress(Q, K, V, P.tolist())
    torch.cuda.synchronize()
    p_gpu = cache.scores(w.context).cpu().numpy()[0, 0]
    u = oc.units[(0, 0)]
    n_s = u.segments[0].hi.n
    idx = cache.segment(0, 0, 0)[0].cpu().numpy()[0, 0]
    assert tl.salient_sets_match(p_gpu, u.segments[0].p_tilde, idx, u.segments[0].hi.idx, n_s) == 0
    assert tl.compare_segment(cache, oc, 0) == 0


def test_quantize_operands_outside_the_kept_reciprocal_range():
    """The prefill quantiser divides by kept reciprocals only while every operand of the warp
    lies in 2^-40 .. 2^40 and takes the IEEE division otherwise: zeros, tiny and huge values in
    single elements, whole tokens and whole channels must give the oracle's bits all the same."""
    def edit(K, V):
        K[0, 0, 3, 17] = 0.0                 # one zero element: the token's warp leaves the fast path
        K[0, 0, 9, :] = 2.0 ** -50           # tiny constant token
        K[0, 0, 12, 40] = 2.0 ** -60         # tiny element
        V[0, 0, 20, 5] = 2.0 ** 50           # huge element (its channel's c = 2^25 stays inside)
        V[0, 0, :, 64] *= 2.0 ** 90          # channel whose c = 2^45-ish lies outside
        V[0, 1, 33, :] *= 2.0 ** -45         # token whose scale s lies outside
        K[0, 1, :, 100] *= 2.0 ** -90        # channel with a tiny c
    _staged_quant_case(tl.small_workload(dtype="bf16", context=300, n_q_heads=2, n_kv_heads=2,
                                         saliency_ratio=0.5, outlier_fixed=0), edit)


def test_division_by_a_kept_reciprocal_is_the_ieee_division():
    """zc_div_by (the quantiser's a / b from RN(1 / b), two residual steps) against the
    hardware's IEEE division on 4e9 pseudo-random pairs: operands over the whole admitted range,
    operands of like magnitude, and quotients at and beside integers and halves, where a wrong
    last bit would flip a code."""
    import ctypes as C
    import os
    import sys
    sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), "helpers"))
    import build_helpers
    helper = C.CDLL(build_helpers.build())
    helper.zct_div_check.restype = C.c_int
    helper.zct_div_check.argtypes = [C.c_longlong, C.c_ulonglong, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
    bad = torch.zeros(1, dtype=torch.int64, device=tl.DEV)
    first = torch.zeros(2, dtype=torch.float32, device=tl.DEV)
    st = torch.cuda.current_stream().cuda_stream
    for seed, span in ((1, 40), (2, 20), (3, 3), (4, 0)):
        assert helper.zct_div_check(1_000_000_000, seed, span, bad.data_ptr(), first.data_ptr(), st) == 0
    torch.cuda.synchronize()
    assert int(bad.item()) == 0, f"first differing pair: a={first[0].item()!r} b={first[1].item()!r}"


@pytest.mark.parametrize("kw", [
    dict(context=512, n_q_heads=4, n_kv_heads=4),
    dict(context=777, batch=2, n_q_heads=8, n_kv_heads=2, dtype="bf16", outlier_fixed=0),
    dict(context=64, n_q_heads=8, n_kv_heads=1, rho_recent=0.3, rho_random=0.3),
    dict(context=1, n_q_heads=2, n_kv_heads=1),
    dict(context=1300, n_q_heads=2, n_kv_heads=2, band=20, saliency_ratio=0.3),
    # every row a probe row: more than the workspace keeps a dense copy of, so the column-sum
    # kernel gathers its probe tiles itself
    dict(context=1100, n_q_heads=4, n_kv_heads=2, rho_recent=0.5, rho_random=0.5),
])
def test_normalized_scores_and_salient_sets(kw):
    w = tl.small_workload(**kw)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w)
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    cache = tl.make_cache(w)
    cache.prefill_compress(Q, K, V, P.tolist())
    torch.cuda.synchronize()
    p_gpu = cache.scores(w.context).cpu().numpy()
    idx_hi = cache.segment(0, 0, 0)[0].cpu().numpy()
    idx_lo = cache.segment(0, 0, 1)[0].cpu().numpy()
    swaps = 0
    for (bi, kv), u in oc.units.items():
        ref = u.segments[0].p_tilde
        rel = np.abs(p_gpu[bi, kv] - ref) / np.maximum(np.abs(ref), 1e-30)
        assert rel.max() <= 1e-4, rel.max()
        n_s = u.segments[0].hi.n
        swaps += tl.salient_sets_match(p_gpu[bi, kv], ref, idx_hi[bi, kv], u.segments[0].hi.idx, n_s)
        got = np.concatenate([idx_hi[bi, kv], idx_lo[bi, kv]])
        assert sorted(got.tolist()) == list(range(w.context))
        assert np.all(np.diff(idx_hi[bi, kv]) > 0) and np.all(np.diff(idx_lo[bi, kv]) > 0)
    assert swaps == 0   # no near-ties expected at these sizes


def test_topk_ties_prefer_lower_index():
    """Q = 0 makes every probe row uniform, so many columns tie exactly."""
    w = tl.small_workload(context=200, n_q_heads=1, n_kv_heads=1, rho_recent=0.05, rho_random=0.0)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    Q.zero_()
    P = tl.probes_for(w)
    oc = tl.make_oracle(w)
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    cache = tl.make_cache(w)
    cache.prefill_compress(Q, K, V, P.tolist())
    torch.cuda.synchronize()
    p_gpu = cache.scores(w.context).cpu().numpy()[0, 0]
    # the GPU's own scores, split by the oracle's rule, must give the GPU's lists
    sal, reg = zo.split_salient(p_gpu.astype(np.float64), 80)
    np.testing.assert_array_equal(cache.segment(0, 0, 0)[0].cpu().numpy()[0, 0], sal)
    np.testing.assert_array_equal(cache.segment(0, 0, 1)[0].cpu().numpy()[0, 0], reg)


@pytest.mark.parametrize("kw,steps", [
    (dict(context=512, n_q_heads=4, n_kv_heads=4), 16),
    (dict(context=300, batch=2, n_q_heads=8, n_kv_heads=2, dtype="bf16", outlier_fixed=0), 6),
    (dict(context=70, n_q_heads=8, n_kv_heads=1, saliency_ratio=0.5), 4),
    (dict(context=129, n_q_heads=2, n_kv_heads=2, saliency_ratio=0.0), 3),
    (dict(context=129, n_q_heads=2, n_kv_heads=2, saliency_ratio=1.0), 3),
    (dict(context=1, n_q_heads=1, n_kv_heads=1), 2),
    (dict(context=200, n_q_heads=4, n_kv_heads=1, bits_hi=4, bits_lo=4), 3),
    (dict(context=200, n_q_heads=4, n_kv_heads=1, bits_hi=2, bits_lo=2), 3),
    # 8-bit codes (a build of the decode kernel of their own), with each of the other widths
    (dict(context=200, n_q_heads=4, n_kv_heads=1, bits_hi=8, bits_lo=8), 3),
    (dict(context=333, batch=2, n_q_heads=8, n_kv_heads=2, bits_hi=8, bits_lo=4, dtype="bf16", outlier_fixed=0), 4),
    (dict(context=515, n_q_heads=4, n_kv_heads=4, bits_hi=8, bits_lo=2), 5),
    (dict(context=70, n_q_heads=2, n_kv_heads=2, bits_hi=4, bits_lo=8, saliency_ratio=0.5), 3),
    (dict(context=300, n_q_heads=4, n_kv_heads=2, bits_hi=8, bits_lo=2, k_scheme="channel"), 4),
])
def test_decode_attention_parity(kw, steps):
    w = tl.small_workload(**kw)
    tl.run_decode_parity(w, steps)      # outputs are checked step by step inside


@pytest.mark.parametrize("window,steps,ratio", [
    (16, 40, 0.4), (100, 105, 0.4),
    (16, 100, 0.4),                   # six windows: more partials per unit than the merge keeps in registers
    (100, 105, 0.8),                  # 80 salient tokens: more than one tile in a class
    (16, 20, 0.0), (16, 20, 1.0),     # an empty class
    (128, 130, 0.5),                  # the largest window, both tiles full
    (8, 323, 0.4),                    # forty windows: 82 items per unit and call at the end
])
def test_decode_across_window_recompression(window, steps, ratio):
    """The tail is re-compressed after `window` steps: new segment codes must be bit-exact
    (given equal salient sets) and attention must stay within tolerance."""
    w = tl.small_workload(context=150, n_q_heads=4, n_kv_heads=2, window=window,
                          rho_recent=0.1, rho_random=0.1, saliency_ratio=ratio)
    worst, cache, oc = tl.run_decode_parity(w, steps)
    import paper_2405_14256_b200 as zc
    n_seg = zc.zc_num_segments(cache.handle)
    assert n_seg == 1 + steps // window
    for seg in range(1, n_seg):
        p_gpu = None
        # window scores are exported only for the latest compression
        if seg == n_seg - 1:
            p_gpu = cache.scores(window).cpu().numpy()
        idx_hi = cache.segment(seg, 0, 0)[0].cpu().numpy()
        for (bi, kv), u in oc.units.items():
            s = u.segments[seg]
            if p_gpu is not None:
                rel = np.abs(p_gpu[bi, kv] - s.p_tilde) / np.maximum(s.p_tilde, 1e-30)
                assert rel.max() <= tl.WINDOW_SCORE_RTOL
                tl.salient_sets_match(p_gpu[bi, kv], s.p_tilde, idx_hi[bi, kv], s.hi.idx, s.hi.n)
            assert set(idx_hi[bi, kv].tolist()) == set(s.hi.idx.tolist())
        assert tl.compare_segment(cache, oc, seg) == 0


def test_end_to_end_config1_all_units():
    w = get_config(1)
    worst, cache, oc = tl.run_decode_parity(w, w.decode_steps, staged=False)
    assert worst <= tl.TOL_OUT      # fp16, outputs below 1: the plain bound holds on the stored output
    assert tl.compare_segment(cache, oc, 0) == 0


def test_run_to_run_determinism():
    """Three runs from zeroed buffers: outputs and the WHOLE cache buffer (codes, parameters,
    channel factors, index lists, tail, window statistics, scores) are bitwise identical."""
    from workloads import make_decode_step
    w = tl.small_workload(context=400, n_q_heads=8, n_kv_heads=2, batch=2, window=16)
    runs = []
    for _ in range(3):
        Q, K, V = make_prefill(w, 0, tl.DEV)
        P = tl.probes_for(w)
        cache = tl.make_cache(w, max_new=40)
        cache.mem.zero_()
        cache.prefill_compress(Q, K, V, P.tolist())
        outs = []
        for step in range(20):      # crosses one re-compressed window
            q, k, v = make_decode_step(w, 0, step, tl.DEV)
            cache.append(k, v)
            outs.append(cache.decode_attention(q, step % 3 == 0).clone())
        torch.cuda.synchronize()
        runs.append((torch.stack(outs), cache.mem.clone()))
    for o, m in runs[1:]:
        assert torch.equal(o, runs[0][0])
        assert torch.equal(m, runs[0][1])


FULL_SIZE = [
    (2, [(0, 0), (5, 3), (7, 7)], 3),
    (3, [(0, 0), (11, 5)], 2),
    (4, [(0, 0), (17, 13), (31, 31)], 3),
    (5, [(2, 6)], 2),
]


@pytest.mark.parametrize("cfg_id,units,steps", FULL_SIZE)
def test_full_size_configs_on_sampled_units(cfg_id, units, steps):
    """The benchmark's shapes at full size (one layer), end to end through the C ABI with the
    default plan (one call at a time, separate append launch); the oracle follows a seeded
    sample of units: normalised scores, salient sets, packed codes, parameters and decode
    outputs."""
    w = get_config(cfg_id)
    worst, cache, oc = tl.run_decode_parity(w, steps, units=units, staged=False)
    swaps, clean, rel = tl.compare_prefill_segment(w, cache, oc, units)
    tl.record("full size, default plan", config=cfg_id, units=len(units), steps=steps,
              max_abs_out=worst, near_tie_swaps=swaps, units_code_exact=clean, score_rel=rel)


@pytest.mark.parametrize("cfg_id,units,steps", FULL_SIZE)
def test_full_size_staged_codes_bit_exact(cfg_id, units, steps):
    """Full size, staged: the GPU quantiser is fed the oracle's salient lists, so packed codes,
    parameters and channel factors of every sampled unit must be bit-exact whatever near-ties
    the scores have."""
    w = get_config(cfg_id)
    worst, cache, oc = tl.run_decode_parity(w, 1, units=units, staged=True)
    assert tl.compare_segment(cache, oc, 0, units=units) == 0
    tl.record("full size, staged quantiser", config=cfg_id, units=len(units), steps=1,
              max_abs_out=worst, code_mismatches=0)


@pytest.mark.parametrize("cfg_id,units,steps,graph", [
    (2, [(0, 0), (5, 3), (7, 7)], 105, True),     # through the re-compression at step 100, replayed as a graph
    (2, [(1, 2), (6, 5)], 305, False),            # three re-compressed windows
    (3, [(0, 0), (11, 5)], 4, False),
    (4, [(0, 0), (17, 13), (31, 31)], 4, False),
    (5, [(2, 6)], 3, False),                      # items of 820 and 1229 sub-tiles, one CTA per unit
    (5, [(1, 1)], 3, True),
])
def test_full_size_in_the_benchmark_configuration(cfg_id, units, steps, graph):
    """What the benchmark times: two layers sharing a workspace, ZC_FLAG_OVERLAP_CALLS (one CTA
    per unit working through every item) and ZC_FLAG_DEFER_APPEND, all calls issued back to
    back on one stream (as a replayed CUDA graph where marked), compared with the oracle on
    sampled units: outputs at every step, prefill scores / sets / codes, the re-compressed
    windows' codes."""
    w = get_config(cfg_id)
    r = tl.run_benchmark_mode(w, units, steps, layers=2, graph=graph)
    assert r["excess"] <= 0.0, r
    swaps, clean = r["near_tie_swaps"], r["units_code_exact"]
    tl.record("full size, benchmark configuration" + (" (CUDA graph)" if graph else ""), config=cfg_id,
              units=2 * len(units), steps=steps, max_abs_out=r["worst"],
              max_abs_out_vs_rounded_oracle=r["worst_rounded"], near_tie_swaps=swaps,
              units_code_exact=clean, window_set_swaps=r["window_set_mismatches"])


@pytest.mark.parametrize("cfg_id,units,steps", [
    (1, None, 16), (2, [(0, 0), (5, 3), (7, 7)], 4), (3, [(0, 0), (11, 5)], 3),
    (4, [(0, 0), (17, 13), (31, 31)], 3), (5, [(2, 6)], 2),
])
def test_kernel_arithmetic_within_2e3_of_the_oracle_on_every_config(cfg_id, units, steps):
    """With ZC_FLAG_OUT_F32 the result is stored before its rounding to the 16-bit type, so
    the kernel's own arithmetic can be held to the plain bound on all five configurations:
    max |out - oracle| <= 2e-3 with nothing subtracted (a bf16 output of magnitude 1 to 4, as
    these workloads produce, is by itself up to 4e-3 to 8e-3 away from any exact value)."""
    w = get_config(cfg_id)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w, units)
    oc.prefill_compress(*tl.oracle_inputs(w, Q, K, V, units), P)
    import paper_2405_14256_b200 as zc
    from workloads import make_decode_step, decode_probe_flags
    worst = {}
    for overlap in (False, True):
        cache = zc.ZipCache(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context, steps,
                            w.saliency_ratio, w.bits_hi, w.bits_lo, w.window, device=tl.DEV,
                            defer_append=overlap, overlap_calls=overlap, out_f32=True)
        cache.prefill_compress(Q, K, V, P.tolist())
        oc2 = tl.make_oracle(w, units)
        for u in oc.unit_ids:
            oc2.units[u].segments = list(oc.units[u].segments)
        flags = decode_probe_flags(w, 0, steps)
        worst[overlap] = 0.0
        for s in range(steps):
            q, k, v = make_decode_step(w, 0, s, tl.DEV)
            cache.append(k, v)
            out = cache.decode_attention(q, flags[s])
            assert out.dtype == torch.float32
            q64, k64, v64 = tl.oracle_step_inputs(w, q, k, v, units)
            oc2.append(k64, v64)
            ref = oc2.decode_attention(q64, flags[s])
            got = out.double().cpu().numpy()
            for (bi, kv), o in ref.items():
                worst[overlap] = max(worst[overlap], tl.output_error(got[bi, kv * w.group:(kv + 1) * w.group], o))
        assert worst[overlap] <= tl.TOL_OUT, worst
    tl.record("fp32 output (ZC_FLAG_OUT_F32), raw bound", config=cfg_id,
              units=len(oc.unit_ids), steps=steps, max_abs_out=max(worst.values()))


@pytest.mark.parametrize("cfg_id,units,steps", [(2, [(3, 1), (4, 6)], 4), (4, [(9, 30)], 3)])
def test_full_size_one_call_at_a_time(cfg_id, units, steps):
    """The other launch mode the benchmark reports (no ZC_FLAG_OVERLAP_CALLS): every call waits
    for the kernel before it, items sized for a call that has the GPU to itself (workload 4: one
    CTA per unit), deferred append, calls issued back to back."""
    w = get_config(cfg_id)
    r = tl.run_benchmark_mode(w, units, steps, layers=2, overlap_calls=False)
    assert r["excess"] <= 0.0, r
    tl.record("full size, one call at a time (benchmark mode `dependent`)", config=cfg_id, units=2 * len(units),
              steps=steps, max_abs_out=r["worst"], max_abs_out_vs_rounded_oracle=r["worst_rounded"])


@pytest.mark.parametrize("kw,steps", [
    (dict(context=512, n_q_heads=4, n_kv_heads=4), 16),
    (dict(context=300, batch=2, n_q_heads=8, n_kv_heads=2, dtype="bf16", outlier_fixed=0), 6),
    (dict(context=70, n_q_heads=8, n_kv_heads=1, saliency_ratio=0.5), 4),
    (dict(context=150, n_q_heads=4, n_kv_heads=2, window=16, rho_recent=0.1, rho_random=0.1), 40),
    (dict(context=150, n_q_heads=4, n_kv_heads=2, window=100, rho_recent=0.1, rho_random=0.1), 105),
])
def test_deferred_append_gives_the_same_results(kw, steps):
    """With ZC_FLAG_DEFER_APPEND the new row is consumed from the caller's buffers by the
    decode kernel and stored into the tail there: outputs, re-compressed windows and the
    tail must match the oracle exactly as with the separate append launch."""
    w = tl.small_workload(**kw)
    worst, cache, oc = tl.run_decode_parity(w, steps, defer_append=True)
    import paper_2405_14256_b200 as zc
    for seg in range(1, zc.zc_num_segments(cache.handle)):
        assert tl.compare_segment(cache, oc, seg) == 0
    assert zc.zc_device_status() == 0


def test_deferred_append_is_performed_by_any_other_call():
    """Two appends in a row, and an export between append and decode: the pending row must
    reach the tail through its own launch, and the result must equal the undeferred path."""
    from workloads import make_decode_step
    w = tl.small_workload(context=200, n_q_heads=4, n_kv_heads=2, batch=2)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w).tolist()
    outs = []
    for defer in (False, True):
        cache = tl.make_cache(w, max_new=8, defer_append=defer)
        cache.mem.zero_()
        cache.prefill_compress(Q, K, V, P)
        q0, k0, v0 = make_decode_step(w, 0, 0, tl.DEV)
        q1, k1, v1 = make_decode_step(w, 0, 1, tl.DEV)
        q2, k2, v2 = make_decode_step(w, 0, 2, tl.DEV)
        cache.append(k0, v0)
        cache.append(k1, v1)            # performs the first one
        o1 = cache.decode_attention(q1, True)
        cache.append(k2, v2)
        cache.scores(w.context)         # an export performs the pending append
        o2 = cache.decode_attention(q2, False)
        torch.cuda.synchronize()
        outs.append((o1.clone(), o2.clone(), cache.mem.clone()))
    assert torch.equal(outs[0][0], outs[1][0])
    assert torch.equal(outs[0][1], outs[1][1])
    assert torch.equal(outs[0][2], outs[1][2])


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_prefill_accepts_token_major_inputs(dtype):
    """Q, K, V handed over as views of [batch, token, head, d] buffers (the layout projection
    kernels usually write): strides instead of copies.  Scores, salient sets and packed codes
    must equal those of the contiguous [batch, head, token, d] call bit for bit, and match the
    oracle."""
    w = tl.small_workload(dtype=dtype, context=700, batch=2, n_q_heads=8, n_kv_heads=2)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    views = [t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) for t in (Q, K, V)]
    assert not views[1].is_contiguous() and torch.equal(views[1], K)
    results = []
    for q_, k_, v_ in ((Q, K, V), views):
        cache = tl.make_cache(w)
        cache.mem.zero_()
        cache.prefill_compress(q_, k_, v_, P.tolist())
        torch.cuda.synchronize()
        results.append((cache.scores(w.context).clone(), cache.mem.clone(), cache))
    assert torch.equal(results[0][0], results[1][0])
    assert torch.equal(results[0][1], results[1][1])
    oc = tl.make_oracle(w)
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    assert tl.compare_segment(results[1][2], oc, 0) == 0
    import paper_2405_14256_b200 as zc
    assert zc.zc_device_status() == 0


# ------------------------------------------------------------------ channelwise keys (ZC_K_CHANNEL)
@pytest.mark.parametrize("l", [1, 17, 100, 513])
@pytest.mark.parametrize("ratio", [0.0, 0.4, 1.0])
def test_channelwise_keys_codes_bit_exact(l, ratio):
    """Keys by ChannelQuant (Sec. 4.1, Alg. 2), values by CSTQuant: K codes and the per-channel
    (s, z), V codes, per-token (s, z) and channel factors equal the oracle's bit for bit."""
    _staged_quant_case(tl.small_workload(context=l, saliency_ratio=ratio, n_q_heads=2, n_kv_heads=2,
                                         rho_recent=0.2, rho_random=0.2, k_scheme="channel"))


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("bits", [(4, 2), (4, 4), (2, 2)])
def test_channelwise_keys_bit_pairs(dtype, bits):
    _staged_quant_case(tl.small_workload(dtype=dtype, context=333, batch=2, n_q_heads=8, n_kv_heads=2,
                                         bits_hi=bits[0], bits_lo=bits[1], outlier_fixed=0,
                                         k_scheme="channel"))


def test_channelwise_keys_with_an_offset_channel():
    """A key channel that lies far from zero gets a large negative zero point: codes must
    still be the oracle's and decode attention must stay within tolerance."""
    w = tl.small_workload(context=300, n_q_heads=4, n_kv_heads=2, k_scheme="channel")
    Q, K, V = make_prefill(w, 0, tl.DEV)
    K[:, :, :, 5] += 9.0
    K[:, :, :, 77] -= 6.5
    P = tl.probes_for(w)
    oc = tl.make_oracle(w)
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    cache = tl.make_cache(w, max_new=4)
    cache.prefill_compress(Q, K, V, P.tolist())
    torch.cuda.synchronize()
    assert tl.compare_segment(cache, oc, 0) == 0
    from workloads import make_decode_step
    for step in range(3):
        q, k, v = make_decode_step(w, 0, step, tl.DEV)
        cache.append(k, v)
        out = tl.to64(cache.decode_attention(q, False))
        oc.append(tl.to64(k), tl.to64(v))
        ref = oc.decode_attention(tl.to64(q), False)
        for (bi, kv), o in ref.items():
            assert tl.output_excess(out[bi, kv * w.group:(kv + 1) * w.group], o, w.torch_dtype) <= 0.0


@pytest.mark.parametrize("kw,steps", [
    (dict(context=512, n_q_heads=4, n_kv_heads=4), 16),
    (dict(context=300, batch=2, n_q_heads=8, n_kv_heads=2, dtype="bf16", outlier_fixed=0), 6),
    (dict(context=129, n_q_heads=2, n_kv_heads=2, saliency_ratio=0.0), 3),
    (dict(context=200, n_q_heads=4, n_kv_heads=1, bits_hi=4, bits_lo=4), 3),
    (dict(context=150, n_q_heads=4, n_kv_heads=2, window=16, rho_recent=0.1, rho_random=0.1), 40),
    (dict(context=150, n_q_heads=16, n_kv_heads=2, window=100, rho_recent=0.1, rho_random=0.1), 105),
])
@pytest.mark.parametrize("defer", [False, True])
def test_channelwise_keys_decode_and_windows(kw, steps, defer):
    """Decode attention over channelwise-key caches, across re-compressed windows, with the
    separate append launch and with the deferred append."""
    w = tl.small_workload(k_scheme="channel", **kw)
    worst, cache, oc = tl.run_decode_parity(w, steps, defer_append=defer)
    import paper_2405_14256_b200 as zc
    for seg in range(1, zc.zc_num_segments(cache.handle)):
        assert tl.compare_segment(cache, oc, seg) == 0
    assert zc.zc_device_status() == 0


@pytest.mark.parametrize("cfg_id,units,steps", [
    (2, [(0, 0), (5, 3)], 105), (3, [(11, 5)], 3), (4, [(17, 13), (31, 31)], 3), (5, [(2, 6)], 2),
])
def test_channelwise_keys_full_size_in_the_benchmark_configuration(cfg_id, units, steps):
    w = get_config(cfg_id).scaled(k_scheme="channel")
    r = tl.run_benchmark_mode(w, units, steps, layers=2)
    assert r["excess"] <= 0.0, r
    tl.record("full size, benchmark configuration, channelwise keys", config=cfg_id, units=2 * len(units),
              steps=steps, max_abs_out=r["worst"], max_abs_out_vs_rounded_oracle=r["worst_rounded"],
              near_tie_swaps=r["near_tie_swaps"], units_code_exact=r["units_code_exact"],
              window_set_swaps=r["window_set_mismatches"])


# ------------------------------------------------------------------ 16-bit classes ("16/16", "16/2")
@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("kw", [
    dict(context=300, n_q_heads=4, n_kv_heads=2),
    dict(context=777, batch=2, n_q_heads=8, n_kv_heads=2, outlier_fixed=0),
    dict(context=1, n_q_heads=1, n_kv_heads=1),
    dict(context=50, n_q_heads=16, n_kv_heads=2),
])
def test_every_token_salient_at_16_bits_is_exact_attention(dtype, kw):
    """The pin the method's statement gives for the CUDA path: with every token salient and
    salient tokens kept at 16 bits, decode attention IS Eq. 4 -- compared with the oracle's
    library-free exact attention over the raw keys and values (fp32 output, 1e-4)."""
    import paper_2405_14256_b200 as zc
    from workloads import make_decode_step
    w = tl.small_workload(dtype=dtype, saliency_ratio=1.0, bits_hi=16, bits_lo=2, **kw)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    cache = zc.ZipCache(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context, 8, 1.0, 16, 2,
                        w.window, device=tl.DEV, out_f32=True)
    cache.prefill_compress(Q, K, V, tl.probes_for(w).tolist())
    K_all, V_all = tl.to64(K), tl.to64(V)
    G = w.group
    for step in range(3):
        q, k, v = make_decode_step(w, 0, step, tl.DEV)
        cache.append(k, v)
        out = cache.decode_attention(q, False).double().cpu().numpy()
        K_all = np.concatenate([K_all, tl.to64(k)[:, :, None, :]], axis=2)
        V_all = np.concatenate([V_all, tl.to64(v)[:, :, None, :]], axis=2)
        q64 = tl.to64(q)
        for bi in range(w.batch):
            for kv in range(w.n_kv_heads):
                ref = zo.exact_attention(q64[bi, kv * G:(kv + 1) * G], K_all[bi, kv], V_all[bi, kv])
                assert np.abs(out[bi, kv * G:(kv + 1) * G] - ref).max() <= 1e-4
    assert zc.zc_device_status() == 0


@pytest.mark.parametrize("bits,ratio", [((16, 2), 0.15), ((16, 4), 0.5), ((4, 16), 0.4), ((16, 16), 0.3)])
@pytest.mark.parametrize("defer", [False, True])
def test_mixed_16_bit_and_quantised_classes(bits, ratio, defer):
    """One class kept at 16 bits beside a quantised one (Table 3's "16/2" setting): rows,
    codes and parameters bit-exact, decode within tolerance, across two re-compressed windows."""
    w = tl.small_workload(context=333, batch=2, n_q_heads=8, n_kv_heads=2, bits_hi=bits[0], bits_lo=bits[1],
                          saliency_ratio=ratio, window=16, rho_recent=0.1, rho_random=0.1)
    worst, cache, oc = tl.run_decode_parity(w, 36, defer_append=defer)
    import paper_2405_14256_b200 as zc
    assert zc.zc_num_segments(cache.handle) == 3
    for seg in range(zc.zc_num_segments(cache.handle)):
        assert tl.compare_segment(cache, oc, seg) == 0
    assert zc.zc_device_status() == 0


def test_16_2_full_size_in_the_benchmark_configuration():
    w = get_config(2).scaled(bits_hi=16, bits_lo=2, saliency_ratio=0.152)
    r = tl.run_benchmark_mode(w, [(0, 0), (5, 3)], 105, layers=2)
    assert r["excess"] <= 0.0, r
    tl.record("full size, benchmark configuration, 16/2 bits at 15.2 % salient", config=2, units=4, steps=105,
              max_abs_out=r["worst"], max_abs_out_vs_rounded_oracle=r["worst_rounded"],
              near_tie_swaps=r["near_tie_swaps"], units_code_exact=r["units_code_exact"],
              window_set_swaps=r["window_set_mismatches"])


# ------------------------------------------------------------------ properties that hold at any size
def test_decode_is_invariant_under_a_permutation_of_the_cached_tokens():
    """Attention is order-free: the prompt's tokens permuted (with the salient list mapped
    along) give the same codes per token and the same decode output up to the kernel's own
    arithmetic noise (fp32 output, 2e-4: the order decides where the running maximum is
    refreshed and so how each weight is scaled before its hi + lo split)."""
    import paper_2405_14256_b200 as zc
    from workloads import make_decode_step
    w = tl.small_workload(context=700, batch=2, n_q_heads=8, n_kv_heads=2, dtype="bf16")
    Q, K, V = make_prefill(w, 0, tl.DEV)
    n_s = zo.salient_count(w.saliency_ratio, w.context)
    g = torch.Generator(device="cpu").manual_seed(5)
    sal = torch.stack([torch.stack([torch.randperm(w.context, generator=g)[:n_s].sort().values
                                    for _ in range(w.n_kv_heads)]) for _ in range(w.batch)]).to(torch.int32)
    perm = torch.randperm(w.context, generator=g)
    inv = torch.empty_like(perm)
    inv[perm] = torch.arange(w.context)
    outs = []
    for permuted in (False, True):
        c = tl.make_cache(w, max_new=4, out_f32=True)
        if permuted:   # token j of the permuted prompt is token perm[j] of the original
            Kp, Vp = K[:, :, perm.to(tl.DEV)].contiguous(), V[:, :, perm.to(tl.DEV)].contiguous()
            salp = inv[sal.long()].sort(dim=2).values.to(torch.int32)
            c.prefill_compress(None, Kp, Vp, None, salient_idx=salp.to(tl.DEV))
        else:
            c.prefill_compress(None, K, V, None, salient_idx=sal.to(tl.DEV))
        q, k, v = make_decode_step(w, 0, 0, tl.DEV)
        c.append(k, v)
        outs.append(c.decode_attention(q, False).clone())
        torch.cuda.synchronize()
        assert c.check_guards()
    assert float((outs[0] - outs[1]).abs().max()) <= 2e-4
    assert zc.zc_device_status() == 0


@pytest.mark.parametrize("cfg_id", [2, 3])
def test_decode_is_invariant_under_the_split_count(cfg_id):
    """The same cache attended with different split-K plans (one CTA per unit and large items;
    items sized for one call at a time; separate and deferred append) gives the same output up
    to the kernel's arithmetic noise (2e-4 on the fp32 output), at full size."""
    import paper_2405_14256_b200 as zc
    from workloads import make_decode_step
    w = get_config(cfg_id)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w).tolist()
    outs = []
    for overlap, defer in ((False, False), (True, True), (False, True)):
        c = tl.make_cache(w, max_new=4, defer_append=defer, overlap_calls=overlap, out_f32=True)
        c.prefill_compress(Q, K, V, P)
        for step in range(2):
            q, k, v = make_decode_step(w, 0, step, tl.DEV)
            c.append(k, v)
            o = c.decode_attention(q, False)
        outs.append(o.clone())
        torch.cuda.synchronize()
        assert c.check_guards()
    assert float((outs[0] - outs[1]).abs().max()) <= 2e-4
    assert float((outs[0] - outs[2]).abs().max()) <= 2e-4
    assert zc.zc_device_status() == 0


def test_a_second_decode_call_on_the_same_tail_leaves_the_window_bookkeeping_alone():
    """Alg. 3 takes one step per generated token.  A re-query (a second decode call without an
    append) must attend the same cache and change nothing: the window still completes after
    `window` tokens and its re-compressed segment equals the oracle's, which never saw the
    extra calls."""
    import paper_2405_14256_b200 as zc
    from workloads import make_decode_step
    w = tl.small_workload(context=200, batch=2, n_q_heads=8, n_kv_heads=2, window=16,
                          rho_recent=0.1, rho_random=0.1)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w)
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    for defer in (False, True):
        cache = tl.make_cache(w, max_new=40, defer_append=defer)
        cache.prefill_compress(Q, K, V, P.tolist())
        oc2 = tl.make_oracle(w)
        for u in oc.unit_ids:
            oc2.units[u].segments = list(oc.units[u].segments)
        for step in range(20):
            q, k, v = make_decode_step(w, 0, step, tl.DEV)
            cache.append(k, v)
            first = cache.decode_attention(q, step % 3 == 0).clone()
            if step % 4 == 1 or step == 15:            # also on the step that completes the window
                again = cache.decode_attention(q, True)
                if step != 15:                          # same cache, same query: same result
                    assert torch.equal(first, again)
            oc2.append(tl.to64(k), tl.to64(v))
            ref = oc2.decode_attention(tl.to64(q), step % 3 == 0)
            got = tl.to64(first)
            for (bi, kv), o in ref.items():
                assert tl.output_excess(got[bi, kv * w.group:(kv + 1) * w.group], o, w.torch_dtype) <= 0.0
        torch.cuda.synchronize()
        assert zc.zc_num_segments(cache.handle) == 2 and zc.zc_tail_tokens(cache.handle) == 4
        assert tl.compare_segment(cache, oc2, 1) == 0
        assert cache.check_guards()


# ------------------------------------------------------------------ prefill attention (Eq. 2) with row log-sum-exp
@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("kw", [
    dict(context=1, n_q_heads=1, n_kv_heads=1),
    dict(context=17, n_q_heads=2, n_kv_heads=2),
    dict(context=128, n_q_heads=4, n_kv_heads=1),
    dict(context=129, n_q_heads=2, n_kv_heads=1),
    dict(context=300, batch=2, n_q_heads=8, n_kv_heads=2),
    dict(context=1000, n_q_heads=4, n_kv_heads=4, outlier_fixed=0),
    # around the kernel's blocks of 256 query rows (two groups of 128) and its 128-key tiles
    dict(context=256, n_q_heads=2, n_kv_heads=1),
    dict(context=257, n_q_heads=2, n_kv_heads=2),
    dict(context=385, n_q_heads=4, n_kv_heads=2),
    dict(context=640, n_q_heads=2, n_kv_heads=1),
])
def test_prefill_attention_output_and_row_lse(dtype, kw):
    """O = causal Softmax(Q K^T / sqrt(d)) V and every row's log-sum-exp against the oracle's
    Eq. 2, head by head.  The weights reach the tensor cores in the input type, so O carries
    their rounding (2^-9 relative for bf16, 2^-12 for fp16) on top of its own storage
    rounding: 2e-2 / 4e-3 absolute on outputs of magnitude up to 4; the log-sum-exp is formed
    in fp32 from unrounded values: 2e-4 (base-2 units)."""
    import paper_2405_14256_b200 as zc
    w = tl.small_workload(dtype=dtype, **kw)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    cache = tl.make_cache(w)
    O, lse = cache.prefill_attention(Q, K, V)
    torch.cuda.synchronize()
    assert zc.zc_device_status() == 0 and cache.check_guards()
    Q64, K64, V64 = tl.to64(Q), tl.to64(K), tl.to64(V)
    O_g, lse_g = tl.to64(O), lse.double().cpu().numpy()
    tol = 2e-2 if dtype == "bf16" else 4e-3
    for bi in range(w.batch):
        for h in range(w.n_q_heads):
            kv = h // w.group
            O_ref, lse_ref = zo.prefill_attention(Q64[bi, h], K64[bi, kv], V64[bi, kv])
            assert np.abs(O_g[bi, h] - O_ref).max() <= tol, (bi, h, np.abs(O_g[bi, h] - O_ref).max())
            assert np.abs(lse_g[bi, h] - lse_ref).max() <= 2e-4, (bi, h, np.abs(lse_g[bi, h] - lse_ref).max())


@pytest.mark.parametrize("kw", [
    dict(context=777, batch=2, n_q_heads=8, n_kv_heads=2, dtype="bf16", outlier_fixed=0),
    dict(context=1300, n_q_heads=2, n_kv_heads=2, band=20, saliency_ratio=0.3),
])
def test_prefill_compress_from_the_attention_kernels_lse(kw):
    """zc_prefill_compress_lse: the probe rows' statistics come from zc_prefill_attention instead
    of the first probe-score pass; scores, salient sets and codes must match the oracle as with
    zc_prefill_compress."""
    w = tl.small_workload(**kw)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w)
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    cache = tl.make_cache(w)
    _, lse = cache.prefill_attention(Q, K, V)
    cache.prefill_compress_lse(Q, K, V, P.tolist(), lse)
    torch.cuda.synchronize()
    swaps, clean, rel = tl.compare_prefill_segment(w, cache, oc, oc.unit_ids)
    assert swaps == 0 and clean == len(oc.unit_ids)
    assert cache.check_guards()


def test_prefill_attention_full_size_config2():
    """Workload 2 at full size on sampled heads."""
    import paper_2405_14256_b200 as zc
    w = get_config(2)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    cache = tl.make_cache(w, max_new=4)
    O, lse = cache.prefill_attention(Q, K, V)
    torch.cuda.synchronize()
    assert zc.zc_device_status() == 0
    worst_o = worst_l = 0.0
    for (bi, h) in [(0, 0), (3, 17), (7, 31)]:
        kv = h // w.group
        O_ref, lse_ref = zo.prefill_attention(tl.to64(Q[bi, h]), tl.to64(K[bi, kv]), tl.to64(V[bi, kv]))
        worst_o = max(worst_o, float(np.abs(tl.to64(O[bi, h]) - O_ref).max()))
        worst_l = max(worst_l, float(np.abs(lse[bi, h].double().cpu().numpy() - lse_ref).max()))
    assert worst_o <= 2e-2 and worst_l <= 2e-4, (worst_o, worst_l)
    tl.record("prefill attention, full size (3 heads)", config=2, max_abs_out=worst_o, score_rel=worst_l)


# ---------------------------------------------------------------- token-level saliency (ZC_SCOPE_TOKEN)
@pytest.mark.parametrize("kw", [
    dict(context=300, batch=2, n_q_heads=8, n_kv_heads=4),
    dict(context=515, batch=1, n_q_heads=8, n_kv_heads=2, dtype="bf16", outlier_fixed=0),
    dict(context=130, batch=2, n_q_heads=4, n_kv_heads=4, k_scheme="channel"),
])
def test_token_scope_prefill_one_split_per_batch_row(kw):
    """ZC_SCOPE_TOKEN: a token's score is the mean of its KV heads' normalised scores, every
    head of a batch row makes the same split, and codes, parameters and factors are the
    oracle's (scope="token") bit for bit."""
    w = tl.small_workload(**kw)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w, scope="token")
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    cache = tl.make_cache(w, token_scope=True)
    cache.prefill_compress(Q, K, V, P.tolist())
    torch.cuda.synchronize()
    p_gpu = cache.scores(w.context).cpu().numpy()
    idx_hi = cache.segment(0, 0, 0)[0].cpu().numpy()
    for bi in range(w.batch):
        for kv in range(w.n_kv_heads):
            s0 = oc.units[(bi, kv)].segments[0]
            rel = np.abs(p_gpu[bi, kv] - s0.p_tilde) / np.maximum(np.abs(s0.p_tilde), 1e-30)
            assert rel.max() <= 1e-4, rel.max()
            np.testing.assert_array_equal(p_gpu[bi, kv], p_gpu[bi, 0])       # one score per token of the row
            np.testing.assert_array_equal(idx_hi[bi, kv], idx_hi[bi, 0])     # one split per row
            assert tl.salient_sets_match(p_gpu[bi, kv], s0.p_tilde, idx_hi[bi, kv], s0.hi.idx, s0.hi.n) == 0
    assert tl.compare_segment(cache, oc, 0) == 0


@pytest.mark.parametrize("defer", [False, True])
def test_token_scope_decode_across_two_windows(defer):
    """The window's re-compression under ZC_SCOPE_TOKEN (kernels of their own after the decode
    kernel of the completing call): outputs within the bound at every step, the two new
    segments' lists, codes and parameters equal to the oracle's, one split per batch row."""
    w = tl.small_workload(context=200, batch=2, n_q_heads=8, n_kv_heads=4, window=16, decode_steps=40,
                          rho_recent=0.2, rho_random=0.2)
    from workloads import make_decode_step
    import paper_2405_14256_b200 as zc
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w, scope="token")
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    cache = tl.make_cache(w, max_new=40, defer_append=defer, token_scope=True)
    cache.prefill_compress(Q, K, V, P.tolist())
    worst = 0.0
    for step in range(36):
        q, k, v = make_decode_step(w, 0, step, tl.DEV)
        probe = step % 3 == 0
        cache.append(k, v)
        out = cache.decode_attention(q, probe)
        oc.append(tl.to64(k), tl.to64(v))
        ref = oc.decode_attention(tl.to64(q), probe)
        torch.cuda.synchronize()
        got = out.float().cpu().numpy()
        for (bi, kv), r in ref.items():
            g = got[bi, kv * oc.G:(kv + 1) * oc.G]
            assert tl.output_excess(g, r, w.torch_dtype) <= 0.0
            worst = max(worst, float(np.abs(g - r).max()))
    assert zc.zc_num_segments(cache.handle) == 3 and zc.zc_tail_tokens(cache.handle) == 4
    assert zc.zc_device_status() == 0
    for seg in (1, 2):
        idx_hi = cache.segment(seg, 0, 0)[0].cpu().numpy()
        for bi in range(w.batch):
            for kv in range(w.n_kv_heads):
                np.testing.assert_array_equal(idx_hi[bi, kv], idx_hi[bi, 0])
        assert tl.compare_segment(cache, oc, seg) == 0
    cache.check_guards()


# ---------------------------------------------------------------- 8-bit codes
@pytest.mark.parametrize("bits,kch", [((8, 4), False), ((8, 8), False), ((2, 8), False), ((8, 2), True)])
@pytest.mark.parametrize("defer", [False, True])
def test_8_bit_classes_across_two_windows(bits, kch, defer):
    """8-bit codes in the prompt and in two re-compressed windows (the in-kernel re-compression
    composes 8-bit tiles too): outputs within the bound at every step, every segment's lists,
    codes and parameters equal to the oracle's."""
    from workloads import make_decode_step
    import paper_2405_14256_b200 as zc
    w = tl.small_workload(context=260, batch=2, n_q_heads=8, n_kv_heads=2, window=16, decode_steps=40,
                          rho_recent=0.2, rho_random=0.2, bits_hi=bits[0], bits_lo=bits[1],
                          k_scheme="channel" if kch else "cst")
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w)
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    cache = tl.make_cache(w, max_new=40, defer_append=defer)
    cache.prefill_compress(Q, K, V, P.tolist())
    for step in range(35):
        q, k, v = make_decode_step(w, 0, step, tl.DEV)
        probe = step % 3 == 0
        cache.append(k, v)
        out = cache.decode_attention(q, probe)
        oc.append(tl.to64(k), tl.to64(v))
        ref = oc.decode_attention(tl.to64(q), probe)
        torch.cuda.synchronize()
        got = out.float().cpu().numpy()
        for (bi, kv), r in ref.items():
            assert tl.output_excess(got[bi, kv * oc.G:(kv + 1) * oc.G], r, w.torch_dtype) <= 0.0
    assert zc.zc_num_segments(cache.handle) == 3 and zc.zc_device_status() == 0
    for seg in range(3):
        assert tl.compare_segment(cache, oc, seg) == 0
    cache.check_guards()


def test_8_bit_full_size_in_the_benchmark_configuration():
    """Workload 2 at 8/4 bits: calls side by side with the append deferred, through one window."""
    w = get_config(2).scaled(bits_hi=8, bits_lo=4)
    r = tl.run_benchmark_mode(w, [(0, 0), (5, 3)], 105, layers=2)
    assert r["excess"] <= 0.0, r
    tl.record("full size, benchmark configuration, 8/4 bits", config=2, units=4, steps=105,
              max_abs_out=r["worst"], max_abs_out_vs_rounded_oracle=r["worst_rounded"],
              near_tie_swaps=r["near_tie_swaps"], units_code_exact=r["units_code_exact"],
              window_set_swaps=r["window_set_mismatches"])


# ---------------------------------------------------------------- 16-bit parameters (ZC_FLAG_PARAMS_F16)
@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("kw", [
    dict(context=333, batch=2, n_q_heads=8, n_kv_heads=2),
    dict(context=64, n_q_heads=2, n_kv_heads=2, saliency_ratio=1.0, bits_hi=4, bits_lo=4),
    dict(context=513, n_q_heads=4, n_kv_heads=4, bits_hi=2, bits_lo=2, outlier_fixed=0),
    dict(context=17, n_q_heads=1, n_kv_heads=1),
])
def test_params_f16_codes_and_parameters_bit_exact(dtype, kw):
    """Scales and channel factors rounded up to fp16 before the codes are formed, zero points as
    16-bit integers: lists, codes, parameters and factors equal to the oracle's
    (param_dtype="f16") bit for bit."""
    w = tl.small_workload(dtype=dtype, **kw)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w, param_dtype="f16")
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    n_s = zo.salient_count(w.saliency_ratio, w.context)
    sal = np.zeros((w.batch, w.n_kv_heads, max(n_s, 1)), dtype=np.int32)
    for (bi, kv), u in oc.units.items():
        sal[bi, kv, :n_s] = u.segments[0].hi.idx
    cache = tl.make_cache(w, params_f16=True)
    cache.prefill_compress(None, K, V, None, salient_idx=torch.tensor(sal, device=tl.DEV))
    torch.cuda.synchronize()
    assert tl.compare_segment(cache, oc, 0) == 0
    cache.check_guards()


@pytest.mark.parametrize("kw", [
    dict(context=260, batch=2, n_q_heads=8, n_kv_heads=2),
    dict(context=150, n_q_heads=4, n_kv_heads=4, dtype="bf16", outlier_fixed=0, bits_hi=4, bits_lo=4),
    dict(context=97, n_q_heads=2, n_kv_heads=1, bits_hi=2, bits_lo=2, saliency_ratio=0.5),
])
@pytest.mark.parametrize("defer", [False, True])
def test_params_f16_decode_across_two_windows(kw, defer):
    """16-bit parameters in the decode loop (fp16 scale and int16 zero point per token and tensor)
    and in two re-compressed windows (by kernels of their own behind the completing call): outputs
    within the bound at every step, every segment equal to the oracle's (param_dtype="f16")."""
    from workloads import make_decode_step
    import paper_2405_14256_b200 as zc
    w = tl.small_workload(window=16, decode_steps=40, rho_recent=0.2, rho_random=0.2, **kw)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w, param_dtype="f16")
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    cache = tl.make_cache(w, max_new=40, defer_append=defer, params_f16=True)
    cache.prefill_compress(Q, K, V, P.tolist())
    for step in range(35):
        q, k, v = make_decode_step(w, 0, step, tl.DEV)
        probe = step % 3 == 0
        cache.append(k, v)
        out = cache.decode_attention(q, probe)
        oc.append(tl.to64(k), tl.to64(v))
        ref = oc.decode_attention(tl.to64(q), probe)
        torch.cuda.synchronize()
        got = out.float().cpu().numpy()
        for (bi, kv), r in ref.items():
            assert tl.output_excess(got[bi, kv * oc.G:(kv + 1) * oc.G], r, w.torch_dtype) <= 0.0
    assert zc.zc_num_segments(cache.handle) == 3 and zc.zc_device_status() == 0
    for seg in range(3):
        assert tl.compare_segment(cache, oc, seg) == 0
    cache.check_guards()


def test_params_f16_full_size_one_call_at_a_time():
    """Workload 2 with 16-bit parameters, the launch mode they admit (every call waits for what
    precedes it), sampled units, through one window."""
    w = get_config(2)
    units = [(0, 0), (5, 3)]
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w, units, param_dtype="f16")
    oc.prefill_compress(*tl.oracle_inputs(w, Q, K, V, units), P)
    cache = tl.make_cache(w, max_new=104, defer_append=True, params_f16=True)
    cache.prefill_compress(Q, K, V, P.tolist())
    from workloads import make_decode_step, decode_probe_flags
    flags = decode_probe_flags(w, 0, 103)
    worst = 0.0
    for step in range(103):
        q, k, v = make_decode_step(w, 0, step, tl.DEV)
        probe = bool(flags[step])
        cache.append(k, v)
        out = cache.decode_attention(q, probe)
        qq, kk, vv = tl.oracle_step_inputs(w, q, k, v, units)
        oc.append(kk, vv)
        ref = oc.decode_attention(qq, probe)
        got = out.float().cpu().numpy()
        for (bi, kv), r in ref.items():
            g = got[bi, kv * oc.G:(kv + 1) * oc.G]
            assert tl.output_excess(g, r, w.torch_dtype) <= 0.0
            worst = max(worst, float(np.abs(g - r).max()))
    import paper_2405_14256_b200 as zc
    assert zc.zc_num_segments(cache.handle) == 2 and zc.zc_device_status() == 0
    for seg in range(2):
        assert tl.compare_segment(cache, oc, seg, units) == 0
    tl.record("full size, 16-bit parameters, one call at a time", config=2, units=len(units), steps=103,
              max_abs_out=worst)


# ---------------------------------------------------------------- token groups over all heads (ZC_FLAG_GROUP_ALL_HEADS)
@pytest.mark.parametrize("kw,p16", [
    (dict(context=260, batch=2, n_q_heads=8, n_kv_heads=4), False),
    (dict(context=150, n_q_heads=8, n_kv_heads=2, dtype="bf16", outlier_fixed=0, bits_hi=4, bits_lo=4), False),
    (dict(context=97, n_q_heads=4, n_kv_heads=4, bits_hi=8, bits_lo=2, saliency_ratio=0.5), False),
    (dict(context=200, batch=2, n_q_heads=8, n_kv_heads=2, k_scheme="channel"), False),
    (dict(context=130, n_q_heads=8, n_kv_heads=4), True),
])
def test_token_groups_over_all_heads_across_two_windows(kw, p16):
    """Alg. 1 on X in R^{l x hd}: one (s, z) per token over the channels of all KV heads of its
    batch row, in the prompt and in two re-compressed windows: every head's tiles carry the
    row's pair, codes, parameters and factors equal to the oracle's (scope="token",
    group="all_heads"), decode within the bound at every step."""
    from workloads import make_decode_step
    import paper_2405_14256_b200 as zc
    w = tl.small_workload(window=16, decode_steps=40, rho_recent=0.2, rho_random=0.2, **kw)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    K[:, -1] *= 5.0            # heads of unlike range: the shared scale is the widest head's
    P = tl.probes_for(w)
    oc = tl.make_oracle(w, scope="token", group="all_heads", param_dtype="f16" if p16 else "f32")
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    cache = tl.make_cache(w, max_new=40, token_scope=True, group_all_heads=True, params_f16=p16)
    cache.prefill_compress(Q, K, V, P.tolist())
    torch.cuda.synchronize()
    assert tl.compare_segment(cache, oc, 0) == 0
    sz = cache.segment(0, 1, 0)[2].cpu().numpy()          # V parameters of the salient subset
    for bi in range(w.batch):
        for kv in range(1, w.n_kv_heads):
            np.testing.assert_array_equal(sz[bi, kv], sz[bi, 0])      # one pair per token for every head
    for step in range(35):
        q, k, v = make_decode_step(w, 0, step, tl.DEV)
        probe = step % 3 == 0
        cache.append(k, v)
        out = cache.decode_attention(q, probe)
        oc.append(tl.to64(k), tl.to64(v))
        ref = oc.decode_attention(tl.to64(q), probe)
        torch.cuda.synchronize()
        got = out.float().cpu().numpy()
        for (bi, kv), r in ref.items():
            assert tl.output_excess(got[bi, kv * oc.G:(kv + 1) * oc.G], r, w.torch_dtype) <= 0.0
    assert zc.zc_num_segments(cache.handle) == 3 and zc.zc_device_status() == 0
    for seg in (1, 2):
        assert tl.compare_segment(cache, oc, seg) == 0
    cache.check_guards()


def test_token_scope_all_heads_full_size_one_call_at_a_time():
    """Workload 2 with one split per token and one (s, z) per token over all KV heads, in the
    launch mode they admit, on every head of one batch row (the oracle needs the whole row),
    through one re-compressed window."""
    from workloads import make_decode_step, decode_probe_flags
    import paper_2405_14256_b200 as zc
    w = get_config(2)
    units = [(5, kv) for kv in range(w.n_kv_heads)]
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w, units, scope="token", group="all_heads")
    oc.prefill_compress(*tl.oracle_inputs(w, Q, K, V, units), P)
    cache = tl.make_cache(w, max_new=104, defer_append=True, token_scope=True, group_all_heads=True)
    cache.prefill_compress(Q, K, V, P.tolist())
    torch.cuda.synchronize()
    p_gpu = cache.scores(w.context).cpu().numpy()
    idx_hi = cache.segment(0, 0, 0)[0].cpu().numpy()
    s0 = oc.units[units[0]].segments[0]
    assert (np.abs(p_gpu[5, 0] - s0.p_tilde) / np.maximum(np.abs(s0.p_tilde), 1e-30)).max() <= 1e-4
    swaps = tl.salient_sets_match(p_gpu[5, 0], s0.p_tilde, idx_hi[5, 0], s0.hi.idx, s0.hi.n)
    flags = decode_probe_flags(w, 0, 103)
    worst = 0.0
    for step in range(103):
        q, k, v = make_decode_step(w, 0, step, tl.DEV)
        probe = bool(flags[step])
        cache.append(k, v)
        out = cache.decode_attention(q, probe)
        qq, kk, vv = tl.oracle_step_inputs(w, q, k, v, units)
        oc.append(kk, vv)
        ref = oc.decode_attention(qq, probe)
        if swaps:
            continue
        got = out.float().cpu().numpy()
        for (bi, kv), r in ref.items():
            g = got[bi, kv * oc.G:(kv + 1) * oc.G]
            assert tl.output_excess(g, r, w.torch_dtype) <= 0.0
            worst = max(worst, float(np.abs(g - r).max()))
    assert zc.zc_num_segments(cache.handle) == 2 and zc.zc_device_status() == 0
    exact = 0
    if swaps == 0:
        assert tl.compare_segment(cache, oc, 0, units) == 0
        exact = len(units)
        sg = oc.units[units[0]].segments[1]
        ihi = cache.segment(1, 0, 0)[0].cpu().numpy()
        if set(ihi[5, 0].tolist()) == set(sg.hi.idx.tolist()):
            assert tl.compare_segment(cache, oc, 1, units) == 0
    tl.record("full size, token scope and token groups over all heads, one call at a time", config=2,
              units=len(units), steps=103, max_abs_out=worst, near_tie_swaps=swaps, units_code_exact=exact)


@pytest.mark.parametrize("opts", [
    dict(token_scope=True), dict(params_f16=True),
    dict(token_scope=True, group_all_heads=True, params_f16=True),
])
def test_window_recompression_by_kernels_behind_the_call_inside_a_cuda_graph(opts):
    """Token scope and 16-bit parameters re-compress a window by kernels launched behind the
    decode kernel of the completing call.  36 steps (two windows) captured into one CUDA graph
    and replayed must leave the same outputs and the same cache, byte for byte, as the same calls
    issued directly (which the tests above compare with the oracle)."""
    import paper_2405_14256_b200 as zc
    from workloads import make_decode_step
    w = tl.small_workload(context=260, batch=2, n_q_heads=8, n_kv_heads=2, window=16, rho_recent=0.2,
                          rho_random=0.2)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w).tolist()
    n = 36
    ins = [make_decode_step(w, 0, s, tl.DEV) for s in range(n)]
    res = {}
    for mode in ("direct", "graph"):
        c = tl.make_cache(w, max_new=40, defer_append=True, **opts)
        c.mem.zero_()
        c.prefill_compress(Q, K, V, P)
        outs = [torch.empty_like(ins[0][0]) for _ in range(n)]

        def issue():
            for s in range(n):
                q, k, v = ins[s]
                c.append(k, v)
                c.decode_attention(q, s % 3 == 0, out=outs[s])

        torch.cuda.synchronize()
        if mode == "graph":
            st = torch.cuda.Stream()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.stream(st):
                with torch.cuda.graph(g, stream=st):
                    issue()
                g.replay()
        else:
            issue()
        torch.cuda.synchronize()
        assert zc.zc_num_segments(c.handle) == 3 and zc.zc_device_status() == 0
        assert c.check_guards()
        res[mode] = (torch.stack(outs).clone(), c.mem.clone())
    assert torch.equal(res["direct"][0], res["graph"][0])
    assert torch.equal(res["direct"][1], res["graph"][1])


@pytest.mark.parametrize("graph", [False, True])
def test_forty_windows_with_calls_side_by_side(graph):
    """A long generation in the benchmark's launch mode: window 8, 323 steps, so every unit's
    one CTA ends up working through 82 items per call; outputs within the bound at every step,
    all 41 segments equal to the oracle's (up to near-tie splits, which are counted)."""
    w = tl.small_workload(context=150, batch=2, n_q_heads=4, n_kv_heads=2, window=8, rho_recent=0.1,
                          rho_random=0.1)
    units = [(bi, kv) for bi in range(w.batch) for kv in range(w.n_kv_heads)]
    r = tl.run_benchmark_mode(w, units, 323, layers=2, graph=graph)
    assert r["excess"] <= 0.0, r["excess"]
    import paper_2405_14256_b200 as zc
    assert all(zc.zc_num_segments(c.handle) == 41 for c in r["caches"])


@pytest.mark.parametrize("l,G,rho", [(262144, 2, 0.002), (1 << 20, 1, 0.0005)])
def test_longest_prompts(l, G, rho):
    """One unit at 2^18 tokens and at 2^20, the largest max_prefill the library accepts (about a
    thousand probe rows, so that the oracle finishes in seconds): scores, the split, every packed
    code and parameter, and three decode steps over the whole cache."""
    import paper_2405_14256_b200 as zc
    from workloads import make_decode_step
    w = tl.small_workload(context=l, batch=1, n_q_heads=G, n_kv_heads=1, dtype="bf16", rho_recent=rho,
                          rho_random=rho, decode_steps=4)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    cache = tl.make_cache(w, max_new=4, defer_append=True)
    cache.prefill_compress(Q, K, V, P.tolist())
    torch.cuda.synchronize()
    assert zc.zc_device_status() == 0
    oc = tl.make_oracle(w)
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    swaps, clean, rel = tl.compare_prefill_segment(w, cache, oc, [(0, 0)])
    worst = 0.0
    for step in range(3):
        q, k, v = make_decode_step(w, 0, step, tl.DEV)
        cache.append(k, v)
        out = cache.decode_attention(q, step == 1)
        oc.append(tl.to64(k), tl.to64(v))
        ref = oc.decode_attention(tl.to64(q), step == 1)
        torch.cuda.synchronize()
        if swaps == 0:
            g = out.float().cpu().numpy()[0]
            worst = max(worst, tl.output_error(g, ref[(0, 0)]))
            assert worst <= tl.TOL_OUT, (step, worst)
    assert zc.zc_device_status() == 0 and cache.check_guards()
    tl.record(f"one unit, {l} tokens", units=1, steps=3, max_abs_out=worst, near_tie_swaps=swaps,
              units_code_exact=clean, score_rel=rel)


def test_many_units():
    """4096 units (batch 512 x 8 KV heads, 32 query heads) of 300 tokens through one re-compressed
    window: several times more units than CTA slots on the GPU; sampled units against the oracle."""
    w = tl.small_workload(context=300, batch=512, n_q_heads=32, n_kv_heads=8, window=16, rho_recent=0.1,
                          rho_random=0.1, dtype="bf16")
    units = [(0, 0), (1, 7), (255, 3), (256, 4), (511, 0), (511, 7)]
    worst, cache, oc = tl.run_decode_parity(w, 20, units=units, staged=False, defer_append=True)
    import paper_2405_14256_b200 as zc
    assert zc.zc_num_segments(cache.handle) == 2 and zc.zc_device_status() == 0
    assert tl.compare_segment(cache, oc, 0, units) == 0


def test_prefill_attention_statistics_at_2_18_tokens():
    """zc_prefill_attention over 2^18 tokens: its row statistics, given to
    zc_prefill_compress_lse, must lead to the oracle's scores, split and codes (every probe row's
    log-sum-exp is then right to the score tolerance), and O's first 300 rows must be the
    oracle's attention over the same prefix (causal: later tokens do not touch them)."""
    import paper_2405_14256_b200 as zc
    l = 262144
    w = tl.small_workload(context=l, batch=1, n_q_heads=2, n_kv_heads=1, dtype="bf16", rho_recent=0.002,
                          rho_random=0.002)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    cache = tl.make_cache(w, max_new=4)
    O, lse = cache.prefill_attention(Q, K, V)
    cache.prefill_compress_lse(Q, K, V, P.tolist(), lse)
    torch.cuda.synchronize()
    assert zc.zc_device_status() == 0 and cache.check_guards()
    oc = tl.make_oracle(w)
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    swaps, clean, rel = tl.compare_prefill_segment(w, cache, oc, [(0, 0)])
    n = 300
    for h in range(2):
        O_ref, lse_ref = zo.prefill_attention(tl.to64(Q[0, h, :n]), tl.to64(K[0, 0, :n]), tl.to64(V[0, 0, :n]))
        assert np.abs(tl.to64(O[0, h, :n]) - O_ref).max() <= 2e-2
        assert np.abs(lse[0, h, :n].double().cpu().numpy() - lse_ref).max() <= 2e-4
    tl.record("prefill attention statistics, 262144 tokens", units=1, near_tie_swaps=swaps, units_code_exact=clean,
              score_rel=rel)
