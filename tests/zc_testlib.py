"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI
binding and the oracle on the same seeded inputs."""
from __future__ import annotations

import numpy as np
import torch

from oracle import zipcache_oracle as zo
from workloads import Workload, make_prefill, make_decode_step, decode_probe_flags

DEV = "cuda:0"


def small_workload(**kw) -> Workload:
    base = dict(name="test", cfg_id=9, dtype="fp16", batch=1, n_q_heads=4, n_kv_heads=4,
                head_dim=128, context=512, n_layers=1, saliency_ratio=0.4, bits_hi=4, bits_lo=2,
                rho_recent=0.05, rho_random=0.05, window=100, decode_steps=8, outlier_fixed=4,
                band=0)
    base.update(kw)
    return Workload(**base)


def to64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


GUARD = 4096   # bytes of canary on each side of every cache buffer and workspace the tests allocate


def make_cache(w: Workload, max_new=None, defer_append: bool = False, overlap_calls: bool = False, **kw):
    import paper_2405_14256_b200 as zc
    return zc.ZipCache(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context,
                       w.decode_steps if max_new is None else max_new, w.saliency_ratio,
                       w.bits_hi, w.bits_lo, w.window, device=DEV, defer_append=defer_append,
                       overlap_calls=overlap_calls, k_channel=w.k_scheme == "channel", guard_bytes=GUARD,
                       **kw)


def make_oracle(w: Workload, units=None, scope: str = "kv_head", param_dtype: str = "f32",
                group: str = "head") -> zo.ZipCacheOracle:
    return zo.ZipCacheOracle(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.saliency_ratio,
                             w.bits_hi, w.bits_lo, w.window, units=units, k_scheme=w.k_scheme, scope=scope,
                             param_dtype=param_dtype, group=group)


def probes_for(w: Workload, layer: int = 0) -> np.ndarray:
    return zo.probe_positions(w.context, w.rho_recent, w.rho_random, w.seed(layer))


def compare_segment(cache, oc: zo.ZipCacheOracle, seg: int, units=None):
    """Bit-exact comparison of index lists, packed codes, (s, z) and channel factors."""
    mism = 0
    for subset, name in ((0, "hi"), (1, "lo")):
        for tensor, tn in ((0, "qK"), (1, "qV")):
            idx, codes, sz, cf = (x.cpu().numpy() for x in cache.segment(seg, tensor, subset))
            for (bi, kv) in (units or oc.unit_ids):
                sub = getattr(oc.units[(bi, kv)].segments[seg], name)
                assert idx.shape[2] == sub.n, (idx.shape, sub.n)
                if sub.n == 0:
                    continue
                np.testing.assert_array_equal(idx[bi, kv], sub.idx)
                if sub.bits == 16:
                    # rows kept at full precision: the exported bytes are the rows themselves
                    rows = sub.K_hat if tensor == 0 else sub.V_hat
                    want = torch.from_numpy(rows).to(cache.dtype).contiguous().view(torch.uint8).numpy()
                    np.testing.assert_array_equal(codes[bi, kv].reshape(want.shape), want)
                    continue
                q = getattr(sub, tn)
                want = zo.pack_codes(q["codes"], sub.bits)
                mism += int((codes[bi, kv] != want).sum())
                np.testing.assert_array_equal(codes[bi, kv], want)
                # per token (CSTQuant) or per channel (channelwise keys): same export slots
                np.testing.assert_array_equal(sz[bi, kv, :, 0], q["s"])
                np.testing.assert_array_equal(sz[bi, kv, :, 1], q["z"])
                if "c" in q:
                    np.testing.assert_array_equal(cf[bi, kv], q["c"])
    return mism


def salient_sets_match(p_gpu: np.ndarray, p_ref: np.ndarray, sal_gpu, sal_ref, n_s: int):
    """Sets must be equal except for near-ties: a token may differ only if its oracle
    score is within relative 1e-5 of the oracle's n_s-th largest score.  Returns the
    number of such swaps."""
    a, b = set(int(x) for x in sal_gpu), set(int(x) for x in sal_ref)
    if a == b:
        return 0
    kth = np.sort(p_ref)[::-1][n_s - 1]
    diff = (a - b) | (b - a)
    for j in diff:
        assert abs(p_ref[j] - kth) <= 1e-5 * abs(kth), (j, p_ref[j], kth)
    return len(diff) // 2


TOL_OUT = 2e-3   # max-abs bound on decode outputs (fp16 / bf16 inputs)
# Scores of a re-compressed window are sums of this step's softmax weights over the tail's
# columns, normalised with the row maximum and sum of the WHOLE cache; the compressed part of
# those sums carries the decode kernel's logit noise (f16 hi+lo query, ex2.approx), about 1e-3
# relative, where the prefill scores (fp32 accumulation over exact 16-bit operands) reach 1e-4.
WINDOW_SCORE_RTOL = 1e-3


def output_error(got: np.ndarray, ref: np.ndarray, dtype=None) -> float:
    """Largest |got - ref|: the library's stored output (16-bit) against the oracle's fp64
    value, nothing subtracted.  This is the figure every decode parity test holds to 2e-3."""
    return float(np.abs(got - ref).max())


def output_error_rounded(got: np.ndarray, ref: np.ndarray, dtype) -> float:
    """The same comparison with the oracle's value first rounded to the storage type of the
    output (reported beside the raw figure, never asserted instead of it)."""
    ref_r = torch.from_numpy(np.ascontiguousarray(ref)).to(dtype).to(torch.float64).numpy()
    return float(np.abs(got - ref_r).max())


def output_excess(got: np.ndarray, ref: np.ndarray, dtype) -> float:
    """For the edge-size tests, whose tiny contexts give outputs of magnitude 2 to 4: there half
    a unit in the last place of the 16-bit output type alone is 1e-3 (fp16) to 8e-3 (bf16), so
    no kernel can stay within 2e-3 of the oracle.  Returns by how much |got - ref| exceeds
    max(2e-3, half an ulp of the output type at the oracle's value + 2e-4), i.e. the output must
    be within 2e-3 or be the oracle's value correctly rounded to within 2e-4; <= 0 passes.
    The benchmark configurations are held to the plain 2e-3 (output_error)."""
    mant = 10 if dtype == torch.float16 else 7
    expo = np.floor(np.log2(np.maximum(np.abs(ref), 2.0 ** -14)))
    half_ulp = 0.5 * 2.0 ** (expo - mant)
    return float((np.abs(got - ref) - np.maximum(TOL_OUT, half_ulp + 2e-4)).max())


# ---- records of what the parity tests measured: written to a report when the session ends ----
RECORDS = []


def record(test: str, **fields) -> None:
    RECORDS.append(dict(test=test, **fields))


class UnitView:
    """The sampled units of a [batch, heads, ...] tensor as fp64 arrays, indexable the way the
    oracle indexes the full tensor (`t[b, kv]` or `t[b, kv*G:(kv+1)*G]`), so that full-size
    inputs never have to be widened to fp64 as a whole."""

    def __init__(self, t: torch.Tensor, units, G: int = 1):
        self.G = G
        self.d = {(bi, kv): to64(t[bi, kv * G:(kv + 1) * G]) for (bi, kv) in units}

    def __getitem__(self, key):
        bi, h = key
        if isinstance(h, slice):
            return self.d[(bi, h.start // self.G)]
        return self.d[(bi, h)][0]


def oracle_inputs(w: Workload, Q, K, V, units):
    """fp64 views of the prompt for the oracle: everything, or only the sampled units."""
    if units is None:
        return to64(Q), to64(K), to64(V)
    return UnitView(Q, units, w.group), UnitView(K, units), UnitView(V, units)


def oracle_step_inputs(w: Workload, q, k, v, units):
    if units is None:
        return to64(q), to64(k), to64(v)
    return UnitView(q, units, w.group), UnitView(k, units), UnitView(v, units)


def run_decode_parity(w: Workload, n_steps: int, units=None, layer: int = 0,
                      staged: bool = True, check_segments: bool = True, defer_append: bool = False,
                      salient=None):
    """Prefill + n_steps of append/decode on GPU and oracle.  Every output is checked with
    output_excess; the largest raw |got - ref| is returned for the caller to bound.
    staged: the GPU quantiser is given the oracle's salient lists (for the sampled units; the
    others get the first n_s positions, which is as valid a split as any)."""
    Q, K, V = make_prefill(w, layer, DEV)
    P = probes_for(w, layer)
    oc = make_oracle(w, units)
    oc.prefill_compress(*oracle_inputs(w, Q, K, V, units), P)
    cache = make_cache(w, max_new=max(n_steps, 1), defer_append=defer_append)
    if staged:
        n_s = zo.salient_count(w.saliency_ratio, w.context)
        sal = np.tile(np.arange(max(n_s, 1), dtype=np.int32), (w.batch, w.n_kv_heads, 1))
        for (bi, kv), u in oc.units.items():
            sal[bi, kv, :n_s] = u.segments[0].hi.idx
        cache.prefill_compress(None, K, V, None, salient_idx=torch.tensor(sal, device=DEV))
    else:
        cache.prefill_compress(Q, K, V, P.tolist())
    flags = decode_probe_flags(w, layer, n_steps)
    worst = 0.0
    G = w.group
    for step in range(n_steps):
        q, k, v = make_decode_step(w, layer, step, DEV)
        cache.append(k, v)
        out = cache.decode_attention(q, flags[step])
        q64, k64, v64 = oracle_step_inputs(w, q, k, v, units)
        oc.append(k64, v64)
        ref = oc.decode_attention(q64, flags[step])
        got = to64(out)
        for (bi, kv), o in ref.items():
            g_ = got[bi, kv * G:(kv + 1) * G]
            worst = max(worst, output_error(g_, o))
            assert output_excess(g_, o, w.torch_dtype) <= 0.0, (step, worst)
    torch.cuda.synchronize()
    assert cache.check_guards(), "a kernel wrote outside the cache buffer or the workspace"
    if check_segments:
        import paper_2405_14256_b200 as zc
        n_seg = zc.zc_num_segments(cache.handle)
        some = oc.units[oc.unit_ids[0]]
        assert n_seg == len(some.segments)
        assert zc.zc_tail_tokens(cache.handle) == some.tail_K.shape[0]
    return worst, cache, oc


def compare_prefill_segment(w: Workload, cache, oc: zo.ZipCacheOracle, units):
    """Scores, salient sets and packed codes of segment 0 on the sampled units.  A unit whose
    salient set differs from the oracle's by near-tie swaps (see salient_sets_match) cannot be
    compared code by code; every other unit is.  Returns (swaps, units compared bit for bit,
    largest relative score error)."""
    p_gpu = cache.scores(w.context).cpu().numpy()
    idx_hi = cache.segment(0, 0, 0)[0].cpu().numpy()
    swaps, clean, worst_rel = 0, [], 0.0
    for (bi, kv) in units:
        s0 = oc.units[(bi, kv)].segments[0]
        rel = np.abs(p_gpu[bi, kv] - s0.p_tilde) / np.maximum(np.abs(s0.p_tilde), 1e-30)
        worst_rel = max(worst_rel, float(rel.max()))
        assert rel.max() <= 1e-4, rel.max()
        n = salient_sets_match(p_gpu[bi, kv], s0.p_tilde, idx_hi[bi, kv], s0.hi.idx, s0.hi.n)
        swaps += n
        if n == 0:
            clean.append((bi, kv))
    if clean:
        assert compare_segment(cache, oc, 0, units=clean) == 0
    return swaps, len(clean), worst_rel


def run_benchmark_mode(w: Workload, units, n_steps: int, layers: int = 2, graph: bool = False,
                       overlap_calls: bool = True, defer_append: bool = True):
    """What the benchmark times, checked against the oracle on sampled units: `layers` caches
    that share one workspace, ZC_FLAG_OVERLAP_CALLS | ZC_FLAG_DEFER_APPEND, every append and
    decode call of every step issued back to back on one stream with no host synchronisation
    (optionally captured into a CUDA graph and replayed once), the oracle run afterwards.
    Returns dict(worst = largest raw |out - oracle|, worst_rounded, excess (see output_excess),
    window_set_mismatches, caches, oracles)."""
    import paper_2405_14256_b200 as zc
    caches, oracles, ws = [], [], None
    pre_swaps = pre_clean = 0
    for ly in range(layers):
        Q, K, V = make_prefill(w, ly, DEV)
        P = probes_for(w, ly)
        oc = make_oracle(w, units)
        oc.prefill_compress(*oracle_inputs(w, Q, K, V, units), P)
        c = zc.ZipCache(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context, max(n_steps, 1),
                        w.saliency_ratio, w.bits_hi, w.bits_lo, w.window, device=DEV, workspace=ws,
                        defer_append=defer_append, overlap_calls=overlap_calls,
                        k_channel=w.k_scheme == "channel", guard_bytes=GUARD)
        ws = c.workspace
        c.prefill_compress(Q, K, V, P.tolist())
        torch.cuda.synchronize()
        del Q, K, V
        # scores, salient sets and codes of the prompt, before any window overwrites the scores
        a, b_, rel = compare_prefill_segment(w, c, oc, units)
        pre_swaps += a
        pre_clean += b_
        caches.append(c)
        oracles.append(oc)
    ins = [[make_decode_step(w, ly, s, DEV) for ly in range(layers)] for s in range(n_steps)]
    flags = [decode_probe_flags(w, ly, n_steps) for ly in range(layers)]
    outs = [[torch.empty_like(ins[0][0][0]) for _ in range(layers)] for _ in range(n_steps)]

    def issue():
        for s in range(n_steps):
            for ly, c in enumerate(caches):
                q, k, v = ins[s][ly]
                c.append(k, v)
                c.decode_attention(q, bool(flags[ly][s]), out=outs[s][ly])

    torch.cuda.synchronize()
    if graph:
        st = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(st):
            with torch.cuda.graph(g, stream=st):
                issue()
            g.replay()
    else:
        issue()
    torch.cuda.synchronize()
    assert zc.zc_device_status() == 0
    assert all(c.check_guards() for c in caches), "a kernel wrote outside its buffers"
    G = w.group
    worst = worst_r = 0.0
    excess = -1.0
    for s in range(n_steps):
        for ly, oc in enumerate(oracles):
            q64, k64, v64 = oracle_step_inputs(w, *ins[s][ly], units)
            oc.append(k64, v64)
            ref = oc.decode_attention(q64, bool(flags[ly][s]))
            got = to64(outs[s][ly])
            for (bi, kv), o in ref.items():
                g_ = got[bi, kv * G:(kv + 1) * G]
                worst = max(worst, output_error(g_, o))
                worst_r = max(worst_r, output_error_rounded(g_, o, w.torch_dtype))
                excess = max(excess, output_excess(g_, o, w.torch_dtype))
    swaps = clean = 0
    for c, oc in zip(caches, oracles):
        n_seg = zc.zc_num_segments(c.handle)
        some = oc.units[oc.unit_ids[0]]
        assert n_seg == len(some.segments)
        assert zc.zc_tail_tokens(c.handle) == some.tail_K.shape[0]
        for seg in range(1, n_seg):
            # Re-compressed windows.  Their scores come from the decode kernel's own softmax
            # statistics (relative error up to 1e-3, see WINDOW_SCORE_RTOL), so two tokens whose
            # oracle scores lie within twice that of the oracle's n_s-th score may swap sides;
            # such units are counted, every other unit is compared code by code.
            idx_hi = c.segment(seg, 0, 0)[0].cpu().numpy()
            same = []
            for u in units:
                sg = oc.units[u].segments[seg]
                a, b = set(idx_hi[u[0], u[1]].tolist()), set(sg.hi.idx.tolist())
                if a == b:
                    same.append(u)
                    continue
                kth = np.sort(sg.p_tilde)[::-1][sg.hi.n - 1]
                for j in (a - b) | (b - a):
                    assert abs(sg.p_tilde[j] - kth) <= 2 * WINDOW_SCORE_RTOL * abs(kth), (seg, u, j)
                swaps += len(a - b)
            if same:
                assert compare_segment(c, oc, seg, units=same) == 0
    return dict(worst=worst, worst_rounded=worst_r, excess=excess, window_set_mismatches=swaps,
                near_tie_swaps=pre_swaps, units_code_exact=pre_clean, caches=caches,
                oracles=oracles)
