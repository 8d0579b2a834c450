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


def make_cache(w: Workload, max_new=None, defer_append: bool = False, overlap_calls: bool = False):
    import paper_2405_14256_b200 as zc
    return zc.ZipCache(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context,
                       w.decode_steps if max_new is None else max_new, w.saliency_ratio,
                       w.bits_hi, w.bits_lo, w.window, device=DEV, defer_append=defer_append,
                       overlap_calls=overlap_calls)


def make_oracle(w: Workload, units=None) -> zo.ZipCacheOracle:
    return zo.ZipCacheOracle(w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.saliency_ratio,
                             w.bits_hi, w.bits_lo, w.window, units=units)


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
                q = getattr(sub, tn)
                want = zo.pack_codes(q["codes"], sub.bits)
                mism += int((codes[bi, kv] != want).sum())
                np.testing.assert_array_equal(codes[bi, kv], want)
                np.testing.assert_array_equal(sz[bi, kv, :, 0], q["s"])
                np.testing.assert_array_equal(sz[bi, kv, :, 1], q["z"])
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


def output_error(got: np.ndarray, ref: np.ndarray, dtype) -> float:
    """Largest |got - ref| beyond the rounding of the output itself: the library stores its
    result in the 16-bit input type, which alone moves a value by up to half a unit in the
    last place (bf16: 2^-9 at |o| in [0.5, 1)); that half-ulp is not the kernel's error and
    is subtracted before comparing with the 2e-3 bound."""
    mant = 10 if dtype == torch.float16 else 7
    expo = np.floor(np.log2(np.maximum(np.abs(ref), 2.0 ** -14)))
    half_ulp = 0.5 * 2.0 ** (expo - mant)
    return float(np.maximum(np.abs(got - ref) - half_ulp, 0.0).max())


def run_decode_parity(w: Workload, n_steps: int, tol: float = 2e-3, units=None, layer: int = 0,
                      staged: bool = True, check_segments: bool = True, defer_append: bool = False):
    """Prefill + n_steps of append/decode on GPU and oracle; returns max abs output error."""
    Q, K, V = make_prefill(w, layer, DEV)
    P = probes_for(w, layer)
    oc = make_oracle(w, units)
    Qh, Kh, Vh = to64(Q), to64(K), to64(V)
    oc.prefill_compress(Qh, Kh, Vh, P)
    cache = make_cache(w, max_new=max(n_steps, 1), defer_append=defer_append)
    if staged:
        n_s = zo.salient_count(w.saliency_ratio, w.context)
        sal = np.zeros((w.batch, w.n_kv_heads, max(n_s, 1)), dtype=np.int32)
        full = make_oracle(w) if units is not None else oc
        if units is not None:
            full.prefill_compress(Qh, Kh, Vh, P)
        for (bi, kv), u in full.units.items():
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
        oc.append(to64(k), to64(v))
        ref = oc.decode_attention(to64(q), flags[step])
        got = to64(out)
        for (bi, kv), o in ref.items():
            worst = max(worst, output_error(got[bi, kv * G:(kv + 1) * G], o, w.torch_dtype))
        assert worst <= tol, (step, worst)
    torch.cuda.synchronize()
    if check_segments:
        import paper_2405_14256_b200 as zc
        n_seg = zc.zc_num_segments(cache.handle)
        some = oc.units[oc.unit_ids[0]]
        assert n_seg == len(some.segments)
        assert zc.zc_tail_tokens(cache.handle) == some.tail_K.shape[0]
    return worst, cache, oc
