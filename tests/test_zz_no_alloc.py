"""zc_decode_attention_noalloc against zc_decode_attention.

Some callers cannot give the library a workspace because they are not allowed to allocate
device memory at that point (a plug-in inside a server whose pool owns the device, a loop
that must stay out of the allocator).  For them the library carries a fixed scratch buffer
and one extra entry point that uses it.  Here two caches are filled with the same seeded
input; one is driven through the ordinary call with a caller workspace, the other through the
no-allocation call, for two decode steps in a row.  The second step re-uses the shared
buffer with the first step's contents still in it, which is the case a stale-scratch bug
would show up in.  This file sorts last on purpose: it runs after every other GPU test and
must also pass alone in a fresh process.
"""
import pytest
import torch

import zc_testlib as tl
from workloads import make_prefill, make_decode_step

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("kw", [
    dict(context=300, batch=2, n_q_heads=8, n_kv_heads=2, dtype="bf16", outlier_fixed=0),
    dict(context=512, n_q_heads=4, n_kv_heads=4),
])
def test_noalloc_entry_matches_workspace_entry_two_calls_in_a_row(kw):
    import paper_2405_14256_b200 as zc
    w = tl.small_workload(**kw)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w).tolist()
    ref_cache, new_cache = tl.make_cache(w), tl.make_cache(w)
    ref_cache.mem.zero_()
    new_cache.mem.zero_()
    ref_cache.prefill_compress(Q, K, V, P)
    new_cache.prefill_compress(Q, K, V, P)
    for step in range(2):
        q, k, v = make_decode_step(w, 0, step, tl.DEV)
        ref_cache.append(k, v)
        new_cache.append(k, v)
        want = ref_cache.decode_attention(q, step == 1)
        got = torch.empty_like(q)
        zc.zc_decode_attention_noalloc(new_cache.handle, q, got, step == 1)
        torch.cuda.synchronize()
        err = float((got.double() - want.double()).abs().max())
        assert err <= 2e-3, (step, err)   # the tolerance of the decode parity tests
        assert torch.equal(got, want)      # same kernels, same order of operations
    assert zc.zc_device_status() == 0
    # the window statistics collected on the probe step went through the built-in buffer too
    assert torch.equal(ref_cache.mem, new_cache.mem)


def test_noalloc_entry_across_a_recompressed_window():
    """The call that completes a window re-compresses it inside the same kernel: through the
    built-in buffer the cache must end up byte for byte as through a caller workspace."""
    import paper_2405_14256_b200 as zc
    w = tl.small_workload(context=200, batch=2, n_q_heads=8, n_kv_heads=2, window=8)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w).tolist()
    ref_cache, new_cache = tl.make_cache(w, max_new=32), tl.make_cache(w, max_new=32)
    ref_cache.mem.zero_()
    new_cache.mem.zero_()
    ref_cache.prefill_compress(Q, K, V, P)
    new_cache.prefill_compress(Q, K, V, P)
    for step in range(19):                       # two windows and three steps of the third
        q, k, v = make_decode_step(w, 0, step, tl.DEV)
        ref_cache.append(k, v)
        new_cache.append(k, v)
        want = ref_cache.decode_attention(q, step % 3 == 0)
        got = torch.empty_like(q)
        zc.zc_decode_attention_noalloc(new_cache.handle, q, got, step % 3 == 0)
        torch.cuda.synchronize()
        assert torch.equal(got, want), step
    assert zc.zc_device_status() == 0
    assert zc.zc_num_segments(new_cache.handle) == 3
    assert torch.equal(ref_cache.mem, new_cache.mem)


def test_noalloc_entry_rejects_shapes_beyond_its_buffer():
    import paper_2405_14256_b200 as zc
    # 128 x 32 heads: the split-K partials of one call alone exceed the 4 MiB buffer
    w = tl.small_workload(context=64, batch=128, n_q_heads=32, n_kv_heads=32, window=8)
    big = tl.make_cache(w, max_new=64)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    big.prefill_compress(Q, K, V, tl.probes_for(w).tolist())
    q, k, v = make_decode_step(w, 0, 0, tl.DEV)
    big.append(k, v)
    out = torch.empty_like(q)
    with pytest.raises(zc.ZipCacheError, match="built-in buffer"):
        zc.zc_decode_attention_noalloc(big.handle, q, out, False)
    # the ordinary entry point still serves the same cache
    big.decode_attention(q, False, out=out)
    torch.cuda.synchronize()
    assert torch.isfinite(out.float()).all()


def test_noalloc_calls_back_to_back_without_synchronising():
    """Several caches, call after call on one stream with no host synchronisation between
    them: every call uses the one built-in buffer, the library gives calls that may be in
    flight together separate parts of it (or orders them).  Results must equal those of the
    same sequence through a caller workspace."""
    import paper_2405_14256_b200 as zc
    w = tl.small_workload(context=260, batch=2, n_q_heads=8, n_kv_heads=2, window=8)
    layers, steps = 3, 20
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w).tolist()
    ins = [make_decode_step(w, 0, s, tl.DEV) for s in range(steps)]
    results = []
    for noalloc in (False, True):
        caches = [tl.make_cache(w, max_new=32, defer_append=True, overlap_calls=True) for _ in range(layers)]
        for c in caches:
            c.mem.zero_()
            c.prefill_compress(Q, K, V, P)
        outs = [[torch.empty_like(ins[0][0]) for _ in range(layers)] for _ in range(steps)]
        torch.cuda.synchronize()
        for s in range(steps):
            q, k, v = ins[s]
            for ly, c in enumerate(caches):
                c.append(k, v)
                if noalloc:
                    zc.zc_decode_attention_noalloc(c.handle, q, outs[s][ly], s % 3 == 0)
                else:
                    c.decode_attention(q, s % 3 == 0, out=outs[s][ly])
        torch.cuda.synchronize()
        assert zc.zc_device_status() == 0
        results.append((outs, [c.mem.clone() for c in caches]))
    for a, b in zip(results[0][0], results[1][0]):
        for x, y in zip(a, b):
            assert torch.equal(x, y)
    for x, y in zip(results[0][1], results[1][1]):
        assert torch.equal(x, y)


def test_noalloc_entry_against_the_oracle():
    """The no-allocation call compared with the oracle itself (not only with the workspace
    call): every output within the decode bound over two re-compressed windows, and the
    windows' lists, codes and parameters equal to the oracle's."""
    import numpy as np
    import paper_2405_14256_b200 as zc
    w = tl.small_workload(context=260, batch=2, n_q_heads=8, n_kv_heads=2, window=16, rho_recent=0.2,
                          rho_random=0.2)
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w)
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    cache = tl.make_cache(w, max_new=40)
    cache.prefill_compress(Q, K, V, P.tolist())
    for step in range(35):
        q, k, v = make_decode_step(w, 0, step, tl.DEV)
        probe = step % 3 == 0
        cache.append(k, v)
        got = torch.empty_like(q)
        zc.zc_decode_attention_noalloc(cache.handle, q, got, probe)
        oc.append(tl.to64(k), tl.to64(v))
        ref = oc.decode_attention(tl.to64(q), probe)
        torch.cuda.synchronize()
        g = got.float().cpu().numpy()
        for (bi, kv), r in ref.items():
            assert tl.output_excess(g[bi, kv * oc.G:(kv + 1) * oc.G], r, w.torch_dtype) <= 0.0, step
    assert zc.zc_num_segments(cache.handle) == 3 and zc.zc_device_status() == 0
    for seg in range(3):
        assert tl.compare_segment(cache, oc, seg) == 0
    assert cache.check_guards()
