"""Randomly drawn small configurations for the GPU parity tests: every combination of bit
pair, key scheme, saliency scope, parameter width, token grouping, window, context length,
head layout, append mode and launch mode that the library accepts, each run against the oracle
on inputs seeded by the case.  Holds no arithmetic of the method."""
from __future__ import annotations

import numpy as np
import torch

import zc_testlib as tl
from workloads import make_prefill, make_decode_step

BIT_PAIRS = [(4, 2), (4, 4), (2, 2), (2, 4), (16, 2), (16, 4), (4, 16), (16, 16), (8, 8), (8, 4), (8, 2),
             (4, 8), (2, 8)]
EDGE_LENGTHS = [1, 2, 15, 16, 17, 31, 33, 100, 127, 128, 129, 255, 256, 257, 300, 383, 385, 511, 512,
                513, 640, 700]


def draw(seed: int) -> dict:
    """One case: the workload's fields and the cache's options (only combinations the library
    accepts: 16-bit parameters with CSTQuant at 2 / 4 bits, token groups over all heads with
    token scope and no 16-bit class, calls side by side with neither)."""
    rng = np.random.default_rng(seed)
    n_kv = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([1, 2, 4, 8]))
    hi, lo = BIT_PAIRS[int(rng.integers(len(BIT_PAIRS)))]
    kch = bool(rng.random() < 0.3)
    token = bool(rng.random() < 0.35)
    p16 = bool(rng.random() < 0.3) and not kch and hi in (2, 4) and lo in (2, 4)
    ga = token and bool(rng.random() < 0.5) and 16 not in (hi, lo)
    l = int(rng.choice(EDGE_LENGTHS)) if rng.random() < 0.5 else int(rng.integers(1, 700))
    if rng.random() < 0.12:
        l = int(rng.integers(700, 3000))
    window = int(rng.choice([8, 9, 16, 17, 31, 32, 100, 128])) if rng.random() < 0.7 else int(rng.integers(8, 129))
    steps = int(min(rng.integers(1, int(2.4 * window) + 2), 140))
    ratio = float(rng.choice([0.0, 0.15, 0.3, 0.4, 0.5, 1.0, round(float(rng.random()), 3)]))
    return dict(
        w=dict(dtype=str(rng.choice(["fp16", "bf16"])), batch=int(rng.integers(1, 4)), n_q_heads=n_kv * G,
               n_kv_heads=n_kv, context=l, saliency_ratio=ratio, bits_hi=hi, bits_lo=lo, window=window,
               decode_steps=steps, rho_recent=float(rng.choice([0.05, 0.1, 0.2])),
               rho_random=float(rng.choice([0.05, 0.1, 0.2])), outlier_fixed=int(rng.choice([0, 4])),
               band=int(rng.choice([0, 0, 3])), k_scheme="channel" if kch else "cst",
               cfg_id=int(rng.integers(10, 1000))),
        token=token, p16=p16, ga=ga, defer=bool(rng.random() < 0.5), steps=steps,
        overlap=(not token and not p16 and bool(rng.random() < 0.4)), layers=int(rng.integers(2, 4)),
        graph=bool(rng.random() < 0.5))


def _near_tie(p_ref, got, want, n, rtol) -> int:
    """0: same set; > 0: that many tokens swapped, all within rtol of the n-th largest oracle
    score; -1: the sets differ by more than near ties."""
    a, b = set(map(int, got)), set(map(int, want))
    if a == b:
        return 0
    kth = np.sort(p_ref)[::-1][n - 1]
    if any(abs(p_ref[j] - kth) > rtol * abs(kth) for j in (a - b) | (b - a)):
        return -1
    return len(a - b)


def _check_prompt(w, cache, oc) -> bool:
    """Scores within 1e-4, the split (up to near ties at 1e-5) and, unless a near tie swapped
    tokens, every packed code and parameter of the prompt's segment.  False: a near tie, the case
    cannot be compared any further."""
    p_gpu = cache.scores(w.context).cpu().numpy()
    idx_hi = cache.segment(0, 0, 0)[0].cpu().numpy()
    for (bi, kv), u in oc.units.items():
        s0 = u.segments[0]
        rel = np.abs(p_gpu[bi, kv] - s0.p_tilde) / np.maximum(np.abs(s0.p_tilde), 1e-30)
        assert rel.max() <= 1e-4, ("score", rel.max())
        if s0.hi.n:
            t = _near_tie(s0.p_tilde, idx_hi[bi, kv][:s0.hi.n], s0.hi.idx, s0.hi.n, 1e-5)
            assert t >= 0, "the salient set differs by more than near ties"
            if t > 0:
                return False
    assert tl.compare_segment(cache, oc, 0) == 0
    return True


def _check_window(cache, oc, seg) -> bool:
    """A re-compressed window: the split up to near ties (window scores carry the decode
    kernel's noise: see zc_testlib.WINDOW_SCORE_RTOL), then codes and parameters bit for bit."""
    idx_hi = cache.segment(seg, 0, 0)[0].cpu().numpy()
    for (bi, kv), u in oc.units.items():
        sg = u.segments[seg]
        if sg.hi.n and sg.lo.n:
            t = _near_tie(sg.p_tilde, idx_hi[bi, kv][:sg.hi.n], sg.hi.idx, sg.hi.n, 3 * tl.WINDOW_SCORE_RTOL)
            assert t >= 0, ("a window's salient set differs by more than near ties", seg)
            if t > 0:
                return False
    assert tl.compare_segment(cache, oc, seg) == 0
    return True


def _check_output(w, got, ref, step, beyond: list) -> None:
    """The decode bound of the edge-size tests (zc_testlib.output_excess).  The random inputs
    include contexts of a few tokens with outlier channels, whose outputs reach magnitude 5; the
    kernel's contraction runs on 16-bit operands (probabilities rounded to f16, relative 2^-11),
    so there its error grows with the output: such a case is counted in `beyond` and must stay
    within 2e-3 + half an ulp of the output type + 1e-3 x the head's largest output."""
    if tl.output_excess(got, ref, w.torch_dtype) <= 0.0:
        return
    err = np.abs(got - ref)
    k = np.unravel_index(err.argmax(), err.shape)
    mag = float(np.abs(ref).max())
    mant = 10 if w.torch_dtype == torch.float16 else 7
    half_ulp = 0.5 * 2.0 ** (np.floor(np.log2(max(abs(ref[k]), 2.0 ** -14))) - mant)
    assert err.max() <= 2e-3 + half_ulp + 1e-3 * mag, ("decode", step, float(err.max()), float(ref[k]), mag)
    beyond.append(float(err.max()))


def _one_call_at_a_time(case, w, zc) -> str:
    Q, K, V = make_prefill(w, 0, tl.DEV)
    P = tl.probes_for(w)
    oc = tl.make_oracle(w, scope="token" if case["token"] else "kv_head",
                        param_dtype="f16" if case["p16"] else "f32",
                        group="all_heads" if case["ga"] else "head")
    oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
    cache = tl.make_cache(w, max_new=case["steps"], defer_append=case["defer"], token_scope=case["token"],
                          params_f16=case["p16"], group_all_heads=case["ga"])
    cache.prefill_compress(Q, K, V, P.tolist())
    torch.cuda.synchronize()
    if not _check_prompt(w, cache, oc):
        return "near tie"
    rng = np.random.default_rng(w.cfg_id)
    n_seg, beyond = 1, []
    for step in range(case["steps"]):
        q, k, v = make_decode_step(w, 0, step, tl.DEV)
        probe = bool(rng.random() < 0.3)
        cache.append(k, v)
        out = cache.decode_attention(q, probe)
        oc.append(tl.to64(k), tl.to64(v))
        ref = oc.decode_attention(tl.to64(q), probe)
        torch.cuda.synchronize()
        got = out.float().cpu().numpy()
        for (bi, kv), r in ref.items():
            _check_output(w, got[bi, kv * oc.G:(kv + 1) * oc.G], r, step, beyond)
        some = oc.units[oc.unit_ids[0]]
        assert zc.zc_num_segments(cache.handle) == len(some.segments), ("segments", step)
        assert zc.zc_tail_tokens(cache.handle) == some.tail_K.shape[0], ("tail", step)
        if len(some.segments) > n_seg:
            n_seg += 1
            if not _check_window(cache, oc, n_seg - 1):
                return "near tie"
    assert zc.zc_device_status() == 0
    assert cache.check_guards(), "a kernel wrote outside the cache buffer or the workspace"
    return "beyond" if beyond else "ok"


def _side_by_side(case, w, zc) -> str:
    """ZC_FLAG_OVERLAP_CALLS: 2 or 3 caches on one workspace, every call of every step issued
    back to back (or captured in a graph and replayed), the oracle run afterwards."""
    layers, n_steps = case["layers"], case["steps"]
    caches, oracles, ws = [], [], None
    for ly in range(layers):
        Q, K, V = make_prefill(w, ly, tl.DEV)
        P = tl.probes_for(w, ly)
        oc = tl.make_oracle(w)
        oc.prefill_compress(tl.to64(Q), tl.to64(K), tl.to64(V), P)
        c = zc.ZipCache(w.torch_dtype, w.batch, w.n_q_heads, w.n_kv_heads, w.context, max(n_steps, 1),
                        w.saliency_ratio, w.bits_hi, w.bits_lo, w.window, device=tl.DEV, workspace=ws,
                        defer_append=case["defer"], overlap_calls=True,
                        k_channel=w.k_scheme == "channel", guard_bytes=tl.GUARD)
        ws = c.workspace
        c.prefill_compress(Q, K, V, P.tolist())
        torch.cuda.synchronize()
        if not _check_prompt(w, c, oc):
            return "near tie"
        caches.append(c)
        oracles.append(oc)
    rng = np.random.default_rng(w.cfg_id)
    ins = [[make_decode_step(w, ly, s, tl.DEV) for ly in range(layers)] for s in range(n_steps)]
    flags = [[bool(rng.random() < 0.3) for _ in range(n_steps)] for _ in range(layers)]
    outs = [[torch.empty_like(ins[0][0][0]) for _ in range(layers)] for _ in range(n_steps)]

    def issue():
        for s in range(n_steps):
            for ly, c in enumerate(caches):
                q, k, v = ins[s][ly]
                c.append(k, v)
                c.decode_attention(q, flags[ly][s], out=outs[s][ly])

    torch.cuda.synchronize()
    if case["graph"]:
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
    refs = []
    for s in range(n_steps):
        for ly, oc in enumerate(oracles):
            q, k, v = ins[s][ly]
            oc.append(tl.to64(k), tl.to64(v))
            refs.append((s, ly, oc.decode_attention(tl.to64(q), flags[ly][s])))
    # windows first: a near tie in a window's split changes the outputs that follow it
    for c, oc in zip(caches, oracles):
        some = oc.units[oc.unit_ids[0]]
        assert zc.zc_num_segments(c.handle) == len(some.segments)
        assert zc.zc_tail_tokens(c.handle) == some.tail_K.shape[0]
        for seg in range(1, len(some.segments)):
            if not _check_window(c, oc, seg):
                return "near tie"
    beyond = []
    for s, ly, ref in refs:
        got = outs[s][ly].float().cpu().numpy()
        G = oracles[ly].G
        for (bi, kv), r in ref.items():
            _check_output(w, got[bi, kv * G:(kv + 1) * G], r, s, beyond)
    return "beyond" if beyond else "ok"


def run_case(seed: int) -> str:
    """Runs case `seed`; returns "ok", "beyond" (see _check_output) or "near tie" (a split
    differed by tokens within the score tolerance of the threshold: nothing after it can be
    compared); raises on any mismatch."""
    import paper_2405_14256_b200 as zc
    case = draw(seed)
    w = tl.small_workload(**case["w"])
    return _side_by_side(case, w, zc) if case["overlap"] else _one_call_at_a_time(case, w, zc)
