"""Randomly drawn configurations (tests/zc_random_cases.py) against the oracle: scores, splits,
packed codes and parameters of the prompt and of every re-compressed window bit for bit, every
decode output within the bound, the device status clean and the guard bands intact."""
import pytest

import zc_random_cases as rc
import zc_testlib as tl

CASES_PER_TEST = 30


@pytest.mark.gpu
@pytest.mark.parametrize("first", [20000 + CASES_PER_TEST * i for i in range(8)])
def test_random_configurations_match_the_oracle(first):
    tally = {}
    for seed in range(first, first + CASES_PER_TEST):
        try:
            r = rc.run_case(seed)
        except AssertionError as e:
            raise AssertionError(f"case {seed}: {rc.draw(seed)}: {e!r}") from e
        tally[r] = tally.get(r, 0) + 1
    # near ties are rare by construction of the inputs; most cases must be compared to the end
    assert tally.get("ok", 0) + tally.get("beyond", 0) >= CASES_PER_TEST - 3, tally
    tl.record(f"random configurations, cases {first}-{first + CASES_PER_TEST - 1}", cases=CASES_PER_TEST,
              compared_to_the_end=tally.get("ok", 0) + tally.get("beyond", 0),
              beyond_strict_output_bound=tally.get("beyond", 0), near_tie_cases=tally.get("near tie", 0))


def test_drawn_cases_cover_every_option():
    """The 240 cases above reach every bit pair, both key schemes, both scopes, 16-bit parameters,
    token groups over all heads, both append modes, calls side by side with and without a graph,
    contexts from 1 token to several tiles and at least two windows."""
    cases = [rc.draw(s) for s in range(20000, 20000 + 8 * CASES_PER_TEST)]
    assert {(c["w"]["bits_hi"], c["w"]["bits_lo"]) for c in cases} == set(rc.BIT_PAIRS)
    for key in ("token", "p16", "ga", "defer", "overlap"):
        assert {c[key] for c in cases} == {False, True}, key
    assert {c["graph"] for c in cases if c["overlap"]} == {False, True}
    assert {c["w"]["k_scheme"] for c in cases} == {"cst", "channel"}
    assert min(c["w"]["context"] for c in cases) <= 2 and max(c["w"]["context"] for c in cases) > 1024
    assert any(c["steps"] >= 2 * c["w"]["window"] for c in cases)
    assert {c["w"]["dtype"] for c in cases} == {"fp16", "bf16"}


ATTENTION_LENGTHS = [1, 2, 63, 64, 65, 127, 128, 129, 191, 255, 256, 257, 383, 384, 385, 511, 512, 513, 767, 768,
                     769, 1023, 1024, 1025]


@pytest.mark.gpu
@pytest.mark.parametrize("first", [30000, 30020, 30040])
def test_random_prefill_attention_shapes(first):
    """zc_prefill_attention on random lengths (tile boundaries and anything up to 2600), head
    layouts and input types: O and every row's log-sum-exp against the oracle.  O's bound is the
    one of test_prefill_attention_output_and_row_lse, stated there for outputs of magnitude up
    to 4 and scaled with the head's largest output beyond that."""
    import numpy as np
    import torch
    import paper_2405_14256_b200 as zc
    from oracle import zipcache_oracle as zo
    from workloads import make_prefill
    worst_o = worst_l = 0.0
    for seed in range(first, first + 20):
        rng = np.random.default_rng(seed)
        n_kv, G = int(rng.choice([1, 2, 4])), int(rng.choice([1, 2, 4, 8]))
        l = int(rng.choice(ATTENTION_LENGTHS)) if rng.random() < 0.5 else int(rng.integers(1, 2600))
        w = tl.small_workload(dtype=str(rng.choice(["fp16", "bf16"])), batch=int(rng.integers(1, 3)),
                              n_q_heads=n_kv * G, n_kv_heads=n_kv, context=l, outlier_fixed=int(rng.choice([0, 4])),
                              band=int(rng.choice([0, 3])), cfg_id=int(rng.integers(10, 1000)))
        Q, K, V = make_prefill(w, 0, tl.DEV)
        cache = tl.make_cache(w)
        O, lse = cache.prefill_attention(Q, K, V)
        torch.cuda.synchronize()
        assert zc.zc_device_status() == 0 and cache.check_guards(), seed
        heads = [(bi, h) for bi in range(w.batch) for h in range(w.n_q_heads)]
        if l > 1200:   # the oracle's l x l attention: three heads of the long cases
            heads = [heads[j] for j in rng.choice(len(heads), size=min(3, len(heads)), replace=False)]
        tol = 2e-2 if w.dtype == "bf16" else 4e-3
        for bi, h in heads:
            kv = h // w.group
            O_ref, lse_ref = zo.prefill_attention(tl.to64(Q[bi, h]), tl.to64(K[bi, kv]), tl.to64(V[bi, kv]))
            e_o = float(np.abs(tl.to64(O[bi, h]) - O_ref).max())
            e_l = float(np.abs(lse[bi, h].double().cpu().numpy() - lse_ref).max())
            assert e_o <= tol * max(1.0, float(np.abs(O_ref).max()) / 4.0), (seed, l, bi, h, e_o)
            assert e_l <= 2e-4, (seed, l, bi, h, e_l)
            worst_o, worst_l = max(worst_o, e_o), max(worst_l, e_l)
    tl.record(f"random prefill attention shapes, cases {first}-{first + 19}", cases=20, max_abs_out=worst_o,
              score_rel=worst_l)
