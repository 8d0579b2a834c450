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
