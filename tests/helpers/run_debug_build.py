"""Runs a handful of parity cases against the bounds-checked build of the library
(libzipcache_debug.so, -DZC_DEBUG) in a process of its own: every index check in the kernels
must pass (zc_device_status() == 0) and results must still match the oracle."""
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))


def main():
    from paper_2405_14256_b200 import build
    path = build.build(debug=True)
    import paper_2405_14256_b200 as zc
    zc.load_library(path)
    import zc_testlib as tl
    cases = [
        (dict(context=512, n_q_heads=4, n_kv_heads=4), 8, False),
        (dict(context=150, n_q_heads=4, n_kv_heads=2, window=16, rho_recent=0.1, rho_random=0.1), 40, True),
        (dict(context=300, batch=2, n_q_heads=8, n_kv_heads=2, dtype="bf16", k_scheme="channel"), 6, True),
        (dict(context=333, batch=2, n_q_heads=8, n_kv_heads=2, bits_hi=16, bits_lo=2, saliency_ratio=0.15,
              window=16), 36, False),
        (dict(context=129, n_q_heads=2, n_kv_heads=2, saliency_ratio=1.0), 3, False),
    ]
    for kw, steps, defer in cases:
        w = tl.small_workload(**kw)
        _, cache, oc = tl.run_decode_parity(w, steps, staged=False, defer_append=defer)
        for seg in range(zc.zc_num_segments(cache.handle)):
            assert tl.compare_segment(cache, oc, seg) == 0
        assert zc.zc_device_status() == 0, "an index check of the bounds-checked build failed"
    from workloads import get_config
    r = tl.run_benchmark_mode(get_config(2), [(0, 0)], 3, layers=2)
    assert r["excess"] <= 0.0 and zc.zc_device_status() == 0
    print("debug build ok")


if __name__ == "__main__":
    main()
