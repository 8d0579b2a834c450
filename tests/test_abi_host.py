"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
include/zipcache.h declares, sizes caches, samples probes like the oracle and rejects bad
arguments and out-of-order calls before any device work."""
import ctypes as C
import os
import re

import numpy as np
import pytest
import torch

from oracle import zipcache_oracle as zo

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def zc():
    from paper_2405_14256_b200 import build
    build.build()
    import paper_2405_14256_b200 as mod
    mod.load_library()
    return mod


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "zipcache.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(zc_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(zc):
    names = _declared_symbols()
    assert {"zc_prefill_compress", "zc_append", "zc_decode_attention"} <= set(names)
    lib = zc.lib()
    for n in names:
        assert hasattr(lib, n), n


def test_binding_covers_every_declared_symbol(zc):
    from paper_2405_14256_b200 import binding
    for n in _declared_symbols():
        assert n in binding._SIGS, n
        assert hasattr(binding, n), n


def test_cache_bytes_cover_the_algorithmic_bytes(zc):
    for (b, hq, hkv, l, r) in [(8, 32, 8, 4096, 0.4), (1, 4, 4, 512, 0.4), (16, 32, 8, 8192, 0.3)]:
        cfg = zc.ZcConfig.make(torch.bfloat16, b, hq, hkv, l, 128, r)
        cache, ws = zc.zc_cache_bytes(cfg)
        n_s = int(np.floor(r * l))
        algorithmic = b * hkv * (n_s * 144 + (l - n_s) * 80)
        assert cache >= algorithmic
        assert cache <= 1.25 * algorithmic + b * hkv * (2 * 100 * 256 + 8 * l + 65536)
        assert ws > 0 and ws % 256 == 0 and cache % 256 == 0


@pytest.mark.parametrize("bad", [
    dict(head_dim=64), dict(bits_hi=5), dict(bits_lo=3), dict(bits_hi=16, bits_lo=8), dict(k_scheme=2), dict(window=4), dict(window=129),
    dict(saliency_ratio=1.5), dict(n_q_heads=6), dict(batch=0), dict(n_q_heads=72, n_kv_heads=8),
    dict(scope=2), dict(scope=1, flags=2),   # token scope cannot be combined with ZC_FLAG_OVERLAP_CALLS (2)
    # ZC_FLAG_PARAMS_F16 (8): not with overlapping calls, channelwise keys, or classes other than 2 / 4 bits
    dict(flags=8 | 2), dict(flags=8, k_scheme=1), dict(flags=8, bits_hi=16), dict(flags=8, bits_lo=8), dict(flags=32),
    # ZC_FLAG_GROUP_ALL_HEADS (16): needs token scope, no 16-bit class
    dict(flags=16), dict(flags=16, scope=1, bits_hi=16),
])
def test_invalid_configurations_are_rejected(zc, bad):
    kw = dict(dtype=torch.float16, batch=2, n_q_heads=8, n_kv_heads=8, max_prefill=256,
              max_new_tokens=16, saliency_ratio=0.4, bits_hi=4, bits_lo=2, window=100, head_dim=128)
    kw.update(bad)
    cfg = zc.ZcConfig.make(**kw)
    with pytest.raises(zc.ZipCacheError, match="invalid argument"):
        zc.zc_cache_bytes(cfg)


@pytest.mark.parametrize("l", [1, 2, 19, 20, 21, 100, 512, 4096, 32768])
def test_default_probes_equal_the_oracle_sampler(zc, l):
    for seed in (1, 0x5A1F + 2000, 2 ** 63 + 11):
        got = zc.zc_default_probes(l, 0.05, 0.05, seed)
        want = zo.probe_positions(l, 0.05, 0.05, seed)
        assert got == want.tolist()
        assert zc.zc_probe_count(l, 0.05, 0.05) == len(got)
        assert got[-1] == l - 1 and all(a < b for a, b in zip(got, got[1:]))


def test_calls_out_of_order_and_bad_pointers_fail_on_the_host(zc):
    """A handle over a fake (never dereferenced) device address: every call below must be
    refused by the host-side checks, so nothing reaches a GPU."""
    cfg = zc.ZcConfig.make(torch.float16, 1, 4, 4, 64, 8, 0.5)
    nbytes, ws = zc.zc_cache_bytes(cfg)
    lib = zc.lib()
    h = C.c_void_p(0)
    assert lib.zc_cache_init(C.c_void_p(0), nbytes, C.byref(cfg), C.byref(h)) == -1      # null
    assert lib.zc_cache_init(C.c_void_p(0x1010), nbytes, C.byref(cfg), C.byref(h)) == -4  # alignment
    assert lib.zc_cache_init(C.c_void_p(0x10000), nbytes - 1, C.byref(cfg), C.byref(h)) == -2
    assert lib.zc_cache_init(C.c_void_p(0x10000), nbytes, C.byref(cfg), C.byref(h)) == 0
    try:
        fake = C.c_void_p(0x20000)
        assert lib.zc_append(h, fake, fake, None) == -3                      # before prefill
        assert lib.zc_decode_attention(h, fake, fake, 0, fake, ws, None) == -3
        assert lib.zc_decode_attention_noalloc(h, fake, fake, 0, None) == -3
        assert lib.zc_num_segments(h) == 0 and lib.zc_tail_tokens(h) == 0
        assert lib.zc_decode_bytes(h) == 0
        ks = (C.c_int64 * 3)(4 * 64 * 128, 64 * 128, 128)
        pp = (C.c_int32 * 2)(5, 63)
        # too long, misaligned K, probe list not ending at the last token, descending list
        assert lib.zc_prefill_compress(h, fake, fake, fake, 65, ks, ks, pp, 2, None, fake, ws, None) == -2
        assert lib.zc_prefill_compress(h, fake, C.c_void_p(0x20008), fake, 64, ks, ks, pp, 2, None, fake, ws, None) == -4
        bad = (C.c_int32 * 2)(5, 62)
        assert lib.zc_prefill_compress(h, fake, fake, fake, 64, ks, ks, bad, 2, None, fake, ws, None) == -1
        bad = (C.c_int32 * 2)(63, 5)
        assert lib.zc_prefill_compress(h, fake, fake, fake, 64, ks, ks, bad, 2, None, fake, ws, None) == -1
        odd = (C.c_int64 * 3)(4 * 64 * 128, 64 * 128, 132)
        assert lib.zc_prefill_compress(h, fake, fake, fake, 64, ks, odd, pp, 2, None, fake, ws, None) == -1
        assert lib.zc_prefill_compress(h, fake, fake, fake, 64, ks, ks, pp, 2, None, fake, 16, None) == -2
    finally:
        lib.zc_cache_free(h)
    for code, word in [(0, "ok"), (-1, "invalid"), (-2, "capacity"), (-3, "order"), (-4, "aligned"),
                       (-6, "built-in buffer"), (-99, "unknown")]:
        assert word in zc.zc_strerror(code)


def test_missing_library_fails_loudly(zc, tmp_path):
    with pytest.raises(zc.ZipCacheError, match="no CPU or PyTorch fallback"):
        zc.load_library(str(tmp_path / "libzipcache.so"))
    zc.load_library()
