"""B200 (sm_100a) quantize-and-attend library for a mixed-precision KV cache.

The compute lives in ``libzipcache.so`` (hand-written CUDA, C ABI declared in
``include/zipcache.h``); this package is the ctypes binding plus a small
convenience class that lets PyTorch own the device memory and the stream.
There is no CPU path: importing works anywhere, calling needs the library
and a CUDA device.
"""
from .binding import (  # noqa: F401
    ZC_F16, ZC_BF16, ZC_FLAG_DEFER_APPEND, ZC_FLAG_OVERLAP_CALLS, ZC_FLAG_OUT_F32, ZC_FLAG_PARAMS_F16, ZC_FLAG_GROUP_ALL_HEADS, ZC_K_CST, ZC_K_CHANNEL, ZC_SCOPE_KV_HEAD, ZC_SCOPE_TOKEN, ZcConfig, ZipCacheError, lib, load_library,
    zc_cache_bytes, zc_cache_init, zc_cache_free, zc_probe_count, zc_default_probes,
    zc_prefill_compress, zc_prefill_attention, zc_prefill_compress_lse, zc_append, zc_decode_attention, zc_decode_attention_noalloc,
    zc_export_scores,
    zc_export_segment, zc_segment_tokens, zc_num_segments, zc_tail_tokens,
    zc_decode_bytes, zc_launch_count, zc_strerror, zc_device_status, ZipCache,
    zc_order_model_reset, zc_order_model_call,
)
