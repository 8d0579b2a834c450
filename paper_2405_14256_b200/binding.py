"""ctypes binding of libzipcache.so: the same names as the C ABI, argument
marshalling only.  Every step of the path runs in the library's kernels."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libzipcache.so")

ZC_F16, ZC_BF16 = 0, 1
ZC_FLAG_DEFER_APPEND = 1
ZC_FLAG_OVERLAP_CALLS = 2
ZC_FLAG_OUT_F32 = 4
ZC_FLAG_PARAMS_F16 = 8
ZC_FLAG_GROUP_ALL_HEADS = 16
ZC_K_CST, ZC_K_CHANNEL = 0, 1
ZC_SCOPE_KV_HEAD, ZC_SCOPE_TOKEN = 0, 1


class ZipCacheError(RuntimeError):
    pass


class ZcConfig(C.Structure):
    _fields_ = [
        ("struct_size", C.c_int32), ("dtype", C.c_int32), ("batch", C.c_int32),
        ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("max_prefill", C.c_int32), ("max_new_tokens", C.c_int32), ("window", C.c_int32),
        ("bits_hi", C.c_int32), ("bits_lo", C.c_int32), ("flags", C.c_int32),
        ("saliency_ratio", C.c_double), ("k_scheme", C.c_int32), ("scope", C.c_int32),
    ]

    @classmethod
    def make(cls, dtype, batch, n_q_heads, n_kv_heads, max_prefill, max_new_tokens,
             saliency_ratio, bits_hi=4, bits_lo=2, window=100, head_dim=128,
             flags=0, k_scheme=0, scope=0) -> "ZcConfig":
        code = {torch.float16: ZC_F16, torch.bfloat16: ZC_BF16}.get(dtype, dtype)
        return cls(C.sizeof(cls), code, batch, n_q_heads, n_kv_heads, head_dim, max_prefill,
                   max_new_tokens, window, bits_hi, bits_lo, flags, float(saliency_ratio),
                   int(k_scheme), int(scope))


_lib = None

_SIGS = {
    "zc_cache_bytes": (C.c_int, [C.POINTER(ZcConfig), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "zc_cache_init": (C.c_int, [C.c_void_p, C.c_size_t, C.POINTER(ZcConfig), C.POINTER(C.c_void_p)]),
    "zc_cache_free": (None, [C.c_void_p]),
    "zc_probe_count": (C.c_int, [C.c_int, C.c_double, C.c_double]),
    "zc_default_probes": (C.c_int, [C.c_int, C.c_double, C.c_double, C.c_uint64,
                                    C.POINTER(C.c_int32), C.POINTER(C.c_int)]),
    "zc_prefill_compress": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                      C.POINTER(C.c_int64), C.POINTER(C.c_int64),
                                      C.POINTER(C.c_int32), C.c_int, C.c_void_p, C.c_void_p,
                                      C.c_size_t, C.c_void_p]),
    "zc_prefill_attention": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                       C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.c_void_p, C.c_void_p,
                                       C.c_void_p]),
    "zc_prefill_compress_lse": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                          C.POINTER(C.c_int64), C.POINTER(C.c_int64),
                                          C.POINTER(C.c_int32), C.c_int, C.c_void_p, C.c_void_p,
                                          C.c_size_t, C.c_void_p]),
    "zc_append": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "zc_decode_attention": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p,
                                      C.c_size_t, C.c_void_p]),
    "zc_decode_attention_noalloc": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]),
    "zc_export_scores": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p]),
    "zc_segment_tokens": (C.c_int, [C.c_void_p, C.c_int, C.c_int]),
    "zc_num_segments": (C.c_int, [C.c_void_p]),
    "zc_tail_tokens": (C.c_int, [C.c_void_p]),
    "zc_export_segment": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                    C.c_void_p, C.c_void_p, C.c_void_p]),
    "zc_decode_bytes": (C.c_int64, [C.c_void_p]),
    "zc_launch_count": (C.c_int64, [C.c_void_p]),
    "zc_device_status": (C.c_int, [C.POINTER(C.c_int)]),
    "zc_order_model_reset": (None, []),
    "zc_order_model_call": (C.c_int, [C.c_uint64, C.c_int, C.POINTER(C.c_uint64), C.c_uint64, C.c_uint64,
                                      C.c_int, C.c_uint64, C.c_uint64, C.c_uint64, C.c_uint64,
                                      C.POINTER(C.c_int)]),
    "zc_strerror": (C.c_char_p, [C.c_int]),
}


def load_library(path: Optional[str] = None):
    """Load libzipcache.so and declare its signatures.  Fails loudly when the
    library has not been built: there is no fallback path."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise ZipCacheError(
            f"{p} is missing: build it with `python -m paper_2405_14256_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    lib_ = C.CDLL(p)
    for name, (res, args) in _SIGS.items():
        fn = getattr(lib_, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib_
    return lib_


def lib():
    return load_library()


def _check(rc: int, what: str) -> int:
    if rc < 0:
        raise ZipCacheError(f"{what}: {zc_strerror(rc)} ({rc})")
    return rc


def _ptr(t) -> int:
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def zc_strerror(status: int) -> str:
    return lib().zc_strerror(status).decode()


def zc_cache_bytes(cfg: ZcConfig):
    cb, wb = C.c_size_t(0), C.c_size_t(0)
    _check(lib().zc_cache_bytes(C.byref(cfg), C.byref(cb), C.byref(wb)), "zc_cache_bytes")
    return cb.value, wb.value


def zc_cache_init(dev_mem, nbytes: int, cfg: ZcConfig) -> int:
    h = C.c_void_p(0)
    _check(lib().zc_cache_init(_ptr(dev_mem), nbytes, C.byref(cfg), C.byref(h)), "zc_cache_init")
    return h.value


def zc_cache_free(handle: int) -> None:
    lib().zc_cache_free(handle)


def zc_probe_count(l: int, rho_recent: float, rho_random: float) -> int:
    return _check(lib().zc_probe_count(l, rho_recent, rho_random), "zc_probe_count")


def zc_default_probes(l: int, rho_recent: float, rho_random: float, seed: int):
    n = zc_probe_count(l, rho_recent, rho_random)
    buf = (C.c_int32 * n)()
    n_out = C.c_int(0)
    _check(lib().zc_default_probes(l, rho_recent, rho_random, seed, buf, C.byref(n_out)),
           "zc_default_probes")
    return list(buf[: n_out.value])


def zc_prefill_compress(handle, Q, K, V, l: int, probe_pos: Optional[Sequence[int]],
                        salient_idx=None, workspace=None, stream=None) -> None:
    qs = (C.c_int64 * 3)(*(Q.stride()[:3] if Q is not None else (0, 0, 0)))
    ks = (C.c_int64 * 3)(*K.stride()[:3])
    if K.stride() != V.stride():
        raise ZipCacheError("K and V must share strides")
    n_probe = 0 if probe_pos is None else len(probe_pos)
    pp = (C.c_int32 * max(1, n_probe))(*(probe_pos if probe_pos is not None else [0]))
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().zc_prefill_compress(handle, _ptr(Q), _ptr(K), _ptr(V), l, qs, ks, pp, n_probe,
                                     _ptr(salient_idx), _ptr(workspace), ws_bytes,
                                     _stream(stream)), "zc_prefill_compress")


def zc_prefill_attention(handle, Q, K, V, l: int, O, row_lse, stream=None) -> None:
    qs = (C.c_int64 * 3)(*Q.stride()[:3])
    ks = (C.c_int64 * 3)(*K.stride()[:3])
    if K.stride() != V.stride():
        raise ZipCacheError("K and V must share strides")
    _check(lib().zc_prefill_attention(handle, _ptr(Q), _ptr(K), _ptr(V), l, qs, ks, _ptr(O), _ptr(row_lse),
                                      _stream(stream)), "zc_prefill_attention")


def zc_prefill_compress_lse(handle, Q, K, V, l: int, probe_pos: Sequence[int], row_lse, workspace,
                            stream=None) -> None:
    qs = (C.c_int64 * 3)(*Q.stride()[:3])
    ks = (C.c_int64 * 3)(*K.stride()[:3])
    if K.stride() != V.stride():
        raise ZipCacheError("K and V must share strides")
    pp = (C.c_int32 * max(1, len(probe_pos)))(*probe_pos)
    ws_bytes = workspace.numel() * workspace.element_size()
    _check(lib().zc_prefill_compress_lse(handle, _ptr(Q), _ptr(K), _ptr(V), l, qs, ks, pp, len(probe_pos),
                                         _ptr(row_lse), _ptr(workspace), ws_bytes, _stream(stream)),
           "zc_prefill_compress_lse")


def zc_append(handle, k_new, v_new, stream=None) -> None:
    _check(lib().zc_append(handle, _ptr(k_new), _ptr(v_new), _stream(stream)), "zc_append")


def zc_decode_attention(handle, q, out, is_probe_step: bool, workspace, stream=None) -> None:
    ws_bytes = workspace.numel() * workspace.element_size()
    _check(lib().zc_decode_attention(handle, _ptr(q), _ptr(out), int(bool(is_probe_step)),
                                     _ptr(workspace), ws_bytes, _stream(stream)),
           "zc_decode_attention")


def zc_decode_attention_noalloc(handle, q, out, is_probe_step: bool, stream=None) -> None:
    """zc_decode_attention with the library's built-in scratch buffer instead of a caller
    workspace (for callers that cannot allocate device memory)."""
    _check(lib().zc_decode_attention_noalloc(handle, _ptr(q), _ptr(out), int(bool(is_probe_step)),
                                             _stream(stream)), "zc_decode_attention_noalloc")


def zc_export_scores(handle, p_tilde, stream=None) -> None:
    _check(lib().zc_export_scores(handle, _ptr(p_tilde), _stream(stream)), "zc_export_scores")


def zc_segment_tokens(handle, segment: int, subset: int) -> int:
    return _check(lib().zc_segment_tokens(handle, segment, subset), "zc_segment_tokens")


def zc_num_segments(handle) -> int:
    return _check(lib().zc_num_segments(handle), "zc_num_segments")


def zc_tail_tokens(handle) -> int:
    return _check(lib().zc_tail_tokens(handle), "zc_tail_tokens")


def zc_export_segment(handle, segment, tensor, subset, idx=None, codes=None, sz=None, cf=None,
                      stream=None) -> None:
    _check(lib().zc_export_segment(handle, segment, tensor, subset, _ptr(idx), _ptr(codes),
                                   _ptr(sz), _ptr(cf), _stream(stream)), "zc_export_segment")


def zc_decode_bytes(handle) -> int:
    return lib().zc_decode_bytes(handle)


def zc_launch_count(handle) -> int:
    return lib().zc_launch_count(handle)


def zc_device_status() -> int:
    code = C.c_int(0)
    _check(lib().zc_device_status(C.byref(code)), "zc_device_status")
    return code.value


ORDER_FIELDS = ("epoch_start", "e", "need_start", "need_end", "slot", "tag", "record", "drain")


def zc_order_model_reset() -> None:
    lib().zc_order_model_reset()


def zc_order_model_call(stream_id, cache_id, q, k_new, v_new, out, io_bytes, kv_bytes, collect,
                        ws_addr, ws_bytes, need, capture_id=0) -> dict:
    """Books one call in the host-only model of the call ordering; addresses are integers."""
    addr = (C.c_uint64 * 4)(q, k_new, v_new, out)
    res = (C.c_int * 8)()
    _check(lib().zc_order_model_call(stream_id, cache_id, addr, io_bytes, kv_bytes, int(collect),
                                     ws_addr, ws_bytes, need, capture_id, res), "zc_order_model_call")
    return dict(zip(ORDER_FIELDS, list(res)))


class ZipCache:
    """Owns the device buffers (allocated by PyTorch) of one attention layer's cache and
    forwards to the C ABI.  Marshalling and allocation only."""

    def __init__(self, dtype, batch, n_q_heads, n_kv_heads, max_prefill, max_new_tokens,
                 saliency_ratio, bits_hi=4, bits_lo=2, window=100, device="cuda:0",
                 workspace: Optional[torch.Tensor] = None, defer_append: bool = False,
                 overlap_calls: bool = False, out_f32: bool = False, k_channel: bool = False,
                 guard_bytes: int = 0, token_scope: bool = False, params_f16: bool = False,
                 group_all_heads: bool = False):
        if not torch.cuda.is_available():
            raise ZipCacheError("a CUDA device is required (no CPU fallback)")
        self.cfg = ZcConfig.make(dtype, batch, n_q_heads, n_kv_heads, max_prefill, max_new_tokens,
                                 saliency_ratio, bits_hi, bits_lo, window,
                                 flags=(ZC_FLAG_DEFER_APPEND if defer_append else 0) |
                                 (ZC_FLAG_OVERLAP_CALLS if overlap_calls else 0) |
                                 (ZC_FLAG_OUT_F32 if out_f32 else 0) |
                                 (ZC_FLAG_PARAMS_F16 if params_f16 else 0) |
                                 (ZC_FLAG_GROUP_ALL_HEADS if group_all_heads else 0),
                                 k_scheme=ZC_K_CHANNEL if k_channel else ZC_K_CST,
                                 scope=ZC_SCOPE_TOKEN if token_scope else ZC_SCOPE_KV_HEAD)
        self.k_channel = bool(k_channel)
        self.out_dtype = torch.float32 if out_f32 else dtype
        self.dtype, self.device = dtype, torch.device(device)
        self.batch, self.n_q_heads, self.n_kv_heads = batch, n_q_heads, n_kv_heads
        self.cache_bytes, self.workspace_bytes = zc_cache_bytes(self.cfg)
        # guard_bytes > 0 (a multiple of 256): the cache buffer and a workspace allocated here sit
        # between two bands filled with 0xA5, which check_guards() verifies (a debugging aid:
        # a kernel that writes outside its buffers shows up there)
        self.guard_bytes = int(guard_bytes)
        g = self.guard_bytes
        self._mem_all = torch.full((self.cache_bytes + 2 * g,), 0xA5, dtype=torch.uint8, device=self.device) \
            if g else torch.empty(self.cache_bytes, dtype=torch.uint8, device=self.device)
        self.mem = self._mem_all[g:g + self.cache_bytes]
        self._ws_all = None
        if workspace is None:
            self._ws_all = torch.full((self.workspace_bytes + 2 * g,), 0xA5, dtype=torch.uint8, device=self.device) \
                if g else torch.empty(self.workspace_bytes, dtype=torch.uint8, device=self.device)
            workspace = self._ws_all[g:g + self.workspace_bytes]
        self.workspace = workspace
        if self.workspace.numel() * self.workspace.element_size() < self.workspace_bytes:
            raise ZipCacheError("shared workspace too small")
        self.handle = zc_cache_init(self.mem, self.cache_bytes, self.cfg)

    def check_guards(self) -> bool:
        """True when the guard bands around the cache buffer (and the workspace, if this object
        allocated it) still hold their fill pattern."""
        g = self.guard_bytes
        if not g:
            return True
        ok = True
        for buf in (self._mem_all, self._ws_all):
            if buf is not None:
                ok = ok and bool((buf[:g] == 0xA5).all()) and bool((buf[-g:] == 0xA5).all())
        return ok

    def close(self):
        if getattr(self, "handle", None):
            zc_cache_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def prefill_compress(self, Q, K, V, probe_pos=None, salient_idx=None, stream=None):
        zc_prefill_compress(self.handle, Q, K, V, K.shape[2], probe_pos, salient_idx,
                            self.workspace, stream)

    def prefill_attention(self, Q, K, V, stream=None):
        """Causal attention output O and the rows' log-sum-exp (Alg. 2's attention-output line)."""
        l = K.shape[2]
        O = torch.empty((self.batch, self.n_q_heads, l, 128), dtype=self.dtype, device=self.device)
        lse = torch.empty((self.batch, self.n_q_heads, l), dtype=torch.float32, device=self.device)
        zc_prefill_attention(self.handle, Q, K, V, l, O, lse, stream)
        return O, lse

    def prefill_compress_lse(self, Q, K, V, probe_pos, row_lse, stream=None):
        zc_prefill_compress_lse(self.handle, Q, K, V, K.shape[2], probe_pos, row_lse, self.workspace, stream)

    def append(self, k_new, v_new, stream=None):
        zc_append(self.handle, k_new, v_new, stream)

    def decode_attention(self, q, is_probe_step=False, out=None, stream=None):
        if out is None:
            out = torch.empty(q.shape, dtype=self.out_dtype, device=q.device)
        zc_decode_attention(self.handle, q, out, is_probe_step, self.workspace, stream)
        return out

    # ---- exports (canonical layouts) ----
    def scores(self, n: int):
        out = torch.empty((self.batch, self.n_kv_heads, n), dtype=torch.float32, device=self.device)
        zc_export_scores(self.handle, out)
        return out

    def segment(self, segment: int, tensor: int, subset: int):
        n = zc_segment_tokens(self.handle, segment, subset)
        bits = self.cfg.bits_hi if subset == 0 else self.cfg.bits_lo
        b, h = self.batch, self.n_kv_heads
        dev = self.device
        idx = torch.zeros((b, h, n), dtype=torch.int32, device=dev)
        codes = torch.zeros((b, h, n, 16 * bits), dtype=torch.uint8, device=dev)
        # channelwise keys: (scale, zero point) per channel instead of per token
        sz = torch.zeros((b, h, 128 if (self.k_channel and tensor == 0) else n, 2), dtype=torch.float32,
                         device=dev)
        cf = torch.zeros((b, h, 128), dtype=torch.float32, device=dev)
        if n > 0:
            zc_export_segment(self.handle, segment, tensor, subset, idx, codes, sz, cf)
        return idx, codes, sz, cf
