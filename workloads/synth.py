"""Seeded synthetic Q/K/V with the value structure of LLM attention layers.

Stand-in for the LLaMA / Mistral workloads the paper evaluates on (shapes and
value structure only): Gaussian states, a few outlier key channels per KV head,
a "sink" first token whose key is aligned with the mean query direction, and
optionally a band of heavy columns.  Values are built in fp32 and cast to the
storage dtype last; the cast values are the ground truth for every consumer.

Nothing here performs any of the method's arithmetic.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Iterator, List, Tuple

import numpy as np
import torch

MU = 4.0  # length of the mean-query offset added to every query


@dataclass(frozen=True)
class Workload:
    name: str
    cfg_id: int
    dtype: str            # "fp16" | "bf16"
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    context: int          # prefill length l
    n_layers: int
    saliency_ratio: float
    bits_hi: int
    bits_lo: int
    rho_recent: float
    rho_random: float
    window: int
    decode_steps: int
    outlier_fixed: int    # >0: exactly this many outlier channels, x15
    band: int             # number of extra heavy columns (0 = none)
    k_scheme: str = "cst"  # "cst": CSTQuant for keys and values; "channel": channelwise keys

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float16 if self.dtype == "fp16" else torch.bfloat16

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def units_per_layer(self) -> int:
        return self.batch * self.n_kv_heads

    def seed(self, layer: int = 0) -> int:
        return 0x5A1F + 1000 * self.cfg_id + layer

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


def _w(name, cfg_id, dtype, b, hq, hkv, l, layers, r, steps, fixed=0, band=0):
    return Workload(name, cfg_id, dtype, b, hq, hkv, 128, l, layers, r, 4, 2,
                    0.05, 0.05, 100, steps, fixed, band)


CONFIGS = {
    1: _w("tiny-mha-512", 1, "fp16", 1, 4, 4, 512, 1, 0.4, 16, fixed=4),
    2: _w("llama3-8b-layer-b8-l4096", 2, "bf16", 8, 32, 8, 4096, 1, 0.4, 128),
    3: _w("mistral-7b-layer-b16-l8192", 3, "fp16", 16, 32, 8, 8192, 1, 0.3, 256, band=20),
    4: _w("llama2-7b-layer-b32-l4096", 4, "fp16", 32, 32, 32, 4096, 1, 0.4, 128),
    5: _w("llama3-8b-32layers-b4-l32768", 5, "bf16", 4, 32, 8, 32768, 32, 0.4, 64),
}


def get_config(cfg_id: int) -> Workload:
    return CONFIGS[cfg_id]


def splitmix64_stream(seed: int) -> Iterator[int]:
    """Plain splitmix64 output stream (a public-domain mixing generator)."""
    mask = (1 << 64) - 1
    state = seed & mask
    while True:
        state = (state + 0x9E3779B97F4A7C15) & mask
        z = state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & mask
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & mask
        yield z ^ (z >> 31)


def decode_probe_flags(w: Workload, layer: int, n_steps: int) -> List[bool]:
    """One coin flip per decode step: True with probability 5 % (the random
    part of the decode-phase probe choice); drawn once, fed to every consumer."""
    gen = splitmix64_stream(w.seed(layer) ^ 0xD3C0DE)
    return [(next(gen) % 100) < 5 for _ in range(n_steps)]


def _head_structure(w: Workload, layer: int):
    """Per-KV-head small draws: mean query direction, outlier channels and their
    gains, heavy-band positions.  Always drawn on the host so that they do not
    depend on the device the big tensors are generated on."""
    rs = np.random.RandomState(w.seed(layer) % (2 ** 31))
    d = w.head_dim
    u = rs.standard_normal((w.n_kv_heads, d))
    u /= np.linalg.norm(u, axis=1, keepdims=True)
    gains = np.ones((w.n_kv_heads, d), dtype=np.float64)
    for kv in range(w.n_kv_heads):
        if w.outlier_fixed > 0:
            ch = rs.choice(d, size=w.outlier_fixed, replace=False)
            gains[kv, ch] = 15.0
        else:
            n_out = int(rs.randint(2, 7))
            ch = rs.choice(d, size=n_out, replace=False)
            gains[kv, ch] = rs.uniform(10.0, 20.0, size=n_out)
    band_pos = None
    if w.band > 0:
        band_pos = np.sort(rs.choice(np.arange(1, w.context), size=min(w.band, w.context - 1),
                                     replace=False))
    return u, gains, band_pos


def make_prefill(w: Workload, layer: int = 0, device: str = "cpu"
                 ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """Q [b,h_q,l,d], K and V [b,h_kv,l,d] in the workload's storage dtype."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed(w.seed(layer))
    u_np, gains_np, band_pos = _head_structure(w, layer)
    u = torch.tensor(u_np, dtype=torch.float32, device=dev)            # [h_kv, d]
    gains = torch.tensor(gains_np, dtype=torch.float32, device=dev)    # [h_kv, d]
    b, hq, hkv, l, d = w.batch, w.n_q_heads, w.n_kv_heads, w.context, w.head_dim
    dt = w.torch_dtype
    Q = torch.empty((b, hq, l, d), dtype=dt, device=dev)
    K = torch.empty((b, hkv, l, d), dtype=dt, device=dev)
    V = torch.empty((b, hkv, l, d), dtype=dt, device=dev)
    u_q = u.repeat_interleave(w.group, dim=0)                           # [h_q, d]
    sink = (6.0 * np.sqrt(d) / MU) * u                                  # [h_kv, d]
    for bi in range(b):
        q = torch.randn((hq, l, d), generator=g, device=dev, dtype=torch.float32)
        q += MU * u_q[:, None, :]
        Q[bi] = q.to(dt)
        del q
        k = torch.randn((hkv, l, d), generator=g, device=dev, dtype=torch.float32)
        k *= gains[:, None, :]
        k[:, 0, :] = sink
        if band_pos is not None:
            pos = torch.tensor(band_pos, device=dev, dtype=torch.long)
            noise = torch.randn((hkv, len(band_pos), d), generator=g, device=dev,
                                dtype=torch.float32)
            k[:, pos, :] = (3.0 * np.sqrt(d) / MU) * u[:, None, :] + 0.1 * noise
        K[bi] = k.to(dt)
        del k
        v = torch.randn((hkv, l, d), generator=g, device=dev, dtype=torch.float32)
        V[bi] = v.to(dt)
        del v
    return Q, K, V


def make_decode_step(w: Workload, layer: int, step: int, device: str = "cpu"
                     ) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """Fresh N(0,1) q [b,h_q,d], k and v [b,h_kv,d] for one decode step."""
    dev = torch.device(device)
    g = torch.Generator(device=dev)
    g.manual_seed((w.seed(layer) * 7919 + 104729 * (step + 1)) % (2 ** 63))
    dt = w.torch_dtype
    q = torch.randn((w.batch, w.n_q_heads, w.head_dim), generator=g, device=dev,
                    dtype=torch.float32).to(dt)
    k = torch.randn((w.batch, w.n_kv_heads, w.head_dim), generator=g, device=dev,
                    dtype=torch.float32).to(dt)
    v = torch.randn((w.batch, w.n_kv_heads, w.head_dim), generator=g, device=dev,
                    dtype=torch.float32).to(dt)
    return q, k, v
