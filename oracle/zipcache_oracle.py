"""CPU oracle for the ZipCache quantize-and-attend path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, step-by-step restatement of what the paper defines, in NumPy.
It shares no code with the CUDA library and must never be imported by the
product path: only the tests, the smoke check and the benchmark's CPU-baseline
leg may use it.

Arithmetic: everything is fp64 on inputs widened exactly from fp16/bf16, except
the quantiser (CSTQuant), which follows one fixed fp32 sequence with
round-to-nearest-even and no fused operations so that integer codes can be
compared bit for bit.

Passages followed (paper section / equation / algorithm):
  probe selection ............ Sec. 4.3 "random+recent" strategy, Alg. 2 line 1
  probe attention ............ Eq. 9 (with the causal mask of Eq. 2 / Sec. 4.2)
  prefill attention output ... Eq. 2, Alg. 2 "O = FlashAttention(Q, K, V)" (causal), with the
                               row log-sum-exp a fast-attention kernel keeps beside it
  accumulated score .......... Eq. 7
  normalised score ........... Eq. 8
  split by saliency ratio .... Alg. 2 "Split"
  uniform quantisation ....... Eq. 5 (dequantisation subtracts the zero point)
  channel normalisation ...... Eq. 6
  CSTQuant ................... Alg. 1
  ChannelQuant (keys) ........ Sec. 4.1 last paragraph, Table 1 last row, Alg. 2
  16-bit quantisation params . Appendix A (parameters counted at 16 bits)
  token-level saliency ....... Sec. 4.2 / Alg. 2 read literally: one score per token
  decode concat / attention .. Eq. 3, Eq. 4, Alg. 3
  streaming re-compression ... Alg. 3 (every `window` = 100 generated tokens)
  overhead accounting ........ Appendix A, Eq. (A)-(C)

Pins (see tests/test_oracle_pins.py): brute-force l x l causal attention, the
Q = 0 harmonic-number closed form, row-sum invariants, the half-step bound,
textbook per-row affine quantisation when all channel factors are 1, exact
attention at 16 bits, permutation and split invariance, Appendix A's printed
ratios.  Conventions that no printed value or closed form fixes are marked
"parity unpinned" where they are made:
  * GQA aggregation of Eq. 8 over the query heads of one KV head and the
    splitmix64 probe sampler                       -- parity unpinned
  * floor() rounding of the salient / probe counts -- parity unpinned
  * integer zero point (vs. a float offset)         -- parity unpinned
  * streaming-flush semantics (which 100 tokens, the 100th step being a probe
    step)                                           -- parity unpinned
  * rounding of 16-bit scales (up, so that the half-step bound survives) and the
    scope of channelwise parameters (per batch, KV head and subset) -- parity unpinned
  * token-level saliency as the mean of the per-KV-head scores     -- parity unpinned
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

_M64 = (1 << 64) - 1


# --------------------------------------------------------------------------
# Probe selection (Sec. 4.3, "random+recent tokens")
# --------------------------------------------------------------------------
def _splitmix64(seed: int):
    state = seed & _M64
    while True:
        state = (state + 0x9E3779B97F4A7C15) & _M64
        z = state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
        yield z ^ (z >> 31)


def probe_counts(l: int, rho_recent: float, rho_random: float) -> Tuple[int, int]:
    """(n_recent, n_random): floor of ratio*l in double; at least one recent
    probe so that the last token is always a probe.  parity unpinned (rounding)."""
    n_rec = min(l, max(1, int(math.floor(rho_recent * l))))
    n_rnd = min(l - n_rec, int(math.floor(rho_random * l)))
    return n_rec, n_rnd


def probe_positions(l: int, rho_recent: float, rho_random: float, seed: int) -> np.ndarray:
    """Ascending probe positions: the last n_recent tokens plus n_random tokens
    drawn without replacement from the rest by a partial Fisher-Yates shuffle
    driven by splitmix64(seed).  parity unpinned (sampler is a convention)."""
    n_rec, n_rnd = probe_counts(l, rho_recent, rho_random)
    pool = l - n_rec
    perm = list(range(pool))
    gen = _splitmix64(seed)
    for i in range(n_rnd):
        j = i + next(gen) % (pool - i)
        perm[i], perm[j] = perm[j], perm[i]
    chosen = sorted(perm[:n_rnd])
    return np.asarray(chosen + list(range(pool, l)), dtype=np.int32)


# --------------------------------------------------------------------------
# Saliency (Eq. 7, 8, 9)
# --------------------------------------------------------------------------
def probe_attention(Qp: np.ndarray, K: np.ndarray, P: Sequence[int]) -> np.ndarray:
    """Eq. 9 for one head: rows of Softmax(Q_probe K^T / sqrt(d_k)) under the
    causal mask (row of position p sees columns j <= p).  Qp [n_p,d], K [l,d]."""
    Qp = np.asarray(Qp, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    l, d = K.shape
    S = (Qp @ K.T) / math.sqrt(d)
    A = np.zeros_like(S)
    for r, p in enumerate(P):
        row = S[r, : p + 1]
        e = np.exp(row - row.max())
        A[r, : p + 1] = e / e.sum()
    return A


def prefill_attention(Q: np.ndarray, K: np.ndarray, V: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 2 for one head under the causal mask: O = Softmax(Q K^T / sqrt(d_k)) V with row i
    seeing columns j <= i (Alg. 2's attention-output line).  Also returns, per row, the
    base-2 log-sum-exp of its scaled logits, log2(sum_j 2^(s_ij log2 e)) -- the one number per
    row from which any entry of the row's softmax can be rebuilt (Eq. 9's rows included).
    Q, K, V [l, d]."""
    Q = np.asarray(Q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    l, d = K.shape
    S = (Q @ K.T) / math.sqrt(d)
    O = np.zeros((l, V.shape[1]))
    lse2 = np.zeros(l)
    for i in range(l):
        row = S[i, : i + 1]
        mx = row.max()
        e = np.exp(row - mx)
        O[i] = (e / e.sum()) @ V[: i + 1]
        lse2[i] = (mx + math.log(e.sum())) / math.log(2.0)
    return O, lse2


def accumulated_scores(A_list: Sequence[np.ndarray]) -> np.ndarray:
    """Eq. 7: column sums of the attention matrix (summed over the given heads)."""
    return sum(A.sum(axis=0) for A in A_list)


def structural_nnz(P: Sequence[int], l: int) -> np.ndarray:
    """Number of probe rows whose causal span contains column j: #{r : p_r >= j}."""
    P = np.asarray(P)
    return np.asarray([(P >= j).sum() for j in range(l)], dtype=np.int64)


def normalized_scores(Q_heads: np.ndarray, K: np.ndarray, P: Sequence[int]) -> np.ndarray:
    """Eq. 8 with A replaced by A_probe (Eq. 9), for one KV head.

    Q_heads [G,l,d] are the G query heads that read this KV head (GQA: their
    column sums are added and the count is G * nnz; reduces to Eq. 8 when G=1).
    """
    Q_heads = np.asarray(Q_heads, dtype=np.float64)
    l = K.shape[0]
    G = Q_heads.shape[0]
    P = np.asarray(P, dtype=np.int64)
    if len(P) == 0 or P[-1] != l - 1:
        raise ValueError("probe list must end at the last token")
    col = accumulated_scores([probe_attention(Q_heads[g][P], K, P) for g in range(G)])
    return col / (G * structural_nnz(P, l))


def split_salient(p_tilde: np.ndarray, n_s: int) -> Tuple[np.ndarray, np.ndarray]:
    """Alg. 2 Split: the n_s tokens with the largest score are salient (ties go
    to the lower index); both index lists are returned ascending."""
    order = np.argsort(-np.asarray(p_tilde, dtype=np.float64), kind="stable")
    sal = np.sort(order[:n_s]).astype(np.int32)
    reg = np.sort(order[n_s:]).astype(np.int32)
    return sal, reg


def salient_count(ratio: float, n: int) -> int:
    """floor(ratio * n) in double.  parity unpinned (rounding convention)."""
    return int(math.floor(ratio * n))


# --------------------------------------------------------------------------
# CSTQuant (Alg. 1, Eq. 5, Eq. 6) -- normative fp32 sequence
# --------------------------------------------------------------------------
def cst_quant(X: np.ndarray, bits: int) -> Dict[str, np.ndarray]:
    """Channel-separable tokenwise quantisation of X [n_tokens, d] to `bits`.

    Every operation below is a single IEEE fp32 operation rounded to nearest
    even; nothing is fused.  Returns c [d], s [n], z [n] (integer-valued fp32)
    and codes [n,d] (uint8, 0..2^bits-1).
    """
    f32 = np.float32
    X = np.asarray(X, dtype=f32)
    n, d = X.shape
    L = f32((1 << bits) - 1)
    # Eq. 6: c_i = sqrt(max |X_i|) over the tokens of this subset; all-zero channel -> 1
    m = np.abs(X).max(axis=0) if n > 0 else np.zeros(d, dtype=f32)
    c = np.sqrt(m, dtype=f32)
    c = np.where(m == f32(0), f32(1), c).astype(f32)
    # Alg. 1: normalise each channel
    Y = (X / c[None, :]).astype(f32)
    # TokenQuant = Eq. 5 with min/max over one token's channels
    mn = Y.min(axis=1) if n > 0 else np.zeros(0, dtype=f32)
    mx = Y.max(axis=1) if n > 0 else np.zeros(0, dtype=f32)
    s = ((mx - mn).astype(f32) / L).astype(f32)
    flat = mx == mn
    s = np.where(flat, np.where(mn != f32(0), np.abs(mn), f32(1)), s).astype(f32)
    z = (-np.rint((mn / s).astype(f32))).astype(f32)
    q = (np.rint((Y / s[:, None]).astype(f32)).astype(f32) + z[:, None]).astype(f32)
    codes = np.minimum(np.maximum(q, f32(0)), L).astype(np.uint8)
    return {"c": c, "s": s, "z": z, "codes": codes, "bits": bits, "pre_round": (Y / s[:, None]).astype(f32)}


def cst_dequant(qd: Dict[str, np.ndarray]) -> np.ndarray:
    """x_hat = c * ((code - z) * s) in fp64 (Eq. 5 read with the zero point
    subtracted, then Alg. 1's rescale)."""
    c = qd["c"].astype(np.float64)
    s = qd["s"].astype(np.float64)
    z = qd["z"].astype(np.float64)
    codes = qd["codes"].astype(np.float64)
    return c[None, :] * ((codes - z[:, None]) * s[:, None])


def token_quant_reference_fp64(Y: np.ndarray, bits: int) -> np.ndarray:
    """Eq. 5 per row in fp64 (used only to cross-check fp32 codes away from
    rounding boundaries).  Returns the pre-clipping real value y/s + z."""
    Y = np.asarray(Y, dtype=np.float64)
    L = (1 << bits) - 1
    mn = Y.min(axis=1)
    mx = Y.max(axis=1)
    s = (mx - mn) / L
    flat = mx == mn
    s = np.where(flat, np.where(mn != 0, np.abs(mn), 1.0), s)
    z = -np.rint(mn / s)
    return Y / s[:, None] + z[:, None]


# --------------------------------------------------------------------------
# ChannelQuant (Sec. 4.1: channelwise quantisation, the paper's choice for keys)
# --------------------------------------------------------------------------
def channel_quant(X: np.ndarray, bits: int) -> Dict[str, np.ndarray]:
    """Channelwise uniform quantisation of X [n_tokens, d] to `bits`: Eq. 5 with the minimum
    and maximum taken over the tokens of one channel, so that there is one (s, z) pair per
    channel (2 h d parameters per tensor, Table 1) and none per token.

    Normative fp32 sequence, one IEEE operation per step, round to nearest even:
    mn_i, mx_i over the tokens; s_i = (mx_i - mn_i) / L, or |mn_i| (1 if 0) for a constant
    channel; z_i = -rint(mn_i / s_i); code = clamp(rint(x / s_i) + z_i, 0, L)."""
    f32 = np.float32
    X = np.asarray(X, dtype=f32)
    n, d = X.shape
    L = f32((1 << bits) - 1)
    mn = X.min(axis=0) if n > 0 else np.zeros(d, dtype=f32)
    mx = X.max(axis=0) if n > 0 else np.zeros(d, dtype=f32)
    s = ((mx - mn).astype(f32) / L).astype(f32)
    flat = mx == mn
    s = np.where(flat, np.where(mn != f32(0), np.abs(mn), f32(1)), s).astype(f32)
    z = (-np.rint((mn / s).astype(f32))).astype(f32)
    pre = (X / s[None, :]).astype(f32)
    q = (np.rint(pre).astype(f32) + z[None, :]).astype(f32)
    codes = np.minimum(np.maximum(q, f32(0)), L).astype(np.uint8)
    return {"s": s, "z": z, "codes": codes, "bits": bits, "pre_round": pre, "scheme": "channel"}


def channel_dequant(qd: Dict[str, np.ndarray]) -> np.ndarray:
    """x_hat = (code - z_i) * s_i in fp64 (Eq. 5 with the zero point subtracted)."""
    s = qd["s"].astype(np.float64)
    z = qd["z"].astype(np.float64)
    return (qd["codes"].astype(np.float64) - z[None, :]) * s[None, :]


# --------------------------------------------------------------------------
# 16-bit quantisation parameters (Appendix A counts every parameter at 16 bits)
# --------------------------------------------------------------------------
def round_up_to_f16(x: np.ndarray) -> np.ndarray:
    """Smallest fp16 value >= x, element by element (x >= 0, within fp16 range)."""
    x = np.asarray(x, dtype=np.float32)
    h = x.astype(np.float16)
    low = h.astype(np.float32) < x
    return np.where(low, np.nextafter(h, np.float16(np.inf)), h).astype(np.float16)


def cst_quant_f16_params(X: np.ndarray, bits: int) -> Dict[str, np.ndarray]:
    """CSTQuant whose stored parameters fit 16 bits each: the channel factors c and the token
    scales s are fp16 values, the zero points z small integers.

    The scale is rounded UP to fp16 before the codes are formed, so the codes of a token span
    at most the same range as with the fp32 scale and the error bound |y - (code - z) s| <= s/2
    holds for the stored scale (a scale rounded down no longer covers the row: the token's
    maximum then lies beyond the top code).  Everything else follows cst_quant."""
    f32 = np.float32
    X = np.asarray(X, dtype=f32)
    n, d = X.shape
    L = f32((1 << bits) - 1)
    m = np.abs(X).max(axis=0) if n > 0 else np.zeros(d, dtype=f32)
    c = np.sqrt(m, dtype=f32)
    c = np.where(m == f32(0), f32(1), c).astype(f32)
    c = round_up_to_f16(c).astype(f32)                    # stored factor: fp16
    Y = (X / c[None, :]).astype(f32)
    mn = Y.min(axis=1) if n > 0 else np.zeros(0, dtype=f32)
    mx = Y.max(axis=1) if n > 0 else np.zeros(0, dtype=f32)
    s = ((mx - mn).astype(f32) / L).astype(f32)
    flat = mx == mn
    s = np.where(flat, np.where(mn != f32(0), np.abs(mn), f32(1)), s).astype(f32)
    s = round_up_to_f16(s).astype(f32)                    # stored scale: fp16, never below the exact one
    z = (-np.rint((mn / s).astype(f32))).astype(f32)
    pre = (Y / s[:, None]).astype(f32)
    q = (np.rint(pre).astype(f32) + z[:, None]).astype(f32)
    codes = np.minimum(np.maximum(q, f32(0)), L).astype(np.uint8)
    return {"c": c, "s": s, "z": z, "codes": codes, "bits": bits, "pre_round": pre}


def pack_codes(codes: np.ndarray, bits: int) -> np.ndarray:
    """Canonical packing of codes [n,d] -> bytes [n, d*bits/8]: 4-bit element
    2m in the low nibble and 2m+1 in the high nibble of byte m; 2-bit element
    4m+j in bits [2j, 2j+1] of byte m."""
    codes = np.asarray(codes, dtype=np.uint8)
    n, d = codes.shape
    if bits == 4:
        return (codes[:, 0::2] | (codes[:, 1::2] << 4)).astype(np.uint8)
    if bits == 2:
        return (codes[:, 0::4] | (codes[:, 1::4] << 2) | (codes[:, 2::4] << 4)
                | (codes[:, 3::4] << 6)).astype(np.uint8)
    if bits == 8:
        return codes.copy()
    raise ValueError("bits must be 2, 4 or 8")


def unpack_codes(packed: np.ndarray, bits: int, d: int) -> np.ndarray:
    packed = np.asarray(packed, dtype=np.uint8)
    n = packed.shape[0]
    out = np.zeros((n, d), dtype=np.uint8)
    per = 8 // bits
    mask = (1 << bits) - 1
    for j in range(per):
        out[:, j::per] = (packed >> (bits * j)) & mask
    return out


# --------------------------------------------------------------------------
# Appendix A: storage accounting
# --------------------------------------------------------------------------
def quant_param_count(granularity: str, b: int, hd: int, l: int, n: int = 32) -> float:
    """Number of quantisation parameters for ONE tensor X in R^{b x h x l x d}
    (hd = h*d), as counted in Sec. 4.1 and Table 1: tokenwise 2bl, groupwise
    2bhld/n, channelwise 2hd, channel-separable tokenwise hd + 2bl."""
    if granularity == "token":
        return 2 * b * l
    if granularity == "group":
        return 2 * b * hd * l / n
    if granularity == "channel":
        return 2 * hd
    if granularity == "cst":
        return hd + 2 * b * l
    raise ValueError(granularity)


def compression_ratio(k_granularity: str, v_granularity: str, b: int, hd: int, l: int,
                      bits: int = 4, n: int = 32, param_bits: int = 16) -> float:
    """Appendix A, Eq. (A)-(C): bits of the 16-bit K and V over bits of the
    quantised K and V plus their quantisation parameters."""
    full = 2 * b * hd * l * 16
    data = 2 * b * hd * l * bits
    params = (quant_param_count(k_granularity, b, hd, l, n)
              + quant_param_count(v_granularity, b, hd, l, n))
    return full / (data + params * param_bits)


def mixed_precision_ratio(b: int, hd: int, l: int, ratio_salient: float, bits_hi: int, bits_lo: int,
                          k_granularity: str = "channel", v_granularity: str = "cst",
                          param_bits: int = 16, n: int = 32) -> float:
    """Compression ratio of a cache whose salient share is kept at bits_hi and the rest at
    bits_lo, each subset quantised on its own (Alg. 2), in the counting of Appendix A: per-channel
    parameters once per subset (no batch factor), per-token parameters once per token."""
    full = 2 * b * hd * l * 16
    l_hi = ratio_salient * l
    data = 2 * b * hd * (l_hi * bits_hi + (l - l_hi) * bits_lo)
    params = 0.0
    for gran in (k_granularity, v_granularity):
        for l_sub in (l_hi, l - l_hi):
            if l_sub > 0:               # an empty subset stores nothing
                params += quant_param_count(gran, b, hd, l_sub, n)
    return full / (data + params * param_bits)


def cache_footprint_bytes(b: int, h_kv: int, d: int, n_hi: int, n_lo: int, bits_hi: int, bits_lo: int,
                          k_scheme: str = "cst", param_bytes: int = 4) -> int:
    """Bytes of the compressed cache in the granularity this repository stores it in: per
    (batch, KV head) unit and subset, codes of K and V, one (s, z) pair per token for every
    tensor quantised tokenwise, per-channel parameters for every (unit, subset, tensor):
    c for CSTQuant, (s, z) for ChannelQuant."""
    total = 0
    for n_tok, bits in ((n_hi, bits_hi), (n_lo, bits_lo)):
        if n_tok == 0:
            continue
        codes = 2 * n_tok * d * bits // 8
        token_params = n_tok * 2 * param_bytes * (1 if k_scheme == "channel" else 2)
        channel_params = d * param_bytes * (3 if k_scheme == "channel" else 2)
        total += codes + token_params + channel_params
    return total * b * h_kv


# --------------------------------------------------------------------------
# One (batch, KV head) unit of the mixed-precision cache (Alg. 2, Alg. 3)
# --------------------------------------------------------------------------
class _Subset:
    """Tokens of one precision class inside one segment."""

    def __init__(self, idx: np.ndarray, K: np.ndarray, V: np.ndarray, bits: int,
                 k_scheme: str = "cst", param_dtype: str = "f32"):
        self.idx = idx.astype(np.int32)
        self.bits = bits
        self.n = len(idx)
        if bits == 16:
            self.qK = self.qV = None
            self.K_hat = np.asarray(K, dtype=np.float64)[idx]
            self.V_hat = np.asarray(V, dtype=np.float64)[idx]
            return
        cst = cst_quant_f16_params if param_dtype == "f16" else cst_quant
        self.qV = cst(np.asarray(V, dtype=np.float32)[idx], bits)
        self.V_hat = cst_dequant(self.qV)
        if k_scheme == "channel":     # Alg. 2: ChannelQuant for keys, CSTQuant for values
            self.qK = channel_quant(np.asarray(K, dtype=np.float32)[idx], bits)
            self.K_hat = channel_dequant(self.qK)
        else:
            self.qK = cst(np.asarray(K, dtype=np.float32)[idx], bits)
            self.K_hat = cst_dequant(self.qK)


class _Segment:
    def __init__(self, K, V, p_tilde, ratio, bits_hi, bits_lo, k_scheme="cst", param_dtype="f32"):
        n = K.shape[0]
        self.n = n
        self.p_tilde = np.asarray(p_tilde, dtype=np.float64)
        self.k_scheme, self.param_dtype = k_scheme, param_dtype
        n_s = salient_count(ratio, n)
        sal, reg = split_salient(self.p_tilde, n_s)
        self.impose(K, V, sal, reg, bits_hi, bits_lo)

    def impose(self, K, V, sal, reg, bits_hi, bits_lo):
        self.hi = _Subset(sal, K, V, bits_hi, self.k_scheme, self.param_dtype)
        self.lo = _Subset(reg, K, V, bits_lo, self.k_scheme, self.param_dtype)


class UnitCache:
    """Mixed-precision cache of one (batch, KV head) with its G query heads."""

    def __init__(self, G: int, d: int, ratio: float, bits_hi: int = 4, bits_lo: int = 2,
                 window: int = 100, k_scheme: str = "cst", param_dtype: str = "f32"):
        self.G, self.d, self.ratio = G, d, ratio
        self.bits_hi, self.bits_lo, self.window = bits_hi, bits_lo, window
        self.k_scheme, self.param_dtype = k_scheme, param_dtype
        self.segments: List[_Segment] = []
        self.tail_K = np.zeros((0, d), dtype=np.float64)
        self.tail_V = np.zeros((0, d), dtype=np.float64)
        self.i = 0
        self.tail_colsum = np.zeros(window, dtype=np.float64)
        self.tail_nnz = np.zeros(window, dtype=np.int64)
        self.last_attention: Optional[np.ndarray] = None

    # ---- Alg. 2 (without its FlashAttention output line) ----
    def prefill_compress(self, Q_heads: np.ndarray, K: np.ndarray, V: np.ndarray,
                         P: Sequence[int], salient_idx: Optional[np.ndarray] = None,
                         p_tilde: Optional[np.ndarray] = None) -> None:
        """p_tilde given: the saliency was decided outside the unit (token-level scope)."""
        K = np.asarray(K, dtype=np.float64)
        V = np.asarray(V, dtype=np.float64)
        if p_tilde is None:
            p_tilde = normalized_scores(Q_heads, K, P)
        seg = _Segment(K, V, p_tilde, self.ratio, self.bits_hi, self.bits_lo, self.k_scheme,
                       self.param_dtype)
        if salient_idx is not None:  # staged tests: impose a given split
            sal = np.sort(np.asarray(salient_idx, dtype=np.int32))
            reg = np.setdiff1d(np.arange(K.shape[0], dtype=np.int32), sal)
            seg.impose(K, V, sal, reg, self.bits_hi, self.bits_lo)
        self.segments = [seg]
        self.tail_K = np.zeros((0, self.d), dtype=np.float64)
        self.tail_V = np.zeros((0, self.d), dtype=np.float64)
        self.i = 0
        self.tail_colsum[:] = 0
        self.tail_nnz[:] = 0

    # ---- Eq. 3 / Alg. 3: the new token joins the cache at full precision ----
    def append(self, k: np.ndarray, v: np.ndarray) -> None:
        if self.tail_K.shape[0] >= self.window:
            raise RuntimeError("tail full: flush must have happened")
        self.tail_K = np.vstack([self.tail_K, np.asarray(k, dtype=np.float64)[None, :]])
        self.tail_V = np.vstack([self.tail_V, np.asarray(v, dtype=np.float64)[None, :]])

    def _all_kv(self) -> Tuple[np.ndarray, np.ndarray]:
        Ks = [sub.K_hat for seg in self.segments for sub in (seg.hi, seg.lo)]
        Vs = [sub.V_hat for seg in self.segments for sub in (seg.hi, seg.lo)]
        return np.vstack(Ks + [self.tail_K]), np.vstack(Vs + [self.tail_V])

    # ---- Eq. 4 / Alg. 3: attention over every cached token, then bookkeeping ----
    def decode_attention(self, q_heads: np.ndarray, is_probe_step: bool,
                         defer_flush: bool = False) -> np.ndarray:
        """defer_flush: the caller re-compresses the completed window itself (token-level scope:
        the window's scores are first combined over the heads of the batch row)."""
        q = np.asarray(q_heads, dtype=np.float64)             # [G,d]
        K_all, V_all = self._all_kv()
        logits = (q @ K_all.T) / math.sqrt(self.d)             # [G,n]
        logits -= logits.max(axis=1, keepdims=True)
        e = np.exp(logits)
        a = e / e.sum(axis=1, keepdims=True)
        o = a @ V_all
        self.last_attention = a
        n_tail = self.tail_K.shape[0]
        self.i += 1
        # the last five steps of a window are always probe steps (this includes
        # the window's final step, taken before the re-compression)
        if self.i > self.window - 5 or is_probe_step:
            if n_tail > 0:
                self.tail_colsum[:n_tail] += a[:, a.shape[1] - n_tail:].sum(axis=0)
                self.tail_nnz[:n_tail] += 1
        if self.i == self.window and not defer_flush:
            self._flush()
        return o

    def window_scores(self) -> np.ndarray:
        n = self.tail_K.shape[0]
        return self.tail_colsum[:n] / (self.G * self.tail_nnz[:n])

    def _flush(self, p_tilde: Optional[np.ndarray] = None) -> None:
        n = self.tail_K.shape[0]
        assert n == self.window
        if p_tilde is None:
            p_tilde = self.window_scores()
        self.segments.append(_Segment(self.tail_K, self.tail_V, p_tilde, self.ratio,
                                      self.bits_hi, self.bits_lo, self.k_scheme, self.param_dtype))
        self.tail_K = np.zeros((0, self.d), dtype=np.float64)
        self.tail_V = np.zeros((0, self.d), dtype=np.float64)
        self.i = 0
        self.tail_colsum[:] = 0
        self.tail_nnz[:] = 0


def exact_attention(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """Eq. 4 written out: softmax(q K^T / sqrt(d)) V for q [G,d]."""
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    logits = (q @ K.T) / math.sqrt(K.shape[1])
    logits -= logits.max(axis=1, keepdims=True)
    e = np.exp(logits)
    return (e / e.sum(axis=1, keepdims=True)) @ V


# --------------------------------------------------------------------------
# Whole-tensor convenience wrapper: [b, h, ...] tensors -> independent units
# --------------------------------------------------------------------------
class ZipCacheOracle:
    """All (batch, KV head) units of one attention layer; units are independent."""

    def __init__(self, batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int, ratio: float,
                 bits_hi: int = 4, bits_lo: int = 2, window: int = 100,
                 units: Optional[Sequence[Tuple[int, int]]] = None, k_scheme: str = "cst",
                 param_dtype: str = "f32", scope: str = "kv_head", group: str = "head"):
        """scope "kv_head": one saliency decision per (batch, KV head).  scope "token": the
        paper's literal reading, one decision per token of a batch row shared by all heads --
        the score of a token is the mean of its per-KV-head normalised scores (all units of the
        batch row are then needed).  parity unpinned (how heads are combined is a convention).
        group "head": a token's (s, z) are taken over the d channels of one KV head (2 b h l
        parameters per tensor).  group "all_heads": Alg. 1 as printed, X in R^{l x hd}: one (s, z)
        per token over the channels of ALL KV heads of its batch row (Sec. 4.1's 2 b l parameters);
        the heads must then agree on the subsets, so it needs scope "token"."""
        if group not in ("head", "all_heads"):
            raise ValueError("group must be 'head' or 'all_heads'")
        if group == "all_heads" and scope != "token":
            raise ValueError("token groups over all heads need one split per token (scope='token')")
        self.b, self.hq, self.hkv, self.d = batch, n_q_heads, n_kv_heads, head_dim
        self.G = n_q_heads // n_kv_heads
        self.scope = scope
        self.group = group
        self.unit_ids = list(units) if units is not None else [
            (bi, kv) for bi in range(batch) for kv in range(n_kv_heads)]
        self.units = {u: UnitCache(self.G, head_dim, ratio, bits_hi, bits_lo, window, k_scheme,
                                   param_dtype)
                      for u in self.unit_ids}

    def prefill_compress(self, Q, K, V, P, salient_idx=None) -> None:
        """Q [b,h_q,l,d], K,V [b,h_kv,l,d] (float arrays); P ascending probe list."""
        shared = {}
        if self.scope == "token":
            for bi in sorted({u[0] for u in self.unit_ids}):
                per_head = [normalized_scores(Q[bi, kv * self.G:(kv + 1) * self.G],
                                              np.asarray(K[bi, kv], dtype=np.float64), P)
                            for kv in range(self.hkv)]
                shared[bi] = sum(per_head) / self.hkv
        for (bi, kv) in self.unit_ids:
            sal = None if salient_idx is None else salient_idx[bi][kv]
            self.units[(bi, kv)].prefill_compress(
                Q[bi, kv * self.G:(kv + 1) * self.G], K[bi, kv], V[bi, kv], P, sal,
                p_tilde=shared.get(bi))
        if self.group == "all_heads":
            for bi in sorted({u[0] for u in self.unit_ids}):
                self._quantise_row_jointly(bi, [K[bi, kv] for kv in range(self.hkv)],
                                           [V[bi, kv] for kv in range(self.hkv)])

    def _quantise_row_jointly(self, bi: int, Ks, Vs) -> None:
        """Alg. 1 on X in R^{n x (h d)}: the newest segment's subsets of every KV head of batch row
        bi are quantised again as ONE matrix per tensor whose columns are the channels of all the
        heads, so a token has one (s, z) for all of them; every head keeps its own columns of the
        codes and of the channel factors.  (Channelwise keys have no token parameters: their K
        stays as it is.)"""
        row = [self.units[(bi, kv)] for kv in range(self.hkv)]
        d = self.d
        for name in ("hi", "lo"):
            subs = [getattr(u.segments[-1], name) for u in row]
            if subs[0].bits == 16 or subs[0].n == 0:
                continue
            idx = subs[0].idx
            for sub in subs:
                assert np.array_equal(sub.idx, idx), "token groups need the same subsets in every head"
            cst = cst_quant_f16_params if row[0].param_dtype == "f16" else cst_quant
            for tensor, Xs in (("V", Vs), ("K", Ks)):
                if tensor == "K" and row[0].k_scheme == "channel":
                    continue
                X = np.concatenate([np.asarray(x, dtype=np.float32)[idx] for x in Xs], axis=1)
                q = cst(X, subs[0].bits)
                for kv, sub in enumerate(subs):
                    part = {"c": q["c"][kv * d:(kv + 1) * d], "s": q["s"], "z": q["z"],
                            "codes": q["codes"][:, kv * d:(kv + 1) * d], "bits": q["bits"],
                            "pre_round": q["pre_round"][:, kv * d:(kv + 1) * d]}
                    if tensor == "V":
                        sub.qV, sub.V_hat = part, cst_dequant(part)
                    else:
                        sub.qK, sub.K_hat = part, cst_dequant(part)

    def append(self, k, v) -> None:
        for (bi, kv) in self.unit_ids:
            self.units[(bi, kv)].append(k[bi, kv], v[bi, kv])

    def decode_attention(self, q, is_probe_step: bool) -> Dict[Tuple[int, int], np.ndarray]:
        out = {}
        token_scope = self.scope == "token"
        for (bi, kv) in self.unit_ids:
            out[(bi, kv)] = self.units[(bi, kv)].decode_attention(
                q[bi, kv * self.G:(kv + 1) * self.G], is_probe_step, defer_flush=token_scope)
        if token_scope:
            for bi in sorted({u[0] for u in self.unit_ids}):
                row = [self.units[(bi, kv)] for kv in range(self.hkv)]
                if row[0].i == row[0].window:
                    shared = sum(u.window_scores() for u in row) / self.hkv
                    tails = [(u.tail_K.copy(), u.tail_V.copy()) for u in row]
                    for u in row:
                        u._flush(shared)
                    if self.group == "all_heads":
                        self._quantise_row_jointly(bi, [t[0] for t in tails], [t[1] for t in tails])
        return out
