// CSTQuant (Alg. 1, Eq. 5) of one token row and the composition of packed cache tiles: shared
// by the prefill compression kernels and the window re-compression inside the decode kernel.
#pragma once

#include "zc_internal.h"
#include "zc_layout.cuh"

// Normative fp32 sequence (each step one IEEE operation, round to nearest even, nothing
// fused): c = sqrt(max|x|) (1 if the channel is all zero); y = x / c; per token mn, mx over
// the 128 channels; s = (mx - mn) / L, or |mn| (1 if mn == 0) when mx == mn;
// z = -rint(mn / s); code = clamp(rint(y / s) + z, 0, L).
// P16 (ZC_FLAG_PARAMS_F16): the scale is rounded UP to the next fp16 value before z and the codes
// are formed (the caller has done the same to c).
// mm (ZC_FLAG_GROUP_ALL_HEADS): the token's minimum and maximum of y over the channels of all KV
// heads of its batch row, taken beforehand, in place of this head's own.
template <bool P16 = false>
static __device__ __forceinline__ void quant_token(const float (&x)[4], const float (&c)[4], float L,
                                            float* s_out, float* z_out, unsigned* codes4,
                                            const float* mm = nullptr) {
  float y[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) y[e] = __fdiv_rn(x[e], c[e]);
  float mn = fminf(fminf(y[0], y[1]), fminf(y[2], y[3]));
  float mx = fmaxf(fmaxf(y[0], y[1]), fmaxf(y[2], y[3]));
  if (mm) {
    mn = mm[0];
    mx = mm[1];
  } else {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
  }
  float s = __fdiv_rn(__fsub_rn(mx, mn), L);
  if (mx == mn) s = mn != 0.f ? fabsf(mn) : 1.f;
  if (P16) s = __half2float(__float2half_ru(s));
  const float z = -rintf(__fdiv_rn(mn, s));
  unsigned packed = 0;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    float q = __fadd_rn(rintf(__fdiv_rn(y[e], s)), z);
    q = fminf(fmaxf(q, 0.f), L);
    packed |= ((unsigned)(int)q) << (8 * e);
  }
  *s_out = s;
  *z_out = z;
  *codes4 = packed;
}

// a / b, correctly rounded, from b's correctly rounded reciprocal rb = __frcp_rn(b), for a
// divisor that serves many dividends (a channel's c, a token's s, the level count L).  With
// q0 = RN(a rb), each step q <- RN(q + (a - b q) rb) takes the residual by one FMA: the first
// step leaves q within one unit in the last place of a / b, and from there the residual is exact
// and the second step yields RN(a / b) (Markstein's theorem on division by a correctly rounded
// reciprocal).  That needs every intermediate to stay a normal number, which the callers see to:
// 2^-40 <= |a|, b <= 2^40 (zc_mid), or the bounds stated where it is called.  Anything else
// (zeros, subnormals, infinities, NaN) takes __fdiv_rn.
static __device__ __forceinline__ float zc_div_by(float a, float b, float rb) {
  float q = __fmul_rn(a, rb);
  q = __fmaf_rn(__fmaf_rn(-b, q, a), rb, q);
  return __fmaf_rn(__fmaf_rn(-b, q, a), rb, q);
}
static __device__ __forceinline__ bool zc_mid(float a) {
  const float m = fabsf(a);
  return m >= 0x1p-40f && m <= 0x1p40f;   // false for NaN
}

// quant_token for a caller that keeps its channels over many tokens: rc[e] = __frcp_rn(c[e]),
// c_mid = every c[e] passes zc_mid, rL = __frcp_rn(L).  Bit for bit quant_token's results: the
// same sequence with the divisions taken by zc_div_by where the whole warp's operands allow it
// (|y| = |x / c| then lies in [2^-80, 2^80], mx - mn is 0 or at least an ulp of 2^-80, and with
// s in [2^-40, 2^40] the codes' quotients stay below 2^120), by quant_token otherwise.
static __device__ __noinline__ float4 quant_token_ieee(float4 xv, float4 cv, float L, bool p16) {   // (s, z, codes, -)
  const float x[4] = {xv.x, xv.y, xv.z, xv.w}, c[4] = {cv.x, cv.y, cv.z, cv.w};
  float s, z;
  unsigned pk;
  if (p16) quant_token<true>(x, c, L, &s, &z, &pk);
  else quant_token<false>(x, c, L, &s, &z, &pk);
  return make_float4(s, z, __uint_as_float(pk), 0.f);
}
static __device__ __noinline__ float4 quant_token_ieee_shared(float4 xv, float4 cv, float L, bool p16, float mn_sh,
                                                              float mx_sh) {
  const float x[4] = {xv.x, xv.y, xv.z, xv.w}, c[4] = {cv.x, cv.y, cv.z, cv.w};
  const float mm[2] = {mn_sh, mx_sh};
  float s, z;
  unsigned pk;
  if (p16) quant_token<true>(x, c, L, &s, &z, &pk, mm);
  else quant_token<false>(x, c, L, &s, &z, &pk, mm);
  return make_float4(s, z, __uint_as_float(pk), 0.f);
}
static __device__ __forceinline__ void quant_token_rc(const float (&x)[4], const float (&c)[4], const float (&rc)[4],
                                                      bool c_mid, float L, float rL, float* s_out, float* z_out,
                                                      unsigned* codes4, bool p16 = false, bool shared = false,
                                                      float mn_sh = 0.f, float mx_sh = 0.f) {
  const bool mine = c_mid && zc_mid(x[0]) && zc_mid(x[1]) && zc_mid(x[2]) && zc_mid(x[3]);
  if (__all_sync(0xffffffffu, mine)) {
    float y[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) y[e] = zc_div_by(x[e], c[e], rc[e]);
    float mn = fminf(fminf(y[0], y[1]), fminf(y[2], y[3]));
    float mx = fmaxf(fmaxf(y[0], y[1]), fmaxf(y[2], y[3]));
    bool range_ok = true;
    if (shared) {   // the row's statistics over all heads: other heads' values must be in range as well
      mn = mn_sh;
      mx = mx_sh;
      range_ok = zc_mid(mn) && zc_mid(mx);
    } else {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      }
    }
    float s = zc_div_by(__fsub_rn(mx, mn), L, rL);   // 0 when mx == mn, replaced below
    if (mx == mn) s = fabsf(mn);                     // mn != 0 here
    if (p16) s = __half2float(__float2half_ru(s));   // stored as fp16: never below the exact scale
    if (range_ok && zc_mid(s)) {                     // the same for every lane
      const float rs = __frcp_rn(s);
      const float z = -rintf(zc_div_by(mn, s, rs));
      unsigned packed = 0;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        float q = __fadd_rn(rintf(zc_div_by(y[e], s, rs)), z);
        q = fminf(fmaxf(q, 0.f), L);
        packed |= ((unsigned)(int)q) << (8 * e);
      }
      *s_out = s;
      *z_out = z;
      *codes4 = packed;
      return;
    }
  }
  const float4 xv = make_float4(x[0], x[1], x[2], x[3]), cv = make_float4(c[0], c[1], c[2], c[3]);
  const float4 r = shared ? quant_token_ieee_shared(xv, cv, L, p16, mn_sh, mx_sh) : quant_token_ieee(xv, cv, L, p16);
  *s_out = r.x;
  *z_out = r.y;
  *codes4 = __float_as_uint(r.z);
}

// ChannelQuant (Eq. 5 per channel, Sec. 4.1) of one token's four channels, whose (s, z) the
// caller holds: code = clamp(rint(x / s_i) + z_i, 0, L), each step one IEEE operation.
static __device__ __forceinline__ unsigned quant_channel4(const float (&x)[4], const float (&s)[4],
                                                          const float (&z)[4], float L) {
  unsigned packed = 0;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    float q = __fadd_rn(rintf(__fdiv_rn(x[e], s[e])), z[e]);
    q = fminf(fmaxf(q, 0.f), L);
    packed |= ((unsigned)(int)q) << (8 * e);
  }
  return packed;
}
// quant_channel4 with rs[e] = __frcp_rn(s[e]) and s_mid = every s[e] passes zc_mid: the same
// codes, the divisions by zc_div_by where this thread's operands allow it.
static __device__ __forceinline__ unsigned quant_channel4_rc(const float (&x)[4], const float (&s)[4],
                                                             const float (&rs)[4], bool s_mid,
                                                             const float (&z)[4], float L) {
  if (!(s_mid && zc_mid(x[0]) && zc_mid(x[1]) && zc_mid(x[2]) && zc_mid(x[3]))) return quant_channel4(x, s, z, L);
  unsigned packed = 0;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    float q = __fadd_rn(rintf(zc_div_by(x[e], s[e], rs[e])), z[e]);
    q = fminf(fmaxf(q, 0.f), L);
    packed |= ((unsigned)(int)q) << (8 * e);
  }
  return packed;
}
// Channel parameters from the channel's minimum and maximum over the subset (Eq. 5):
// s = (mx - mn) / L, or |mn| (1 if 0) for a constant channel; z = -rint(mn / s).
static __device__ __forceinline__ void channel_params(float mn, float mx, float L, float* s_out, float* z_out) {
  float s = __fdiv_rn(__fsub_rn(mx, mn), L);
  if (mx == mn) s = mn != 0.f ? fabsf(mn) : 1.f;
  *s_out = s;
  *z_out = -rintf(__fdiv_rn(mn, s));
}

// One 16-byte vector v of a cache tile from byte codes and per-token (s, z), the arrays holding
// the tile's tokens from token row0 on: K codes in canonical order, V codes in fragment order, then the parameters, per
// 16-token sub-block.
// kch: channelwise keys, the parameter block holds (sV, zV) per token only.
static __device__ __forceinline__ uint4 compose_vec(int bits, int kch, int v, int row0,
                                             const unsigned char (*codesK)[ZC_D],
                                             const unsigned char (*codesV)[ZC_D], const float (*parK)[2],
                                             const float (*parV)[2]) {
  const int sub_words = zc_sub_bytes(bits, kch) / 4;
  const int kw = 64 * bits;                           // K-code words per sub-block (= V-code words)
  const int per = 32 / bits;                          // codes per word
  unsigned out[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int wi = 4 * v + q;
    const int st = wi / sub_words, wl = wi % sub_words;
    unsigned word = 0;
    if (wl < kw) {
      // K: canonical order, token row of 4*bits words
      const int words_per_row = 4 * bits;
      const int tok = 16 * st - row0 + wl / words_per_row, wr = wl % words_per_row;
      for (int e = 0; e < per; ++e) word |= (unsigned)codesK[tok][wr * per + e] << (bits * e);
    } else if (wl < 2 * kw) {
      // V: fragment order of the 16-token sub-tile
      const int wv = wl - kw;
      if (bits == 4) {
        const int qd = wv >> 7, ln = (wv >> 2) & 31, jj = wv & 3;
        const int j = 4 * qd + jj, g = ln >> 2, t = ln & 3;
        for (int p = 0; p < 8; ++p) {
          const int hi_row = p & 1, isB = (p >> 1) & 1, is1 = p >> 2;
          const int ch = 16 * j + g + 8 * hi_row, tau = 2 * t + isB + 8 * is1;
          word |= (unsigned)codesV[16 * st - row0 + tau][ch] << (4 * p);
        }
      } else {
        const int ln = wv >> 2, m = wv & 3, g = ln >> 2, t = ln & 3;
        for (int i = 0; i < 16; ++i) {
          const int is1 = i >> 3, pp = i & 7, e2 = pp >> 2, hi_row = (pp >> 1) & 1, isB = pp & 1;
          const int j = 2 * m + e2;
          const int ch = 16 * j + g + 8 * hi_row, tau = 2 * t + isB + 8 * is1;
          word |= (unsigned)codesV[16 * st - row0 + tau][ch] << (2 * i);
        }
      }
    } else {
      const int wp = wl - 2 * kw;  // params: (sK, zK, sV, zV) per token, or (sV, zV)
      if (kch) {
        word = __float_as_uint(parV[16 * st - row0 + (wp >> 1)][wp & 1]);
      } else {
        const int tk = 16 * st - row0 + (wp >> 2), f = wp & 3;
        word = __float_as_uint(f < 2 ? parK[tk][f] : parV[tk][f - 2]);
      }
    }
    out[q] = word;
  }
  return make_uint4(out[0], out[1], out[2], out[3]);
}


// Word wv of the V codes of one 16-token sub-block (fragment order, as compose_vec lays them
// out) from the sub-block's byte codes cv[token][channel]; bits is a constant where it is called.
static __device__ __forceinline__ unsigned zc_v_word(int bits, const unsigned char (*cv)[ZC_D], int wv) {
  unsigned word = 0;
  if (bits == 8) {
    const int q = wv >> 7, ln = (wv >> 2) & 31, i = wv & 3;
    const int ch = 16 * (2 * q + (i >> 1)) + (ln >> 2) + 8 * (i & 1), t = ln & 3;
    word = (unsigned)cv[2 * t][ch] | (unsigned)cv[2 * t + 1][ch] << 8 | (unsigned)cv[2 * t + 8][ch] << 16 |
           (unsigned)cv[2 * t + 9][ch] << 24;
  } else if (bits == 4) {
    const int qd = wv >> 7, ln = (wv >> 2) & 31, jj = wv & 3;
    const int j = 4 * qd + jj, g = ln >> 2, t = ln & 3;
#pragma unroll
    for (int p = 0; p < 8; ++p) {
      const int hi_row = p & 1, isB = (p >> 1) & 1, is1 = p >> 2;
      word |= (unsigned)cv[2 * t + isB + 8 * is1][16 * j + g + 8 * hi_row] << (4 * p);
    }
  } else {
    const int ln = wv >> 2, m = wv & 3, g = ln >> 2, t = ln & 3;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int is1 = i >> 3, pp = i & 7, e2 = pp >> 2, hi_row = (pp >> 1) & 1, isB = pp & 1;
      word |= (unsigned)cv[2 * t + isB + 8 * is1][16 * (2 * m + e2) + g + 8 * hi_row] << (2 * i);
    }
  }
  return word;
}

// The K codes of two tokens a and b (each lane: its four channels' codes of either, a byte each)
// as words of the canonical order (a token's row of 4 * bits words, codes ascending from bit 0).
// Returns this lane's word; *tok_b says which token it belongs to and *wr which word of the
// row; *owner is false in the lanes that hold no word (2-bit codes: half of them).
static __device__ __forceinline__ unsigned zc_k_words(int bits, unsigned pk_a, unsigned pk_b, int lane, bool* tok_b,
                                                      int* wr, bool* owner) {
  if (bits == 4) {
    // four codes -> 16 bits per token; the neighbour lane holds the other half of the word
    const unsigned ta = pk_a | (pk_a >> 4), tb = pk_b | (pk_b >> 4);
    const unsigned hh = __byte_perm(ta, tb, 0x6420);            // [a: 16 bits][b: 16 bits]
    const unsigned other = __shfl_xor_sync(0xffffffffu, hh, 1);
    const bool odd = lane & 1;
    *tok_b = odd;
    *wr = lane >> 1;
    *owner = true;
    // even lane: a's word = own low half | neighbour's low half << 16; odd lane: b's word =
    // neighbour's high half | own high half << 16
    return __byte_perm(hh, other, odd ? 0x3276 : 0x5410);
  }
  // four codes -> 8 bits per token; four lanes hold a word
  const unsigned ta = pk_a | (pk_a >> 6), tb = pk_b | (pk_b >> 6);
  const unsigned ua = ta | (ta >> 12), ub = tb | (tb >> 12);
  const unsigned mine = __byte_perm(ua, ub, 0x0040);             // [a byte][b byte][unused][unused]
  const unsigned nb = __shfl_xor_sync(0xffffffffu, mine, 1);
  // both lanes of a pair: [a even lane][b even lane][a odd lane][b odd lane]
  const unsigned v = (lane & 1) ? __byte_perm(nb, mine, 0x5410) : __byte_perm(mine, nb, 0x5410);
  const unsigned v2 = __shfl_xor_sync(0xffffffffu, v, 2);
  *tok_b = lane & 1;
  *wr = lane >> 2;
  *owner = (lane & 2) == 0;
  return __byte_perm(v, v2, (lane & 1) ? 0x7531 : 0x6420);
}

// compose_vec for 8-bit codes (a K row is the codes themselves, four to a word; V words as
// zc_vcode_pos lays them out).  Kept apart so that the builds without an 8-bit class stay as
// they are.
static __device__ __forceinline__ uint4 compose_vec8(int kch, int v, int row0, const unsigned char (*codesK)[ZC_D],
                                                     const unsigned char (*codesV)[ZC_D], const float (*parK)[2],
                                                     const float (*parV)[2]) {
  const int sub_words = zc_sub_bytes(8, kch) / 4;
  unsigned out[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int wi = 4 * v + q;
    const int st = wi / sub_words, wl = wi % sub_words;
    unsigned word;
    if (wl < 512) {
      const int tok = 16 * st - row0 + (wl >> 5);
      word = *reinterpret_cast<const unsigned*>(&codesK[tok][4 * (wl & 31)]);
    } else if (wl < 1024) {
      word = zc_v_word(8, codesV + (16 * st - row0), wl - 512);
    } else {
      const int wp = wl - 1024;
      if (kch) {
        word = __float_as_uint(parV[16 * st - row0 + (wp >> 1)][wp & 1]);
      } else {
        const int tk = 16 * st - row0 + (wp >> 2), f = wp & 3;
        word = __float_as_uint(f < 2 ? parK[tk][f] : parV[tk][f - 2]);
      }
    }
    out[q] = word;
  }
  return make_uint4(out[0], out[1], out[2], out[3]);
}
