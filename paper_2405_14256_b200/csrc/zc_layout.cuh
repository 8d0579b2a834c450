// Device-side layout helpers: where a (token, channel) code lives inside a tile.
//
// K codes keep the canonical order per token row.  V codes are stored in the
// register order of the m16n8k16 MMA A-fragment of V^T (rows = channels,
// k = tokens), so that the decode kernel can turn a 32-bit word into fragment
// registers with masks only:
//   lane = g*4 + t, g = 0..7, t = 0..3;  M-tile j = channels 16j..16j+15;
//   fragment rows g (scale 1) and g+8 (scale 16) <-> channels 16j+g, 16j+g+8;
//   fragment k-pairs A = (2t, 2t+1) <-> tokens (2t, 2t+8), B = (2t+8, 2t+9) <->
//   tokens (2t+1, 2t+9) of the 16-token sub-tile.
// 4-bit: word j of the lane (8 nibbles) serves M-tile j; nibble p = hi_row + 2*isB + 4*is1.
// 2-bit: word m of the lane (16 crumbs) serves M-tiles 2m and 2m+1;
//        crumb i = 8*is1 + 4*(j&1) + 2*hi_row + isB.
#pragma once
#include "zc_internal.h"

// A tile is four self-contained sub-blocks of 16 tokens, so that one bulk copy brings
// everything a warp needs for one MMA sub-tile:
//   [K codes 16 rows x 16*bits B][V codes, fragment order][(sK, zK, sV, zV) x 16]
// kch: keys quantised channelwise, the parameter block is [(sV, zV) x 16].
// bits = 16: the tokens are kept as they came (no codes, no parameters): [K rows 16 x 256 B][V rows 16 x 256 B].
// p16: the parameters are 16 bits each (fp16 scale, int16 zero point): half the block.
__host__ __device__ inline int zc_sub_bytes(int bits, int kch, int p16 = 0) {
  return bits == 16 ? ZC_SUB * 2 * ZC_D * 2 : ZC_SUB * (32 * bits + ((kch ? 8 : 16) >> (p16 ? 1 : 0)));
}
__host__ __device__ inline int zc_tile_bytes(int bits, int kch, int p16 = 0) {
  return (ZC_TILE / ZC_SUB) * zc_sub_bytes(bits, kch, p16);
}
__host__ __device__ inline int zc_sub_off_vcodes(int bits) { return 256 * bits; }
__host__ __device__ inline int zc_sub_off_par(int bits) { return 512 * bits; }

// Position of V code (token tau of a 16-token sub-tile, channel ch) inside the
// sub-tile's block: returns the 32-bit word index and the bit shift in the word.
__host__ __device__ inline void zc_vcode_pos(int bits, int tau, int ch, int* word, int* shift) {
  int j = ch >> 4, rho = ch & 15, g = rho & 7, hi_row = rho >> 3;
  int is1 = tau >> 3, tp = tau & 7, t = tp >> 1, isB = tp & 1;
  int lane = g * 4 + t;
  if (bits == 8) {
    // two words per lane and 16-channel group: channel row g, then g + 8; bytes = tokens 2t, 2t+1, 2t+8, 2t+9
    *word = (j >> 1) * 128 + lane * 4 + 2 * (j & 1) + hi_row;
    *shift = 8 * (isB + 2 * is1);
  } else if (bits == 4) {
    int p = hi_row + 2 * isB + 4 * is1;
    *word = (j >> 2) * 128 + lane * 4 + (j & 3);
    *shift = 4 * p;
  } else {
    int i = 8 * is1 + 4 * (j & 1) + 2 * hi_row + isB;
    *word = lane * 4 + (j >> 1);
    *shift = 2 * i;
  }
}

template <typename T> __device__ inline float zc_to_float(T v);
template <> __device__ inline float zc_to_float<__half>(__half v) { return __half2float(v); }
template <> __device__ inline float zc_to_float<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ inline T zc_from_float(float v);
template <> __device__ inline __half zc_from_float<__half>(float v) { return __float2half_rn(v); }
template <> __device__ inline __nv_bfloat16 zc_from_float<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// 4 consecutive elements (8 bytes) -> floats
template <typename T> __device__ inline void zc_load4(const T* p, float* out) {
  uint2 raw = *reinterpret_cast<const uint2*>(p);
  const T* e = reinterpret_cast<const T*>(&raw);
  out[0] = zc_to_float<T>(e[0]); out[1] = zc_to_float<T>(e[1]);
  out[2] = zc_to_float<T>(e[2]); out[3] = zc_to_float<T>(e[3]);
}

// Order-preserving map of floats onto unsigned keys (and back), for minima and maxima by
// integer atomics: key(a) < key(b) exactly when a < b.
__device__ inline unsigned zc_float_key(float x) {
  const unsigned b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ inline float zc_key_float(unsigned k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

#ifdef ZC_DEBUG
// one word per translation unit (no relocatable device code): zc_debug_code_* read them
static __device__ int g_zc_debug_fault = 0;
__device__ inline bool zc_debug_check(bool ok, int code) {
  if (!ok) atomicCAS(&g_zc_debug_fault, 0, code);
  return ok;
}
#endif

__device__ inline char* zc_unit_base(char* base, const ZcLayout& lay, int unit) {
  return base + (long long)unit * lay.unit_stride;
}
