// Split by saliency (Alg. 2 "Split"), channel factors (Eq. 6), CSTQuant (Alg. 1, Eq. 5)
// and packing into cache tiles, for the prefill compression.
#include "zc_internal.h"
#include "zc_layout.cuh"
#include "zc_quant.cuh"

namespace {

// ------------------------------------------------------------------ top-k split
// One CTA per unit.  Keys are the bit patterns of the (non-negative) scores, so unsigned
// integer order equals float order.  An MSB-first 8-bit radix select finds the n_s-th
// largest key T and how many keys equal to T belong to the top set (lowest index first);
// a second sweep writes both index lists in ascending order.
constexpr int kTopkThreads = 1024;

__device__ int block_exclusive_scan(int v, int* warp_sums, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int x = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int y = __shfl_up_sync(0xffffffffu, x, o);
    if (lane >= o) x += y;
  }
  if (lane == 31) warp_sums[warp] = x;
  __syncthreads();
  if (warp == 0) {
    int w = warp_sums[lane];
    int xs = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int y = __shfl_up_sync(0xffffffffu, xs, o);
      if (lane >= o) xs += y;
    }
    warp_sums[lane] = xs - w;  // exclusive
    if (lane == 31) *total = xs;
  }
  __syncthreads();
  int r = warp_sums[warp] + x - v;
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(kTopkThreads) k_topk_split(char* cache, ZcLayout lay, int n, int n_s,
                                                             int idx_off,
                                                             const int32_t* __restrict__ given) {
  __shared__ int hist[256];
  __shared__ int warp_sums[32];
  __shared__ int s_total;
  __shared__ unsigned s_prefix;
  __shared__ int s_krem;
  extern __shared__ unsigned flags[];  // bitset, used when the salient set is given
  const int unit = blockIdx.x, tid = threadIdx.x;
  char* ub = zc_unit_base(cache, lay, unit);
  const unsigned* keys = reinterpret_cast<const unsigned*>(ub + lay.off_scores);
  int32_t* idx = reinterpret_cast<int32_t*>(ub + lay.off_idx) + idx_off;
  int32_t* idx_sal = idx;
  int32_t* idx_reg = idx + n_s;

  unsigned T = 0;
  int need_eq = 0;
  if (given) {
    const int words = (n + 31) / 32;
    for (int i = tid; i < words; i += kTopkThreads) flags[i] = 0u;
    __syncthreads();
    const int32_t* mine = given + (long long)unit * n_s;
    for (int i = tid; i < n_s; i += kTopkThreads) {
      const int j = mine[i];
      if (j >= 0 && j < n) atomicOr(&flags[j >> 5], 1u << (j & 31));
    }
    __syncthreads();
  } else if (n_s > 0 && n_s < n) {
    if (tid == 0) { s_prefix = 0u; s_krem = n_s; }
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      const unsigned prefix = s_prefix;
      const unsigned mask_hi = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
      for (int i = tid; i < n; i += kTopkThreads) {
        const unsigned k = keys[i];
        if ((k & mask_hi) == prefix) atomicAdd(&hist[(k >> shift) & 255], 1);
      }
      __syncthreads();
      // the bin, from the top, at which the count reaches the krem keys still wanted: lane l
      // of warp 0 owns bins 255 - 8l down to 248 - 8l
      if (tid < 32) {
        const int krem = s_krem, top = 255 - 8 * tid;
        int cnt[8], sum = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { cnt[j] = hist[top - j]; sum += cnt[j]; }
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int y = __shfl_up_sync(0xffffffffu, incl, o);
          if (tid >= o) incl += y;
        }
        const int excl = incl - sum;
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        if ((excl < krem && krem <= incl) || (tid == 31 && total < krem)) {
          int r = krem - excl, b = top;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            b = top - j;
            if (b == 0 || cnt[j] >= r) break;
            r -= cnt[j];
          }
          s_prefix = prefix | ((unsigned)b << shift);
          s_krem = r;
        }
      }
      __syncthreads();
    }
    T = s_prefix;
    need_eq = s_krem;
  }
  // contiguous chunk per thread keeps index order
  const int chunk = (n + kTopkThreads - 1) / kTopkThreads;
  const int lo = min(n, tid * chunk), hi = min(n, lo + chunk);
  int eq_before = 0;
  if (!given && n_s > 0 && n_s < n) {
    int eq = 0;
    for (int i = lo; i < hi; ++i) eq += keys[i] == T;
    eq_before = block_exclusive_scan(eq, warp_sums, &s_total);
  }
  auto is_sal = [&](int i, int& eq_rank) -> bool {
    if (given) return (flags[i >> 5] >> (i & 31)) & 1u;
    if (n_s <= 0) return false;
    if (n_s >= n) return true;
    const unsigned k = keys[i];
    if (k > T) return true;
    if (k == T) return eq_rank++ < need_eq;
    return false;
  };
  int cnt = 0, er = eq_before;
  for (int i = lo; i < hi; ++i) cnt += is_sal(i, er) ? 1 : 0;
  const int sal_before = block_exclusive_scan(cnt, warp_sums, &s_total);
  int s_pos = sal_before, r_pos = lo - sal_before;
  er = eq_before;
  for (int i = lo; i < hi; ++i) {
    if (is_sal(i, er)) {
      if (ZC_CHECKED(s_pos < n_s, ZC_DBG_TOPK_INDEX) && s_pos < n_s) idx_sal[s_pos] = i;
      ++s_pos;
    } else {
      if (ZC_CHECKED(r_pos < n - n_s, ZC_DBG_TOPK_INDEX) && r_pos < n - n_s) idx_reg[r_pos] = i;
      ++r_pos;
    }
  }
}

// ------------------------------------------------------------------ channel |x| max (Eq. 6)
// grid.x: groups of kAbsTiles tiles of class 0, then of class 1; grid.y: unit.  blockDim 256.
// A CTA folds several tiles before it touches the unit's shared maxima: one atomic per
// channel and CTA.
constexpr int kAbsTiles = 4;

// Channelwise keys (lay.kch): the same pass takes the signed minimum and maximum of every key
// channel instead of the maximum of its magnitude.
template <typename T>
__global__ void __launch_bounds__(256) k_channel_absmax(char* cache, ZcLayout lay, ZcSrc src, ZcSeg seg) {
  __shared__ float red[3][8][ZC_D];
  const int unit = blockIdx.y, b = unit / lay.n_kv, kv = unit % lay.n_kv;
  const int groups_c0 = zc_ceil_div(zc_ceil_div(seg.n_tok[0], ZC_TILE), kAbsTiles);
  const int cls = (int)blockIdx.x < groups_c0 ? 0 : 1;
  if (lay.bits[cls] == 16) return;   // tokens kept as they are: no factors
  const int grp = cls == 0 ? blockIdx.x : blockIdx.x - groups_c0;
  char* ub = zc_unit_base(cache, lay, unit);
  const int32_t* idx = reinterpret_cast<const int32_t*>(ub + lay.off_idx) + seg.idx_off +
                       (cls == 0 ? 0 : seg.n_tok[0]);
  const T* Kb = reinterpret_cast<const T*>(src.K) + b * src.sb + kv * src.sh;
  const T* Vb = reinterpret_cast<const T*>(src.V) + b * src.sb + kv * src.sh;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const bool kch = lay.kch != 0;
  const float k0 = kch ? -INFINITY : 0.f;
  float mk[4] = {k0, k0, k0, k0}, mv[4] = {0.f, 0.f, 0.f, 0.f};
  float nk[4] = {INFINITY, INFINITY, INFINITY, INFINITY};
  const int t_lo = grp * kAbsTiles * ZC_TILE;
  const int t_hi = min(seg.n_tok[cls], t_lo + kAbsTiles * ZC_TILE);
#pragma unroll 4
  for (int tt = t_lo + w; tt < t_hi; tt += 8) {
    const long long row = (long long)idx[tt] * src.sl;
    float x[4];
    zc_load4<T>(Kb + row + 4 * lane, x);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      mk[e] = fmaxf(mk[e], kch ? x[e] : fabsf(x[e]));
      nk[e] = fminf(nk[e], x[e]);
    }
    zc_load4<T>(Vb + row + 4 * lane, x);
#pragma unroll
    for (int e = 0; e < 4; ++e) mv[e] = fmaxf(mv[e], fabsf(x[e]));
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    red[0][w][4 * lane + e] = mk[e];
    red[1][w][4 * lane + e] = mv[e];
    red[2][w][4 * lane + e] = nk[e];
  }
  __syncthreads();
  unsigned* cmax = reinterpret_cast<unsigned*>(ub + lay.off_cmax) + cls * 3 * ZC_D;
  for (int a = threadIdx.x; a < (kch ? 3 : 2) * ZC_D; a += 256) {
    const int ten = a >> 7, ch = a & 127;
    float m = red[ten][0][ch];
#pragma unroll
    for (int i = 1; i < 8; ++i) m = ten == 2 ? fminf(m, red[ten][i][ch]) : fmaxf(m, red[ten][i][ch]);
    // ordered keys: integer order is float order for signed values too
    if (ten == 2) atomicMin(&cmax[ten * ZC_D + ch], zc_float_key(m));
    else atomicMax(&cmax[ten * ZC_D + ch], zc_float_key(m));
  }
}

__global__ void k_clear_cmax(char* cache, ZcLayout lay, ZcSeg seg) {
  char* ub = zc_unit_base(cache, lay, blockIdx.x);
  unsigned* cmax = reinterpret_cast<unsigned*>(ub + lay.off_cmax);
  // maxima start below every key, minima above (per class: K max, V max, K min)
  for (int i = threadIdx.x; i < 6 * ZC_D; i += blockDim.x) cmax[i] = ((i / ZC_D) % 3 == 2) ? 0xffffffffu : 0u;
  float* fac = reinterpret_cast<float*>(ub + lay.off_fac);
  if (threadIdx.x < 2) fac[(seg.run0 + threadIdx.x) * ZC_FAC_FLOATS + 2 * ZC_D] = 0.f;  // smaxV
}

// ------------------------------------------------------------------ token-level saliency (ZC_SCOPE_TOKEN)
// scores[b][kv][j] <- mean over the KV heads of batch row b of scores[b][.][j], j < n: every head
// of the row then makes the same split.  grid.x: blocks of 256 tokens; grid.y: batch row.
__global__ void k_share_scores(char* cache, ZcLayout lay, int n) {
  const int j = blockIdx.x * 256 + threadIdx.x, b = blockIdx.y;
  if (j >= n) return;
  float sum = 0.f;
  for (int kv = 0; kv < lay.n_kv; ++kv)
    sum = __fadd_rn(sum, reinterpret_cast<const float*>(zc_unit_base(cache, lay, b * lay.n_kv + kv) + lay.off_scores)[j]);
  const float mean = __fdiv_rn(sum, (float)lay.n_kv);
  for (int kv = 0; kv < lay.n_kv; ++kv)
    reinterpret_cast<float*>(zc_unit_base(cache, lay, b * lay.n_kv + kv) + lay.off_scores)[j] = mean;
}

// The completed window's normalised scores of every unit (Eq. 8 on the collected probe rows:
// column sum / (G * rows that saw the token)); the statistics start from zero for the next
// window.  The same two steps open the re-compression inside the decode kernel.
__global__ void k_window_scores(char* cache, ZcLayout lay, ZcFlushArgs fl) {
  char* ub = zc_unit_base(cache, lay, blockIdx.x);
  const int tid = threadIdx.x;
  if (tid >= lay.window) return;
  float* colsum = reinterpret_cast<float*>(ub + lay.off_colsum);
  reinterpret_cast<float*>(ub + lay.off_scores)[tid] = __fdiv_rn(colsum[tid], (float)(lay.G * max(1, (int)fl.nnz[tid])));
  colsum[tid] = 0.f;
}

// ------------------------------------------------------------------ token groups over all heads (ZC_FLAG_GROUP_ALL_HEADS)
// Channel factor of Alg. 1 from the subset's channel maximum: c = sqrt(max |x|), 1 for an all-zero
// channel; with 16-bit parameters the fp16 value at or above it.
__device__ __forceinline__ float channel_factor(unsigned key, bool p16) {
  const float m = zc_key_float(key);
  float c = m == 0.f ? 1.f : __fsqrt_rn(m);
  if (p16) c = __half2float(__float2half_ru(c));
  return c;
}

template <typename T> __device__ __forceinline__ void raw4_load(float (&x)[4], const T* p) {
  const uint2 raw = *reinterpret_cast<const uint2*>(p);
  const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) x[i] = zc_to_float<T>(e[i]);
}

// Per token of a subset: minimum and maximum of y = x / c over the channels of ALL KV heads of
// its batch row, for K and for V (Alg. 1 on X in R^{n x hd}).  One warp per token; the row's
// first unit keeps the results.  grid: (tokens / 8, batch, class).
template <typename T>
__global__ void k_token_minmax(char* cache, ZcLayout lay, ZcSrc src, ZcSeg seg) {
  const int cls = blockIdx.z, n_c = seg.n_tok[cls];
  const int lane = threadIdx.x & 31, t = blockIdx.x * 8 + (threadIdx.x >> 5), b = blockIdx.y;
  if (t >= n_c || lay.bits[cls] == 16) return;
  char* ub0 = zc_unit_base(cache, lay, b * lay.n_kv);
  const int32_t* idx = reinterpret_cast<const int32_t*>(ub0 + lay.off_idx) + seg.idx_off + (cls == 0 ? 0 : seg.n_tok[0]);
  const long long row = (long long)idx[t] * src.sl;
  float mnK = INFINITY, mxK = -INFINITY, mnV = INFINITY, mxV = -INFINITY;
  for (int kv = 0; kv < lay.n_kv; ++kv) {
    const char* ub = zc_unit_base(cache, lay, b * lay.n_kv + kv);
    const unsigned* cmax = reinterpret_cast<const unsigned*>(ub + lay.off_cmax) + cls * 3 * ZC_D;
    const T* Kb = reinterpret_cast<const T*>(src.K) + b * src.sb + kv * src.sh + row + 4 * lane;
    const T* Vb = reinterpret_cast<const T*>(src.V) + b * src.sb + kv * src.sh + row + 4 * lane;
    float xk[4], xv[4];
    raw4_load<T>(xk, Kb);
    raw4_load<T>(xv, Vb);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (!lay.kch) {   // channelwise keys have no token parameters
        const float y = __fdiv_rn(xk[e], channel_factor(cmax[4 * lane + e], lay.p16 != 0));
        mnK = fminf(mnK, y);
        mxK = fmaxf(mxK, y);
      }
      const float y = __fdiv_rn(xv[e], channel_factor(cmax[ZC_D + 4 * lane + e], lay.p16 != 0));
      mnV = fminf(mnV, y);
      mxV = fmaxf(mxV, y);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mnK = fminf(mnK, __shfl_xor_sync(0xffffffffu, mnK, o));
    mxK = fmaxf(mxK, __shfl_xor_sync(0xffffffffu, mxK, o));
    mnV = fminf(mnV, __shfl_xor_sync(0xffffffffu, mnV, o));
    mxV = fmaxf(mxV, __shfl_xor_sync(0xffffffffu, mxV, o));
  }
  if (lane == 0)
    reinterpret_cast<float4*>(ub0 + lay.off_tokmm)[(cls == 0 ? 0 : seg.n_tok[0]) + t] = make_float4(mnK, mxK, mnV, mxV);
}

// ------------------------------------------------------------------ CSTQuant + pack (arithmetic in zc_quant.cuh)
template <typename T> __device__ __forceinline__ void raw4(float (&x)[4], uint2 raw) {
  const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
  for (int i = 0; i < 4; ++i) x[i] = zc_to_float<T>(e[i]);
}

// One warp = one 16-token sub-block of a tile at a time (a lane: four channels of every token),
// `rounds` sub-blocks per warp.  K codes leave the registers as words of the canonical order
// (a shuffle joins the lanes of a word); V codes pass through the warp's own 2 KB of shared
// memory, from which each lane gathers its words of the fragment order; the tokens' (s, z) are
// kept by the lane of the token's number.  No barrier of the CTA.
// grid.x: CTAs of class 0 (8 * rounds sub-blocks each), then of class 1; grid.y: unit.
// GA: token groups over all heads (the row's statistics come from k_token_minmax); P16: 16-bit
// parameters; B8: a class of 8-bit codes.  Template parameters, so that the plain build carries none of them.
template <typename T, bool GA, bool P16, bool B8>
__global__ void __launch_bounds__(256, 4) k_quantize_pack(char* cache, ZcLayout lay, ZcSrc src, ZcSeg seg, int rounds) {
  __shared__ __align__(16) unsigned char stageV[8][ZC_SUB][ZC_D];
  const int unit = blockIdx.y, b = unit / lay.n_kv, kv = unit % lay.n_kv;
  const int per_tile = ZC_TILE / ZC_SUB;
  const int subs0 = per_tile * zc_ceil_div(seg.n_tok[0], ZC_TILE);
  const int ctas0 = zc_ceil_div(subs0, 8 * rounds);
  const int cls = (int)blockIdx.x < ctas0 ? 0 : 1;
  const int cta = cls == 0 ? blockIdx.x : blockIdx.x - ctas0;
  const int subs = per_tile * zc_ceil_div(seg.n_tok[cls], ZC_TILE);   // whole tiles: rows past the end are zero
  const int bits = lay.bits[cls];
  const float L = (float)((1 << bits) - 1);
  char* ub = zc_unit_base(cache, lay, unit);
  const int32_t* idx = reinterpret_cast<const int32_t*>(ub + lay.off_idx) + seg.idx_off +
                       (cls == 0 ? 0 : seg.n_tok[0]);
  const T* Kb = reinterpret_cast<const T*>(src.K) + b * src.sb + kv * src.sh;
  const T* Vb = reinterpret_cast<const T*>(src.V) + b * src.sb + kv * src.sh;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const bool kch = lay.kch != 0;
  constexpr bool p16 = P16;
  const int sub_bytes = zc_sub_bytes(bits, lay.kch, P16 ? 1 : 0);
  char* tiles = ub + lay.off_tiles[cls] + (long long)seg.tile0[cls] * lay.tile_bytes[cls];
  if (bits == 16) {
    // 16-bit "quantisation" (the 16/16 and 16/2 settings): the subset's rows are gathered into
    // the tile as they are, [K rows][V rows] per 16-token sub-block; rows past the end are zero
    for (int r = 0; r < rounds; ++r) {
      const int sb = (cta * rounds + r) * 8 + w;
      if (sb >= subs) break;
      char* sub = tiles + (long long)(sb / per_tile) * lay.tile_bytes[cls] + (sb % per_tile) * sub_bytes;
      for (int i = 0; i < ZC_SUB; ++i) {
        const int tt = sb * ZC_SUB + i;
        uint2 k = make_uint2(0, 0), v = make_uint2(0, 0);
        if (tt < seg.n_tok[cls]) {
          const long long row = (long long)idx[tt] * src.sl;
          k = *reinterpret_cast<const uint2*>(Kb + row + 4 * lane);
          v = *reinterpret_cast<const uint2*>(Vb + row + 4 * lane);
        }
        reinterpret_cast<uint2*>(sub + i * ZC_D * 2)[lane] = k;
        reinterpret_cast<uint2*>(sub + (ZC_SUB + i) * ZC_D * 2)[lane] = v;
      }
    }
    return;
  }
  const unsigned* cmax = reinterpret_cast<const unsigned*>(ub + lay.off_cmax) + cls * 3 * ZC_D;
  float* fac = reinterpret_cast<float*>(ub + lay.off_fac) + (seg.run0 + cls) * ZC_FAC_FLOATS;
  float cK[4], cV[4], zK[4];   // channelwise keys: cK holds the channel scales, zK the zero points
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const float mk = zc_key_float(cmax[4 * lane + e]);
    const float mv = zc_key_float(cmax[ZC_D + 4 * lane + e]);
    if (kch) {
      channel_params(zc_key_float(cmax[2 * ZC_D + 4 * lane + e]), mk, L, &cK[e], &zK[e]);
    } else {
      cK[e] = channel_factor(cmax[4 * lane + e], p16);
      zK[e] = 0.f;
    }
    cV[e] = channel_factor(cmax[ZC_D + 4 * lane + e], p16);
  }
  // the divisors that stay for all of the CTA's tokens: their correctly rounded reciprocals once
  float rK[4], rV[4];
  bool midK = true, midV = true;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    rK[e] = __frcp_rn(cK[e]);
    rV[e] = __frcp_rn(cV[e]);
    midK = midK && zc_mid(cK[e]);
    midV = midV && zc_mid(cV[e]);
  }
  const float rL = __frcp_rn(L);
  if (cta == 0 && w == 0) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      fac[4 * lane + e] = cK[e];
      fac[ZC_D + 4 * lane + e] = cV[e];
      if (kch) fac[ZC_FAC_ZK + 4 * lane + e] = zK[e];
    }
  }
  // token groups over all heads: the row's statistics, kept by its first unit
  const float4* tokmm = GA ? reinterpret_cast<const float4*>(zc_unit_base(cache, lay, b * lay.n_kv) + lay.off_tokmm) +
                                 (cls == 0 ? 0 : seg.n_tok[0])
                           : nullptr;
  const int k_row_bytes = 16 * bits;            // a token's K codes
  const int v_off = ZC_SUB * k_row_bytes;       // the sub-block's V codes follow its K codes, then the parameters
  float smax = 0.f;
  for (int r = 0; r < rounds; ++r) {
    const int sb = (cta * rounds + r) * 8 + w;
    if (sb >= subs) break;   // the same for the whole warp
    if (!ZC_CHECKED(seg.tile0[cls] + sb / per_tile < lay.cap_tiles[cls], ZC_DBG_QUANT_TILE)) break;
    char* sub = tiles + (long long)(sb / per_tile) * lay.tile_bytes[cls] + (sb % per_tile) * sub_bytes;
    float4 par = make_float4(0.f, 0.f, 0.f, 0.f);   // lane t < 16: (sK, zK, sV, zV) of the sub-block's token t
    // lane t < 16: the source row of the sub-block's token t (-1 past the end of the subset)
    int my_row = -1;
    if (lane < ZC_SUB && sb * ZC_SUB + lane < seg.n_tok[cls]) {
      my_row = idx[sb * ZC_SUB + lane];
      if (!ZC_CHECKED(my_row >= 0 && my_row < src.l, ZC_DBG_QUANT_ROW)) my_row = -1;
    }
    auto prefetch_batch = [&](int bat) {   // the batch's rows on their way while the one before is quantised
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int rowi = __shfl_sync(0xffffffffu, my_row, 4 * bat + i);
        if (rowi >= 0) {
          const long long row = (long long)rowi * src.sl;
          asm volatile("prefetch.global.L1 [%0];\n" ::"l"(Kb + row + 4 * lane));
          asm volatile("prefetch.global.L1 [%0];\n" ::"l"(Vb + row + 4 * lane));
        }
      }
    };
    prefetch_batch(0);
    // the sub-block's 16 token rows in four batches of four: gather a batch (memory-level
    // parallelism), then quantise it two rows at a time
#pragma unroll 1
    for (int bat = 0; bat < 4; ++bat) {
      uint2 rawK[4], rawV[4];
      if (bat + 1 < 4) prefetch_batch(bat + 1);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int rowi = __shfl_sync(0xffffffffu, my_row, 4 * bat + i);
        if (rowi >= 0) {
          const long long row = (long long)rowi * src.sl;
          rawK[i] = *reinterpret_cast<const uint2*>(Kb + row + 4 * lane);
          rawV[i] = *reinterpret_cast<const uint2*>(Vb + row + 4 * lane);
        } else {
          rawK[i] = make_uint2(0, 0);
          rawV[i] = make_uint2(0, 0);
        }
      }
      // one copy of the pair's code for the batch's two pairs (the kernel is straight-line code
      // executed once per warp and waits for instruction fetch when it grows)
#pragma unroll 1
      for (int pr = 0; pr < 2; ++pr) {
        const int ta = 4 * bat + 2 * pr;                       // the pair's tokens within the sub-block: ta, ta + 1
        const bool live_a = sb * ZC_SUB + ta < seg.n_tok[cls], live_b = sb * ZC_SUB + ta + 1 < seg.n_tok[cls];
        const uint2 rk_a = pr == 0 ? rawK[0] : rawK[2], rk_b = pr == 0 ? rawK[1] : rawK[3];
        const uint2 rv_a = pr == 0 ? rawV[0] : rawV[2], rv_b = pr == 0 ? rawV[1] : rawV[3];
        float x[4], sKa = 0.f, zKa = 0.f, sKb = 0.f, zKb = 0.f, sVa, zVa, sVb, zVb;
        unsigned kA, kB, vA, vB;
        // token groups over all heads: the row's (min, max) of y for the pair's tokens
        constexpr bool shared = GA;
        float4 mmA = make_float4(0.f, 0.f, 0.f, 0.f), mmB = mmA;
        if (shared) {
          if (live_a) mmA = tokmm[sb * ZC_SUB + ta];
          if (live_b) mmB = tokmm[sb * ZC_SUB + ta + 1];
        }
        raw4<T>(x, rk_a);
        if (kch) kA = quant_channel4_rc(x, cK, rK, midK, zK, L);
        else quant_token_rc(x, cK, rK, midK, L, rL, &sKa, &zKa, &kA, p16, shared, mmA.x, mmA.y);
        raw4<T>(x, rk_b);
        if (kch) kB = quant_channel4_rc(x, cK, rK, midK, zK, L);
        else quant_token_rc(x, cK, rK, midK, L, rL, &sKb, &zKb, &kB, p16, shared, mmB.x, mmB.y);
        raw4<T>(x, rv_a);
        quant_token_rc(x, cV, rV, midV, L, rL, &sVa, &zVa, &vA, p16, shared, mmA.z, mmA.w);
        raw4<T>(x, rv_b);
        quant_token_rc(x, cV, rV, midV, L, rL, &sVb, &zVb, &vB, p16, shared, mmB.z, mmB.w);
        if (!live_a) { kA = 0u; vA = 0u; sKa = zKa = sVa = zVa = 0.f; }
        if (!live_b) { kB = 0u; vB = 0u; sKb = zKb = sVb = zVb = 0.f; }
        smax = fmaxf(smax, fmaxf(sVa, sVb));
        if (lane == ta) par = make_float4(sKa, zKa, sVa, zVa);
        if (lane == ta + 1) par = make_float4(sKb, zKb, sVb, zVb);
        // K: straight from the registers
        if (B8 && bits == 8) {   // a lane's four codes are a word of the row
          *reinterpret_cast<unsigned*>(sub + ta * k_row_bytes + 4 * lane) = kA;
          *reinterpret_cast<unsigned*>(sub + (ta + 1) * k_row_bytes + 4 * lane) = kB;
        } else {
          bool tok_b, owner;
          int wr;
          const unsigned kw = bits == 4 ? zc_k_words(4, kA, kB, lane, &tok_b, &wr, &owner)
                                        : zc_k_words(2, kA, kB, lane, &tok_b, &wr, &owner);
          if (owner) *reinterpret_cast<unsigned*>(sub + (ta + (tok_b ? 1 : 0)) * k_row_bytes + 4 * wr) = kw;
        }
        // V: byte codes into the warp's staging rows
        *reinterpret_cast<unsigned*>(&stageV[w][ta][4 * lane]) = vA;
        *reinterpret_cast<unsigned*>(&stageV[w][ta + 1][4 * lane]) = vB;
      }
    }
    __syncwarp();
    // V: this lane's words of the fragment order, 16 bytes at a time
    if (B8 && bits == 8) {
#pragma unroll 1
      for (int q = 0; q < 4; ++q) {
        uint4 o;
        o.x = zc_v_word(8, stageV[w], q * 128 + lane * 4 + 0);
        o.y = zc_v_word(8, stageV[w], q * 128 + lane * 4 + 1);
        o.z = zc_v_word(8, stageV[w], q * 128 + lane * 4 + 2);
        o.w = zc_v_word(8, stageV[w], q * 128 + lane * 4 + 3);
        *reinterpret_cast<uint4*>(sub + v_off + (q * 128 + lane * 4) * 4) = o;
      }
    } else if (bits == 4) {
#pragma unroll
      for (int qd = 0; qd < 2; ++qd) {
        uint4 o;
        o.x = zc_v_word(4, stageV[w], qd * 128 + lane * 4 + 0);
        o.y = zc_v_word(4, stageV[w], qd * 128 + lane * 4 + 1);
        o.z = zc_v_word(4, stageV[w], qd * 128 + lane * 4 + 2);
        o.w = zc_v_word(4, stageV[w], qd * 128 + lane * 4 + 3);
        *reinterpret_cast<uint4*>(sub + v_off + (qd * 128 + lane * 4) * 4) = o;
      }
    } else {
      uint4 o;
      o.x = zc_v_word(2, stageV[w], lane * 4 + 0);
      o.y = zc_v_word(2, stageV[w], lane * 4 + 1);
      o.z = zc_v_word(2, stageV[w], lane * 4 + 2);
      o.w = zc_v_word(2, stageV[w], lane * 4 + 3);
      *reinterpret_cast<uint4*>(sub + v_off + lane * 16) = o;
    }
    // the tokens' parameters: (sK, zK, sV, zV), or (sV, zV) with channelwise keys
    if (lane < ZC_SUB) {
      if (p16) {   // (fp16 scale, int16 zero point) per tensor
        const unsigned k2 = (unsigned)__half_as_ushort(__float2half_rn(par.x)) | (unsigned)(unsigned short)(short)par.y << 16;
        const unsigned v2 = (unsigned)__half_as_ushort(__float2half_rn(par.z)) | (unsigned)(unsigned short)(short)par.w << 16;
        *reinterpret_cast<uint2*>(sub + 2 * v_off + lane * 8) = make_uint2(k2, v2);
      } else if (kch) {
        *reinterpret_cast<float2*>(sub + 2 * v_off + lane * 8) = make_float2(par.z, par.w);
      } else {
        *reinterpret_cast<float4*>(sub + 2 * v_off + lane * 16) = par;
      }
    }
    __syncwarp();   // the staging rows are free for the next sub-block
  }
  if (lane == 0 && smax > 0.f) atomicMax(reinterpret_cast<unsigned*>(&fac[2 * ZC_D]), __float_as_uint(smax));
}

}  // namespace

int zc_launch_topk(zc_cache* c, int n, int n_s, int idx_off, const int32_t* given_sal,
                   cudaStream_t st) {
  const int smem = given_sal ? ((n + 31) / 32) * 4 : 0;
  if (smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(k_topk_split, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
  }
  k_topk_split<<<c->lay.units, kTopkThreads, (size_t)smem, st>>>(c->base, c->lay, n, n_s, idx_off, given_sal);
  c->launches += 1;
  return (int)cudaGetLastError();
}

int zc_launch_share_scores(zc_cache* c, int n, cudaStream_t st) {
  k_share_scores<<<dim3(zc_ceil_div(n, 256), c->cfg.batch), 256, 0, st>>>(c->base, c->lay, n);
  c->launches += 1;
  return (int)cudaGetLastError();
}

int zc_launch_window_scores(zc_cache* c, const ZcFlushArgs& fl, cudaStream_t st) {
  k_window_scores<<<c->lay.units, ZC_MAX_WINDOW, 0, st>>>(c->base, c->lay, fl);
  c->launches += 1;
  return (int)cudaGetLastError();
}

int zc_launch_quantize(zc_cache* c, const ZcSrc& src, const ZcSeg& seg, cudaStream_t st) {
  const int tiles = zc_ceil_div(seg.n_tok[0], ZC_TILE) + zc_ceil_div(seg.n_tok[1], ZC_TILE);
  k_clear_cmax<<<c->lay.units, 128, 0, st>>>(c->base, c->lay, seg);
  c->launches += 1;
  if (tiles > 0) {
    // sub-blocks per warp of the quantiser: more than one once the grid is many waves deep (the
    // set-up of a CTA, its channels' factors and their reciprocals, is then paid less often)
    const int per_tile = ZC_TILE / ZC_SUB;
    const long long ctas1 = (long long)zc_ceil_div(tiles * per_tile, 8) * c->lay.units;
    const long long slots = (long long)c->n_sm * 4;
    const int rounds = ctas1 >= 16 * slots ? 4 : ctas1 >= 8 * slots ? 2 : 1;
    dim3 grid(zc_ceil_div(per_tile * zc_ceil_div(seg.n_tok[0], ZC_TILE), 8 * rounds) +
                  zc_ceil_div(per_tile * zc_ceil_div(seg.n_tok[1], ZC_TILE), 8 * rounds),
              c->lay.units);
    dim3 grid_max(zc_ceil_div(zc_ceil_div(seg.n_tok[0], ZC_TILE), kAbsTiles) +
                      zc_ceil_div(zc_ceil_div(seg.n_tok[1], ZC_TILE), kAbsTiles),
                  c->lay.units);
    const dim3 grid_mm(zc_ceil_div(std::max(seg.n_tok[0], seg.n_tok[1]), 8), c->cfg.batch, 2);
#define ZC_QUANT_GO(T)                                                                                   \
  do {                                                                                                 \
    const bool b8 = c->lay.bits[0] == 8 || c->lay.bits[1] == 8;   /* never together with 16-bit parameters */ \
    k_channel_absmax<T><<<grid_max, 256, 0, st>>>(c->base, c->lay, src, seg);                          \
    if (c->lay.grp_all) k_token_minmax<T><<<grid_mm, 256, 0, st>>>(c->base, c->lay, src, seg);         \
    if (c->lay.grp_all && c->lay.p16)                                                                  \
      k_quantize_pack<T, true, true, false><<<grid, 256, 0, st>>>(c->base, c->lay, src, seg, rounds);  \
    else if (c->lay.grp_all && b8)                                                                     \
      k_quantize_pack<T, true, false, true><<<grid, 256, 0, st>>>(c->base, c->lay, src, seg, rounds);  \
    else if (c->lay.grp_all)                                                                           \
      k_quantize_pack<T, true, false, false><<<grid, 256, 0, st>>>(c->base, c->lay, src, seg, rounds); \
    else if (c->lay.p16)                                                                               \
      k_quantize_pack<T, false, true, false><<<grid, 256, 0, st>>>(c->base, c->lay, src, seg, rounds); \
    else if (b8)                                                                                       \
      k_quantize_pack<T, false, false, true><<<grid, 256, 0, st>>>(c->base, c->lay, src, seg, rounds); \
    else                                                                                               \
      k_quantize_pack<T, false, false, false><<<grid, 256, 0, st>>>(c->base, c->lay, src, seg, rounds); \
  } while (0)
    if (c->cfg.dtype == ZC_F16) ZC_QUANT_GO(__half);
    else ZC_QUANT_GO(__nv_bfloat16);
#undef ZC_QUANT_GO
    c->launches += c->lay.grp_all ? 3 : 2;
  }
  return (int)cudaGetLastError();
}

int zc_debug_code_compress(int* out) {
#ifdef ZC_DEBUG
  return (int)cudaMemcpyFromSymbol(out, g_zc_debug_fault, sizeof(int));
#else
  *out = 0;
  return (int)cudaSuccess;
#endif
}
