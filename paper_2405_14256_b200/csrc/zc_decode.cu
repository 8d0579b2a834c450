// Append (Eq. 3) and single-query attention over the mixed-precision cache (Eq. 4, Alg. 3).
//
// Split-K: every unit's cache is cut into items (a tile range of one precision class of one
// segment, or the full-precision tail); one CTA per item produces a partial (m, l, acc) per
// query head, and a combine kernel merges the partials in a fixed order, writes the output
// and, on probe steps, adds the step's attention over the tail's tokens to the window
// statistics.
//
// Dequantisation is folded so that it is never done per element:
//   q . k_hat_t = s_t (q' . code_t - z_t sum(q')),  q' = q * c^K        (per run)
//   o = c^V * (sum_t w_t code_t - sum_t w_t z_t),    w_t = a_t s_t
#include "zc_internal.h"
#include "zc_layout.cuh"
#include "zc_mma.cuh"

namespace {

constexpr float kLog2e = 1.4426950408889634f;

struct ItemDesc {
  int kind;      // 0 = compressed run, 1 = tail
  int cls, run;  // precision class, factor-block index
  int tile_lo, tile_hi;  // absolute tile range inside the class region
  int tok_lo, tok_hi;    // token range relative to the run's first tile
  int run_tile0;
};

__device__ inline ItemDesc decode_item(const ZcDecodePlan& p, int it) {
  ItemDesc d;
  d.kind = 0;
  int base = 0;
  for (int k = 0; k < 2; ++k) {
    if (it < base + p.split0[k]) {
      const int i = it - base;
      d.cls = k; d.run = k; d.run_tile0 = 0;
      const int lo = i * p.tpi0[k], hi = min(p.tiles0[k], lo + p.tpi0[k]);
      d.tile_lo = lo; d.tile_hi = max(lo, hi);
      d.tok_lo = lo * ZC_TILE; d.tok_hi = min(p.n0[k], hi * ZC_TILE);
      return d;
    }
    base += p.split0[k];
  }
  const int i2 = it - base;
  if (i2 < 2 * (p.n_seg - 1)) {
    const int seg = 1 + i2 / 2, k = i2 & 1;
    d.cls = k; d.run = 2 * seg + k;
    d.run_tile0 = p.tiles0[k] + (seg - 1) * p.tilesw[k];
    d.tile_lo = d.run_tile0; d.tile_hi = d.run_tile0 + p.tilesw[k];
    d.tok_lo = 0; d.tok_hi = p.nw[k];
    return d;
  }
  d.kind = 1; d.cls = 0; d.run = 0; d.run_tile0 = 0;
  d.tile_lo = d.tile_hi = 0; d.tok_lo = 0; d.tok_hi = p.n_tail;
  return d;
}

template <typename T>
__global__ void k_append(char* cache, ZcLayout lay, const T* __restrict__ k_new,
                         const T* __restrict__ v_new, int pos) {
  const int unit = blockIdx.x;
  char* ub = zc_unit_base(cache, lay, unit);
  T* tk = reinterpret_cast<T*>(ub + lay.off_tailK) + pos * ZC_D;
  T* tv = reinterpret_cast<T*>(ub + lay.off_tailV) + pos * ZC_D;
  const int i = threadIdx.x;  // 32 threads x 16 bytes = one 256-byte row per tensor
  if (i < 16)
    reinterpret_cast<uint4*>(tk)[i] = reinterpret_cast<const uint4*>(k_new + (long long)unit * ZC_D)[i];
  else
    reinterpret_cast<uint4*>(tv)[i - 16] =
        reinterpret_cast<const uint4*>(v_new + (long long)unit * ZC_D)[i - 16];
}

// ---------------------------------------------------------------------------------------
// Reference-grade item kernel: one warp per token, scalar FMAs.
// ---------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(128) k_decode_items(char* cache, ZcLayout lay, ZcDecodePlan plan,
                                                      const T* __restrict__ q, float* __restrict__ part,
                                                      float* __restrict__ tail_logits) {
  __shared__ float qp[ZC_MAX_G][ZC_D];
  __shared__ float qsum[ZC_MAX_G];
  __shared__ float red_m[4][ZC_MAX_G], red_l[4][ZC_MAX_G];
  __shared__ float red_acc[4][ZC_D];
  const int unit = blockIdx.y, it = blockIdx.x;
  const int b = unit / lay.n_kv, kv = unit % lay.n_kv, G = lay.G;
  const ItemDesc d = decode_item(plan, it);
  char* ub = zc_unit_base(cache, lay, unit);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const float* fac = reinterpret_cast<const float*>(ub + lay.off_fac) + d.run * ZC_FAC_FLOATS;
  const float scale = kLog2e * rsqrtf((float)ZC_D);
  const bool has = d.tok_hi > d.tok_lo;
  {
    const float cK = (d.kind == 0 && has) ? fac[tid] : 1.f;
    for (int g = 0; g < G; ++g)
      qp[g][tid] = zc_to_float<T>(q[((long long)b * lay.n_kv * G + kv * G + g) * ZC_D + tid]) * cK * scale;
  }
  __syncthreads();
  if (tid < G) {
    float s = 0.f;
    for (int i = 0; i < ZC_D; ++i) s += qp[tid][i];
    qsum[tid] = s;
  }
  __syncthreads();
  float m[ZC_MAX_G], l[ZC_MAX_G], zacc[ZC_MAX_G], acc[ZC_MAX_G][4];
#pragma unroll
  for (int g = 0; g < ZC_MAX_G; ++g) {
    m[g] = -INFINITY; l[g] = 0.f; zacc[g] = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[g][e] = 0.f;
  }
  const int bits = lay.bits[d.cls];
  const char* tiles = ub + lay.off_tiles[d.cls];
  for (int tok = d.tok_lo + warp; tok < d.tok_hi; tok += 4) {
    float kc[4], vc[4], sK = 1.f, zK = 0.f, sV = 1.f, zV = 0.f;
    if (d.kind == 0) {
      const int tile = d.run_tile0 + tok / ZC_TILE, tl = tok % ZC_TILE;
      const char* tp = tiles + (long long)tile * lay.tile_bytes[d.cls];
      const float* pk = reinterpret_cast<const float*>(tp + zc_tile_off_kpar(bits)) + 2 * tl;
      const float* pv = reinterpret_cast<const float*>(tp + zc_tile_off_vpar(bits)) + 2 * tl;
      sK = pk[0]; zK = pk[1]; sV = pv[0]; zV = pv[1];
      const unsigned char* krow = reinterpret_cast<const unsigned char*>(tp) + tl * 16 * bits;
      const unsigned* vblk = reinterpret_cast<const unsigned*>(tp + zc_tile_off_vcodes(bits)) +
                             (tl / ZC_SUB) * (64 * bits);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int ch = 4 * lane + e;
        const unsigned byte = krow[ch * bits / 8];
        kc[e] = (float)((byte >> ((ch * bits) & 7)) & ((1u << bits) - 1u));
        int word, shift;
        zc_vcode_pos(bits, tl % ZC_SUB, ch, &word, &shift);
        vc[e] = (float)((vblk[word] >> shift) & ((1u << bits) - 1u));
      }
    } else {
      const T* tk = reinterpret_cast<const T*>(ub + lay.off_tailK) + tok * ZC_D + 4 * lane;
      const T* tv = reinterpret_cast<const T*>(ub + lay.off_tailV) + tok * ZC_D + 4 * lane;
      zc_load4<T>(tk, kc);
      zc_load4<T>(tv, vc);
    }
    for (int g = 0; g < G; ++g) {
      float dot = 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) dot += qp[g][4 * lane + e] * kc[e];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
      const float logit = sK * (dot - zK * qsum[g]);
      if (d.kind == 1 && lane == 0)
        tail_logits[((long long)unit * G + g) * ZC_MAX_WINDOW + tok] = logit;
      const float mn = fmaxf(m[g], logit);
      const float corr = zc_exp2(m[g] - mn);
      const float p = zc_exp2(logit - mn);
      const float w = p * sV;
      l[g] = l[g] * corr + p;
      zacc[g] = zacc[g] * corr + w * zV;
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[g][e] = acc[g][e] * corr + w * vc[e];
      m[g] = mn;
    }
  }
  // merge the 4 warps, apply c^V, write the partial
  float cV[4];
#pragma unroll
  for (int e = 0; e < 4; ++e) cV[e] = (d.kind == 0 && has) ? fac[ZC_D + 4 * lane + e] : 1.f;
  float* my = part + (((long long)unit * plan.items + it) * G) * ZC_PART_STRIDE;
  for (int g = 0; g < G; ++g) {
    if (lane == 0) { red_m[warp][g] = m[g]; red_l[warp][g] = l[g]; }
    __syncthreads();
    float ms = fmaxf(fmaxf(red_m[0][g], red_m[1][g]), fmaxf(red_m[2][g], red_m[3][g]));
    const float cw = ms == -INFINITY ? 0.f : zc_exp2(m[g] - ms);
    for (int w2 = 0; w2 < 4; ++w2) {
      __syncthreads();
      if (warp == w2) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float v = (acc[g][e] - zacc[g]) * cw * cV[e];
          if (w2 == 0) red_acc[0][4 * lane + e] = v; else red_acc[0][4 * lane + e] += v;
        }
      }
    }
    __syncthreads();
    if (tid == 0) {
      float ls = 0.f;
      for (int w2 = 0; w2 < 4; ++w2)
        ls += red_l[w2][g] * (ms == -INFINITY ? 0.f : zc_exp2(red_m[w2][g] - ms));
      my[g * ZC_PART_STRIDE + 0] = ms;
      my[g * ZC_PART_STRIDE + 1] = ls;
    }
    my[g * ZC_PART_STRIDE + 4 + tid] = red_acc[0][tid];
    __syncthreads();
  }
}

template <typename T>
__global__ void __launch_bounds__(128) k_decode_combine(char* cache, ZcLayout lay, int items, int n_tail,
                                                        int collect, const float* __restrict__ part,
                                                        const float* __restrict__ tail_logits,
                                                        T* __restrict__ out) {
  __shared__ float s_m[ZC_MAX_G], s_l[ZC_MAX_G];
  const int unit = blockIdx.x, tid = threadIdx.x, G = lay.G;
  const int b = unit / lay.n_kv, kv = unit % lay.n_kv;
  const float* mine = part + (long long)unit * items * G * ZC_PART_STRIDE;
  if (tid < G) {
    float ms = -INFINITY;
    for (int i = 0; i < items; ++i) ms = fmaxf(ms, mine[(i * G + tid) * ZC_PART_STRIDE]);
    float ls = 0.f;
    for (int i = 0; i < items; ++i) {
      const float* p = mine + (i * G + tid) * ZC_PART_STRIDE;
      ls += p[1] * zc_exp2(p[0] - ms);
    }
    s_m[tid] = ms;
    s_l[tid] = ls;
  }
  __syncthreads();
  for (int g = 0; g < G; ++g) {
    float o = 0.f;
    for (int i = 0; i < items; ++i) {
      const float* p = mine + (i * G + g) * ZC_PART_STRIDE;
      o += p[4 + tid] * zc_exp2(p[0] - s_m[g]);
    }
    out[((long long)b * lay.n_kv * G + kv * G + g) * ZC_D + tid] = zc_from_float<T>(o / s_l[g]);
  }
  if (collect && tid < n_tail) {
    float a = 0.f;
    for (int g = 0; g < G; ++g)
      a += zc_exp2(tail_logits[((long long)unit * G + g) * ZC_MAX_WINDOW + tid] - s_m[g]) / s_l[g];
    float* colsum = reinterpret_cast<float*>(zc_unit_base(cache, lay, unit) + lay.off_colsum);
    colsum[tid] += a;
  }
}

}  // namespace

int zc_launch_append(zc_cache* c, const void* k_new, const void* v_new, int pos, cudaStream_t st) {
  if (c->cfg.dtype == ZC_F16)
    k_append<__half><<<c->lay.units, 32, 0, st>>>(c->base, c->lay, (const __half*)k_new,
                                                  (const __half*)v_new, pos);
  else
    k_append<__nv_bfloat16><<<c->lay.units, 32, 0, st>>>(c->base, c->lay, (const __nv_bfloat16*)k_new,
                                                         (const __nv_bfloat16*)v_new, pos);
  c->launches += 1;
  return cudaGetLastError();
}

int zc_launch_decode(zc_cache* c, const ZcDecodePlan& plan, const void* q, void* out, int collect,
                     float* ws, cudaStream_t st) {
  const int G = c->lay.G;
  float* part = ws;
  float* tail_logits = ws + (size_t)c->lay.units * plan.items * G * ZC_PART_STRIDE;
  dim3 grid(plan.items, c->lay.units);
  if (c->cfg.dtype == ZC_F16) {
    k_decode_items<__half><<<grid, 128, 0, st>>>(c->base, c->lay, plan, (const __half*)q, part,
                                                 tail_logits);
    k_decode_combine<__half><<<c->lay.units, 128, 0, st>>>(c->base, c->lay, plan.items, plan.n_tail,
                                                           collect, part, tail_logits, (__half*)out);
  } else {
    k_decode_items<__nv_bfloat16><<<grid, 128, 0, st>>>(c->base, c->lay, plan,
                                                        (const __nv_bfloat16*)q, part, tail_logits);
    k_decode_combine<__nv_bfloat16><<<c->lay.units, 128, 0, st>>>(
        c->base, c->lay, plan.items, plan.n_tail, collect, part, tail_logits, (__nv_bfloat16*)out);
  }
  c->launches += 2;
  return cudaGetLastError();
}
