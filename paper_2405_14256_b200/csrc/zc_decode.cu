// Append (Eq. 3) and single-query attention over the mixed-precision cache (Eq. 4, Alg. 3).
//
// Split-K: every unit's cache is cut into items (a range of 16-token sub-tiles of one
// precision class of one segment, or the full-precision tail); one CTA per item produces a
// partial (m, l, acc) per query head, and a combine kernel merges the partials in a fixed
// order, writes the output and, on probe steps, adds the step's attention over the tail's
// tokens to the window statistics.
//
// Dequantisation is folded so that it is never done per element:
//   q . k_hat_t = s_t (q' . code_t - z_t sum(q')),  q' = q * c^K        (per run)
//   o = c^V * (sum_t w_t code_t - sum_t w_t z_t),    w_t = a_t s_t
// Both contractions run on tensor cores (warp-level m16n8k16, f16 operands, f32 accumulate)
// with M = tokens for q'.code and M = channels for sum_t w_t code_t, N = the G query heads
// of the KV head.  A masked 32-bit word of packed codes IS a pair of f16 subnormals
// (code * 2^-24, times 16 / 4 / 64 for codes that sit higher in the word), which the
// tensor cores multiply exactly; the power-of-two factors are folded into q' (per channel),
// into the softmax weights (per token) and into the output rows.
//
// Each warp owns a ring of shared-memory stages filled by bulk asynchronous copies (one per
// 16-token sub-block, completion on an mbarrier), so a CTA needs no block-wide barrier in
// its main loop.  Every wait is bounded; a wait that runs out records an error code.
#include "zc_internal.h"
#include "zc_layout.cuh"
#include "zc_mma.cuh"

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kStages = 4;                 // ring depth per warp
constexpr int kStageBytes = 2304;          // largest sub-block (4-bit)
constexpr int kWarps = 4;
constexpr int kRingBytes = kWarps * kStages * kStageBytes;   // 36864
constexpr int kWaitLimit = 1 << 22;
constexpr float kPScale = 32768.f;         // 2^15: softmax weights are sent to f16 as p * s/smax * 2^15

__device__ int g_zc_error = 0;

struct ItemDesc {
  int kind;      // 0 = compressed run, 1 = tail
  int cls, run;  // precision class, factor-block index
  int sub_lo, sub_hi;  // absolute sub-tile range inside the class region
  int run_sub0;        // first sub-tile of the run
  int n_tok;           // tokens of the run (kind 0) or of the tail (kind 1)
};

__device__ inline ItemDesc decode_item(const ZcDecodePlan& p, int it) {
  ItemDesc d;
  d.kind = 0;
  int base = 0;
  for (int k = 0; k < 2; ++k) {
    if (it < base + p.split0[k]) {
      const int i = it - base;
      const int subs = (p.n0[k] + ZC_SUB - 1) / ZC_SUB;
      d.cls = k; d.run = k; d.run_sub0 = 0; d.n_tok = p.n0[k];
      d.sub_lo = min(subs, i * p.spi0[k]);
      d.sub_hi = min(subs, d.sub_lo + p.spi0[k]);
      return d;
    }
    base += p.split0[k];
  }
  const int i2 = it - base;
  if (i2 < 2 * (p.n_seg - 1)) {
    const int seg = 1 + i2 / 2, k = i2 & 1;
    d.cls = k; d.run = 2 * seg + k; d.n_tok = p.nw[k];
    d.run_sub0 = (ZC_TILE / ZC_SUB) * (p.tiles0[k] + (seg - 1) * p.tilesw[k]);
    d.sub_lo = d.run_sub0;
    d.sub_hi = d.run_sub0 + (p.nw[k] + ZC_SUB - 1) / ZC_SUB;
    return d;
  }
  d.kind = 1; d.cls = 0; d.run = 0; d.run_sub0 = 0;
  d.sub_lo = d.sub_hi = 0; d.n_tok = p.n_tail;
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

// ---- mbarrier / bulk-copy primitives ----
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(zc_smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, int bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(zc_smem_u32(bar)),
               "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, int parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      " selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(zc_smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, int bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n" ::"r"(
          zc_smem_u32(dst)),
      "l"(src), "r"(bytes), "r"(zc_smem_u32(bar))
      : "memory");
}

// q' B-fragment geometry: channel offset (inside the lane's 32-channel slice) and the power
// of two the matching A element carries, for MMA k-step ks and slot (0,1 -> b0; 2,3 -> b1).
template <int BITS> __device__ __forceinline__ void qfrag_geom(int ks, int slot, int* ch, float* inv_sigma) {
  if (BITS == 4) {
    const int jw = ks >> 1, hb = ks & 1;
    const int odd = slot >> 1, hi = slot & 1;           // b1 <-> nibbles 2hb+1, 2hb+5 (x16)
    *ch = 8 * jw + 2 * hb + odd + 4 * hi;
    *inv_sigma = odd ? (1.f / 16.f) : 1.f;
  } else {
    const int jw = ks >> 2, e = ks & 3, hb = e >> 1, pr = e & 1;
    const int odd = slot >> 1, hi = slot & 1;           // crumbs 4hb+2pr(+1), +8
    *ch = 16 * jw + 4 * hb + 2 * pr + odd + 8 * hi;
    const int pw = 2 * pr + odd;                         // sigma = 4^pw
    *inv_sigma = pw == 0 ? 1.f : (pw == 1 ? 0.25f : (pw == 2 ? (1.f / 16.f) : (1.f / 64.f)));
  }
}

// The compressed-run part of one item, for one warp.  A CTA serves up to four query heads
// (h0 .. h0+Gl-1).  q' is split into two f16 numbers, q' = hi + lo, carried in MMA columns
// n = head (hi) and n = 4 + head (lo): f16 alone would put ~1e-3 of rounding noise on the
// logits of outlier key channels.
template <int BITS>
__device__ __forceinline__ void run_subtiles(const ItemDesc& d, const char* class_base, char* ring,
                                             uint64_t* bars, const float* qp /*[G][128] smem*/,
                                             const float* hscale /*[8] smem*/, float inv_smax, int h0,
                                             int Gl, int warp, int lane, float (&oacc)[8][4],
                                             float (&m)[2], float (&l)[2], float (&zacc)[2], int* err) {
  constexpr int SB = ZC_SUB * (32 * BITS + 16);
  const int g = lane >> 2, t = lane & 3;
  // ---- B fragments of q' for column n = g, and sum(q') consistent with the f16 rounding ----
  uint32_t qb[8][2];
  float qsum_mine = 0.f;
  {
    const int hl = g & 3, is_lo = g >> 2;
    const bool live = hl < Gl;
    const float hs = live ? hscale[h0 + hl] : 0.f;
    const float* qrow = qp + (live ? h0 + hl : 0) * ZC_D + 32 * t;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        __half hv[2];
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          int ch; float is;
          qfrag_geom<BITS>(ks, 2 * r + e, &ch, &is);
          const float x = live ? qrow[ch] * hs * is : 0.f;
          const __half hi = __float2half_rn(x);
          const __half lo = __float2half_rn(x - __half2float(hi));
          hv[e] = is_lo ? lo : hi;
          qsum_mine += __half2float(hv[e]) * (1.f / is);   // exact: is is a power of two
        }
        const __half2 h2 = __halves2half2(hv[0], hv[1]);
        qb[ks][r] = *reinterpret_cast<const uint32_t*>(&h2);
      }
    }
  }
  qsum_mine += __shfl_xor_sync(0xffffffffu, qsum_mine, 1);
  qsum_mine += __shfl_xor_sync(0xffffffffu, qsum_mine, 2);
  // after the hi+lo columns are added, this thread holds local heads 2(t&1) and 2(t&1)+1
  float zq[2], isc[2];
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int hl = 2 * (t & 1) + e;
    const float hs = hl < Gl ? hscale[h0 + hl] : 1.f;
    const float qs = __shfl_sync(0xffffffffu, qsum_mine, hl * 4) +
                     __shfl_sync(0xffffffffu, qsum_mine, (hl + 4) * 4);
    isc[e] = 16777216.f / hs;           // D * 2^24 / head scale = q' . code
    zq[e] = hl < Gl ? qs / hs : 0.f;    // sum(q')
  }

  const int n_sub = d.sub_hi - d.sub_lo;
  const int my_n = (n_sub - warp + kWarps - 1) / kWarps;     // sub-tiles of this warp
  char* my_ring = ring + warp * kStages * kStageBytes;
  uint64_t* my_bar = bars + warp * kStages;
  const char* src0 = class_base + (long long)(d.sub_lo + warp) * SB;
  if (lane == 0) {
    for (int s = 0; s < kStages && s < my_n; ++s) {
      mbar_expect_tx(&my_bar[s], SB);
      bulk_copy_g2s(my_ring + s * kStageBytes, src0 + (long long)s * kWarps * SB, SB, &my_bar[s]);
    }
  }
  bool dead = false;
  for (int i = 0; i < my_n; ++i) {
    const int s = i % kStages, parity = (i / kStages) & 1;
    if (!dead) {
      int spins = 0;
      while (!mbar_try_wait(&my_bar[s], parity)) {
        if (++spins > kWaitLimit) { dead = true; atomicExch(err, 1); break; }
      }
    }
    const char* st = my_ring + s * kStageBytes;
    const int tok0 = (d.sub_lo - d.run_sub0 + warp + i * kWarps) * ZC_SUB;   // first token of the sub-tile
    // ---- loads: K words of tokens g and g+8, V words, parameters ----
    uint32_t kw[2][BITS];   // 4-bit: 4 words per token, 2-bit: 2 words per token
    uint32_t vw[2 * BITS];  // 4-bit: 8 words, 2-bit: 4 words
    if (BITS == 4) {
      const uint4 a = *reinterpret_cast<const uint4*>(st + lane * 16);
      const uint4 b = *reinterpret_cast<const uint4*>(st + 512 + lane * 16);
      kw[0][0] = a.x; kw[0][1] = a.y; kw[0][2] = a.z; kw[0][3] = a.w;
      kw[1][0] = b.x; kw[1][1] = b.y; kw[1][2] = b.z; kw[1][3] = b.w;
      const uint4 c = *reinterpret_cast<const uint4*>(st + 1024 + lane * 16);
      const uint4 e = *reinterpret_cast<const uint4*>(st + 1536 + lane * 16);
      vw[0] = c.x; vw[1] = c.y; vw[2] = c.z; vw[3] = c.w;
      vw[4] = e.x; vw[5] = e.y; vw[6] = e.z; vw[7] = e.w;
    } else {
      const uint2 a = *reinterpret_cast<const uint2*>(st + lane * 8);
      const uint2 b = *reinterpret_cast<const uint2*>(st + 256 + lane * 8);
      kw[0][0] = a.x; kw[0][1] = a.y;
      kw[1][0] = b.x; kw[1][1] = b.y;
      const uint4 c = *reinterpret_cast<const uint4*>(st + 512 + lane * 16);
      vw[0] = c.x; vw[1] = c.y; vw[2] = c.z; vw[3] = c.w;
    }
    const float2 pk0 = *reinterpret_cast<const float2*>(st + 512 * BITS + g * 8);
    const float2 pk1 = *reinterpret_cast<const float2*>(st + 512 * BITS + (g + 8) * 8);
    const float2 pv0 = *reinterpret_cast<const float2*>(st + 512 * BITS + 128 + g * 8);
    const float2 pv1 = *reinterpret_cast<const float2*>(st + 512 * BITS + 128 + (g + 8) * 8);

    // ---- S^T = codes(16 tokens x 128) . q'^T : 8 k-steps ----
    float dacc[4] = {0.f, 0.f, 0.f, 0.f};
    if (BITS == 4) {
#pragma unroll
      for (int jw = 0; jw < 4; ++jw) {
        const uint32_t w0 = kw[0][jw], w1 = kw[1][jw];
        const uint32_t a0[4] = {w0 & 0x000F000Fu, w1 & 0x000F000Fu, w0 & 0x00F000F0u, w1 & 0x00F000F0u};
        zc_mma16816<__half>(dacc, a0, qb[2 * jw][0], qb[2 * jw][1]);
        const uint32_t x0 = w0 >> 8, x1 = w1 >> 8;
        const uint32_t a1[4] = {x0 & 0x000F000Fu, x1 & 0x000F000Fu, x0 & 0x00F000F0u, x1 & 0x00F000F0u};
        zc_mma16816<__half>(dacc, a1, qb[2 * jw + 1][0], qb[2 * jw + 1][1]);
      }
    } else {
#pragma unroll
      for (int jw = 0; jw < 2; ++jw) {
#pragma unroll
        for (int hb = 0; hb < 2; ++hb) {
          const uint32_t w0 = kw[0][jw] >> (8 * hb), w1 = kw[1][jw] >> (8 * hb);
          const uint32_t a0[4] = {w0 & 0x00030003u, w1 & 0x00030003u, w0 & 0x000C000Cu, w1 & 0x000C000Cu};
          zc_mma16816<__half>(dacc, a0, qb[4 * jw + 2 * hb][0], qb[4 * jw + 2 * hb][1]);
          const uint32_t a1[4] = {w0 & 0x00300030u, w1 & 0x00300030u, w0 & 0x00C000C0u, w1 & 0x00C000C0u};
          zc_mma16816<__half>(dacc, a1, qb[4 * jw + 2 * hb + 1][0], qb[4 * jw + 2 * hb + 1][1]);
        }
      }
    }
    // columns n and n+4 (hi and lo parts of q') live in lanes t and t^2: add them
#pragma unroll
    for (int e = 0; e < 4; ++e) dacc[e] += __shfl_xor_sync(0xffffffffu, dacc[e], 2);
    // ---- logits (base 2), online softmax for local heads 2(t&1), +1 over tokens g, g+8 ----
    const bool v0 = tok0 + g < d.n_tok, v1 = tok0 + g + 8 < d.n_tok;
    float lg[2][2];  // [token slot][head]
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      lg[0][e] = v0 ? pk0.x * (dacc[e] * isc[e] - pk0.y * zq[e]) : -INFINITY;
      lg[1][e] = v1 ? pk1.x * (dacc[2 + e] * isc[e] - pk1.y * zq[e]) : -INFINITY;
    }
    float mx[2] = {fmaxf(lg[0][0], lg[1][0]), fmaxf(lg[0][1], lg[1][1])};
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
      mx[0] = fmaxf(mx[0], __shfl_xor_sync(0xffffffffu, mx[0], o));
      mx[1] = fmaxf(mx[1], __shfl_xor_sync(0xffffffffu, mx[1], o));
    }
    const float mn0 = fmaxf(m[0], mx[0]), mn1 = fmaxf(m[1], mx[1]);
    if (mn0 > m[0] || mn1 > m[1]) {
      const float c0 = zc_exp2(m[0] - mn0), c1 = zc_exp2(m[1] - mn1);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        oacc[j][0] *= c0; oacc[j][1] *= c1; oacc[j][2] *= c0; oacc[j][3] *= c1;
      }
      l[0] *= c0; l[1] *= c1; zacc[0] *= c0; zacc[1] *= c1;
      m[0] = mn0; m[1] = mn1;
    }
    float p[2][2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      p[0][e] = zc_exp2(lg[0][e] - m[e]);
      p[1][e] = zc_exp2(lg[1][e] - m[e]);
      l[e] += p[0][e] + p[1][e];
    }
    // weights to f16: w' = p * s^V / smax * 2^15 (/4 for odd tokens at 2 bits)
    const float sig = (BITS == 2 && (g & 1)) ? 0.25f : 1.f;
    const float ws0 = pv0.x * inv_smax * kPScale * sig, ws1 = pv1.x * inv_smax * kPScale * sig;
    const float zs0 = pv0.y / sig, zs1 = pv1.y / sig;   // zero points times sigma'
    uint32_t X[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const __half2 h2 = __floats2half2_rn(p[0][e] * ws0, p[1][e] * ws1);   // (token g, token g+8)
      const float2 back = __half22float2(h2);
      zacc[e] += back.x * zs0 + back.y * zs1;
      X[e] = *reinterpret_cast<const uint32_t*>(&h2);
    }
    // B fragment of P^T for column n = g (local head g & 3, held by lanes t' = (g & 3) >> 1):
    // (tokens 2t, 2t+8) and (tokens 2t+1, 2t+9)
    const uint32_t sendA = (g & 1) ? X[1] : X[0];
    const uint32_t sendB = (g & 1) ? X[0] : X[1];
    const int odd = g & 1;
    const int srcA = ((2 * t + odd) << 2) | ((g & 3) >> 1);
    const int srcB = ((2 * t + 1 - odd) << 2) | ((g & 3) >> 1);
    const uint32_t rA = __shfl_sync(0xffffffffu, sendA, srcA);
    const uint32_t rB = __shfl_sync(0xffffffffu, sendB, srcB);
    const uint32_t pb0 = odd ? rB : rA, pb1 = odd ? rA : rB;
    // ---- O^T += V^T(128 channels x 16 tokens) . P^T : 8 M-tiles ----
    if (BITS == 4) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t w = vw[j], x = w >> 8;
        const uint32_t a[4] = {w & 0x000F000Fu, w & 0x00F000F0u, x & 0x000F000Fu, x & 0x00F000F0u};
        zc_mma16816<__half>(oacc[j], a, pb0, pb1);
      }
    } else {
#pragma unroll
      for (int mw = 0; mw < 4; ++mw) {
#pragma unroll
        for (int e2 = 0; e2 < 2; ++e2) {
          const uint32_t w = vw[mw] >> (8 * e2);
          const uint32_t a[4] = {w & 0x00030003u, w & 0x00300030u, w & 0x000C000Cu, w & 0x00C000C0u};
          zc_mma16816<__half>(oacc[2 * mw + e2], a, pb0, pb1);
        }
      }
    }
    // ---- refill this stage ----
    __syncwarp();
    if (lane == 0 && i + kStages < my_n) {
      mbar_expect_tx(&my_bar[s], SB);
      bulk_copy_g2s(my_ring + s * kStageBytes, src0 + (long long)(i + kStages) * kWarps * SB, SB,
                    &my_bar[s]);
    }
  }
}

template <typename T>
__global__ void __launch_bounds__(128, 4) k_decode_items(char* cache, ZcLayout lay, ZcDecodePlan plan,
                                                         const T* __restrict__ q, float* __restrict__ part,
                                                         float* __restrict__ tail_logits) {
  extern __shared__ __align__(128) char smem[];
  char* ring = smem;                                               // kRingBytes, reused for the merge
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kRingBytes);  // kWarps * kStages
  float* qp = reinterpret_cast<float*>(smem + kRingBytes + 128);    // [8][128]
  float* hscale = qp + ZC_MAX_G * ZC_D;                             // [8]
  float* wm = hscale + 8;                                           // [4 warps][4 heads] maxima
  float* wl = wm + 32;                                              // [4 warps][4 heads] sums
  const int unit = blockIdx.y, it = blockIdx.x;
  const int b = unit / lay.n_kv, kv = unit % lay.n_kv, G = lay.G;
  const int h0 = 4 * blockIdx.z, Gl = min(4, G - h0);              // this CTA's query heads
  const ItemDesc d = decode_item(plan, it);
  char* ub = zc_unit_base(cache, lay, unit);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, t = lane & 3;
  const float* fac = reinterpret_cast<const float*>(ub + lay.off_fac) + d.run * ZC_FAC_FLOATS;
  const float scale = kLog2e * rsqrtf((float)ZC_D);
  const bool has = d.kind == 0 ? d.sub_hi > d.sub_lo : d.n_tok > 0;
  float* my = part + (((long long)unit * plan.items + it) * G) * ZC_PART_STRIDE;

  if (tid == 0) {
    for (int i = 0; i < kWarps * kStages; ++i) mbar_init(&bars[i], 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
  }
  {
    const float cK = (d.kind == 0 && has) ? fac[tid] : 1.f;
    for (int h = 0; h < Gl; ++h)
      qp[(h0 + h) * ZC_D + tid] =
          zc_to_float<T>(q[((long long)b * lay.n_kv * G + kv * G + h0 + h) * ZC_D + tid]) * cK * scale;
  }
  __syncthreads();
  // per-head power-of-two scale that brings max |q'| under 2^14
  for (int h = h0 + warp; h < h0 + Gl; h += kWarps) {
    float mxq = 0.f;
#pragma unroll
    for (int e = 0; e < 4; ++e) mxq = fmaxf(mxq, fabsf(qp[h * ZC_D + lane + 32 * e]));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mxq = fmaxf(mxq, __shfl_xor_sync(0xffffffffu, mxq, o));
    if (lane == 0) hscale[h] = mxq > 0.f ? exp2f(floorf(14.f - log2f(mxq)) - 1.f) : 1.f;
  }
  __syncthreads();

  float* mbuf = reinterpret_cast<float*>(ring);   // [kWarps][4 heads][128], after the main loop
  if (d.kind == 0) {
    float oacc[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) oacc[j][e] = 0.f;
    float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f}, zacc[2] = {0.f, 0.f};
    if (has) {
      const float smax = fac[2 * ZC_D];
      const float inv_smax = smax > 0.f ? 1.f / smax : 0.f;
      const char* class_base = ub + lay.off_tiles[d.cls];
      if (lay.bits[d.cls] == 4)
        run_subtiles<4>(d, class_base, ring, bars, qp, hscale, inv_smax, h0, Gl, warp, lane, oacc, m,
                        l, zacc, &g_zc_error);
      else
        run_subtiles<2>(d, class_base, ring, bars, qp, hscale, inv_smax, h0, Gl, warp, lane, oacc, m,
                        l, zacc, &g_zc_error);
      // bring the accumulators to true units:
      //   o[ch][h] = c^V[ch] * smax * 2^-15 * (oacc * 2^24 / sigma(row) - zacc)
#pragma unroll
      for (int e = 0; e < 2; ++e) {
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) {
          l[e] += __shfl_xor_sync(0xffffffffu, l[e], o);
          zacc[e] += __shfl_xor_sync(0xffffffffu, zacc[e], o);
        }
      }
      const float k0 = smax / kPScale;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float c_lo = fac[ZC_D + 16 * j + g] * k0, c_hi = fac[ZC_D + 16 * j + g + 8] * k0;
        oacc[j][0] = c_lo * (oacc[j][0] * 16777216.f - zacc[0]);
        oacc[j][1] = c_lo * (oacc[j][1] * 16777216.f - zacc[1]);
        oacc[j][2] = c_hi * (oacc[j][2] * 1048576.f - zacc[0]);
        oacc[j][3] = c_hi * (oacc[j][3] * 1048576.f - zacc[1]);
      }
    }
    __syncthreads();   // the ring is free: every warp consumed all of its copies
    // lanes t = 0, 1 hold local heads 2t, 2t+1 in accumulator columns 2t, 2t+1
    if (t < 2) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int hl = 2 * t + e;
        if (hl < Gl) {
          if (g == 0) { wm[warp * 4 + hl] = m[e]; wl[warp * 4 + hl] = l[e]; }
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            mbuf[(warp * 4 + hl) * ZC_D + 16 * j + g] = oacc[j][e];
            mbuf[(warp * 4 + hl) * ZC_D + 16 * j + g + 8] = oacc[j][2 + e];
          }
        }
      }
    }
  } else {
    // ---- full-precision tail: one warp per token, lanes over channels, scalar FMAs ----
    float tm[4], tl_[4], tacc[4][4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      tm[h] = -INFINITY; tl_[h] = 0.f;
#pragma unroll
      for (int e = 0; e < 4; ++e) tacc[h][e] = 0.f;
    }
    for (int tok = warp; tok < d.n_tok; tok += kWarps) {
      float kc[4], vc[4];
      zc_load4<T>(reinterpret_cast<const T*>(ub + lay.off_tailK) + tok * ZC_D + 4 * lane, kc);
      zc_load4<T>(reinterpret_cast<const T*>(ub + lay.off_tailV) + tok * ZC_D + 4 * lane, vc);
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        if (h < Gl) {
          float dot = 0.f;
#pragma unroll
          for (int e = 0; e < 4; ++e) dot += qp[(h0 + h) * ZC_D + 4 * lane + e] * kc[e];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
          if (lane == 0) tail_logits[((long long)unit * G + h0 + h) * ZC_MAX_WINDOW + tok] = dot;
          const float mn = fmaxf(tm[h], dot);
          const float corr = zc_exp2(tm[h] - mn), pp = zc_exp2(dot - mn);
          tl_[h] = tl_[h] * corr + pp;
#pragma unroll
          for (int e = 0; e < 4; ++e) tacc[h][e] = tacc[h][e] * corr + pp * vc[e];
          tm[h] = mn;
        }
      }
    }
    __syncthreads();
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      if (h < Gl) {
        if (lane == 0) { wm[warp * 4 + h] = tm[h]; wl[warp * 4 + h] = tl_[h]; }
#pragma unroll
        for (int e = 0; e < 4; ++e) mbuf[(warp * 4 + h) * ZC_D + 4 * lane + e] = tacc[h][e];
      }
    }
  }
  __syncthreads();
  // merge the warps: thread = channel
  for (int h = 0; h < Gl; ++h) {
    float ms = -INFINITY;
#pragma unroll
    for (int w2 = 0; w2 < kWarps; ++w2) ms = fmaxf(ms, wm[w2 * 4 + h]);
    float ls = 0.f, o = 0.f;
#pragma unroll
    for (int w2 = 0; w2 < kWarps; ++w2) {
      const float mw = wm[w2 * 4 + h];
      const float cw = mw == -INFINITY ? 0.f : zc_exp2(mw - ms);
      ls += wl[w2 * 4 + h] * cw;
      o += mbuf[(w2 * 4 + h) * ZC_D + tid] * cw;
    }
    float* dst = my + (h0 + h) * ZC_PART_STRIDE;
    if (tid == 0) { dst[0] = ms; dst[1] = ls; }
    dst[4 + tid] = o;
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

constexpr int kDecodeSmem = kRingBytes + 128 + (ZC_MAX_G * ZC_D + 8 + 64) * 4;

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
  dim3 grid(plan.items, c->lay.units, (G + 3) / 4);
  cudaError_t e;
  if (c->cfg.dtype == ZC_F16) {
    e = cudaFuncSetAttribute(k_decode_items<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             kDecodeSmem);
    if (e != cudaSuccess) return e;
    k_decode_items<__half><<<grid, 128, kDecodeSmem, st>>>(c->base, c->lay, plan, (const __half*)q,
                                                           part, tail_logits);
    k_decode_combine<__half><<<c->lay.units, 128, 0, st>>>(c->base, c->lay, plan.items, plan.n_tail,
                                                           collect, part, tail_logits, (__half*)out);
  } else {
    e = cudaFuncSetAttribute(k_decode_items<__nv_bfloat16>,
                             cudaFuncAttributeMaxDynamicSharedMemorySize, kDecodeSmem);
    if (e != cudaSuccess) return e;
    k_decode_items<__nv_bfloat16><<<grid, 128, kDecodeSmem, st>>>(
        c->base, c->lay, plan, (const __nv_bfloat16*)q, part, tail_logits);
    k_decode_combine<__nv_bfloat16><<<c->lay.units, 128, 0, st>>>(
        c->base, c->lay, plan.items, plan.n_tail, collect, part, tail_logits, (__nv_bfloat16*)out);
  }
  c->launches += 2;
  return cudaGetLastError();
}

int zc_device_error_code(int* out) {
  return (int)cudaMemcpyFromSymbol(out, g_zc_error, sizeof(int));
}
