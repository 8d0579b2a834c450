// Append (Eq. 3) and single-query attention over the mixed-precision cache (Eq. 4, Alg. 3).
//
// Split-K: every unit's compressed cache is cut into items (a range of 16-token sub-tiles of
// one precision class of one segment); a CTA works through one or more items and stores a
// partial (m, l, acc) per item and query head.  The attention over the full-precision tail runs
// on tensor cores in the input type, in a CTA of its own or in the unit's first item CTA.  The
// CTA of a unit that finishes last (an arrival counter tells) merges the unit's partials in a
// fixed order, writes the output and, on probe steps, adds the step's attention over the
// tail's tokens to the window statistics; when the call completes a window, the same CTA then
// re-compresses the unit's tail into a new segment (Alg. 3).  One kernel per call, nothing
// spins on another CTA.
// Consecutive calls on a stream are chained by programmatic dependent launch and run side by
// side; what orders them where they touch the same memory is described at ZcOrder and at
// zc_launch_decode.
//
// Dequantisation is folded so that it is never done per element:
//   q . k_hat_t = s_t (q' . code_t - z_t sum(q')),  q' = q * c^K        (per run)
//   o = c^V * (sum_t w_t code_t - sum_t w_t z_t),    w_t = a_t s_t
// Both contractions run on tensor cores (warp-level m16n8k16, f16 operands, f32 accumulate)
// with M = tokens for q'.code and M = channels for sum_t w_t code_t, N = the query heads of
// the KV head.  A masked 32-bit word of packed codes IS a pair of f16 subnormals
// (code * 2^-24, times 16 / 4 / 64 for codes that sit higher in the word), which the
// tensor cores multiply exactly; the power-of-two factors are folded into q' (per channel),
// into the softmax weights (per token) and into the output rows.
//
// Each warp owns a ring of shared-memory stages filled by bulk asynchronous copies (one per
// 16-token sub-block, completion on an mbarrier), so a CTA needs no block-wide barrier in
// its main loop.  Every wait is bounded; a wait that runs out records an error code.
#include <atomic>
#include <mutex>
#include "zc_internal.h"
#include "zc_layout.cuh"
#include "zc_mma.cuh"
#include "zc_order.h"
#include "zc_quant.cuh"

namespace {

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kMaxStages = 5;              // ring depth per warp: 3 pairs at 4 bits, 5 at 2 bits
constexpr int kWarps = 4;
// Two builds of the kernel: 3 CTAs per SM with a 13824-byte ring per warp (3 pairs in flight
// at 4 bits, 5 at 2 bits) for calls whose CTAs fit one or two waves, and 4 CTAs per SM with a
// 9216-byte ring (2 / 3 pairs) for calls of many waves and for calls that share the GPU with
// their neighbours, where more resident warps hide the set-up and merge of the others.
constexpr int kRingWide = 13824, kRingNarrow = 9216;
constexpr int kWaitLimit = 1 << 22;
constexpr int kPExp = 12;      // softmax weights go to f16 as p * s^V * 2^kPExp / 2^ceil(log2 smax)
constexpr float kTau = 3.5f;   // the running maximum is refreshed only when a logit exceeds it by this
constexpr unsigned kFull = 0xffffffffu;

// shared-memory map of an item CTA: small arrays first, then the warps' rings
constexpr int kOffBars = 0;                          // kWarps * kMaxStages mbarriers
constexpr int kOffQfrag = kOffBars + 256;            // q' B-fragments, 4 x 32 x uint4
constexpr int kOffRed = kOffQfrag + 2048;            // [kWarps] |q'| maxima as bits
constexpr int kOffWm = kOffRed + 64;                 // [kWarps][4] running maxima
constexpr int kOffWl = kOffWm + 64;                  // [kWarps][4] sums
constexpr int kOffWz = kOffWl + 64;                  // [kWarps][4] zero-point sums
constexpr int kOffCw = kOffWz + 64;                  // [4 heads][kWarps] merge weights
constexpr int kOffHead = kOffCw + 64;                // [4 heads] x (M, L, Z, -)
constexpr int kOffZq = kOffHead + 128;               // [kWarps][4 heads] partial sums of q' . z (channelwise keys)
constexpr int kOffRing = kOffZq + 128;               // kWarps rings
constexpr int decode_smem(int ring) { return kOffRing + kWarps * ring; }

__device__ int g_zc_error = 0;

struct ItemDesc {
  int kind;      // 0 = compressed run
  int cls, run;  // precision class, factor-block index
  int sub_lo, sub_hi;  // absolute sub-tile range inside the class region
  int run_sub0;        // first sub-tile of the run
  int n_tok;           // tokens of the run
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
  // not reached for it < plan.items
  d.kind = 1; d.cls = 0; d.run = 0; d.run_sub0 = 0; d.sub_lo = d.sub_hi = 0; d.n_tok = 0;
  return d;
}

// Programmatic dependent launch: the next kernel in the stream may start once every CTA has
// passed launch_dependents; wait() returns when the previous kernel has completed and its
// writes are visible.
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }

// Ordering between decode calls that run side by side on a stream.  One word per stream,
// (epoch tag << 20) | n, says that the first n calls of the epoch have completed; it is written
// by one CTA per kernel after that kernel's predecessor has completed.  A call that must not
// touch something before an earlier call of its epoch is done waits for the word to reach that
// call's number.  The calls waited for are always resident or finished (a kernel starts only
// after every CTA of its predecessor has started), so the wait ends; it is bounded all the same.
struct ZcOrder {
  unsigned* done;     // the stream's word
  unsigned tag;       // epoch tag
  int e;              // number of this call within its epoch
  int need_start;     // calls that must have completed before this call reads its inputs
  int need_end;       // ... before it writes partials, the output and the window statistics
  int epoch_start;    // launched without early start: everything before it has completed
};
__device__ __forceinline__ unsigned ld_order(const unsigned* p) {
  unsigned v;
  asm volatile("ld.volatile.global.u32 %0, [%1];\n" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// The same read as an acquire: what the thread loads afterwards is ordered behind it, without
// the cost of a fence.
__device__ __forceinline__ unsigned ld_order_acquire(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];\n" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ bool order_ok(unsigned v, unsigned tag, int need) {
  return (v >> 20) == tag && (int)(v & 0xFFFFFu) >= need;
}
__device__ __noinline__ void order_wait_slow(const unsigned* p, unsigned tag, int need, int* err) {
  if (*reinterpret_cast<volatile int*>(err) == 2) return;   // a wait already ran out: do not add to it
  for (int spins = 0; spins < (1 << 20); ++spins) {
    if (order_ok(ld_order(p), tag, need)) { __threadfence(); return; }
    __nanosleep(256);
  }
  atomicExch(err, 2);
}
// `first` is the value the thread read when it started: with ld_order_acquire if it goes on to
// READ what the earlier call wrote (need_start), so those loads are ordered behind the
// observation; stores and read-modify-writes issued after a wait need no such ordering.
__device__ __forceinline__ void order_wait(const ZcOrder& o, unsigned first, int need, int* err) {
  if (need <= 0 || order_ok(first, o.tag, need)) return;
  order_wait_slow(o.done, o.tag, need, err);
}

template <typename T>
__global__ void k_append(char* cache, ZcLayout lay, const T* __restrict__ k_new,
                         const T* __restrict__ v_new, int pos) {
  pdl_launch_dependents();
  pdl_wait();   // k_new / v_new may come from the previous kernel; the tail may still be read by it
  const int unit = blockIdx.x;
  if (!ZC_CHECKED(pos >= 0 && pos < lay.window, ZC_DBG_TAIL_ROW)) return;
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
__device__ __forceinline__ void mbar_inval(uint64_t* bar) {
  asm volatile("mbarrier.inval.shared::cta.b64 [%0];\n" ::"r"(zc_smem_u32(bar)) : "memory");
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
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;\n" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}

// Where channel `off` (0..31) of a lane's 32-channel slice of a K-code row sits in the MMA:
// B-fragment register (2 * k-step + {0: k = 2t,2t+1; 1: k = 2t+8,2t+9}), half e of it, and the
// inverse of the power of two that the matching masked code carries.
template <int BITS> __device__ __forceinline__ void chan_slot(int off, int* reg, int* e, float* inv_sigma) {
  if (BITS == 8) {
    // a word = four channels = one k-step: bytes 0, 2 are k = 2t, 2t+1; bytes 1, 3 are k = 2t+8, 2t+9
    const int jw = off >> 2, b = off & 3;
    *reg = 2 * jw + (b & 1);
    *e = b >> 1;
    *inv_sigma = 1.f;
  } else if (BITS == 4) {
    const int jw = off >> 3, hi = (off >> 2) & 1, hb = (off >> 1) & 1, odd = off & 1;
    *reg = 2 * (2 * jw + hb) + odd;
    *e = hi;
    *inv_sigma = odd ? (1.f / 16.f) : 1.f;
  } else {
    const int jw = off >> 4, hi = (off >> 3) & 1, hb = (off >> 2) & 1, pr = (off >> 1) & 1, odd = off & 1;
    *reg = 2 * (4 * jw + 2 * hb + pr) + odd;
    *e = hi;
    const int pw = 2 * pr + odd;   // sigma = 4^pw
    *inv_sigma = pw == 0 ? 1.f : (pw == 1 ? 0.25f : (pw == 2 ? (1.f / 16.f) : (1.f / 64.f)));
  }
}

__device__ __forceinline__ uint32_t shr8(uint32_t w) { return w >> 8; }

// expect_tx + bulk copy by one lane without a divergent branch
__device__ __forceinline__ void refill_if(bool pred, uint64_t* bar, void* dst, const void* src, int bytes) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %0, 0;\n"
      " @p mbarrier.arrive.expect_tx.shared::cta.b64 _, [%1], %2;\n"
      " @p cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%3], [%4], %2, [%1];\n}\n" ::"r"(
          (int)pred),
      "r"(zc_smem_u32(bar)), "r"(bytes), "r"(zc_smem_u32(dst)), "l"(src)
      : "memory");
}

struct PairState {
  float mu;       // running maximum of u = logit / isc
  float mo_neg;   // logKs - mu * isc
  float uthr;     // mu + kTau / isc
  float l, zacc;
};

// One PAIR of 16-token sub-tiles (one ring stage) for one warp: two independent chains of work
// keep the pipes busy between dependent instructions.  Column n of the q' B-fragments is
// (head n >> 1, part n & 1) with q' = hi + lo in f16, so that lane (g, t) receives both parts
// of head t for tokens g and g + 8 in its accumulator.  LAST: the pair may reach past the end
// of the run (`rem` tokens left from its first token); otherwise it is complete.
// KCH: channelwise keys -- a token has no key parameters (the channel scales are folded into
// q', qs is then sum_i q'_i z_i), its parameter slot holds (sV, zV) only.
// P16: a token's parameters are (fp16 scale, int16 zero point) pairs, 8 bytes (ZC_FLAG_PARAMS_F16).
template <int BITS, bool LAST, bool KCH, bool P16 = false>
__device__ __forceinline__ void pair_step(char* st, int lane, int rem, const uint32_t (&qb)[16],
                                          float qs, float isc, float logKs, float tau_u, int srcA,
                                          int srcB, int c0_src, int c1_src, float (&oacc)[8][4],
                                          PairState& S) {
  constexpr int PARB = (KCH || P16) ? 8 : 16;
  constexpr int SB = ZC_SUB * (32 * BITS + PARB);
  const int g = lane >> 2;
  if (LAST && rem <= ZC_SUB) {
    // the run ends inside the first half: the second half was not copied; its tokens are
    // masked below, its parameters must not hold stale bits
    if (KCH || P16) {
      if (lane < ZC_SUB) *reinterpret_cast<float2*>(st + SB + 512 * BITS + lane * 8) = make_float2(0.f, 0.f);
    } else {
      if (lane < ZC_SUB) *reinterpret_cast<float4*>(st + SB + 512 * BITS + lane * 16) = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    __syncwarp();
  }
  // ---- loads: K words of tokens g and g+8, V words, parameters (sK, zK, sV, zV), both halves ----
  uint32_t kw[2][2][BITS];   // [half][token slot][word]
  uint32_t vw[2][2 * BITS];
  float4 pp[2][2];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const char* sh = st + h * SB;
    if (BITS == 8) {
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const uint4 a = *reinterpret_cast<const uint4*>(sh + lane * 32 + 16 * q);
        const uint4 b = *reinterpret_cast<const uint4*>(sh + 1024 + lane * 32 + 16 * q);
        kw[h][0][4 * q] = a.x; kw[h][0][4 * q + 1] = a.y; kw[h][0][4 * q + 2] = a.z; kw[h][0][4 * q + 3] = a.w;
        kw[h][1][4 * q] = b.x; kw[h][1][4 * q + 1] = b.y; kw[h][1][4 * q + 2] = b.z; kw[h][1][4 * q + 3] = b.w;
      }
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const uint4 c = *reinterpret_cast<const uint4*>(sh + 2048 + q * 512 + lane * 16);
        vw[h][4 * q] = c.x; vw[h][4 * q + 1] = c.y; vw[h][4 * q + 2] = c.z; vw[h][4 * q + 3] = c.w;
      }
    } else if (BITS == 4) {
      const uint4 a = *reinterpret_cast<const uint4*>(sh + lane * 16);
      const uint4 b = *reinterpret_cast<const uint4*>(sh + 512 + lane * 16);
      kw[h][0][0] = a.x; kw[h][0][1] = a.y; kw[h][0][2] = a.z; kw[h][0][3] = a.w;
      kw[h][1][0] = b.x; kw[h][1][1] = b.y; kw[h][1][2] = b.z; kw[h][1][3] = b.w;
      const uint4 c = *reinterpret_cast<const uint4*>(sh + 1024 + lane * 16);
      const uint4 e = *reinterpret_cast<const uint4*>(sh + 1536 + lane * 16);
      vw[h][0] = c.x; vw[h][1] = c.y; vw[h][2] = c.z; vw[h][3] = c.w;
      vw[h][4] = e.x; vw[h][5] = e.y; vw[h][6] = e.z; vw[h][7] = e.w;
    } else {
      const uint2 a = *reinterpret_cast<const uint2*>(sh + lane * 8);
      const uint2 b = *reinterpret_cast<const uint2*>(sh + 256 + lane * 8);
      kw[h][0][0] = a.x; kw[h][0][1] = a.y;
      kw[h][1][0] = b.x; kw[h][1][1] = b.y;
      const uint4 c = *reinterpret_cast<const uint4*>(sh + 512 + lane * 16);
      vw[h][0] = c.x; vw[h][1] = c.y; vw[h][2] = c.z; vw[h][3] = c.w;
    }
    if (P16) {
      const uint2 a = *reinterpret_cast<const uint2*>(sh + 512 * BITS + g * 8);
      const uint2 b = *reinterpret_cast<const uint2*>(sh + 512 * BITS + (g + 8) * 8);
      pp[h][0] = make_float4(__half2float(__ushort_as_half((unsigned short)a.x)), (float)(short)(a.x >> 16),
                             __half2float(__ushort_as_half((unsigned short)a.y)), (float)(short)(a.y >> 16));
      pp[h][1] = make_float4(__half2float(__ushort_as_half((unsigned short)b.x)), (float)(short)(b.x >> 16),
                             __half2float(__ushort_as_half((unsigned short)b.y)), (float)(short)(b.y >> 16));
    } else if (KCH) {
      const float2 a = *reinterpret_cast<const float2*>(sh + 512 * BITS + g * 8);
      const float2 b = *reinterpret_cast<const float2*>(sh + 512 * BITS + (g + 8) * 8);
      pp[h][0] = make_float4(1.f, 1.f, a.x, a.y);
      pp[h][1] = make_float4(1.f, 1.f, b.x, b.y);
    } else {
      pp[h][0] = *reinterpret_cast<const float4*>(sh + 512 * BITS + g * 16);
      pp[h][1] = *reinterpret_cast<const float4*>(sh + 512 * BITS + (g + 8) * 16);
    }
  }
  // ---- S^T = codes(16 tokens x 128) . q'^T per half: 8 k-steps; the halves are independent chains ----
  float u[2][2];   // [half][token slot] logits (base 2) of head t, divided by isc
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    float dacc[4];
    if (BITS == 8) {
#pragma unroll
      for (int jw = 0; jw < 8; ++jw) {   // one word per token = one k-step
        const uint32_t w0 = kw[h][0][jw], w1 = kw[h][1][jw];
        const uint32_t a0[4] = {w0 & 0x00FF00FFu, w1 & 0x00FF00FFu, shr8(w0) & 0x00FF00FFu, shr8(w1) & 0x00FF00FFu};
        if (jw == 0) zc_mma16816_z(dacc, a0, qb[0], qb[1]);
        else zc_mma16816<__half>(dacc, a0, qb[2 * jw], qb[2 * jw + 1]);
      }
    } else if (BITS == 4) {
#pragma unroll
      for (int jw = 0; jw < 4; ++jw) {
        const uint32_t w0 = kw[h][0][jw], w1 = kw[h][1][jw];
        const uint32_t a0[4] = {w0 & 0x000F000Fu, w1 & 0x000F000Fu, w0 & 0x00F000F0u, w1 & 0x00F000F0u};
        if (jw == 0) zc_mma16816_z(dacc, a0, qb[0], qb[1]);
        else zc_mma16816<__half>(dacc, a0, qb[4 * jw], qb[4 * jw + 1]);
        const uint32_t x0 = shr8(w0), x1 = shr8(w1);
        const uint32_t a1[4] = {x0 & 0x000F000Fu, x1 & 0x000F000Fu, x0 & 0x00F000F0u, x1 & 0x00F000F0u};
        zc_mma16816<__half>(dacc, a1, qb[4 * jw + 2], qb[4 * jw + 3]);
      }
    } else {
#pragma unroll
      for (int jw = 0; jw < 2; ++jw) {
#pragma unroll
        for (int hb = 0; hb < 2; ++hb) {
          const uint32_t w0 = hb ? shr8(kw[h][0][jw]) : kw[h][0][jw];
          const uint32_t w1 = hb ? shr8(kw[h][1][jw]) : kw[h][1][jw];
          const int ks = 4 * jw + 2 * hb;
          const uint32_t a0[4] = {w0 & 0x00030003u, w1 & 0x00030003u, w0 & 0x000C000Cu, w1 & 0x000C000Cu};
          if (ks == 0) zc_mma16816_z(dacc, a0, qb[0], qb[1]);
          else zc_mma16816<__half>(dacc, a0, qb[2 * ks], qb[2 * ks + 1]);
          const uint32_t a1[4] = {w0 & 0x00300030u, w1 & 0x00300030u, w0 & 0x00C000C0u, w1 & 0x00C000C0u};
          zc_mma16816<__half>(dacc, a1, qb[2 * ks + 2], qb[2 * ks + 3]);
        }
      }
    }
    // hi and lo parts of q' sit in columns 2t and 2t+1 of this lane
    if (KCH) {
      u[h][0] = (dacc[0] + dacc[1]) - qs;
      u[h][1] = (dacc[2] + dacc[3]) - qs;
    } else {
      u[h][0] = fmaf(-pp[h][0].y, qs, dacc[0] + dacc[1]) * pp[h][0].x;
      u[h][1] = fmaf(-pp[h][1].y, qs, dacc[2] + dacc[3]) * pp[h][1].x;
    }
  }
  if (LAST && rem < 2 * ZC_SUB) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      if (16 * h + g >= rem) u[h][0] = -INFINITY;
      if (16 * h + g + 8 >= rem) u[h][1] = -INFINITY;
    }
  }
  const float mx = fmaxf(fmaxf(u[0][0], u[0][1]), fmaxf(u[1][0], u[1][1]));
  if (__any_sync(kFull, mx > S.uthr)) {
    float mr = mx;
    mr = fmaxf(mr, __shfl_xor_sync(kFull, mr, 4));
    mr = fmaxf(mr, __shfl_xor_sync(kFull, mr, 8));
    mr = fmaxf(mr, __shfl_xor_sync(kFull, mr, 16));
    const float mn = fmaxf(S.mu, mr);
    const float corr = mn == -INFINITY ? 1.f : zc_exp2((S.mu - mn) * isc);
    S.l *= corr; S.zacc *= corr;
    S.mu = mn; S.mo_neg = fmaf(-mn, isc, logKs); S.uthr = mn + tau_u;
    const float c0 = __shfl_sync(kFull, corr, c0_src), c1 = __shfl_sync(kFull, corr, c1_src);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      oacc[j][0] *= c0; oacc[j][1] *= c1; oacc[j][2] *= c0; oacc[j][3] *= c1;
    }
  }
  // p' = p * 2^logKs; weights w = p' * s^V go to the tensor cores as hi + lo in f16 (columns
  // 0..3 and 4..7 of P^T: a single f16 would put a relative error of 2^-11 on every weight,
  // which a few dominant tokens turn into an output error above 1e-3)
  uint32_t pb[2][2];
  const bool lo_col = g >= 4;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const float p0 = zc_exp2(fmaf(u[h][0], isc, S.mo_neg)), p1 = zc_exp2(fmaf(u[h][1], isc, S.mo_neg));
    S.l += p0 + p1;
    const float w0 = p0 * pp[h][0].z, w1 = p1 * pp[h][1].z;
    S.zacc = fmaf(w0, pp[h][0].w, S.zacc);
    S.zacc = fmaf(w1, pp[h][1].w, S.zacc);
    const __half2 h2 = __floats2half2_rn(w0, w1);   // (token g, token g+8)
    const float2 back = __half22float2(h2);
    const __half2 l2 = __floats2half2_rn(w0 - back.x, w1 - back.y);
    const uint32_t Xh = *reinterpret_cast<const uint32_t*>(&h2);
    const uint32_t Xl = *reinterpret_cast<const uint32_t*>(&l2);
    // B fragment of P^T, column n = g: head g & 3, part g >> 2; (tokens 2t, 2t+8) and (2t+1, 2t+9)
    const uint32_t ah = __shfl_sync(kFull, Xh, srcA), al = __shfl_sync(kFull, Xl, srcA);
    const uint32_t bh = __shfl_sync(kFull, Xh, srcB), bl = __shfl_sync(kFull, Xl, srcB);
    pb[h][0] = lo_col ? al : ah;
    pb[h][1] = lo_col ? bl : bh;
  }
  // ---- O^T += V^T(128 channels x 16 tokens) . P^T per half: 8 M-tiles ----
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    if (BITS == 8) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {   // channel rows g and g + 8 in a word each; bytes = tokens 2t, 2t+1, 2t+8, 2t+9
        const uint32_t w0 = vw[h][2 * j], w1 = vw[h][2 * j + 1];
        const uint32_t a[4] = {w0 & 0x00FF00FFu, w1 & 0x00FF00FFu, shr8(w0) & 0x00FF00FFu, shr8(w1) & 0x00FF00FFu};
        zc_mma16816<__half>(oacc[j], a, pb[h][0], pb[h][1]);
      }
    } else if (BITS == 4) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint32_t w = vw[h][j], x = shr8(w);
        const uint32_t a[4] = {w & 0x000F000Fu, w & 0x00F000F0u, x & 0x000F000Fu, x & 0x00F000F0u};
        zc_mma16816<__half>(oacc[j], a, pb[h][0], pb[h][1]);
      }
    } else {
#pragma unroll
      for (int mw = 0; mw < 4; ++mw) {
#pragma unroll
        for (int e2 = 0; e2 < 2; ++e2) {
          const uint32_t w = e2 ? shr8(vw[h][mw]) : vw[h][mw];
          const uint32_t a[4] = {w & 0x00030003u, w & 0x00300030u, w & 0x000C000Cu, w & 0x00C000C0u};
          zc_mma16816<__half>(oacc[2 * mw + e2], a, pb[h][0], pb[h][1]);
        }
      }
    }
  }
}

// Compressed-run part of one item, one warp: prologue done by the CTA, stages primed.  The
// first my_np - NST iterations refill their stage and need no end-of-run handling; the last
// NST do not refill and the very last pair may be cut short by the end of the run.
template <int BITS, int RING, bool KCH, bool P16 = false>
__device__ __forceinline__ void run_pairs(const ItemDesc& d, const char* class_base, char* my_ring,
                                          uint64_t* my_bar, const uint32_t (&qb)[16], float qs,
                                          float isc, float logK, int my_np, int warp, int lane,
                                          float (&oacc)[8][4], float& m_out, float& l_out,
                                          float& z_out, int* err) {
  constexpr int SB = ZC_SUB * (32 * BITS + ((KCH || P16) ? 8 : 16));
  constexpr int PB = 2 * SB;
  constexpr int NST = (RING / PB) < kMaxStages ? (RING / PB) : kMaxStages;
  const int g = lane >> 2, t = lane & 3;
  const bool odd_tok = BITS == 2 && (g & 1);
  const float logKs = logK - (odd_tok ? 2.f : 0.f);      // weights of odd tokens carry 1/4 at 2 bits
  // columns 4..7 of P^T carry the lo parts of the weights of heads 0..3
  const int srcA = 8 * t + (g & 3), srcB = srcA + 4;
  const int c0_src = (lane & ~3) | ((2 * t) & 3), c1_src = (lane & ~3) | ((2 * t + 1) & 3);
  // Logits are kept divided by isc (u = lg / isc): u costs one multiply less per token.
  PairState S;
  S.mu = -INFINITY; S.mo_neg = 0.f; S.uthr = -INFINITY; S.l = 0.f; S.zacc = 0.f;
  const float tau_u = kTau / isc;
  const int s_first = d.sub_lo + 2 * warp;
  const int rem0 = d.n_tok - (s_first - d.run_sub0) * ZC_SUB;   // tokens from the first pair's first token to the run's end
  const char* src_refill = class_base + (long long)(s_first + 2 * kWarps * NST) * SB;
  int rem_refill = rem0 - 2 * ZC_SUB * kWarps * NST;
  int stage = 0;
  uint32_t parity = 0;
  auto wait_stage = [&](uint64_t* bar) {
    if (!mbar_try_wait(bar, parity)) {
      int spins = 0;
      while (!mbar_try_wait(bar, parity)) {
        if (++spins > kWaitLimit) { atomicExch(err, 1); break; }
      }
    }
  };
  // One loop body for every pair (the end-of-run handling costs two uniform compares per pair;
  // a second copy of the unrolled step for the last pairs would double the loop's code, and the
  // instruction cache is what this loop runs out of first).
  const int n_refill = my_np - NST;
  for (int i = 0; i < my_np; ++i) {
    uint64_t* bar = &my_bar[stage];
    wait_stage(bar);
    char* st = my_ring + stage * PB;
    pair_step<BITS, true, KCH, P16>(st, lane, rem0 - i * (2 * ZC_SUB * kWarps), qb, qs, isc, logKs, tau_u, srcA, srcB,
                               c0_src, c1_src, oacc, S);
    __syncwarp();
    refill_if(lane == 0 && i < n_refill, bar, st, src_refill, rem_refill > ZC_SUB ? PB : SB);
    src_refill += kWarps * PB;
    rem_refill -= 2 * ZC_SUB * kWarps;
    if (++stage == NST) { stage = 0; parity ^= 1u; }
  }
  // sums back to plain units: l' = sum p 2^logKs; zacc' = sum w z with w short by the odd-token 1/4
  const float inv_sig = odd_tok ? 4.f : 1.f;
  l_out = S.l * zc_exp2(-logKs);
  z_out = S.zacc * inv_sig;
  m_out = S.mu * isc;
}

// One compressed item, whole CTA.  On return every warp has put its (m, l, z-sum) and its
// accumulators into shared memory; *chan_factor / *rowscale tell the merge how to bring a
// channel's accumulator to true units.
// Not inlined: the loop inside gets the whole register budget to itself, whatever the caller
// keeps alive around the call.
struct ItemScale { float chan_factor, rowscale; };
template <typename T, int BITS, int RING, bool KCH, bool P16 = false>
__device__ __noinline__ ItemScale compressed_item(ItemDesc d, const char* class_base, const float* fac,
                                                  const T* qbase, int Gl, char* smem, int* err) {
  constexpr int SB = ZC_SUB * (32 * BITS + ((KCH || P16) ? 8 : 16));
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  constexpr int PB = 2 * SB;
  constexpr int NST = (RING / PB) < kMaxStages ? (RING / PB) : kMaxStages;
  char* my_ring = smem + kOffRing + warp * RING;
  uint64_t* my_bar = reinterpret_cast<uint64_t*>(smem + kOffBars) + warp * kMaxStages;
  uint4* qfrag = reinterpret_cast<uint4*>(smem + kOffQfrag);
  unsigned* s_red = reinterpret_cast<unsigned*>(smem + kOffRed);
  float* wm = reinterpret_cast<float*>(smem + kOffWm);
  float* wl = reinterpret_cast<float*>(smem + kOffWl);
  float* wz = reinterpret_cast<float*>(smem + kOffWz);
  const int n_pairs = (d.sub_hi - d.sub_lo + 1) >> 1;
  const int my_np = n_pairs > warp ? (n_pairs - warp + kWarps - 1) / kWarps : 0;
  // ---- the few words the set-up needs go out first, ahead of this CTA's own 55 KB of copies ----
  const float scale = kLog2e * rsqrtf((float)ZC_D);
  const float cK = fac[tid];              // channelwise keys: the channel's scale
  const float cV = fac[ZC_D + tid];
  const float smax = fac[2 * ZC_D];
  const float zK = KCH ? fac[ZC_FAC_ZK + tid] : 0.f;
  T qraw[4];   // used only after the copies below are on their way
#pragma unroll
  for (int h = 0; h < 4; ++h) qraw[h] = qbase[(h < Gl ? h : 0) * ZC_D + tid];
  // ---- then the code copies: their latency covers the q' set-up ----
  if (lane == 0) {
    for (int s = 0; s < NST; ++s) mbar_init(&my_bar[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");   // init visible to the copy engine
    for (int s = 0; s < NST && s < my_np; ++s) {
      const int sn = d.sub_lo + 2 * (warp + s * kWarps);
      const int bytes = sn + 1 < d.sub_hi ? PB : SB;
      mbar_expect_tx(&my_bar[s], bytes);
      bulk_copy_g2s(my_ring + s * PB, class_base + (long long)sn * SB, bytes, &my_bar[s]);
    }
  }
  // ---- q' = q * c^K * log2(e)/sqrt(d); thread = channel ----
  float x[4];
#pragma unroll
  for (int h = 0; h < 4; ++h) x[h] = h < Gl ? zc_to_float<T>(qraw[h]) * cK * scale : 0.f;
  {
    const float ax = fmaxf(fmaxf(fabsf(x[0]), fabsf(x[1])), fmaxf(fabsf(x[2]), fabsf(x[3])));
    const unsigned mb = __reduce_max_sync(kFull, __float_as_uint(ax));
    if (lane == 0) s_red[warp] = mb;
  }
  __syncthreads();
  // one power of two per CTA that brings max |q'| into [2^13, 2^14): keeps the lo parts normal in f16
  const unsigned ex_q = max(max(s_red[0], s_red[1]), max(s_red[2], s_red[3])) >> 23;
  const bool scaled = ex_q >= 14u && ex_q < 255u;
  {
    int reg, e;
    float is;
    chan_slot<BITS>(tid & 31, &reg, &e, &is);
    const int t_l = tid >> 5;
    __half* qh = reinterpret_cast<__half*>(qfrag);
    const float hs_is = (scaled ? __uint_as_float((267u - ex_q) << 23) : 1.f) * is;
    const int base = ((reg >> 2) * 32 + t_l) * 4 + (reg & 3);          // + 4 * (4 * column)
    float zq[4];   // channelwise keys: this channel's share of sum_i q'_i z_i, in the accumulator's units
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      const float xs = x[h] * hs_is;
      const __half hi = __float2half_rn(xs);
      const __half lo = __float2half_rn(xs - __half2float(hi));
      qh[(base + 16 * (2 * h)) * 2 + e] = hi;
      qh[(base + 16 * (2 * h + 1)) * 2 + e] = lo;
      // the operands as the tensor cores see them, times the code's power of two (1 / is), 2^-24
      if (KCH) zq[h] = (__half2float(hi) + __half2float(lo)) * (zK * (5.9604644775390625e-8f / is));
    }
    if (KCH) {
#pragma unroll
      for (int h = 0; h < 4; ++h) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) zq[h] += __shfl_xor_sync(kFull, zq[h], o);
      }
      if (lane == 0) {
        float* zred = reinterpret_cast<float*>(smem + kOffZq);
#pragma unroll
        for (int h = 0; h < 4; ++h) zred[warp * 4 + h] = zq[h];
      }
    }
  }
  __syncthreads();
  uint32_t qb[16];
#pragma unroll
  for (int q4 = 0; q4 < 4; ++q4) {
    const uint4 v = qfrag[q4 * 32 + lane];
    qb[4 * q4] = v.x; qb[4 * q4 + 1] = v.y; qb[4 * q4 + 2] = v.z; qb[4 * q4 + 3] = v.w;
  }
  // sum of q' exactly as the f16 operands represent it: one MMA pass against all-one codes
  float ds[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    uint32_t one_lo, one_hi;
    if (BITS == 8) { one_lo = 0x00010001u; one_hi = 0x00010001u; }
    else if (BITS == 4) { one_lo = 0x00010001u; one_hi = 0x00100010u; }
    else if ((ks & 1) == 0) { one_lo = 0x00010001u; one_hi = 0x00040004u; }
    else { one_lo = 0x00100010u; one_hi = 0x00400040u; }
    const uint32_t a[4] = {one_lo, one_lo, one_hi, one_hi};
    zc_mma16816<__half>(ds[ks & 1], a, qb[2 * ks], qb[2 * ks + 1]);
  }
  float qs = (ds[0][0] + ds[1][0]) + (ds[0][1] + ds[1][1]);
  if (KCH) {
    const float* zred = reinterpret_cast<const float*>(smem + kOffZq);
    qs = (zred[t] + zred[4 + t]) + (zred[8 + t] + zred[12 + t]);   // sum_i q'_i z_i of head t
  }
  // accumulator * 2^24 / CTA scale = q' . code
  const float isc = 16777216.f * (scaled ? __uint_as_float((ex_q - 13u) << 23) : 1.f);
  // weights are scaled by 2^logK = 2^kPExp / 2^ceil(log2 smax) so that w <= 2^(kPExp + kTau)
  const int es = (int)((__float_as_uint(smax) >> 23) & 255u) - 127;
  const float logK = (float)(kPExp - es - 1);

  float oacc[8][4];
#pragma unroll
  for (int j = 0; j < 8; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) oacc[j][e] = 0.f;
  float m, l, z;
  run_pairs<BITS, RING, KCH, P16>(d, class_base, my_ring, my_bar, qb, qs, isc, logK, my_np, warp, lane, oacc, m, l, z, err);
  __syncwarp();
  if (lane == 0)   // every copy has landed and been consumed: retire the barriers
    for (int s = 0; s < NST; ++s) mbar_inval(&my_bar[s]);
#pragma unroll
  for (int o = 4; o < 32; o <<= 1) {
    l += __shfl_xor_sync(kFull, l, o);
    z += __shfl_xor_sync(kFull, z, o);
  }
  if (g == 0) { wm[warp * 4 + t] = m; wl[warp * 4 + t] = l; wz[warp * 4 + t] = z; }
  // columns 4..7 (lanes t >= 2) hold the products of the weights' lo parts for heads 0..3
#pragma unroll
  for (int j = 0; j < 8; ++j)
#pragma unroll
    for (int e = 0; e < 4; ++e) oacc[j][e] += __shfl_xor_sync(kFull, oacc[j][e], 2);
  // the warp's own ring is free (all of its copies were consumed): accumulators go there
  float* mbuf = reinterpret_cast<float*>(my_ring);   // [4 heads][128]
  __syncwarp();
  if (t < 2) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        mbuf[(2 * t + e) * ZC_D + 16 * j + g] = oacc[j][e];
        mbuf[(2 * t + e) * ZC_D + 16 * j + g + 8] = oacc[j][2 + e];
      }
    }
  }
  // o[ch] = c^V[ch] 2^-logK (acc 2^24 / sigma(row) - z sum); rows g+8 of a tile carry sigma = 16
  ItemScale r;
  r.chan_factor = cV * zc_exp2(-logK);
  r.rowscale = (BITS != 8 && (tid & 8)) ? 1048576.f : 16777216.f;   // 8-bit codes carry no power of two
  return r;
}

// Sixteen tokens of the full-precision tail for one warp and up to four query heads, on tensor
// cores in the input type: S^T = K_tail q^T with q exact in its own type, then
// O^T = V_tail^T P^T with P = hi + lo in the input type (columns 0..3 and 4..7).
// The tile is a split-K partial of its own: (row maximum, sum) and the accumulators of head h
// go to dst + h * ZC_PART_STRIDE, the logits (base 2) of the tokens, when the step collects
// probe statistics, to stash [4 heads][ZC_MAX_WINDOW] (global memory).  One warp, no shared
// memory, no barrier: the warps of a CTA take tiles independently.
template <typename T>
__device__ __forceinline__ void tail_tile(const T* tK, const T* tV, int n_tail, int base,
                                          const T* qbase, int Gl, int unit, float* dst, float* stash,
                                          const T* k_new, const T* v_new) {
  const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int nv = min(ZC_SUB, n_tail - base);
  if (nv <= 0) return;
  const int last = n_tail - 1;
  // Deferred append: the newest row is read from the caller's k_new / v_new [unit][128] (the
  // unit's first item CTA stores it into the tail).
  const T* newK = k_new ? k_new + (long long)unit * ZC_D : nullptr;
  const T* newV = v_new ? v_new + (long long)unit * ZC_D : nullptr;
  // rows past the end are read from the last valid row and masked
  const int r0 = min(base + g, last), r1 = min(base + g + 8, last);
  const int va_r = min(base + 2 * t, last), vb_r = min(base + 2 * t + 8, last);
  const int vc_r = min(base + 2 * t + 1, last), vd_r = min(base + 2 * t + 9, last);
  auto krow = [&](int r) -> const T* { return (newK && r == last) ? newK : tK + r * ZC_D; };
  auto vrow = [&](int r) -> const T* { return (newV && r == last) ? newV : tV + r * ZC_D; };
  const T* k0p = krow(r0);
  const T* k1p = krow(r1);
  uint4 qv[4], ka[4], kb[4];
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    qv[c] = g < Gl ? *reinterpret_cast<const uint4*>(qbase + g * ZC_D + 32 * c + 8 * t) : make_uint4(0, 0, 0, 0);
    ka[c] = __ldcg(reinterpret_cast<const uint4*>(k0p + 32 * c + 8 * t));
    kb[c] = __ldcg(reinterpret_cast<const uint4*>(k1p + 32 * c + 8 * t));
  }
  // V: this lane's 16 channels (16g .. 16g+15) of the four tokens its fragments pair up
  const T* vap = vrow(va_r);
  const T* vbp = vrow(vb_r);
  const T* vcp = vrow(vc_r);
  const T* vdp = vrow(vd_r);
  uint4 va[2], vb[2], vc[2], vd[2];
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    va[u] = __ldcg(reinterpret_cast<const uint4*>(vap + 16 * g + 8 * u));
    vb[u] = __ldcg(reinterpret_cast<const uint4*>(vbp + 16 * g + 8 * u));
    vc[u] = __ldcg(reinterpret_cast<const uint4*>(vcp + 16 * g + 8 * u));
    vd[u] = __ldcg(reinterpret_cast<const uint4*>(vdp + 16 * g + 8 * u));
  }
  // ---- S^T: k-step (c, pp) contracts channels 32c + 8t + 4pp + {0,1 | 2,3} ----
  float dacc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    const uint32_t a0[4] = {ka[c].x, kb[c].x, ka[c].y, kb[c].y};
    zc_mma16816<T>(dacc, a0, qv[c].x, qv[c].y);
    const uint32_t a1[4] = {ka[c].z, kb[c].z, ka[c].w, kb[c].w};
    zc_mma16816<T>(dacc, a1, qv[c].z, qv[c].w);
  }
  const float scale = kLog2e * rsqrtf((float)ZC_D);
  const bool v0 = g < nv, v1 = g + 8 < nv;
  float lg[2][2];   // [token slot][head 2t + e]
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    lg[0][e] = dacc[e] * scale;
    lg[1][e] = dacc[2 + e] * scale;
    const int h = 2 * t + e;
    if (stash && t < 2 && h < Gl) {
      if (v0) stash[h * ZC_MAX_WINDOW + base + g] = lg[0][e];
      if (v1) stash[h * ZC_MAX_WINDOW + base + g + 8] = lg[1][e];
    }
    if (!v0) lg[0][e] = -INFINITY;
    if (!v1) lg[1][e] = -INFINITY;
  }
  float mx[2] = {fmaxf(lg[0][0], lg[1][0]), fmaxf(lg[0][1], lg[1][1])};
#pragma unroll
  for (int o = 4; o < 32; o <<= 1) {
    mx[0] = fmaxf(mx[0], __shfl_xor_sync(kFull, mx[0], o));
    mx[1] = fmaxf(mx[1], __shfl_xor_sync(kFull, mx[1], o));
  }
  float ls[2] = {0.f, 0.f};
  uint32_t Xhi[2], Xlo[2];
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const float pa = zc_exp2(lg[0][e] - mx[e]), pb = zc_exp2(lg[1][e] - mx[e]);
    ls[e] = pa + pb;
    const T ha = zc_from_float<T>(pa), hb = zc_from_float<T>(pb);
    const T la = zc_from_float<T>(pa - zc_to_float<T>(ha)), lb = zc_from_float<T>(pb - zc_to_float<T>(hb));
    Xhi[e] = (uint32_t)(*reinterpret_cast<const unsigned short*>(&ha)) |
             ((uint32_t)(*reinterpret_cast<const unsigned short*>(&hb)) << 16);
    Xlo[e] = (uint32_t)(*reinterpret_cast<const unsigned short*>(&la)) |
             ((uint32_t)(*reinterpret_cast<const unsigned short*>(&lb)) << 16);
  }
#pragma unroll
  for (int o = 4; o < 32; o <<= 1) {
    ls[0] += __shfl_xor_sync(kFull, ls[0], o);
    ls[1] += __shfl_xor_sync(kFull, ls[1], o);
  }
  // B fragment of P^T: column n = g is head g & 3, part g >> 2; (tokens 2t, 2t+8) come from
  // lane (2t, head >> 1), (tokens 2t+1, 2t+9) from lane (2t+1, head >> 1)
  const int hh = g & 3, srcA = 8 * t + (hh >> 1), srcB = srcA + 4;
  uint32_t pb0, pb1;
  {
    const uint32_t a_h0 = __shfl_sync(kFull, Xhi[0], srcA), a_h1 = __shfl_sync(kFull, Xhi[1], srcA);
    const uint32_t a_l0 = __shfl_sync(kFull, Xlo[0], srcA), a_l1 = __shfl_sync(kFull, Xlo[1], srcA);
    const uint32_t b_h0 = __shfl_sync(kFull, Xhi[0], srcB), b_h1 = __shfl_sync(kFull, Xhi[1], srcB);
    const uint32_t b_l0 = __shfl_sync(kFull, Xlo[0], srcB), b_l1 = __shfl_sync(kFull, Xlo[1], srcB);
    const bool lo_part = g >= 4, second = hh & 1;
    pb0 = lo_part ? (second ? a_l1 : a_l0) : (second ? a_h1 : a_h0);
    pb1 = lo_part ? (second ? b_l1 : b_l0) : (second ? b_h1 : b_h0);
  }
  // ---- O^T: M-tile i has rows g <-> channel 16g + 2i, g + 8 <-> channel 16g + 2i + 1 ----
  float oacc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const uint32_t ra = (&va[i >> 2].x)[i & 3], rb = (&vb[i >> 2].x)[i & 3];
    const uint32_t rc = (&vc[i >> 2].x)[i & 3], rd = (&vd[i >> 2].x)[i & 3];
    const uint32_t a[4] = {prmt(ra, rb, 0x5410u), prmt(ra, rb, 0x7632u), prmt(rc, rd, 0x5410u),
                           prmt(rc, rd, 0x7632u)};
    oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
    zc_mma16816<T>(oacc[i], a, pb0, pb1);
  }
  // columns 4..7 (lanes t >= 2) hold the lo-part products of heads 0..3: add them in
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int e = 0; e < 4; ++e) oacc[i][e] += __shfl_xor_sync(kFull, oacc[i][e], 2);
  if (t < 2) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      if (2 * t + e < Gl) {
        float* d = dst + (2 * t + e) * ZC_PART_STRIDE;
        if (g == 0) *reinterpret_cast<float2*>(d) = make_float2(mx[e], ls[e]);
#pragma unroll
        for (int i = 0; i < 8; ++i)
          *reinterpret_cast<float2*>(d + 4 + 16 * g + 2 * i) = make_float2(oacc[i][e], oacc[i][2 + e]);
      }
    }
  }
}

// One item of a class kept at 16 bits (the "16/16" and "16/2" settings): its tokens sit in the
// cache as rows of the input type, [K rows 16 x 128][V rows 16 x 128] per sub-tile, and are
// attended like the tail -- on tensor cores in the input type, q exact, probabilities as
// hi + lo -- but with one running (maximum, sum, accumulator) per warp over all its sub-tiles.
// On return every warp has put its (m, l) and accumulators where compressed_item puts them;
// the merge then takes them with unit scales.
template <typename T>
__device__ __noinline__ ItemScale raw_item(ItemDesc d, const char* class_base, const T* qbase, int Gl,
                                           char* smem, int ring_bytes) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  float* wm = reinterpret_cast<float*>(smem + kOffWm);
  float* wl = reinterpret_cast<float*>(smem + kOffWl);
  float* wz = reinterpret_cast<float*>(smem + kOffWz);
  uint4 qv[4];
#pragma unroll
  for (int c = 0; c < 4; ++c)
    qv[c] = g < Gl ? *reinterpret_cast<const uint4*>(qbase + g * ZC_D + 32 * c + 8 * t) : make_uint4(0, 0, 0, 0);
  const float scale = kLog2e * rsqrtf((float)ZC_D);
  float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
  float oacc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  const int hh = g & 3, srcA = 8 * t + (hh >> 1), srcB = srcA + 4;
  const int corr_src = (lane & ~3) | (t & 1);   // the lane that holds the heads of this lane's columns
  for (int s = d.sub_lo + warp; s < d.sub_hi; s += kWarps) {
    const T* tK = reinterpret_cast<const T*>(class_base + (long long)s * (ZC_SUB * 2 * ZC_D * 2));
    const T* tV = tK + ZC_SUB * ZC_D;
    const int nv = min(ZC_SUB, d.n_tok - (s - d.run_sub0) * ZC_SUB);
    const int last = nv - 1;
    const int r0 = min(g, last), r1 = min(g + 8, last);
    uint4 ka[4], kb[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      ka[c] = __ldcg(reinterpret_cast<const uint4*>(tK + r0 * ZC_D + 32 * c + 8 * t));
      kb[c] = __ldcg(reinterpret_cast<const uint4*>(tK + r1 * ZC_D + 32 * c + 8 * t));
    }
    const T* vap = tV + min(2 * t, last) * ZC_D;
    const T* vbp = tV + min(2 * t + 8, last) * ZC_D;
    const T* vcp = tV + min(2 * t + 1, last) * ZC_D;
    const T* vdp = tV + min(2 * t + 9, last) * ZC_D;
    uint4 va[2], vb[2], vc[2], vd[2];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      va[u] = __ldcg(reinterpret_cast<const uint4*>(vap + 16 * g + 8 * u));
      vb[u] = __ldcg(reinterpret_cast<const uint4*>(vbp + 16 * g + 8 * u));
      vc[u] = __ldcg(reinterpret_cast<const uint4*>(vcp + 16 * g + 8 * u));
      vd[u] = __ldcg(reinterpret_cast<const uint4*>(vdp + 16 * g + 8 * u));
    }
    float dacc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint32_t a0[4] = {ka[c].x, kb[c].x, ka[c].y, kb[c].y};
      zc_mma16816<T>(dacc, a0, qv[c].x, qv[c].y);
      const uint32_t a1[4] = {ka[c].z, kb[c].z, ka[c].w, kb[c].w};
      zc_mma16816<T>(dacc, a1, qv[c].z, qv[c].w);
    }
    const bool v0 = g < nv, v1 = g + 8 < nv;
    float lg[2][2];   // [token slot][head 2t + e]
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      lg[0][e] = v0 ? dacc[e] * scale : -INFINITY;
      lg[1][e] = v1 ? dacc[2 + e] * scale : -INFINITY;
    }
    float mx[2] = {fmaxf(lg[0][0], lg[1][0]), fmaxf(lg[0][1], lg[1][1])};
#pragma unroll
    for (int o = 4; o < 32; o <<= 1) {
      mx[0] = fmaxf(mx[0], __shfl_xor_sync(kFull, mx[0], o));
      mx[1] = fmaxf(mx[1], __shfl_xor_sync(kFull, mx[1], o));
    }
    float corr[2];
    uint32_t Xhi[2], Xlo[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const float mn = fmaxf(m[e], mx[e]);            // finite: token 0 of the sub-tile is valid
      corr[e] = m[e] == -INFINITY ? 0.f : zc_exp2(m[e] - mn);
      m[e] = mn;
      const float pa = zc_exp2(lg[0][e] - mn), pb = zc_exp2(lg[1][e] - mn);
      l[e] = l[e] * corr[e] + pa + pb;
      const T ha = zc_from_float<T>(pa), hb = zc_from_float<T>(pb);
      const T la = zc_from_float<T>(pa - zc_to_float<T>(ha)), lb = zc_from_float<T>(pb - zc_to_float<T>(hb));
      Xhi[e] = (uint32_t)(*reinterpret_cast<const unsigned short*>(&ha)) |
               ((uint32_t)(*reinterpret_cast<const unsigned short*>(&hb)) << 16);
      Xlo[e] = (uint32_t)(*reinterpret_cast<const unsigned short*>(&la)) |
               ((uint32_t)(*reinterpret_cast<const unsigned short*>(&lb)) << 16);
    }
    // this lane's accumulator columns 2t, 2t+1 belong to heads (2t) & 3, (2t+1) & 3
    const float c0 = __shfl_sync(kFull, corr[0], corr_src), c1 = __shfl_sync(kFull, corr[1], corr_src);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      oacc[i][0] *= c0; oacc[i][1] *= c1; oacc[i][2] *= c0; oacc[i][3] *= c1;
    }
    uint32_t pb0, pb1;
    {
      const uint32_t a_h0 = __shfl_sync(kFull, Xhi[0], srcA), a_h1 = __shfl_sync(kFull, Xhi[1], srcA);
      const uint32_t a_l0 = __shfl_sync(kFull, Xlo[0], srcA), a_l1 = __shfl_sync(kFull, Xlo[1], srcA);
      const uint32_t b_h0 = __shfl_sync(kFull, Xhi[0], srcB), b_h1 = __shfl_sync(kFull, Xhi[1], srcB);
      const uint32_t b_l0 = __shfl_sync(kFull, Xlo[0], srcB), b_l1 = __shfl_sync(kFull, Xlo[1], srcB);
      const bool lo_part = g >= 4, second = hh & 1;
      pb0 = lo_part ? (second ? a_l1 : a_l0) : (second ? a_h1 : a_h0);
      pb1 = lo_part ? (second ? b_l1 : b_l0) : (second ? b_h1 : b_h0);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const uint32_t ra = (&va[i >> 2].x)[i & 3], rb = (&vb[i >> 2].x)[i & 3];
      const uint32_t rc = (&vc[i >> 2].x)[i & 3], rd = (&vd[i >> 2].x)[i & 3];
      const uint32_t a[4] = {prmt(ra, rb, 0x5410u), prmt(ra, rb, 0x7632u), prmt(rc, rd, 0x5410u),
                             prmt(rc, rd, 0x7632u)};
      zc_mma16816<T>(oacc[i], a, pb0, pb1);
    }
  }
#pragma unroll
  for (int o = 4; o < 32; o <<= 1) {
    l[0] += __shfl_xor_sync(kFull, l[0], o);
    l[1] += __shfl_xor_sync(kFull, l[1], o);
  }
  // columns 4..7 (lanes t >= 2) hold the lo-part products of heads 0..3
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int e = 0; e < 4; ++e) oacc[i][e] += __shfl_xor_sync(kFull, oacc[i][e], 2);
  if (g == 0 && t < 2) {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      wm[warp * 4 + 2 * t + e] = m[e];
      wl[warp * 4 + 2 * t + e] = l[e];
      wz[warp * 4 + 2 * t + e] = 0.f;
    }
  }
  float* mbuf = reinterpret_cast<float*>(smem + kOffRing + warp * ring_bytes);   // [4 heads][128]
  if (t < 2) {
#pragma unroll
    for (int e = 0; e < 2; ++e)
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        // M-tile i: rows g <-> channel 16g + 2i, g + 8 <-> channel 16g + 2i + 1
        mbuf[(2 * t + e) * ZC_D + 16 * g + 2 * i] = oacc[i][e];
        mbuf[(2 * t + e) * ZC_D + 16 * g + 2 * i + 1] = oacc[i][2 + e];
      }
  }
  ItemScale r;
  r.chan_factor = 1.f;
  r.rowscale = 1.f;
  return r;
}

// shared-memory map of the merge phase (it reuses the memory of the item phase, but not the
// mbarriers': memory that holds mbarrier objects is never reused as data -- plain stores
// over a used barrier were observed to be replaced by barrier state)
constexpr int kMaxTailTiles = ZC_MAX_WINDOW / ZC_SUB;
constexpr int kCmbEntries = (ZC_MAX_ITEMS + kMaxTailTiles) * ZC_MAX_G;   // items + tail tiles, per head
constexpr int kCmbOffM = kOffQfrag;                               // [entries] maxima, then weights
constexpr int kCmbOffL = kCmbOffM + kCmbEntries * 4;              // [entries] sums
constexpr int kCmbOffML = kCmbOffL + kCmbEntries * 4;             // [G] x (M, L)
constexpr int kCmbOffFlag = kCmbOffML + 2 * ZC_MAX_G * 4;         // "this CTA arrived last"
constexpr int kCombineSmem = kCmbOffFlag + 16;
static_assert(kCombineSmem <= decode_smem(kRingNarrow), "the merge phase must fit the item phase's memory");

// Attention over the full-precision tail, all query heads of the unit: tile i (16 tokens) is
// taken by warp i mod 4 and becomes split-K partial `first_entry + i`.  Nothing here touches
// shared memory or a barrier.
template <typename T>
__device__ __noinline__ void tail_phase(const T* tK, const T* tV, int G, int n_tail, const T* qunit, int unit,
                                        float* part_unit, int first_entry, float* stash_g, const T* k_new,
                                        const T* v_new, ZcOrder ord, unsigned ord_first, bool free_run, int* err) {
  const int warp = threadIdx.x >> 5;
  if (free_run) order_wait(ord, ord_first, ord.need_end, err);   // the workspace region is free
  for (int base = warp * ZC_SUB; base < n_tail; base += kWarps * ZC_SUB) {
    float* entry = part_unit + (long long)(first_entry + base / ZC_SUB) * G * ZC_PART_STRIDE;
    for (int hg = 0; hg * 4 < G; ++hg)
      tail_tile<T>(tK, tV, n_tail, base, qunit + 4 * hg * ZC_D, min(4, G - 4 * hg), unit,
                   entry + 4 * hg * ZC_PART_STRIDE, stash_g ? stash_g + 4 * hg * ZC_MAX_WINDOW : nullptr, k_new,
                   v_new);
  }
}

// Merge of a unit's split-K partials (items, then the tail's tiles) in a fixed order,
// the output row of every query head and, on probe steps, this step's attention over the
// tail's tokens added to the window statistics.  Run by the CTA of the unit that finished last.
// ------------------------------------------------------------------ window re-compression
// Alg. 3: when a call completes the window, the CTA that merged a unit's partials turns the
// unit's tail into a new segment: scores from the window statistics (which this call was the
// last to add to), split, channel factors (Eq. 6), CSTQuant and packing, sub-block by
// sub-block, with the arithmetic of the prefill kernels.  Everything it touches belongs to
// the unit, so no other CTA is involved; the cache's next call waits for this one.
constexpr int kFlOffCodesK = kOffQfrag;                                  // [16][128] bytes
constexpr int kFlOffCodesV = kFlOffCodesK + ZC_SUB * ZC_D;
constexpr int kFlOffParK = kFlOffCodesV + ZC_SUB * ZC_D;                 // [16][2] floats
constexpr int kFlOffParV = kFlOffParK + ZC_SUB * 2 * 4;
constexpr int kFlOffKey = kFlOffParV + ZC_SUB * 2 * 4;                   // [128] score bits
constexpr int kFlOffTok = kFlOffKey + ZC_MAX_WINDOW * 4;                 // [2][128] token of each class slot
constexpr int kFlOffRed = kFlOffTok + 2 * ZC_MAX_WINDOW * 4;             // [4 warps][3][128] floats
constexpr int kFlOffC = kFlOffRed + kWarps * 3 * ZC_D * 4;               // [3][128] channel factors (cK | sK, cV, zK)
constexpr int kFlOffMask = kFlOffC + 3 * ZC_D * 4;                       // [4] ballots
constexpr int kFlOffSmax = kFlOffMask + 16;                              // [2] V scale maxima as bits
constexpr int kFlushSmem = kFlOffSmax + 16;
static_assert(kFlushSmem <= decode_smem(kRingNarrow), "the re-compression must fit the item phase's memory");
static_assert(ZC_MAX_WINDOW == 32 * kWarps, "one thread per window token");

template <typename T, bool KCH, bool RAW, bool B8>
__device__ __forceinline__ void window_flush_unit(char* ub, const ZcLayout& lay, const ZcFlushArgs& fl, char* smem) {
  auto codesK = reinterpret_cast<unsigned char (*)[ZC_D]>(smem + kFlOffCodesK);
  auto codesV = reinterpret_cast<unsigned char (*)[ZC_D]>(smem + kFlOffCodesV);
  auto parK = reinterpret_cast<float (*)[2]>(smem + kFlOffParK);
  auto parV = reinterpret_cast<float (*)[2]>(smem + kFlOffParV);
  unsigned* s_key = reinterpret_cast<unsigned*>(smem + kFlOffKey);
  auto s_tok = reinterpret_cast<int (*)[ZC_MAX_WINDOW]>(smem + kFlOffTok);
  auto red = reinterpret_cast<float (*)[3][ZC_D]>(smem + kFlOffRed);
  constexpr bool kch = KCH;
  auto s_c = reinterpret_cast<float (*)[ZC_D]>(smem + kFlOffC);   // [3][128]
  unsigned* s_mask = reinterpret_cast<unsigned*>(smem + kFlOffMask);
  unsigned* s_smax = reinterpret_cast<unsigned*>(smem + kFlOffSmax);
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const int n = lay.window, n_s = fl.seg.n_tok[0];

  // ---- scores of the window's tokens; the statistics start from zero for the next window ----
  {
    unsigned key = 0u;
    if (tid < n) {
      float* colsum = reinterpret_cast<float*>(ub + lay.off_colsum);
      const float sc = __fdiv_rn(colsum[tid], (float)(lay.G * max(1, (int)fl.nnz[tid])));
      reinterpret_cast<float*>(ub + lay.off_scores)[tid] = sc;
      colsum[tid] = 0.f;
      key = __float_as_uint(sc);   // scores are non-negative: unsigned order is float order
    }
    s_key[tid] = key;
    if (tid < 2) s_smax[tid] = 0u;
  }
  __syncthreads();
  // ---- split: the n_s largest scores, equal scores by lowest index; both lists ascending ----
  {
    bool sal = false;
    if (tid < n) {
      const unsigned mine = s_key[tid];
      int rank = 0;
      for (int i = 0; i < n; ++i) {
        const unsigned k = s_key[i];
        rank += (k > mine || (k == mine && i < tid)) ? 1 : 0;
      }
      sal = rank < n_s;
    }
    const unsigned m = __ballot_sync(kFull, sal);
    if (lane == 0) s_mask[w] = m;
  }
  __syncthreads();
  if (tid < n) {
    int before = __popc(s_mask[w] & ((1u << lane) - 1u));
    for (int i = 0; i < w; ++i) before += __popc(s_mask[i]);
    const bool sal = (s_mask[w] >> lane) & 1u;
    int32_t* idx = reinterpret_cast<int32_t*>(ub + lay.off_idx) + fl.seg.idx_off;
    if (sal) {
      s_tok[0][before] = tid;
      idx[before] = tid;
    } else {
      s_tok[1][tid - before] = tid;
      idx[n_s + tid - before] = tid;
    }
  }
  __syncthreads();

  const T* tK = reinterpret_cast<const T*>(ub + lay.off_tailK);
  const T* tV = reinterpret_cast<const T*>(ub + lay.off_tailV);
  for (int cls = 0; cls < 2; ++cls) {
    const int n_c = fl.seg.n_tok[cls];
    if (n_c == 0) continue;
    const int bits = lay.bits[cls];
    if (RAW && bits == 16) {
      // a class kept at 16 bits: its rows are gathered into the new tiles as they are
      const int subs16 = (n_c + ZC_SUB - 1) / ZC_SUB;
      for (int r = w; r < subs16 * ZC_SUB; r += kWarps) {
        uint2 k = make_uint2(0, 0), v = make_uint2(0, 0);
        if (r < n_c) {
          const int row = s_tok[cls][r] * ZC_D;
          k = *reinterpret_cast<const uint2*>(tK + row + 4 * lane);
          v = *reinterpret_cast<const uint2*>(tV + row + 4 * lane);
        }
        char* sub = ub + lay.off_tiles[cls] + (long long)fl.seg.tile0[cls] * lay.tile_bytes[cls] +
                    (long long)(r / ZC_SUB) * zc_sub_bytes(16, 0) + (r % ZC_SUB) * ZC_D * 2;
        reinterpret_cast<uint2*>(sub)[lane] = k;
        reinterpret_cast<uint2*>(sub + ZC_SUB * ZC_D * 2)[lane] = v;
      }
      continue;
    }
    // ---- channel |x| maxima over the class (Eq. 6); channelwise keys: their signed min and max ----
    const float L = (float)((1 << bits) - 1);
    {
      const float k0 = kch ? -INFINITY : 0.f;
      float mk[4] = {k0, k0, k0, k0}, mv[4] = {0.f, 0.f, 0.f, 0.f};
      float nk[4] = {INFINITY, INFINITY, INFINITY, INFINITY};
      for (int r = w; r < n_c; r += kWarps) {
        const int row = s_tok[cls][r] * ZC_D;
        float x[4];
        zc_load4<T>(tK + row + 4 * lane, x);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          mk[e] = fmaxf(mk[e], kch ? x[e] : fabsf(x[e]));
          nk[e] = fminf(nk[e], x[e]);
        }
        zc_load4<T>(tV + row + 4 * lane, x);
#pragma unroll
        for (int e = 0; e < 4; ++e) mv[e] = fmaxf(mv[e], fabsf(x[e]));
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        red[w][0][4 * lane + e] = mk[e];
        red[w][1][4 * lane + e] = mv[e];
        red[w][2][4 * lane + e] = nk[e];
      }
    }
    __syncthreads();
    {
      float mk = red[0][0][tid], mv = red[0][1][tid], nk = red[0][2][tid];
#pragma unroll
      for (int i = 1; i < kWarps; ++i) {
        mk = fmaxf(mk, red[i][0][tid]);
        mv = fmaxf(mv, red[i][1][tid]);
        nk = fminf(nk, red[i][2][tid]);
      }
      if (kch) {
        float sk, zk;
        channel_params(nk, mk, L, &sk, &zk);
        s_c[0][tid] = sk;
        s_c[2][tid] = zk;
      } else {
        s_c[0][tid] = mk == 0.f ? 1.f : __fsqrt_rn(mk);
      }
      s_c[1][tid] = mv == 0.f ? 1.f : __fsqrt_rn(mv);
    }
    __syncthreads();
    float cK[4], cV[4], zK[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      cK[e] = s_c[0][4 * lane + e];
      cV[e] = s_c[1][4 * lane + e];
      zK[e] = kch ? s_c[2][4 * lane + e] : 0.f;
    }
    float* fac = reinterpret_cast<float*>(ub + lay.off_fac) + (fl.seg.run0 + cls) * ZC_FAC_FLOATS;
    if (w == 0) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        fac[4 * lane + e] = cK[e];
        fac[ZC_D + 4 * lane + e] = cV[e];
        if (kch) fac[ZC_FAC_ZK + 4 * lane + e] = zK[e];
      }
    }
    // ---- CSTQuant and packing, one 16-token sub-block at a time: four tokens per warp ----
    float smax = 0.f;
    const int subs = (n_c + ZC_SUB - 1) / ZC_SUB;
    const int vecs = zc_sub_bytes(bits, kch) / 16;
    for (int sb = 0; sb < subs; ++sb) {
      uint2 rawK[4], rawV[4];
      bool live[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int tt = ZC_SUB * sb + 4 * w + i;
        live[i] = tt < n_c;
        rawK[i] = make_uint2(0, 0);
        rawV[i] = make_uint2(0, 0);
        if (live[i]) {
          const int row = s_tok[cls][tt] * ZC_D;
          rawK[i] = *reinterpret_cast<const uint2*>(tK + row + 4 * lane);
          rawV[i] = *reinterpret_cast<const uint2*>(tV + row + 4 * lane);
        }
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int tl = 4 * w + i;
        float x[4], sc, z;
        unsigned pk;
        const T* ek = reinterpret_cast<const T*>(&rawK[i]);
#pragma unroll
        for (int e = 0; e < 4; ++e) x[e] = zc_to_float<T>(ek[e]);
        if (kch) {
          pk = quant_channel4(x, cK, zK, L);
        } else {
          quant_token(x, cK, L, &sc, &z, &pk);
          if (lane == 0) { parK[tl][0] = live[i] ? sc : 0.f; parK[tl][1] = live[i] ? z : 0.f; }
        }
        *reinterpret_cast<unsigned*>(&codesK[tl][4 * lane]) = live[i] ? pk : 0u;
        const T* ev = reinterpret_cast<const T*>(&rawV[i]);
#pragma unroll
        for (int e = 0; e < 4; ++e) x[e] = zc_to_float<T>(ev[e]);
        quant_token(x, cV, L, &sc, &z, &pk);
        *reinterpret_cast<unsigned*>(&codesV[tl][4 * lane]) = live[i] ? pk : 0u;
        if (lane == 0) { parV[tl][0] = live[i] ? sc : 0.f; parV[tl][1] = live[i] ? z : 0.f; }
        if (live[i]) smax = fmaxf(smax, sc);
      }
      __syncthreads();
      const int sub_in_tile = sb % (ZC_TILE / ZC_SUB);
      if (!ZC_CHECKED(fl.seg.tile0[cls] + sb / (ZC_TILE / ZC_SUB) < lay.cap_tiles[cls], ZC_DBG_FLUSH_TILE)) break;
      char* tile_ptr = ub + lay.off_tiles[cls] +
                       (long long)(fl.seg.tile0[cls] + sb / (ZC_TILE / ZC_SUB)) * lay.tile_bytes[cls];
      for (int v = tid; v < vecs; v += 128)
        reinterpret_cast<uint4*>(tile_ptr)[sub_in_tile * vecs + v] =
            (B8 && bits == 8)
                ? compose_vec8(kch, sub_in_tile * vecs + v, ZC_SUB * sub_in_tile, codesK, codesV, parK, parV)
                : compose_vec(bits, kch, sub_in_tile * vecs + v, ZC_SUB * sub_in_tile, codesK, codesV, parK, parV);
      __syncthreads();   // the next sub-block reuses the code arrays
    }
    if (lane == 0 && smax > 0.f) atomicMax(&s_smax[cls], __float_as_uint(smax));
  }
  __syncthreads();
  if (tid < 2)
    reinterpret_cast<unsigned*>(ub + lay.off_fac)[(fl.seg.run0 + tid) * ZC_FAC_FLOATS + 2 * ZC_D] = s_smax[tid];
}

template <typename T>
__device__ __noinline__ void merge_unit(float* colsum, int G, int items, int n_tail, T* __restrict__ out_unit,
                                        float* __restrict__ out_unit_f32, const float* mine,
                                        const float* stash_g, int collect, char* smem) {
  float* s_m = reinterpret_cast<float*>(smem + kCmbOffM);
  float* s_l = reinterpret_cast<float*>(smem + kCmbOffL);
  float* s_ML = reinterpret_cast<float*>(smem + kCmbOffML);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int entries = items + (n_tail + ZC_SUB - 1) / ZC_SUB;
  for (int e = tid; e < entries * G; e += 128) {
    const float2 ml = __ldcg(reinterpret_cast<const float2*>(mine + (long long)e * ZC_PART_STRIDE));
    s_m[e] = ml.x;
    s_l[e] = ml.y;
  }
  // each warp owns heads warp, warp + 4: its first rows are requested before the barrier
  constexpr int kChunk = 12;
  float4 acc4[kChunk];
  const int n_first = min(entries, kChunk);
  if (warp < G) {
#pragma unroll
    for (int u = 0; u < kChunk; ++u)
      if (u < n_first)
        acc4[u] = __ldcg(reinterpret_cast<const float4*>(mine + (long long)(u * G + warp) * ZC_PART_STRIDE + 4) + lane);
  }
  __syncthreads();
  for (int h = warp; h < G; h += kWarps) {
    if (h != warp) {
#pragma unroll
      for (int u = 0; u < kChunk; ++u)
        if (u < n_first)
          acc4[u] = __ldcg(reinterpret_cast<const float4*>(mine + (long long)(u * G + h) * ZC_PART_STRIDE + 4) + lane);
    }
    float mxh = -INFINITY;
    for (int i = lane; i < entries; i += 32) mxh = fmaxf(mxh, s_m[i * G + h]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mxh = fmaxf(mxh, __shfl_xor_sync(kFull, mxh, o));
    float lsum = 0.f;
    for (int i = lane; i < entries; i += 32) {
      const float mi = s_m[i * G + h];
      const float sc = mi == -INFINITY ? 0.f : zc_exp2(mi - mxh);
      s_m[i * G + h] = sc;
      lsum += s_l[i * G + h] * sc;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) lsum += __shfl_xor_sync(kFull, lsum, o);
    __syncwarp();
    if (lane == 0) { s_ML[2 * h] = mxh; s_ML[2 * h + 1] = lsum; }
    float4 o4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int u = 0; u < kChunk; ++u) {
      if (u < n_first) {
        const float sc = s_m[u * G + h];
        o4.x += acc4[u].x * sc; o4.y += acc4[u].y * sc; o4.z += acc4[u].z * sc; o4.w += acc4[u].w * sc;
      }
    }
    for (int i = kChunk; i < entries; ++i) {
      const float4 a = __ldcg(reinterpret_cast<const float4*>(mine + (long long)(i * G + h) * ZC_PART_STRIDE + 4) + lane);
      const float sc = s_m[i * G + h];
      o4.x += a.x * sc; o4.y += a.y * sc; o4.z += a.z * sc; o4.w += a.w * sc;
    }
    const float inv = 1.f / lsum;
    if (out_unit_f32) {   // ZC_FLAG_OUT_F32: the result before its rounding to the 16-bit type
      *reinterpret_cast<float4*>(out_unit_f32 + h * ZC_D + 4 * lane) =
          make_float4(o4.x * inv, o4.y * inv, o4.z * inv, o4.w * inv);
    } else {
      T r[4] = {zc_from_float<T>(o4.x * inv), zc_from_float<T>(o4.y * inv), zc_from_float<T>(o4.z * inv),
                zc_from_float<T>(o4.w * inv)};
      *reinterpret_cast<uint2*>(out_unit + h * ZC_D + 4 * lane) = *reinterpret_cast<const uint2*>(r);
    }
  }
  if (collect) {
    __syncthreads();
    if (tid < n_tail) {
      float a = 0.f;
      for (int h = 0; h < G; ++h)
        a += zc_exp2(__ldcg(stash_g + h * ZC_MAX_WINDOW + tid) - s_ML[2 * h]) / s_ML[2 * h + 1];
      colsum[tid] += a;
    }
  }
}

// One decode-attention call as ONE grid.  CTA roles, by linear index: for every unit
// block 0 only waits; then for every unit (items x head groups) item CTAs and one tail CTA.
//   item     streams its range of sub-tiles and stores a partial per query head
//   tail     attention over the full-precision tail, stored as the unit's last partial (with
//            plan.fold_tail there is no such CTA: the unit's first item CTA does it first)
//   either   counts itself in at the unit's arrival counter; the CTA that arrives last merges
//            the unit's partials and writes the output.  Nothing spins on another CTA.
// Every CTA lets the next kernel of the stream start at once and none of the working CTAs
// waits for the previous kernel, so calls on independent caches stream through the GPU like
// one grid; block 0 does nothing but wait for the previous kernel, which
// makes kernels complete in stream order (a launch made without early start then finds every
// earlier call finished) at the price of one idle CTA.  What calls in flight together may
// share is kept apart by the host: each call of an epoch (the launches between two launches
// made without early start) gets its own `slot`, which selects its region of the workspace
// and its arrival counter.
// RAW: the build that also serves a class kept at 16 bits (kept apart so that the 4- and 2-bit
// kernels are compiled exactly as they are without it).
template <typename T, int RING, int NCTA, bool KCH, bool RAW, bool B8 = false, bool P16 = false>
__global__ void __launch_bounds__(128, NCTA) k_decode(char* cache, ZcLayout lay, ZcDecodePlan plan,
                                                      const T* __restrict__ q, T* __restrict__ out,
                                                      float* part, float* stash_all, int slot,
                                                      int collect, const T* k_new, const T* v_new,
                                                      ZcOrder ord, ZcFlushArgs fl) {
  extern __shared__ __align__(128) char smem[];
  const int G = lay.G, zs = (G + 3) >> 2;
  const int groups = (plan.items + plan.cta_items - 1) / plan.cta_items;   // item CTAs per head group
  const int per_unit = groups * zs + (plan.fold_tail ? 0 : 1);
  // Block 0 is the CTA that only waits: it is dispatched first, so it holds a slot even when
  // the rest of a large grid is waiting for what it is going to publish.
  const int idx = (int)blockIdx.x - 1;
  if (idx < 0) {
    // The one CTA that ties this kernel's completion to its predecessor's and publishes it.
    // The first kernel of an epoch resets the word before any later kernel can start.
    if (ord.epoch_start && threadIdx.x == 0) {
      *reinterpret_cast<volatile unsigned*>(ord.done) = ord.tag << 20;
      __threadfence();
    }
    __syncthreads();
    pdl_launch_dependents();
    pdl_wait();
    if (!ord.epoch_start && threadIdx.x == 0)
      *reinterpret_cast<volatile unsigned*>(ord.done) = (ord.tag << 20) | (unsigned)ord.e;
    return;
  }
  const int unit = idx / per_unit, j = idx - unit * per_unit;
  const bool is_tail = !plan.fold_tail && j == per_unit - 1;
  char* ub = zc_unit_base(cache, lay, unit);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (plan.n_tail > 0 && tid < 2 && plan.fold_tail && j == 0) {
    // the tail's rows start their way from DRAM to L2 while the CTA sets up (a CTA that has
    // only the tail to do loads them at once anyway)
    const char* rows = ub + (tid == 0 ? lay.off_tailK : lay.off_tailV);
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(rows), "r"(plan.n_tail * ZC_D * 2) : "memory");
  }
  // the stream's word is requested first and looked at when it is needed
  const bool free_run = plan.chain_free != 0;
  const unsigned ord_first =
      !free_run ? 0u : ord.need_start > 0 ? ld_order_acquire(ord.done) : ord.need_end > 0 ? ld_order(ord.done) : 0u;
  pdl_launch_dependents();
  if (free_run) {
    // The caller promised (ZC_FLAG_OVERLAP_CALLS) that only calls of this library precede this
    // one on the stream: the working CTAs do not wait for the previous kernel, only for what
    // the host found them to depend on (inputs written by an earlier call, a re-compressed
    // window, the previous call's tail row).
    order_wait(ord, ord_first, ord.need_start, &g_zc_error);
  } else {
    // Anything may precede this call on the stream, e.g. the kernel that produces q, and it
    // may have let this kernel start early: everything the stream holds before this launch
    // must have completed before q, k_new, v_new or the cache are read.
    pdl_wait();
  }
  if (k_new && j == 0 && warp == kWarps - 1) {
    // Deferred append: the newest row goes into the tail for the steps to come (this step reads
    // it from k_new / v_new).  The next call on this cache is told to wait for this one.
    const int pos = plan.n_tail - 1;
    T* tk = reinterpret_cast<T*>(ub + lay.off_tailK) + pos * ZC_D;
    T* tv = reinterpret_cast<T*>(ub + lay.off_tailV) + pos * ZC_D;
    if (lane < 16)
      reinterpret_cast<uint4*>(tk)[lane] = reinterpret_cast<const uint4*>(k_new + (long long)unit * ZC_D)[lane];
    else
      reinterpret_cast<uint4*>(tv)[lane - 16] =
          reinterpret_cast<const uint4*>(v_new + (long long)unit * ZC_D)[lane - 16];
  }
  const int b = unit / lay.n_kv, kv = unit % lay.n_kv;
  const T* qunit = q + ((long long)b * lay.n_kv * G + kv * G) * ZC_D;
  const int n_tiles = (plan.n_tail + ZC_SUB - 1) / ZC_SUB;
  float* mine = part + (long long)unit * (plan.items + kMaxTailTiles) * G * ZC_PART_STRIDE;
  float* stash_g = collect ? stash_all + (long long)unit * G * ZC_MAX_WINDOW : nullptr;

  if (n_tiles > 0 && (is_tail || (plan.fold_tail && j == 0))) {
    // The tail is the work of a CTA of its own, or (calls that share the GPU with their
    // neighbours) of the unit's first item CTA before it turns to its codes.
    // without a deferred append the newest tail row comes from the append kernel just before
    if (!k_new && free_run) pdl_wait();
    tail_phase<T>(reinterpret_cast<const T*>(ub + lay.off_tailK), reinterpret_cast<const T*>(ub + lay.off_tailV), G,
                  plan.n_tail, qunit, unit, mine, plan.items, stash_g, k_new, v_new, ord, ord_first, free_run,
                  &g_zc_error);
  }
  if (!is_tail) {
    float* wm = reinterpret_cast<float*>(smem + kOffWm);
    float* wl = reinterpret_cast<float*>(smem + kOffWl);
    float* wz = reinterpret_cast<float*>(smem + kOffWz);
    float* s_cw = reinterpret_cast<float*>(smem + kOffCw);
    float* s_head = reinterpret_cast<float*>(smem + kOffHead);
    const int z = j / groups, gi = j - z * groups;
    const int h0 = 4 * z, Gl = min(4, G - h0);              // this CTA's query heads
    const T* qbase = qunit + h0 * ZC_D;
    const int it_end = min(plan.items, (gi + 1) * plan.cta_items);
    for (int it = gi * plan.cta_items; it < it_end; ++it) {   // usually one item; all of them when calls overlap
    const ItemDesc d = decode_item(plan, it);
    float* my = mine + ((long long)it * G + h0) * ZC_PART_STRIDE;
    ItemScale sc;
    sc.chan_factor = 1.f;
    sc.rowscale = 1.f;
    const bool has = d.sub_hi > d.sub_lo &&
                     ZC_CHECKED(d.sub_hi <= lay.cap_tiles[d.cls] * (ZC_TILE / ZC_SUB) && d.run < lay.max_runs &&
                                    it < ZC_MAX_ITEMS,
                                ZC_DBG_DECODE_ITEM);
    if (has) {
      const float* fac = reinterpret_cast<const float*>(ub + lay.off_fac) + d.run * ZC_FAC_FLOATS;
      const char* class_base = ub + lay.off_tiles[d.cls];
      if (B8 && lay.bits[d.cls] == 8)
        sc = compressed_item<T, 8, RING, KCH>(d, class_base, fac, qbase, Gl, smem, &g_zc_error);
      else if (lay.bits[d.cls] == 4)
        sc = compressed_item<T, 4, RING, KCH, P16>(d, class_base, fac, qbase, Gl, smem, &g_zc_error);
      else if (!RAW || lay.bits[d.cls] == 2)
        sc = compressed_item<T, 2, RING, KCH, P16>(d, class_base, fac, qbase, Gl, smem, &g_zc_error);
      else
        sc = raw_item<T>(d, class_base, qbase, Gl, smem, RING);
    }
    __syncthreads();
    // ---- merge the warps: one thread per head fixes the weights, then thread = channel ----
    if (tid < 4) {
      float ms = -INFINITY;
#pragma unroll
      for (int w2 = 0; w2 < kWarps; ++w2) ms = fmaxf(ms, wm[w2 * 4 + tid]);
      float ls = 0.f, zsum = 0.f;
#pragma unroll
      for (int w2 = 0; w2 < kWarps; ++w2) {
        const float mw = wm[w2 * 4 + tid];
        const float cw = (has && mw != -INFINITY) ? zc_exp2(mw - ms) : 0.f;
        s_cw[tid * 4 + w2] = cw;
        ls += wl[w2 * 4 + tid] * cw;
        zsum += wz[w2 * 4 + tid] * cw;
      }
      s_head[tid * 4] = has ? ms : -INFINITY;
      s_head[tid * 4 + 1] = has ? ls : 0.f;
      s_head[tid * 4 + 2] = has ? zsum : 0.f;
    }
    __syncthreads();
    if (free_run) order_wait(ord, ord_first, ord.need_end, &g_zc_error);   // the workspace region is free
    for (int h = 0; h < Gl; ++h) {
      float o = 0.f;
      if (has) {
        const float4 cw = *reinterpret_cast<const float4*>(s_cw + h * 4);
        const float a0 = reinterpret_cast<const float*>(smem + kOffRing)[h * ZC_D + tid];
        const float a1 = reinterpret_cast<const float*>(smem + kOffRing + RING)[h * ZC_D + tid];
        const float a2 = reinterpret_cast<const float*>(smem + kOffRing + 2 * RING)[h * ZC_D + tid];
        const float a3 = reinterpret_cast<const float*>(smem + kOffRing + 3 * RING)[h * ZC_D + tid];
        o = (sc.rowscale * (((cw.x * a0 + cw.y * a1) + cw.z * a2) + cw.w * a3) - s_head[h * 4 + 2]) * sc.chan_factor;
      }
      float* dst = my + h * ZC_PART_STRIDE;
      if (tid == 0) { dst[0] = s_head[h * 4]; dst[1] = s_head[h * 4 + 1]; }
      dst[4 + tid] = o;
    }
    if (it + 1 < it_end) __syncthreads();   // the next item reuses the rings and the small arrays
    }
  }
  // ---- count in: the barrier orders every thread's stores before thread 0's count; the CTA
  //      that finds all others counted reads their partials from L2 ----
  __syncthreads();
  int* s_last = reinterpret_cast<int*>(smem + kCmbOffFlag);
  if (per_unit == 1) {
    // the unit's only CTA: its own stores are visible to it after the barrier
    if (tid == 0) *s_last = 1;
  } else if (tid == 0) {
    unsigned* cnt = reinterpret_cast<unsigned*>(ub + lay.off_sync) + slot;
    // release: this CTA's stores (the barrier put them before this thread) are visible to whoever
    // sees the count; acquire: the CTA that counts last sees the others' stores
    unsigned old;
    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], 1;\n" : "=r"(old) : "l"(cnt) : "memory");
    const int last = old == (unsigned)(per_unit - 1);
    if (last) *cnt = 0u;  // next used by a later call, after this kernel has completed
    *s_last = last;
  }
  __syncthreads();
  if (*s_last) {
    const long long out_off = ((long long)b * lay.n_kv * G + kv * G) * ZC_D;
    merge_unit<T>(reinterpret_cast<float*>(ub + lay.off_colsum), G, plan.items, plan.n_tail, out + out_off,
                  lay.out_f32 ? reinterpret_cast<float*>(out) + out_off : nullptr, mine, stash_g, collect, smem);
    if (!P16 && fl.on) {   // (16-bit parameters: the host re-compresses by kernels of their own)
      __syncthreads();   // the merge is done with the shared arrays; its additions to the statistics are visible
      window_flush_unit<T, KCH, RAW, B8>(ub, lay, fl, smem);
    }
  }
}

}  // namespace

namespace {

// Launch with the programmatic-stream-serialisation attribute: the kernel may start while the
// previous kernel of the stream is still running and orders itself with pdl_wait().
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                       bool overlap, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = overlap ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// The calls issued so far, per stream (the rules are in zc_order.h / zc_order.cu).
ZcOrderTable g_table;
std::mutex g_table_mutex;

}  // namespace

int zc_launch_append(zc_cache* c, const void* k_new, const void* v_new, int pos, cudaStream_t st) {
  cudaError_t e;
  if (c->cfg.dtype == ZC_F16)
    e = launch_pdl(k_append<__half>, dim3(c->lay.units), dim3(32), 0, st, true, c->base, c->lay,
                   (const __half*)k_new, (const __half*)v_new, pos);
  else
    e = launch_pdl(k_append<__nv_bfloat16>, dim3(c->lay.units), dim3(32), 0, st, true, c->base, c->lay,
                   (const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new, pos);
  c->launches += 1;
  return e != cudaSuccess ? (int)e : (int)cudaGetLastError();
}

size_t zc_decode_scratch_bytes(const zc_cache* c, int items) {
  const size_t part = (size_t)c->lay.units * (items + kMaxTailTiles) * c->lay.G * ZC_PART_STRIDE * 4;
  const size_t stash = (size_t)c->lay.units * c->lay.G * ZC_MAX_WINDOW * 4;
  return ((part + 255) & ~(size_t)255) + ((stash + 255) & ~(size_t)255);
}

// One word per stream record, in the library image (like the built-in scratch below).
// Two per record: calls issued under stream capture use the second, so that replaying a
// captured graph never disturbs the word of the calls issued directly.
static __device__ unsigned g_zc_order_words[2 * kZcStreamRecs];

// Per-device address of a symbol of the library image, looked up once per device; several
// host threads may ask at the same time (the table is guarded by a mutex).
template <typename Sym>
static int symbol_address(const Sym& sym, void** table, std::mutex& guard, void** out) {
  constexpr int kMaxDev = 64;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return (int)e;
  if (dev < 0 || dev >= kMaxDev) return (int)cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(guard);
  if (!table[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, sym);
    if (e != cudaSuccess) return (int)e;
    table[dev] = p;
  }
  if (out) *out = table[dev];
  return (int)cudaSuccess;
}

int zc_order_words(unsigned** ptr) {
  static void* addr[64] = {nullptr};
  static std::mutex guard;
  void* p = nullptr;
  const int rc = symbol_address(g_zc_order_words, addr, guard, &p);
  if (rc == (int)cudaSuccess && ptr) *ptr = (unsigned*)p;
  return rc;
}

int zc_launch_decode(zc_cache* c, const ZcDecodePlan& plan, const void* q, void* out, int collect,
                     char* ws, size_t ws_bytes, const void* k_new, const void* v_new,
                     const ZcFlushArgs* flush, cudaStream_t st) {
  ZcFlushArgs fl;
  if (flush) fl = *flush;
  else memset(&fl, 0, sizeof(fl));
  static_assert(2 * kZcStreamRecs == 32, "two order words per stream record");
  const int G = c->lay.G, zs = (G + 3) / 4;
  const size_t io_bytes = (size_t)c->cfg.batch * c->cfg.n_q_heads * ZC_D * 2;
  const size_t kv_bytes = (size_t)c->lay.units * ZC_D * 2;
  const size_t part_bytes =
      ((size_t)c->lay.units * (plan.items + kMaxTailTiles) * G * ZC_PART_STRIDE * 4 + 255) & ~(size_t)255;
  const size_t need = zc_decode_scratch_bytes(c, plan.items);
  if (need > ws_bytes) return (int)cudaErrorInvalidValue;
  unsigned* words = nullptr;
  {
    const int rc = zc_order_words(&words);
    if (rc != (int)cudaSuccess) return rc;
  }
  int dev = 0;
  cudaGetDevice(&dev);
  cudaStreamCaptureStatus cap_status = cudaStreamCaptureStatusNone;
  unsigned long long cap_id = 0;
  if (cudaStreamGetCaptureInfo(st, &cap_status, &cap_id) != cudaSuccess) {
    cudaGetLastError();
    cap_status = cudaStreamCaptureStatusNone;
    cap_id = 0;
  }
  const int capturing = cap_status == cudaStreamCaptureStatusActive ? 1 : 0;
  ZcOrderCall call{};
  call.st = (const void*)st;
  call.dev = dev;
  call.me.in[0] = zc_range(q, io_bytes);
  call.me.in[1] = zc_range(k_new, kv_bytes);
  call.me.in[2] = zc_range(v_new, kv_bytes);
  call.me.out = zc_range(out, c->lay.out_f32 ? 2 * io_bytes : io_bytes);
  call.cache = c;
  call.collect = collect;
  call.changes_cache = k_new != nullptr || fl.on;
  call.ws = ws;
  call.ws_bytes = ws_bytes;
  call.need = need;
  call.capturing = capturing;
  call.capture_id = cap_id;
  ZcOrder ord;
  int slot = 0;
  size_t ws_off = 0;
  {
    std::lock_guard<std::mutex> lock(g_table_mutex);
    const ZcOrderSlot s = zc_order_next(&g_table, &c->fence, call);
    if (s.drain && !capturing) {
      cudaStreamSynchronize((cudaStream_t)s.drain);
      cudaGetLastError();
    }
    ord.done = words + 2 * s.rec + capturing;
    ord.tag = s.tag;
    ord.e = s.e;
    ord.epoch_start = s.epoch_start;
    ord.need_start = s.need_start;
    ord.need_end = s.need_end;
    slot = s.slot;
    ws_off = s.ws_off;
  }
  const bool overlap = !ord.epoch_start;
  float* part = reinterpret_cast<float*>(ws + ws_off);
  float* stash = reinterpret_cast<float*>(ws + ws_off + part_bytes);
  const int groups = (plan.items + plan.cta_items - 1) / plan.cta_items;
  const dim3 grid((unsigned)(c->lay.units * (groups * zs + (plan.fold_tail ? 0 : 1)) + 1));
  cudaError_t e;
#define ZC_LAUNCH_STEP(T, RING, NCTA, KCH, RAW, B8, P16)                                               \
  do {                                                                                             \
    /* the opt-in to large shared memory is per device and per kernel: one bit per device */       \
    static std::atomic<unsigned long long> attr_done{0};                                           \
    int dev_now = 0;                                                                               \
    cudaGetDevice(&dev_now);                                                                       \
    const unsigned long long bit = 1ull << (dev_now & 63);                                         \
    if (!(attr_done.load(std::memory_order_acquire) & bit)) {                                      \
      e = cudaFuncSetAttribute(k_decode<T, RING, NCTA, KCH, RAW, B8, P16>,                         \
                               cudaFuncAttributeMaxDynamicSharedMemorySize, decode_smem(RING));    \
      if (e != cudaSuccess) return e;                                                              \
      attr_done.fetch_or(bit, std::memory_order_release);                                          \
    }                                                                                              \
    e = launch_pdl(k_decode<T, RING, NCTA, KCH, RAW, B8, P16>, grid, dim3(128), decode_smem(RING), st, \
                   overlap,                                                                        \
                   c->base, c->lay, plan, (const T*)q, (T*)out, part, stash, slot, collect,        \
                   (const T*)k_new, (const T*)v_new, ord, fl);                                     \
  } while (0)
#define ZC_LAUNCH_T(T)                                                                             \
  do {                                                                                             \
    const bool raw = c->lay.bits[0] == 16 || c->lay.bits[1] == 16;                                 \
    const bool b8 = c->lay.bits[0] == 8 || c->lay.bits[1] == 8;                                    \
    if (c->lay.p16) { /* 16-bit parameters: CSTQuant at 2 or 4 bits only */                        \
      if (plan.ctas_per_sm == 4) ZC_LAUNCH_STEP(T, kRingNarrow, 4, false, false, false, true);     \
      else ZC_LAUNCH_STEP(T, kRingWide, 3, false, false, false, true);                             \
    } else if (b8) { /* an 8-bit class: one build (wide rings hold one pair of its sub-tiles, 3 CTAs per SM) */ \
      if (c->lay.kch) ZC_LAUNCH_STEP(T, kRingWide, 3, true, false, true, false);                   \
      else ZC_LAUNCH_STEP(T, kRingWide, 3, false, false, true, false);                             \
    } else if (raw) { /* a class kept at 16 bits: one build (narrow rings, 4 CTAs per SM) */       \
      if (c->lay.kch) ZC_LAUNCH_STEP(T, kRingNarrow, 4, true, true, false, false);                 \
      else ZC_LAUNCH_STEP(T, kRingNarrow, 4, false, true, false, false);                           \
    } else if (c->lay.kch) {                                                                       \
      if (plan.ctas_per_sm == 4) ZC_LAUNCH_STEP(T, kRingNarrow, 4, true, false, false, false);     \
      else ZC_LAUNCH_STEP(T, kRingWide, 3, true, false, false, false);                             \
    } else {                                                                                       \
      if (plan.ctas_per_sm == 4) ZC_LAUNCH_STEP(T, kRingNarrow, 4, false, false, false, false);    \
      else ZC_LAUNCH_STEP(T, kRingWide, 3, false, false, false, false);                            \
    }                                                                                              \
  } while (0)
  if (c->cfg.dtype == ZC_F16) ZC_LAUNCH_T(__half);
  else ZC_LAUNCH_T(__nv_bfloat16);
#undef ZC_LAUNCH_T
#undef ZC_LAUNCH_STEP
  c->launches += 1;
  return e != cudaSuccess ? (int)e : (int)cudaGetLastError();
}

// Scratch of zc_decode_attention_noalloc.  In host code the name below is only a handle for the
// runtime, not a device address: kernels must be given the pointer cudaGetSymbolAddress returns
// for the device that is current.
static __device__ __align__(256) unsigned char g_zc_noalloc_scratch[ZC_NOALLOC_SCRATCH_BYTES];

int zc_static_scratch(void** ptr) {
  static void* addr[64] = {nullptr};
  static std::mutex guard;
  return symbol_address(g_zc_noalloc_scratch, addr, guard, ptr);
}

int zc_debug_code_decode(int* out) {
#ifdef ZC_DEBUG
  return (int)cudaMemcpyFromSymbol(out, g_zc_debug_fault, sizeof(int));
#else
  *out = 0;
  return (int)cudaSuccess;
#endif
}

int zc_device_error_code(int* out) {
  return (int)cudaMemcpyFromSymbol(out, g_zc_error, sizeof(int));
}
