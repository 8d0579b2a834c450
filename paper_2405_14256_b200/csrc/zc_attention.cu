// Causal prefill attention (Eq. 2; Alg. 2's line "O = FlashAttention(Q, K, V)") that also keeps
// every row's log-sum-exp, so that the probe rows' statistics of Eq. 9 need no pass of their own
// (Appendix B: one attention call serves all tokens while the probe scores are computed beside it).
//
// One CTA = 256 consecutive query rows of one query head, as two groups of 128 that share the key
// and value tiles (128 keys each) in shared memory.  Both contractions run on the 5th-generation
// tensor cores (tcgen05.mma, accumulators in tensor memory):
//   S_g = Q_g K^T    A = Q tile, B = key tile, both K-major in shared memory; 128 x 128 fp32
//   O_g += P_g V     A = P_g in tensor memory: the group's 128 worker threads overwrite the first
//                    64 columns of S_g with exp2(s - m) in the input type, two per column;
//                    B = value tile as it comes from memory ([key][d]: the N dimension
//                    contiguous, "MN-major"); 128 x 128 fp32, accumulated over the key tiles
// The MMAs of one CTA execute in the order they are issued, so S_g of the next tile, issued
// after P_g V, may overwrite P_g; while one group turns its S into P, the tensor cores work
// on the other group's tiles.
// Warp 0 issues the MMAs, warp 1 the bulk tensor copies (Q once, K through 3 buffers, V through
// 2); warps 4..7 and 8..11 are the groups.  Row m of an accumulator lives in TMEM lane m, so a
// worker thread owns one query row: its running maximum (refreshed only when a logit exceeds it
// by 8, base 2; O's row is then rescaled in TMEM), its sum, its row of P.  Every wait is bounded.
#include "zc_internal.h"
#include "zc_layout.cuh"
#include "zc_tc.cuh"

namespace {

constexpr int kFaThreads = 384;
constexpr int kFaRows = 2 * kM;                   // query rows per CTA
constexpr int kKS = 3, kVS = 2;                   // key and value buffers
constexpr uint32_t kFaTmemCols = 512;             // S_0 | S_1 | O_0 | O_1
constexpr int kFaTiles = (2 + kKS + kVS) * kTile; // 224 KB
constexpr int kFaSmem = kFaTiles + 1024 + 256;    // + what aligning to 1 KB may take + barriers
constexpr float kFaTau = 8.f;

// B operand whose N dimension is contiguous in memory: rows of the tile are K indices (keys) of
// 128 bytes = 64 elements of N; 8-row groups 1024 bytes apart, the second 64 elements of N one
// k-block (16 KB) further.
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(kKBlock >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// O (+)= P V for one key tile: 8 steps of 16 keys.  A = P from tensor memory (lane = row, a
// column holds two consecutive keys, so a step of 16 keys is 8 columns), B = the value tile.
__device__ __forceinline__ void mma_pv(uint32_t tmem_o, uint32_t tmem_p, uint32_t v_addr, uint32_t idesc,
                                       bool accumulate) {
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    const uint64_t db = smem_desc_mn(v_addr + ks * 16 * 128);
    const uint32_t acc = (accumulate || ks > 0) ? 1u : 0u;
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n}\n" ::"r"(tmem_o),
        "r"(tmem_p + 8u * ks), "l"(db), "r"(idesc), "r"(acc), "r"(0u)
        : "memory");
  }
}
__device__ __forceinline__ void tmem_st32(const uint32_t* r, uint32_t taddr) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(float* v, uint32_t taddr) {
  tmem_ld32_nowait(v, taddr);
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}

// 8 columns of this thread's row, there and back (the rescaling of O goes in small pieces: the
// row of S is live in registers meanwhile)
__device__ __forceinline__ void tmem_ld8(float* v, uint32_t taddr) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void tmem_st8(const float* v, uint32_t taddr) {
  const uint32_t* r = reinterpret_cast<const uint32_t*>(v);
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};\n" ::"r"(taddr), "r"(r[0]),
               "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}

template <typename T> __device__ __forceinline__ uint32_t pack2(float a, float b);
template <> __device__ __forceinline__ uint32_t pack2<__half>(float a, float b) {
  const __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}
template <> __device__ __forceinline__ uint32_t pack2<__nv_bfloat16>(float a, float b) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// grid.x: blocks of 256 query rows, the last (longest) first; grid.y: (batch, query head).
template <typename T>
__global__ void __launch_bounds__(kFaThreads, 1) k_flash_prefill(
    int l, int h_q, int G, T* __restrict__ O, float* __restrict__ lse, const __grid_constant__ CUtensorMap qmap,
    const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap) {
  extern __shared__ __align__(1024) char smem_raw[];
  const uint32_t raw_u = zc_smem_u32(smem_raw);
  const uint32_t base_u = (raw_u + 1023u) & ~1023u;
  char* base = smem_raw + (base_u - raw_u);
  const uint32_t q_addr = base_u, k_addr = base_u + 2 * kTile, v_addr = k_addr + kKS * kTile;
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + kFaTiles);
  uint64_t* q_full = bars;                  // both Q tiles landed
  uint64_t* k_full = bars + 1;              // [kKS] key tile landed
  uint64_t* k_free = k_full + kKS;          // [kKS] both groups' S of that tile completed
  uint64_t* v_full = k_free + kKS;          // [kVS] value tile landed
  uint64_t* v_free = v_full + kVS;          // [kVS] both groups' P V of that tile completed
  uint64_t* s_done = v_free + kVS;          // [2] S_g of a tile completed (and with it the group's earlier P V)
  uint64_t* p_full = s_done + 2;            // [2] the group's four warps have written P_g (and rescaled O_g)
  uint64_t* o_done = p_full + 2;            // [2] the group's last P V completed
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_done + 2);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    bar_init(q_full, 2);   // one arrival per Q tile
    for (int i = 0; i < kKS; ++i) {
      bar_init(&k_full[i], 1);
      bar_init(&k_free[i], 1);
    }
    for (int i = 0; i < kVS; ++i) {
      bar_init(&v_full[i], 1);
      bar_init(&v_free[i], 1);
    }
    for (int g = 0; g < 2; ++g) {
      bar_init(&s_done[g], 1);
      bar_init(&p_full[g], 4);
      bar_init(&o_done[g], 1);
    }
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (warp == 0) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(zc_smem_u32(tmem_slot)),
                 "r"(kFaTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(tmem_slot);

  const int rb = (int)gridDim.x - 1 - (int)blockIdx.x;     // long blocks first
  const int i0 = rb * kFaRows;
  const int b = blockIdx.y / h_q, h = blockIdx.y % h_q, kv = h / G;
  // group g attends key tiles 0 .. 2 rb + g (the last one holds its diagonal), as far as there are keys
  const int n_all = (l + kM - 1) / kM;
  const int n0 = min(2 * rb + 1, n_all), n1 = min(2 * rb + 2, n_all);

  if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 80;\n");
    if (warp == 1 && lane == 0) {
      // ---- copies ----
      tma_key_tile(&qmap, q_addr, q_full, i0, h, b);
      tma_key_tile(&qmap, q_addr + kTile, q_full, i0 + kM, h, b);
      for (int t = 0; t < n1; ++t) {
        const int ks = t % kKS, vs = t % kVS;
        if (t >= kKS) bar_wait(&k_free[ks], (uint32_t)(t / kKS - 1) & 1u);
        tma_key_tile(&kmap, k_addr + ks * kTile, &k_full[ks], t * kM, kv, b);
        if (t >= kVS) bar_wait(&v_free[vs], (uint32_t)(t / kVS - 1) & 1u);
        tma_key_tile(&vmap, v_addr + vs * kTile, &v_full[vs], t * kM, kv, b);
      }
    } else if (warp == 0 && lane == 0) {
      // ---- MMAs ----
      const uint32_t idesc_s = instr_desc<T>();
      const uint32_t idesc_pv = instr_desc<T>() | (1u << 16);   // B with its N dimension contiguous
      const uint32_t tmem_s0 = tmem, tmem_s1 = tmem + kM, tmem_o0 = tmem + 2 * kM, tmem_o1 = tmem + 3 * kM;
      bar_wait(q_full, 0u);
      bar_wait(&k_full[0], 0u);
      mma_tile(tmem_s0, q_addr, k_addr, idesc_s);
      mma_commit(&s_done[0]);
      mma_tile(tmem_s1, q_addr + kTile, k_addr, idesc_s);
      mma_commit(&s_done[1]);
      mma_commit(&k_free[0]);
      for (int j = 0; j < n1; ++j) {
        const int vs = j % kVS, ks1 = (j + 1) % kKS;
        const uint32_t v_tile = v_addr + vs * kTile, k_next = k_addr + ks1 * kTile;
        bool k_ready = false;
        if (j < n0) {
          bar_wait(&p_full[0], (uint32_t)j & 1u);
          bar_wait(&v_full[vs], (uint32_t)(j / kVS) & 1u);
          tc_fence_after();
          mma_pv(tmem_o0, tmem_s0, v_tile, idesc_pv, j > 0);
          if (j + 1 < n0) {
            bar_wait(&k_full[ks1], (uint32_t)((j + 1) / kKS) & 1u);
            k_ready = true;
            mma_tile(tmem_s0, q_addr, k_next, idesc_s);
            mma_commit(&s_done[0]);
          } else {
            mma_commit(&o_done[0]);
          }
        }
        bar_wait(&p_full[1], (uint32_t)j & 1u);
        if (j >= n0) bar_wait(&v_full[vs], (uint32_t)(j / kVS) & 1u);
        tc_fence_after();
        mma_pv(tmem_o1, tmem_s1, v_tile, idesc_pv, j > 0);
        mma_commit(&v_free[vs]);
        if (j + 1 < n1) {
          if (!k_ready) bar_wait(&k_full[ks1], (uint32_t)((j + 1) / kKS) & 1u);
          mma_tile(tmem_s1, q_addr + kTile, k_next, idesc_s);
          mma_commit(&s_done[1]);
          mma_commit(&k_free[ks1]);
        } else {
          mma_commit(&o_done[1]);
        }
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 208;\n");
    const int g = (warp >> 2) - 1, quarter = warp & 3, row = quarter * 32 + lane;
    const int i = i0 + g * kM + row;                          // this thread's query position
    const int n_kt = g ? n1 : n0;
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const uint32_t tmem_s = tmem + lane_off + (uint32_t)g * kM, tmem_o = tmem + lane_off + (uint32_t)(2 + g) * kM;
    const float scale = kLog2e * rsqrtf((float)ZC_D);
    float m_run = -INFINITY, s_run = 0.f;
    for (int kt = 0; kt < n_kt; ++kt) {
      float v[kM];
      bar_wait(&s_done[g], (uint32_t)kt & 1u);
      tc_fence_after();
      tmem_ld128(v, tmem_s);
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      if (kt == n_kt - 1) {
#pragma unroll
        for (int e = 0; e < kM; ++e) {
          if (kt * kM + e > i) v[e] = -INFINITY;             // causal mask on the diagonal tile
          mx4[e & 3] = fmaxf(mx4[e & 3], v[e]);
        }
      } else {
#pragma unroll
        for (int e = 0; e < kM; ++e) mx4[e & 3] = fmaxf(mx4[e & 3], v[e]);
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale;
      const bool grow = mx > m_run + kFaTau || m_run == -INFINITY;
      if (__any_sync(0xffffffffu, grow && kt > 0)) {
        // some row of the warp moves its maximum: its share of O, accumulated with the old one,
        // is rescaled in tensor memory (the previous tile's P V completed before this tile's S)
        const float alpha = grow ? (m_run == -INFINITY ? 0.f : zc_exp2(m_run - mx)) : 1.f;
#pragma unroll 1
        for (int q8 = 0; q8 < 16; ++q8) {
          float o[8];
          tmem_ld8(o, tmem_o + 8 * q8);
#pragma unroll
          for (int e = 0; e < 8; ++e) o[e] *= alpha;
          tmem_st8(o, tmem_o + 8 * q8);
        }
      }
      if (grow) {
        s_run *= m_run == -INFINITY ? 0.f : zc_exp2(m_run - mx);
        m_run = mx;
      }
      // p = 2^(s - m) as the tensor cores will see it (rounded to the input type), summed in fp32
      // from the unrounded values
      float add[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        uint32_t w[32];
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          const float p0 = zc_exp2(fmaf(v[64 * half + 2 * c], scale, -m_run));
          const float p1 = zc_exp2(fmaf(v[64 * half + 2 * c + 1], scale, -m_run));
          add[c & 1] += p0;
          add[2 + (c & 1)] += p1;
          w[c] = pack2<T>(p0, p1);
        }
        tmem_st32(w, tmem_s + 32 * half);
      }
      s_run += (add[0] + add[1]) + (add[2] + add[3]);
      asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory");
      tc_fence_before();
      __syncwarp();
      if (lane == 0) bar_arrive(&p_full[g]);
    }
    // ---- the row's output and log-sum-exp ----
    bar_wait(&o_done[g], 0u);
    tc_fence_after();
    const float inv = 1.f / s_run;
    T* orow = O + ((long long)blockIdx.y * l + i) * ZC_D;
#pragma unroll 1
    for (int q4 = 0; q4 < 4; ++q4) {
      float o[32];
      tmem_ld32(o, tmem_o + 32 * q4);
      if (i < l) {
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {
          const uint4 w = make_uint4(pack2<T>(o[8 * c4] * inv, o[8 * c4 + 1] * inv),
                                     pack2<T>(o[8 * c4 + 2] * inv, o[8 * c4 + 3] * inv),
                                     pack2<T>(o[8 * c4 + 4] * inv, o[8 * c4 + 5] * inv),
                                     pack2<T>(o[8 * c4 + 6] * inv, o[8 * c4 + 7] * inv));
          *reinterpret_cast<uint4*>(orow + 32 * q4 + 8 * c4) = w;
        }
      }
    }
    if (i < l) lse[(long long)blockIdx.y * l + i] = m_run + log2f(s_run);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(kFaTmemCols) : "memory");
}

// lse_probe[b][h][r] = lse_rows[b][h][P[r]]: the probe rows' statistics in the layout the
// column-sum pass reads.
__global__ void k_gather_probe_lse(const float* __restrict__ lse_rows, const int32_t* __restrict__ P, int n_probe,
                                   int l, float* __restrict__ lse_probe) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r < n_probe) lse_probe[(long long)blockIdx.y * n_probe + r] = lse_rows[(long long)blockIdx.y * l + P[r]];
}

}  // namespace

int zc_launch_prefill_attention(zc_cache* c, const void* Q, const void* K, const void* V, int l,
                                const int64_t* qs, const int64_t* ks, void* O, float* lse, cudaStream_t st) {
  const zc_config& cfg = c->cfg;
  CUtensorMap qmap, kmap, vmap;
  memset(&qmap, 0, sizeof(qmap));
  memset(&kmap, 0, sizeof(kmap));
  memset(&vmap, 0, sizeof(vmap));
  if (!make_key_map(&qmap, Q, cfg.dtype, l, cfg.n_q_heads, cfg.batch, qs) ||
      !make_key_map(&kmap, K, cfg.dtype, l, cfg.n_kv_heads, cfg.batch, ks) ||
      !make_key_map(&vmap, V, cfg.dtype, l, cfg.n_kv_heads, cfg.batch, ks))
    return (int)cudaErrorNotSupported;   // the kernel fetches every tile through tensor maps
  const dim3 grid(zc_ceil_div(l, kFaRows), cfg.batch * cfg.n_q_heads);
  cudaError_t e;
  if (cfg.dtype == ZC_F16) {
    e = cudaFuncSetAttribute(k_flash_prefill<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFaSmem);
    if (e != cudaSuccess) return e;
    k_flash_prefill<__half><<<grid, kFaThreads, kFaSmem, st>>>(l, cfg.n_q_heads, c->lay.G, (__half*)O, lse, qmap,
                                                               kmap, vmap);
  } else {
    e = cudaFuncSetAttribute(k_flash_prefill<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFaSmem);
    if (e != cudaSuccess) return e;
    k_flash_prefill<__nv_bfloat16><<<grid, kFaThreads, kFaSmem, st>>>(l, cfg.n_q_heads, c->lay.G,
                                                                       (__nv_bfloat16*)O, lse, qmap, kmap, vmap);
  }
  c->launches += 1;
  return (int)cudaGetLastError();
}

int zc_launch_gather_probe_lse(zc_cache* c, const float* lse_rows, const int32_t* P_dev, int n_probe, int l,
                               float* lse_probe, cudaStream_t st) {
  const dim3 grid(zc_ceil_div(n_probe, 256), c->cfg.batch * c->cfg.n_q_heads);
  k_gather_probe_lse<<<grid, 256, 0, st>>>(lse_rows, P_dev, n_probe, l, lse_probe);
  c->launches += 1;
  return (int)cudaGetLastError();
}

int zc_attention_error_code(int* out) {
  return (int)cudaMemcpyFromSymbol(out, g_zc_tc_error, sizeof(int));
}
