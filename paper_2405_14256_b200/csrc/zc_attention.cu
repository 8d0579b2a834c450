// Causal prefill attention (Eq. 2; Alg. 2's line "O = FlashAttention(Q, K, V)") that also keeps
// every row's log-sum-exp, so that the probe rows' statistics of Eq. 9 need no pass of their own
// (Appendix B: one attention call serves all tokens while the probe scores are computed beside it).
//
// One CTA = 128 consecutive query rows of one query head; key tiles of 128 are streamed.
// Both contractions run on the 5th-generation tensor cores (tcgen05.mma, operands in shared
// memory, accumulators in tensor memory):
//   S = Q K^T      A = Q tile, B = key tile, both K-major; 128 x 128 fp32 in TMEM (two buffers)
//   O += P V       A = P tile (the 128 worker threads write their rows of exp2(s - m) in the
//                  input type), B = value tile as it comes from memory ([key][d]: the N
//                  dimension contiguous, "MN-major"), 128 x 128 fp32 in TMEM, accumulated
//                  over the key tiles
// Row m of either accumulator lives in TMEM lane m, so a worker thread owns one query row: its
// running maximum (refreshed only when a logit exceeds it by 8, base 2; O's row is then rescaled
// in TMEM), its sum, its row of P.  Q, K and V tiles come in by tensor-map bulk copies issued by
// the thread that issues the MMAs.  Every wait is bounded.
#include "zc_internal.h"
#include "zc_layout.cuh"
#include "zc_tc.cuh"

namespace {

constexpr int kFaThreads = 160;                   // warp 0: copies + MMAs; warps 1..4: one query row per thread
constexpr uint32_t kFaTmemCols = 512;             // S0 | S1 | O | (unused)
constexpr int kFaSmem = 6 * kTile + 1024 + 256;   // Q, K x 2, V x 2, P + alignment + barriers
constexpr float kFaTau = 8.f;

// B operand whose N dimension is contiguous in memory: rows of the tile are K indices (keys) of
// 128 bytes = 64 elements of N; 8-row groups 1024 bytes apart, the second 64 elements of N one
// k-block (16 KB) further.
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(kKBlock >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__device__ __forceinline__ void mma_step(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n}\n" ::"r"(tmem_d),
      "l"(da), "l"(db), "r"(idesc), "r"(acc), "r"(0u)
      : "memory");
}
// O (+)= P V for one key tile: 8 steps of 16 keys
__device__ __forceinline__ void mma_pv(uint32_t tmem_o, uint32_t p_addr, uint32_t v_addr, uint32_t idesc, bool accumulate) {
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    const uint64_t da = smem_desc(p_addr + (ks >> 2) * kKBlock + (ks & 3) * 32);
    const uint64_t db = smem_desc_mn(v_addr + ks * 16 * 128);
    mma_step(tmem_o, da, db, idesc, (accumulate || ks > 0) ? 1u : 0u);
  }
}
__device__ __forceinline__ void tmem_st32(const float* v, uint32_t taddr) {
  const uint32_t* r = reinterpret_cast<const uint32_t*>(v);
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

template <typename T> __device__ __forceinline__ uint32_t pack2(float a, float b);
template <> __device__ __forceinline__ uint32_t pack2<__half>(float a, float b) {
  const __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}
template <> __device__ __forceinline__ uint32_t pack2<__nv_bfloat16>(float a, float b) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// grid.x: blocks of 128 query rows, the last (longest) first; grid.y: (batch, query head).
template <typename T>
__global__ void __launch_bounds__(kFaThreads, 1) k_flash_prefill(
    int l, int h_q, int G, T* __restrict__ O, float* __restrict__ lse, const __grid_constant__ CUtensorMap qmap,
    const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap) {
  extern __shared__ char smem_raw[];
  const uint32_t raw_u = zc_smem_u32(smem_raw);
  const uint32_t base_u = (raw_u + 1023u) & ~1023u;
  char* base = smem_raw + (base_u - raw_u);
  const uint32_t q_addr = base_u, k_addr = base_u + kTile, v_addr = base_u + 3 * kTile, p_addr = base_u + 5 * kTile;
  char* Ps = base + 5 * kTile;
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + 6 * kTile);
  uint64_t* q_full = bars;            // Q tile landed
  uint64_t* k_full = bars + 1;        // [2] key tile landed
  uint64_t* v_full = bars + 3;        // [2] value tile landed
  uint64_t* s_done = bars + 5;        // [2] S = Q K^T of a tile completed
  uint64_t* s_free = bars + 7;        // [2] the four worker warps have read that S
  uint64_t* p_full = bars + 9;        // the four worker warps have written their rows of P (and rescaled O)
  uint64_t* pv_done = bars + 10;      // O += P V of a tile completed: P, the V buffer and O's rows are free
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 12);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (tid == 0) {
    bar_init(q_full, 1);
    for (int i = 0; i < 2; ++i) {
      bar_init(&k_full[i], 1);
      bar_init(&v_full[i], 1);
      bar_init(&s_done[i], 1);
      bar_init(&s_free[i], 4);
    }
    bar_init(p_full, 4);
    bar_init(pv_done, 1);
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
  const uint32_t tmem_o = tmem + 2 * kM;

  const int rb = (int)gridDim.x - 1 - (int)blockIdx.x;     // long blocks first
  const int i0 = rb * kM;
  const int b = blockIdx.y / h_q, h = blockIdx.y % h_q, kv = h / G;
  const int n_kt = rb + 1;                                  // key tiles 0 .. rb (the last one holds the diagonal)

  if (warp == 0) {
    if (lane == 0) {
      const uint32_t idesc_s = instr_desc<T>();
      const uint32_t idesc_pv = instr_desc<T>() | (1u << 16);   // B with its N dimension contiguous
      tma_key_tile(&qmap, q_addr, q_full, i0, h, b);
      tma_key_tile(&kmap, k_addr, &k_full[0], 0, kv, b);
      tma_key_tile(&vmap, v_addr, &v_full[0], 0, kv, b);
      if (n_kt > 1) {
        tma_key_tile(&kmap, k_addr + kTile, &k_full[1], kM, kv, b);
        tma_key_tile(&vmap, v_addr + kTile, &v_full[1], kM, kv, b);
      }
      bar_wait(q_full, 0u);
      bar_wait(&k_full[0], 0u);
      async_proxy_fence();
      tc_fence_after();
      mma_tile(tmem, q_addr, k_addr, idesc_s);
      mma_commit(&s_done[0]);
      for (int kt = 0; kt < n_kt; ++kt) {
        const int buf = kt & 1, nb = buf ^ 1;
        // the key buffer of tile kt is free as soon as S of tile kt has completed (it was issued an
        // iteration ago): tile kt + 2 is sent for now, two iterations ahead of its use
        if (kt + 2 < n_kt) {
          bar_wait(&s_done[buf], (uint32_t)(kt >> 1) & 1u);
          tma_key_tile(&kmap, k_addr + buf * kTile, &k_full[buf], (kt + 2) * kM, kv, b);
        }
        // the value buffer of tile kt - 1 is free once its P V has completed: tile kt + 1
        if (kt >= 1 && kt + 1 < n_kt) {
          bar_wait(pv_done, (uint32_t)(kt - 1) & 1u);
          tma_key_tile(&vmap, v_addr + nb * kTile, &v_full[nb], (kt + 1) * kM, kv, b);
        }
        if (kt + 1 < n_kt) {   // S of the next tile, while the workers turn this one into P
          bar_wait(&k_full[nb], (uint32_t)((kt + 1) >> 1) & 1u);
          if (kt + 1 >= 2) bar_wait(&s_free[nb], (uint32_t)((kt - 1) >> 1) & 1u);
          async_proxy_fence();
          tc_fence_after();
          mma_tile(tmem + (uint32_t)nb * kM, q_addr, k_addr + nb * kTile, idesc_s);
          mma_commit(&s_done[nb]);
        }
        bar_wait(p_full, (uint32_t)kt & 1u);
        bar_wait(&v_full[buf], (uint32_t)(kt >> 1) & 1u);
        async_proxy_fence();
        tc_fence_after();
        mma_pv(tmem_o, p_addr, v_addr + buf * kTile, idesc_pv, kt > 0);
        mma_commit(pv_done);
      }
    }
  } else {
    const int quarter = warp & 3, row = quarter * 32 + lane;
    const int i = i0 + row;                                   // this thread's query position
    const uint32_t lane_off = (uint32_t)(quarter * 32) << 16;
    const float scale = kLog2e * rsqrtf((float)ZC_D);
    float m_run = -INFINITY, s_run = 0.f;
    bool o_waited = true;   // has this thread seen the previous tile's P V complete?
    for (int kt = 0; kt < n_kt; ++kt) {
      const int buf = kt & 1;
      float v[kM];
      bar_wait(&s_done[buf], (uint32_t)(kt >> 1) & 1u);
      tc_fence_after();
      tmem_ld128(v, tmem + lane_off + (uint32_t)buf * kM);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) bar_arrive(&s_free[buf]);
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
      o_waited = kt == 0;
      const bool grow = mx > m_run + kFaTau || m_run == -INFINITY;
      if (__any_sync(0xffffffffu, grow && kt > 0)) {
        // some row of the warp moves its maximum: its share of O, accumulated with the old one,
        // is rescaled in tensor memory (after the previous tile's P V has completed)
        bar_wait(pv_done, (uint32_t)(kt - 1) & 1u);
        o_waited = true;
        tc_fence_after();
        const float alpha = grow ? (m_run == -INFINITY ? 0.f : zc_exp2(m_run - mx)) : 1.f;
#pragma unroll 1
        for (int q4 = 0; q4 < 4; ++q4) {
          float o[32];
          tmem_ld32(o, tmem_o + lane_off + 32 * q4);
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] *= alpha;
          tmem_st32(o, tmem_o + lane_off + 32 * q4);
        }
        asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory");
        tc_fence_before();
      }
      if (grow) {
        s_run *= m_run == -INFINITY ? 0.f : zc_exp2(m_run - mx);
        m_run = mx;
      }
      // p = 2^(s - m) as the tensor cores will see it (rounded to the input type), summed in fp32
      // from the unrounded values
      float add[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int e = 0; e < kM; ++e) {
        v[e] = zc_exp2(fmaf(v[e], scale, -m_run));
        add[e & 3] += v[e];
      }
      s_run += (add[0] + add[1]) + (add[2] + add[3]);
      if (!o_waited) bar_wait(pv_done, (uint32_t)(kt - 1) & 1u);   // P is free once the previous P V has read it
#pragma unroll
      for (int ch = 0; ch < 16; ++ch) {
        const uint4 w = make_uint4(pack2<T>(v[8 * ch], v[8 * ch + 1]), pack2<T>(v[8 * ch + 2], v[8 * ch + 3]),
                                   pack2<T>(v[8 * ch + 4], v[8 * ch + 5]), pack2<T>(v[8 * ch + 6], v[8 * ch + 7]));
        *reinterpret_cast<uint4*>(tile_chunk(Ps, row, ch)) = w;
      }
      async_proxy_fence();   // plain stores the tensor core will read
      __syncwarp();
      if (lane == 0) bar_arrive(p_full);
    }
    // ---- the row's output and log-sum-exp ----
    bar_wait(pv_done, (uint32_t)(n_kt - 1) & 1u);
    tc_fence_after();
    const float inv = 1.f / s_run;
    T* orow = O + ((long long)blockIdx.y * l + i) * ZC_D;
#pragma unroll 1
    for (int q4 = 0; q4 < 4; ++q4) {
      float o[32];
      tmem_ld32(o, tmem_o + lane_off + 32 * q4);
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
    tc_fence_before();
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
  const dim3 grid(zc_ceil_div(l, kM), cfg.batch * cfg.n_q_heads);
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
