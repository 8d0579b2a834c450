// Probe attention (Eq. 9) and the normalised attention score (Eq. 8).
//
// Two passes over the probe rows, neither of which stores the n_probe x l matrix:
//   pass 1  per (query head, 64 probe rows): log-sum-exp of each causal row;
//   pass 2  per (KV head, 64 keys): column sums of exp(s - lse) over the G query heads
//           and all probe rows that see the column, divided by G * nnz_j, where
//           nnz_j = #{r : p_r >= j} is the structural count of unmasked rows.
// Both passes are the same tensor-core contraction (warp-level m16n8k16 MMA, fp32
// accumulate): a resident 64 x 128 A tile against streamed 64 x 128 B tiles.
#include "zc_internal.h"
#include "zc_layout.cuh"
#include "zc_mma.cuh"

namespace {

constexpr int kRows = 64;                       // rows per tile
constexpr int kTileBytes = kRows * ZC_D * 2;    // 16 KB
constexpr float kLog2e = 1.4426950408889634f;

// 16-byte chunk `chunk` of row `row` inside a swizzled [64][128] 16-bit tile
__device__ __forceinline__ char* tile_ptr(char* tile, int row, int chunk) {
  return tile + row * 256 + ((chunk ^ (row & 7)) << 4);
}

// Copy one 256-byte row (or zeros) into a tile; 16 threads per row.
__device__ __forceinline__ void load_row_async(char* tile, int row, int chunk, const char* src) {
  if (src) {
    zc_cp_async16(tile_ptr(tile, row, chunk), src + chunk * 16);
  } else {
    *reinterpret_cast<uint4*>(tile_ptr(tile, row, chunk)) = make_uint4(0, 0, 0, 0);
  }
}

__device__ __forceinline__ void load_a_frags(uint32_t (&a)[8][4], char* tile, int warp, int lane) {
#pragma unroll
  for (int ks = 0; ks < 8; ++ks)
    zc_ldmatrix_x4(a[ks], tile_ptr(tile, warp * 16 + (lane & 15), 2 * ks + (lane >> 4)));
}

// acc[nt][.] (16 x 64 per warp) = A(16 x 128) * B(64 x 128)^T
template <typename T>
__device__ __forceinline__ void block_mma(float (&acc)[8][4], const uint32_t (&a)[8][4],
                                          char* btile, int lane) {
#pragma unroll
  for (int nt = 0; nt < 8; ++nt)
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[nt][i] = 0.f;
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
    for (int np = 0; np < 4; ++np) {
      uint32_t b[4];
      const int row = np * 16 + (lane & 7) + ((lane >> 4) << 3);
      zc_ldmatrix_x4(b, tile_ptr(btile, row, 2 * ks + ((lane >> 3) & 1)));
      zc_mma16816<T>(acc[2 * np], a[ks], b[0], b[1]);
      zc_mma16816<T>(acc[2 * np + 1], a[ks], b[2], b[3]);
    }
  }
}

// ---- pass 1: row log-sum-exp (base 2) of the causal probe rows ----
template <typename T>
__global__ void __launch_bounds__(128) k_probe_lse(const T* __restrict__ Q, const T* __restrict__ K,
                                                   const int32_t* __restrict__ P, int n_probe, int l,
                                                   int h_q, int G, long long qsb, long long qsh,
                                                   long long qsl, long long ksb, long long ksh,
                                                   long long ksl, float* __restrict__ lse) {
  extern __shared__ __align__(128) char smem[];
  char* As = smem;
  char* Bs = smem + kTileBytes;  // two buffers
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int r0 = blockIdx.x * kRows;
  const int bh = blockIdx.y, b = bh / h_q, h = bh % h_q, kv = h / G;
  const char* Qb = reinterpret_cast<const char*>(Q + b * qsb + h * qsh);
  const char* Kb = reinterpret_cast<const char*>(K + b * ksb + kv * ksh);
  const int row_ld = tid >> 4, chunk = tid & 15;  // 8 rows per pass of 128 threads

#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = row_ld + 8 * i, r = r0 + row;
    load_row_async(As, row, chunk, r < n_probe ? Qb + (long long)P[r] * qsl * 2 : nullptr);
  }
  const int p_last = P[min(r0 + kRows - 1, n_probe - 1)];
  const int n_cb = p_last / kRows + 1;
  auto load_b = [&](int cb, int buf) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = row_ld + 8 * i, j = cb * kRows + row;
      load_row_async(Bs + buf * kTileBytes, row, chunk, j < l ? Kb + (long long)j * ksl * 2 : nullptr);
    }
  };
  load_b(0, 0);
  zc_cp_async_commit();

  const int g = lane >> 2, t = lane & 3;
  const int ra = r0 + warp * 16 + g, rb = ra + 8;
  const int pa = ra < n_probe ? P[ra] : -1, pb = rb < n_probe ? P[rb] : -1;
  float m_a = -INFINITY, m_b = -INFINITY, s_a = 0.f, s_b = 0.f;
  const float scale = kLog2e * rsqrtf((float)ZC_D);
  uint32_t a[8][4];
  float acc[8][4];
  for (int cb = 0; cb < n_cb; ++cb) {
    if (cb + 1 < n_cb) load_b(cb + 1, (cb + 1) & 1);
    zc_cp_async_commit();
    zc_cp_async_wait<1>();
    __syncthreads();
    if (cb == 0) load_a_frags(a, As, warp, lane);
    block_mma<T>(acc, a, Bs + (cb & 1) * kTileBytes, lane);
    float mx_a = -INFINITY, mx_b = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int j = cb * kRows + nt * 8 + 2 * t + e;
        acc[nt][e] = j <= pa ? acc[nt][e] * scale : -INFINITY;
        acc[nt][2 + e] = j <= pb ? acc[nt][2 + e] * scale : -INFINITY;
        mx_a = fmaxf(mx_a, acc[nt][e]);
        mx_b = fmaxf(mx_b, acc[nt][2 + e]);
      }
    }
    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1));
    mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1));
    mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
    const float mn_a = fmaxf(m_a, mx_a), mn_b = fmaxf(m_b, mx_b);
    // a row with no visible column yet keeps (m, s) = (-inf, 0)
    const float ca = mn_a == -INFINITY ? 0.f : zc_exp2(m_a - mn_a);
    const float cbf = mn_b == -INFINITY ? 0.f : zc_exp2(m_b - mn_b);
    const float ba = mn_a == -INFINITY ? 0.f : mn_a, bb = mn_b == -INFINITY ? 0.f : mn_b;
    float add_a = 0.f, add_b = 0.f;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        add_a += zc_exp2(acc[nt][e] - ba);
        add_b += zc_exp2(acc[nt][2 + e] - bb);
      }
    }
    s_a = s_a * ca + add_a;
    s_b = s_b * cbf + add_b;
    m_a = mn_a;
    m_b = mn_b;
    __syncthreads();
  }
  s_a += __shfl_xor_sync(0xffffffffu, s_a, 1);
  s_a += __shfl_xor_sync(0xffffffffu, s_a, 2);
  s_b += __shfl_xor_sync(0xffffffffu, s_b, 1);
  s_b += __shfl_xor_sync(0xffffffffu, s_b, 2);
  if (t == 0) {
    if (ra < n_probe) lse[(long long)bh * n_probe + ra] = m_a + log2f(s_a);
    if (rb < n_probe) lse[(long long)bh * n_probe + rb] = m_b + log2f(s_b);
  }
}

// ---- pass 2: column sums of the normalised probe rows -> p_tilde ----
template <typename T>
__global__ void __launch_bounds__(128) k_probe_colsum(const T* __restrict__ Q, const T* __restrict__ K,
                                                      const int32_t* __restrict__ P, int n_probe, int l,
                                                      int h_q, int n_kv, int G, long long qsb,
                                                      long long qsh, long long qsl, long long ksb,
                                                      long long ksh, long long ksl,
                                                      const float* __restrict__ lse, char* cache,
                                                      long long unit_stride, long long off_scores) {
  extern __shared__ __align__(128) char smem[];
  char* As = smem;
  char* Bs = smem + kTileBytes;
  int* Pp = reinterpret_cast<int*>(smem + 3 * kTileBytes);          // [2][64]
  float* Ll = reinterpret_cast<float*>(smem + 3 * kTileBytes + 512);  // [2][64]
  __shared__ int s_rstart;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int j0 = blockIdx.x * kRows;
  const int unit = blockIdx.y, b = unit / n_kv, kv = unit % n_kv;
  const char* Kb = reinterpret_cast<const char*>(K + b * ksb + kv * ksh);
  const int row_ld = tid >> 4, chunk = tid & 15;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = row_ld + 8 * i, j = j0 + row;
    load_row_async(As, row, chunk, j < l ? Kb + (long long)j * ksl * 2 : nullptr);
  }
  if (tid == 0) {  // first probe row that sees column j0
    int lo = 0, hi = n_probe;
    while (lo < hi) {
      int mid = (lo + hi) >> 1;
      if (P[mid] < j0) lo = mid + 1; else hi = mid;
    }
    s_rstart = lo;
  }
  __syncthreads();
  const int r_start = s_rstart;
  const int n_rb = (n_probe - r_start + kRows - 1) / kRows;
  const int n_tiles = n_rb * G;
  auto load_b = [&](int tile, int buf) {
    const int gq = tile / n_rb, rb = tile % n_rb;
    const char* Qb = reinterpret_cast<const char*>(Q + b * qsb + (kv * G + gq) * qsh);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = row_ld + 8 * i, r = r_start + rb * kRows + row;
      load_row_async(Bs + buf * kTileBytes, row, chunk,
                     r < n_probe ? Qb + (long long)P[r] * qsl * 2 : nullptr);
    }
    if (tid < kRows) {
      const int r = r_start + rb * kRows + tid;
      Pp[buf * kRows + tid] = r < n_probe ? P[r] : -1;
      Ll[buf * kRows + tid] =
          r < n_probe ? lse[((long long)b * h_q + kv * G + gq) * n_probe + r] : INFINITY;
    }
  };
  if (n_tiles > 0) load_b(0, 0);
  zc_cp_async_commit();
  const int g = lane >> 2, t = lane & 3;
  const int ja = j0 + warp * 16 + g, jb = ja + 8;
  const float scale = kLog2e * rsqrtf((float)ZC_D);
  float sum_a = 0.f, sum_b = 0.f;
  uint32_t a[8][4];
  float acc[8][4];
  for (int tile = 0; tile < n_tiles; ++tile) {
    if (tile + 1 < n_tiles) load_b(tile + 1, (tile + 1) & 1);
    zc_cp_async_commit();
    zc_cp_async_wait<1>();
    __syncthreads();
    if (tile == 0) load_a_frags(a, As, warp, lane);
    const int buf = tile & 1;
    block_mma<T>(acc, a, Bs + buf * kTileBytes, lane);
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int col = nt * 8 + 2 * t + e;
        const int p = Pp[buf * kRows + col];
        const float ls = Ll[buf * kRows + col];
        sum_a += ja <= p ? zc_exp2(acc[nt][e] * scale - ls) : 0.f;
        sum_b += jb <= p ? zc_exp2(acc[nt][2 + e] * scale - ls) : 0.f;
      }
    }
    __syncthreads();
  }
  sum_a += __shfl_xor_sync(0xffffffffu, sum_a, 1);
  sum_a += __shfl_xor_sync(0xffffffffu, sum_a, 2);
  sum_b += __shfl_xor_sync(0xffffffffu, sum_b, 1);
  sum_b += __shfl_xor_sync(0xffffffffu, sum_b, 2);
  if (t == 0) {
    float* scores = reinterpret_cast<float*>(cache + unit * unit_stride + off_scores);
    const int js[2] = {ja, jb};
    const float sums[2] = {sum_a, sum_b};
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int j = js[k];
      if (j < l) {
        int lo = r_start, hi = n_probe;  // rows with p_r >= j
        while (lo < hi) {
          int mid = (lo + hi) >> 1;
          if (P[mid] < j) lo = mid + 1; else hi = mid;
        }
        const int nnz = n_probe - lo;
        scores[j] = __fdiv_rn(sums[k], (float)(G * nnz));
      }
    }
  }
}

}  // namespace

int zc_launch_probe_scores(zc_cache* c, const void* Q, const void* K, int l, const int64_t* qs,
                           const int64_t* ks, const int32_t* P_dev, int n_probe, float* lse_ws,
                           cudaStream_t st) {
  const zc_config& cfg = c->cfg;
  const int G = c->lay.G;
  const int smem1 = 3 * kTileBytes, smem2 = 3 * kTileBytes + 1024;
  dim3 g1(zc_ceil_div(n_probe, kRows), cfg.batch * cfg.n_q_heads);
  dim3 g2(zc_ceil_div(l, kRows), c->lay.units);
  cudaError_t e;
#define ZC_GO(T)                                                                                   \
  do {                                                                                             \
    e = cudaFuncSetAttribute(k_probe_lse<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem1);   \
    if (e != cudaSuccess) return e;                                                                \
    e = cudaFuncSetAttribute(k_probe_colsum<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,        \
                             smem2);                                                               \
    if (e != cudaSuccess) return e;                                                                \
    k_probe_lse<T><<<g1, 128, smem1, st>>>((const T*)Q, (const T*)K, P_dev, n_probe, l,            \
                                           cfg.n_q_heads, G, qs[0], qs[1], qs[2], ks[0], ks[1],    \
                                           ks[2], lse_ws);                                         \
    k_probe_colsum<T><<<g2, 128, smem2, st>>>((const T*)Q, (const T*)K, P_dev, n_probe, l,         \
                                              cfg.n_q_heads, cfg.n_kv_heads, G, qs[0], qs[1],      \
                                              qs[2], ks[0], ks[1], ks[2], lse_ws, c->base,         \
                                              c->lay.unit_stride, c->lay.off_scores);              \
  } while (0)
  if (cfg.dtype == ZC_F16) ZC_GO(__half); else ZC_GO(__nv_bfloat16);
#undef ZC_GO
  c->launches += 2;
  return cudaGetLastError();
}
