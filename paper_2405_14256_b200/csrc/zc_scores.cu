// Probe attention (Eq. 9) and the normalised attention score (Eq. 8) on the 5th-generation
// tensor cores: tcgen05.mma with both operands in shared memory and the 128 x 128 fp32
// score tile in tensor memory (TMEM).
//
// Two passes over the probe rows, neither of which stores the n_probe x l matrix:
//   pass 1  per (group of query heads of one KV head, block of probe rows): log-sum-exp of
//           each causal row.  A tile = 128 rows = Gt heads x 128/Gt probe rows, B tiles = 128
//           keys each, streamed.
//   pass 2  per (KV head, 128 keys): column sums of exp(s - lse) over the G query heads and
//           all probe rows that see the column, divided by G * nnz_j (nnz_j = #{r : p_r >= j},
//           the structural count of unmasked rows).  A tile = 128 keys, B tiles = 128 probe
//           rows of one query head, streamed.
// In both, D[m][n] = A[m] . B[n] lands in TMEM with row m in TMEM lane m, so after
// tcgen05.ld every thread holds one row of the tile: row maxima, row sums (pass 1) and the
// column sums of pass 2 (columns of the score matrix are the rows of its tile) need no
// shuffle.  The MMA of tile i + 1 runs while the threads work on tile i (two TMEM buffers, two
// B buffers).  Operand tiles are [2 k-blocks][128 rows][128 bytes] with the 128-byte swizzle
// of the shared-memory matrix descriptor.  Tiles of consecutive keys come in by tensor-map bulk
// copies (TMA, hardware swizzle) issued by the MMA thread; tiles of gathered probe rows are
// written by the workers with cp.async.  Every wait is bounded; a wait that runs out records
// an error code and the kernel still frees its TMEM.
#include "zc_internal.h"
#include "zc_layout.cuh"
#include "zc_tc.cuh"

namespace {

// What both kernels share: shared memory carved at a 1024-byte boundary, TMEM, barriers.
// 288 threads: lane 0 of warp 0 issues the MMAs, warps 1..8 are the row workers; worker warp w
// may touch TMEM lanes 32 (w mod 4) .. +31, so warps 1..4 cover the 128 rows of a tile and so do
// warps 5..8: the first group works on the even tiles (accumulator 0), the second on the odd
// ones (accumulator 1), a thread taking its row in two halves of 64 columns.  Two threads per
// row: neither pass needs a row's tiles together before its end, where the groups meet once
// through shared memory; and the groups are at different points of their tiles at any time, so
// one group's exponentials run while the other waits or loads (with all eight warps on the same
// tile the exp2 unit idled while they all waited).  A group's 128 threads also copy the tiles of
// its accumulator that do not come by bulk copy (16 bytes per thread and row).
//   a_full        the A tile has landed
//   b_full[b]     B buffer b has been filled: by all 128 workers' copies
//                 (cp.async.mbarrier.arrive) or by the bulk copies (complete_tx)
//   mma_done[b]   the MMA into accumulator b has completed (tcgen05.commit): the workers may
//                 read it, and the B buffer it read may be refilled
//   tmem_free[b]  the four worker warps of group b have read accumulator b: the next MMA may overwrite it
constexpr int kThreads = 288;
constexpr int kHalf = kM / 2;      // columns of a tile per worker thread
struct TcCtx {
  char* As;
  char* Bs;          // two tiles
  uint64_t* mma_done;
  uint64_t* tmem_free;
  uint64_t* b_full;
  uint64_t* a_full;
  uint32_t* tmem_slot;
  char* extra;       // pass 2: per worker warp, probe positions and lse of the rows of kSide B tiles
  uint32_t a_addr, b_addr, tmem;
  bool bad;          // the tiles would not fit behind the alignment padding: nothing was set up
};
constexpr int kSide = 2;           // per-column data of pass 2: two tiles per worker warp (see k_probe_colsum)
constexpr int kTcSlack = 768;      // what aligning the tiles to 1 KB may take (the base is declared 1 KB aligned)
constexpr int kTcSmem = 3 * kTile + kTcSlack + 128 /* barriers, tmem slot */ + 8 * kSide * kM * 8;
static_assert(kTcSmem <= 115712, "two CTAs per SM");

__device__ __forceinline__ TcCtx tc_setup(char* raw, int a_count, int b_count) {
  TcCtx c;
  const uint32_t raw_u = zc_smem_u32(raw);
  const uint32_t base_u = (raw_u + 1023u) & ~1023u;
  c.bad = base_u - raw_u > (uint32_t)kTcSlack;
  if (c.bad) {
    if (threadIdx.x == 0) atomicExch(&g_zc_tc_error, 3);
    return c;
  }
  char* base = raw + (base_u - raw_u);
  c.As = base;
  c.Bs = base + kTile;
  c.mma_done = reinterpret_cast<uint64_t*>(base + 3 * kTile);
  c.tmem_free = c.mma_done + 2;
  c.b_full = c.mma_done + 4;
  c.a_full = c.mma_done + 6;
  c.tmem_slot = reinterpret_cast<uint32_t*>(base + 3 * kTile + 96);
  c.extra = base + 3 * kTile + 128;
  c.a_addr = base_u;
  c.b_addr = base_u + kTile;
  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      bar_init(&c.mma_done[i], 1);
      bar_init(&c.tmem_free[i], 4);
      bar_init(&c.b_full[i], b_count);
    }
    bar_init(c.a_full, a_count);
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
  }
  if (threadIdx.x < 32) {
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(
                     zc_smem_u32(c.tmem_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  c.tmem = *reinterpret_cast<volatile uint32_t*>(c.tmem_slot);
  return c;
}
__device__ __forceinline__ void tc_teardown(const TcCtx& c) {
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(c.tmem), "r"(kTmemCols) : "memory");
}

// Tile `cb` goes into B buffer cb & 1 and accumulator cb & 1.
// The issuing thread: for every tile, wait until its operands are in shared memory and its
// accumulator has been read, then issue its MMAs.  refill(tile, buffer): called once the MMA
// that read `buffer` has completed, for kernels whose B tiles this thread fetches itself.
template <typename Refill>
__device__ __forceinline__ void issue_loop(const TcCtx& c, int n, uint32_t idesc, bool refills, Refill refill) {
  bar_wait(c.a_full, 0u);
  for (int cb = 0; cb < n; ++cb) {
    const int buf = cb & 1;
    bar_wait(&c.b_full[buf], (uint32_t)(cb >> 1) & 1u);
    async_proxy_fence();
    if (cb >= 2) bar_wait(&c.tmem_free[buf], (uint32_t)((cb - 2) >> 1) & 1u);
    tc_fence_after();
    mma_tile(c.tmem + (uint32_t)buf * kM, c.a_addr, c.b_addr + buf * kTile, idesc);
    mma_commit(&c.mma_done[buf]);
    if (refills && cb + 2 < n) {
      bar_wait(&c.mma_done[buf], (uint32_t)(cb >> 1) & 1u);
      refill(cb + 2, buf);
    }
  }
}
// Worker: waits for tile cb's accumulator; fetches one half (64 columns) of this thread's row of
// it; after the second half, gives the accumulator back.
__device__ __forceinline__ void worker_wait(const TcCtx& c, int cb) {
  bar_wait(&c.mma_done[cb & 1], (uint32_t)(cb >> 1) & 1u);
  tc_fence_after();
}
__device__ __forceinline__ void worker_load(const TcCtx& c, int cb, int quarter, int half, float (&v)[kHalf]) {
  const uint32_t t = c.tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)((cb & 1) * kM + half * kHalf);
  tmem_ld32_nowait(v, t);
  tmem_ld32_nowait(v + 32, t + 32);
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void worker_release(const TcCtx& c, int cb) {
  tc_fence_before();
  __syncwarp();
  if ((threadIdx.x & 31) == 0) bar_arrive(&c.tmem_free[cb & 1]);
}

// The eight worker warps meet (warp 0 does not take part).
__device__ __forceinline__ void workers_sync() { asm volatile("bar.sync 1, 256;\n" ::: "memory"); }

// ---- pass 1: row log-sum-exp (base 2) of the causal probe rows ----
// grid.x: blocks of rph = 128 / Gt probe rows, longest first; grid.y: (batch, group of Gt query heads).
template <typename T>
__global__ void __launch_bounds__(kThreads, 2) k_probe_lse(const T* __restrict__ Q, const T* __restrict__ K,
                                                             const int32_t* __restrict__ P, int n_probe, int l,
                                                             int h_q, int G, int Gt, long long qsb,
                                                             long long qsh, long long qsl, long long ksb,
                                                             long long ksh, long long ksl,
                                                             float* __restrict__ lse,
                                                             const __grid_constant__ CUtensorMap kmap,
                                                             int use_tma) {
  extern __shared__ __align__(1024) char smem_raw[];
  // A (gathered probe rows): the 128 workers' copies; B (key tiles): bulk copies, or the workers
  TcCtx c = tc_setup(smem_raw, kM, use_tma ? 1 : kM);
  if (c.bad) return;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int rph = kM / Gt;
  const int r0 = ((int)gridDim.x - 1 - (int)blockIdx.x) * rph;   // rows ascend in position: long blocks first
  const int groups = h_q / Gt;
  const int b = blockIdx.y / groups, hg = blockIdx.y % groups, h0 = hg * Gt, kv = h0 / G;
  const int p_last = P[min(r0 + rph - 1, n_probe - 1)];
  const int n_cb = p_last / kM + 1;
  if (warp == 0) {
    if (lane == 0) {
      auto fetch = [&](int cb, int buf) { tma_key_tile(&kmap, c.b_addr + buf * kTile, &c.b_full[buf], cb * kM, kv, b); };
      if (use_tma) {
        fetch(0, 0);
        if (n_cb > 1) fetch(1, 1);
      }
      issue_loop(c, n_cb, instr_desc<T>(), use_tma != 0, fetch);
    }
  } else {
    const char* Kb = reinterpret_cast<const char*>(K + b * ksb + kv * ksh);
    const int quarter = warp & 3, row = quarter * 32 + lane, grp = (warp - 1) >> 2;   // grp: tiles of this parity
    const int wt = (tid - 32) & (kM - 1), row_ld = wt >> 4, chunk = wt & 15;   // 8 rows per pass of a group's 128 workers
    const bool copier = grp == 0;                                              // of the A tile
    auto load_b = [&](int cb) {   // tile cb's keys into B buffer cb & 1, by the group of that parity
#pragma unroll 4
      for (int i = 0; i < 16; ++i) {
        const int rw = row_ld + 8 * i, j = cb * kM + rw;
        load_row(c.Bs + (cb & 1) * kTile, rw, chunk, j < l ? Kb + (long long)j * ksl * 2 : nullptr);
      }
      copies_arrive(&c.b_full[cb & 1]);
    };
    // A: the block's probe rows of the Gt heads (it lands with tile 0)
    if (copier) {
#pragma unroll 4
      for (int i = 0; i < 16; ++i) {
        const int rw = row_ld + 8 * i, hl = rw / rph, r = r0 + rw % rph;
        const char* src = nullptr;
        if (r < n_probe) src = reinterpret_cast<const char*>(Q + b * qsb + (h0 + hl) * qsh) + (long long)P[r] * qsl * 2;
        load_row(c.As, rw, chunk, src);
      }
      copies_arrive(c.a_full);
    }
    if (!use_tma && grp < n_cb) load_b(grp);
    const int my_r = r0 + row % rph;
    const int my_p = my_r < n_probe ? P[my_r] : -1;
    const float scale = kLog2e * rsqrtf((float)ZC_D);
    float m_run = -INFINITY, s_run = 0.f;
    for (int cb = grp; cb < n_cb; cb += 2) {
      worker_wait(c, cb);
      if (!use_tma && cb + 2 < n_cb) load_b(cb + 2);   // its buffer was read by the MMA that has just completed
#pragma unroll 1
      for (int half = 0; half < 2; ++half) {
        float v[kHalf];
        worker_load(c, cb, quarter, half, v);
        if (half == 1) worker_release(c, cb);
        const int j_base = cb * kM + half * kHalf;
        float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
        if (j_base + kHalf - 1 <= my_p) {
#pragma unroll
          for (int e = 0; e < kHalf; ++e) mx4[e & 3] = fmaxf(mx4[e & 3], v[e]);
        } else {
#pragma unroll
          for (int e = 0; e < kHalf; ++e) {
            if (j_base + e > my_p) v[e] = -INFINITY;
            mx4[e & 3] = fmaxf(mx4[e & 3], v[e]);
          }
        }
        const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
        const float mn = fmaxf(m_run, mx * scale);
        if (mn != -INFINITY) {
          float add[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int e = 0; e < kHalf; ++e) add[e & 3] += zc_exp2(fmaf(v[e], scale, -mn));
          s_run = s_run * zc_exp2(m_run - mn) + ((add[0] + add[1]) + (add[2] + add[3]));
          m_run = mn;
        }
      }
    }
    // the row's two partial results (maximum and sum over the even and over the odd tiles) meet here
    float2* part = reinterpret_cast<float2*>(c.extra);
    if (grp == 1) part[row] = make_float2(m_run, s_run);
    workers_sync();
    if (grp == 0 && my_r < n_probe) {
      const float2 o = part[row];
      const float mn = fmaxf(m_run, o.x);   // key 0 is in tile 0 and every row sees it
      const float tot = s_run * zc_exp2(m_run - mn) + (o.x == -INFINITY ? 0.f : o.y * zc_exp2(o.x - mn));
      lse[((long long)b * h_q + h0 + row / rph) * n_probe + my_r] = mn + log2f(tot);
    }
  }
  tc_teardown(c);
}

// ---- pass 2: column sums of the normalised probe rows -> p_tilde ----
// grid.x: blocks of 128 keys; grid.y: unit (batch, KV head).  B tiles: for every query head of
// the KV head, the probe rows from the first one that sees key j0 on, 128 at a time.
template <typename T>
__global__ void __launch_bounds__(kThreads, 2) k_probe_colsum(
    const T* __restrict__ Q, const T* __restrict__ K, const int32_t* __restrict__ P, int n_probe, int l,
    int h_q, int n_kv, int G, long long qsb, long long qsh, long long qsl, long long ksb, long long ksh,
    long long ksl, const float* __restrict__ lse, char* cache, long long unit_stride, long long off_scores,
    const __grid_constant__ CUtensorMap kmap, int use_tma, const __grid_constant__ CUtensorMap qmap,
    int use_qp) {
  extern __shared__ __align__(1024) char smem_raw[];
  // A (the key block): one bulk copy, or the workers; B (probe rows): bulk copies from the
  // gathered copy of the probe rows when there is one (qmap), else the workers gather them
  TcCtx c = tc_setup(smem_raw, use_tma ? 1 : kM, use_qp ? 1 : kM);
  if (c.bad) return;
  // Per-column data of a B tile (probe position and lse of its 128 rows): every worker warp
  // keeps its own copy of its group's tiles, slot = (tile / 2) mod 2, written while the warp's
  // tile before it is worked on, so the warps need no barrier among themselves.
  const int wq = (threadIdx.x >> 5) > 0 ? (threadIdx.x >> 5) - 1 : 0;
  int* Pp = reinterpret_cast<int*>(c.extra + wq * (kSide * kM * 8));   // [kSide][128]
  float* Ll = reinterpret_cast<float*>(Pp + kSide * kM);                // [kSide][128]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int j0 = blockIdx.x * kM;
  const int unit = blockIdx.y, b = unit / n_kv, kv = unit % n_kv;
  int lo = 0, hi = n_probe;   // first probe row that sees column j0
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (P[mid] < j0) lo = mid + 1; else hi = mid;
  }
  const int r_start = lo;
  const int n_rb = (n_probe - r_start + kM - 1) / kM;
  const int n_tiles = n_rb * G;
  if (warp == 0) {
    if (lane == 0) {
      if (use_tma) tma_key_tile(&kmap, c.a_addr, c.a_full, j0, kv, b);
      auto fetch = [&](int tile, int buf) {
        const int gq = tile / n_rb, rb = tile % n_rb;
        tma_key_tile(&qmap, c.b_addr + buf * kTile, &c.b_full[buf], r_start + rb * kM, kv * G + gq, b);
      };
      if (use_qp) {
        fetch(0, 0);
        if (n_tiles > 1) fetch(1, 1);
      }
      issue_loop(c, n_tiles, instr_desc<T>(), use_qp != 0, fetch);
    }
  } else {
    const char* Kb = reinterpret_cast<const char*>(K + b * ksb + kv * ksh);
    const int quarter = warp & 3, row = quarter * 32 + lane, grp = (warp - 1) >> 2;   // grp: tiles of this parity
    const int wt = (tid - 32) & (kM - 1), row_ld = wt >> 4, chunk = wt & 15;   // 8 rows per pass of a group's 128 workers
    const bool copier = grp == 0;                                              // of the A tile
    auto load_b = [&](int tile) {   // tile's probe rows into B buffer tile & 1 (by the group of that parity), its per-column data into the warp's slot
      const int gq = tile / n_rb, rb = tile % n_rb;
      if (!use_qp) {
        const char* Qb = reinterpret_cast<const char*>(Q + b * qsb + (kv * G + gq) * qsh);
#pragma unroll 4
        for (int i = 0; i < 16; ++i) {
          const int rw = row_ld + 8 * i, r = r_start + rb * kM + rw;
          load_row(c.Bs + (tile & 1) * kTile, rw, chunk, r < n_probe ? Qb + (long long)P[r] * qsl * 2 : nullptr);
        }
        copies_arrive(&c.b_full[tile & 1]);
      }
      const int slot = (tile >> 1) % kSide;
#pragma unroll
      for (int k = 0; k < kM / 32; ++k) {
        const int i = lane + 32 * k, r = r_start + rb * kM + i;
        Pp[slot * kM + i] = r < n_probe ? P[r] : -1;
        Ll[slot * kM + i] = r < n_probe ? lse[((long long)b * h_q + kv * G + gq) * n_probe + r] : INFINITY;
      }
    };
    if (!use_tma && copier) {
#pragma unroll 4
      for (int i = 0; i < 16; ++i) {
        const int rw = row_ld + 8 * i, jj = j0 + rw;
        load_row(c.As, rw, chunk, jj < l ? Kb + (long long)jj * ksl * 2 : nullptr);
      }
      copies_arrive(c.a_full);
    }
    if (grp < n_tiles) load_b(grp);
    __syncwarp();   // per-column data of the warp's first tile is visible to the warp
    const int j = j0 + row;
    const float scale = kLog2e * rsqrtf((float)ZC_D);
    float sum4[4] = {0.f, 0.f, 0.f, 0.f};
    for (int tile = grp; tile < n_tiles; tile += 2) {
      const int slot = (tile >> 1) % kSide;
      worker_wait(c, tile);
      if (tile + 2 < n_tiles) load_b(tile + 2);   // its buffer was read by the MMA that has just completed
      __syncwarp();   // per-column data written here is read in the warp's next iteration
#pragma unroll 1
      for (int half = 0; half < 2; ++half) {
        float v[kHalf];
        worker_load(c, tile, quarter, half, v);
        if (half == 1) worker_release(c, tile);
        const int* pp = Pp + slot * kM + half * kHalf;
        const float* ll = Ll + slot * kM + half * kHalf;
        if (j <= pp[0]) {   // probe rows ascend in position: every row of the half-tile sees column j
#pragma unroll
          for (int e = 0; e < kHalf; ++e) sum4[e & 3] += zc_exp2(fmaf(v[e], scale, -ll[e]));
        } else {
#pragma unroll
          for (int e = 0; e < kHalf; ++e) sum4[e & 3] += j <= pp[e] ? zc_exp2(fmaf(v[e], scale, -ll[e])) : 0.f;
        }
      }
    }
    // the column's two partial sums (over the even and over the odd tiles) meet
    float mine = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
    float* part = reinterpret_cast<float*>(c.extra);
    workers_sync();   // every warp is done with its per-column data: the space is free
    if (grp == 1) part[row] = mine;
    workers_sync();
    if (grp == 0) mine += part[row];
    if (grp == 0 && j < l) {
      int lo2 = r_start, hi2 = n_probe;   // rows with p_r >= j
      while (lo2 < hi2) {
        const int mid = (lo2 + hi2) >> 1;
        if (P[mid] < j) lo2 = mid + 1; else hi2 = mid;
      }
      float* scores = reinterpret_cast<float*>(cache + unit * unit_stride + off_scores);
      scores[j] = __fdiv_rn(mine, (float)(G * (n_probe - lo2)));
    }
  }
  tc_teardown(c);
}

}  // namespace

namespace {

// Dense copy of the probe rows, Qp[b][h][r] = Q[b][h][P[r]]: pass 2 streams its tiles from it
// with bulk copies.  8 rows per CTA, 16 threads x 16 bytes per row.
template <typename T>
__global__ void k_gather_probe_rows(const T* __restrict__ Q, const int32_t* __restrict__ P, int n_probe,
                                    int h_q, long long qsb, long long qsh, long long qsl,
                                    T* __restrict__ Qp) {
  const int r = blockIdx.x * 8 + (threadIdx.x >> 4), ch = threadIdx.x & 15;
  if (r >= n_probe) return;
  const int b = blockIdx.y / h_q, h = blockIdx.y % h_q;
  const uint4 v = *(reinterpret_cast<const uint4*>(Q + b * qsb + h * qsh + (long long)P[r] * qsl) + ch);
  *(reinterpret_cast<uint4*>(Qp + ((long long)blockIdx.y * n_probe + r) * ZC_D) + ch) = v;
}

}  // namespace

int zc_launch_probe_scores(zc_cache* c, const void* Q, const void* K, int l, const int64_t* qs,
                           const int64_t* ks, const int32_t* P_dev, int n_probe, float* lse_ws,
                           void* qp_ws, size_t qp_bytes, const float* lse_rows, cudaStream_t st) {
  const zc_config& cfg = c->cfg;
  const int G = c->lay.G;
  const int Gt = (G % 4 == 0) ? 4 : ((G % 2 == 0) ? 2 : 1);
  const int rph = kM / Gt;
  dim3 g1(zc_ceil_div(n_probe, rph), cfg.batch * (cfg.n_q_heads / Gt));
  dim3 g2(zc_ceil_div(l, kM), c->lay.units);
  CUtensorMap kmap;
  memset(&kmap, 0, sizeof(kmap));
  const int use_tma = make_key_map(&kmap, K, cfg.dtype, l, cfg.n_kv_heads, cfg.batch, ks) ? 1 : 0;
  // the gathered copy of the probe rows, when the workspace has room for it
  CUtensorMap qmap;
  memset(&qmap, 0, sizeof(qmap));
  const size_t qp_need = (size_t)cfg.batch * cfg.n_q_heads * (size_t)n_probe * ZC_D * 2;
  int use_qp = 0;
  if (use_tma && qp_ws && qp_bytes >= qp_need) {
    const int64_t qps[3] = {(int64_t)cfg.n_q_heads * n_probe * ZC_D, (int64_t)n_probe * ZC_D, ZC_D};
    use_qp = make_key_map(&qmap, qp_ws, cfg.dtype, n_probe, cfg.n_q_heads, cfg.batch, qps) ? 1 : 0;
  }
  cudaError_t e;
#define ZC_GO(T)                                                                                       \
  do {                                                                                                 \
    e = cudaFuncSetAttribute(k_probe_lse<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem);  \
    if (e != cudaSuccess) return e;                                                                    \
    e = cudaFuncSetAttribute(k_probe_colsum<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmem); \
    if (e != cudaSuccess) return e;                                                                    \
    if (use_qp)                                                                                        \
      k_gather_probe_rows<T><<<dim3(zc_ceil_div(n_probe, 8), cfg.batch * cfg.n_q_heads), 128, 0, st>>>( \
          (const T*)Q, P_dev, n_probe, cfg.n_q_heads, qs[0], qs[1], qs[2], (T*)qp_ws);                 \
    if (!lse_rows)                                                                                     \
      k_probe_lse<T><<<g1, kThreads, kTcSmem, st>>>((const T*)Q, (const T*)K, P_dev, n_probe, l,    \
                                                       cfg.n_q_heads, G, Gt, qs[0], qs[1], qs[2],      \
                                                       ks[0], ks[1], ks[2], lse_ws, kmap, use_tma);    \
    k_probe_colsum<T><<<g2, kThreads, kTcSmem, st>>>((const T*)Q, (const T*)K, P_dev, n_probe, l,   \
                                                        cfg.n_q_heads, cfg.n_kv_heads, G, qs[0], qs[1], \
                                                        qs[2], ks[0], ks[1], ks[2], lse_ws, c->base,   \
                                                        c->lay.unit_stride, c->lay.off_scores, kmap,   \
                                                        use_tma, qmap, use_qp);                        \
  } while (0)
  if (lse_rows) {
    const int rc = zc_launch_gather_probe_lse(c, lse_rows, P_dev, n_probe, l, lse_ws, st);
    if (rc != (int)cudaSuccess) return rc;
  }
  if (cfg.dtype == ZC_F16) ZC_GO(__half); else ZC_GO(__nv_bfloat16);
#undef ZC_GO
  c->launches += (lse_rows ? 1 : 2) + use_qp;
  return cudaGetLastError();
}

int zc_probe_error_code(int* out) {
  return (int)cudaMemcpyFromSymbol(out, g_zc_tc_error, sizeof(int));
}
