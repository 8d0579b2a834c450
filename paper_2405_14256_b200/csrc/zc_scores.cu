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
#include <cuda.h>
#include <cstring>
#include <type_traits>
#include "zc_internal.h"
#include "zc_layout.cuh"
#include "zc_mma.cuh"

__device__ int g_zc_probe_error = 0;

namespace {

constexpr int kM = 128;                          // rows of a tile (TMEM lanes)
constexpr int kTile = kM * ZC_D * 2;             // 32 KB: [2][128][128 B]
constexpr int kKBlock = kM * 128;                // bytes of one k-block of a tile
constexpr float kLog2e = 1.4426950408889634f;
constexpr int kSpinLimit = 1 << 22;
constexpr uint32_t kTmemCols = 256;              // two 128-column accumulators

// 16-byte chunk `chunk` (0..15) of row `row` inside a tile
__device__ __forceinline__ char* tile_chunk(char* tile, int row, int chunk) {
  return tile + (chunk >> 3) * kKBlock + row * 128 + (((chunk & 7) ^ (row & 7)) << 4);
}
__device__ __forceinline__ void load_row(char* tile, int row, int chunk, const char* src) {
  if (src) zc_cp_async16(tile_chunk(tile, row, chunk), src + chunk * 16);
  else {
    *reinterpret_cast<uint4*>(tile_chunk(tile, row, chunk)) = make_uint4(0, 0, 0, 0);
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");   // a plain store the tensor core will read
  }
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 bytes
// apart; `addr` = shared address of the tile + k-block * kKBlock + (k16 step within it) * 32.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor: fp32 accumulate, A and B of type T (0 = f16, 1 = bf16), both K-major,
// N = 128, M = 128.
template <typename T> __device__ __forceinline__ uint32_t instr_desc() {
  const uint32_t fmt = std::is_same<T, __nv_bfloat16>::value ? 1u : 0u;
  return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

__device__ __forceinline__ void mma_tile(uint32_t tmem_d, uint32_t a_addr, uint32_t b_addr, uint32_t idesc) {
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
    const uint32_t off = (ks >> 2) * kKBlock + (ks & 3) * 32;
    const uint64_t da = smem_desc(a_addr + off), db = smem_desc(b_addr + off);
    const uint32_t acc = ks > 0 ? 1u : 0u;
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n}\n" ::"r"(tmem_d),
        "l"(da), "l"(db), "r"(idesc), "r"(acc), "r"(0u)
        : "memory");
  }
}
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(
                   zc_smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void bar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(zc_smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ bool bar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(zc_smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void bar_wait(uint64_t* bar, uint32_t parity) {
  for (int spins = 0; !bar_try(bar, parity); ++spins) {
    if (spins > kSpinLimit) { atomicExch(&g_zc_probe_error, 1); break; }
    // once a wait has run out somewhere the results are void: do not add to the delay
    if ((spins & 1023) == 1023 && *reinterpret_cast<volatile int*>(&g_zc_probe_error)) break;
  }
}
__device__ __forceinline__ void tmem_ld32_nowait(float* v, uint32_t taddr) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
      "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
// one thread's whole row of a 128-column accumulator: four loads in flight, one wait
__device__ __forceinline__ void tmem_ld128(float (&v)[128], uint32_t taddr) {
#pragma unroll
  for (int q4 = 0; q4 < 4; ++q4) tmem_ld32_nowait(v + 32 * q4, taddr + 32 * q4);
  asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void async_proxy_fence() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }

// What both kernels share: shared memory carved at a 1024-byte boundary, TMEM, barriers.
// 160 threads: lane 0 of warp 0 issues the MMAs, warps 1..4 are the row workers (they also
// copy the tiles into shared memory, 16 bytes per thread and row); worker warp w may touch
// TMEM lanes 32 (w mod 4) .. +31, so together they cover the 128 rows of a tile.
//   a_full        the A tile has landed
//   b_full[b]     B buffer b has been filled: by all 128 workers' copies
//                 (cp.async.mbarrier.arrive) or by the bulk copies (complete_tx)
//   mma_done[b]   the MMA into accumulator b has completed (tcgen05.commit): the workers may
//                 read it, and the B buffer it read may be refilled
//   tmem_free[b]  the four worker warps have read accumulator b: the next MMA may overwrite it
constexpr int kThreads = 160;
struct TcCtx {
  char* As;
  char* Bs;          // two tiles
  uint64_t* mma_done;
  uint64_t* tmem_free;
  uint64_t* b_full;
  uint64_t* a_full;
  uint32_t* tmem_slot;
  char* extra;       // pass 2: per worker warp, probe positions and lse of kSide B tiles
  uint32_t a_addr, b_addr, tmem;
};
constexpr int kSide = 3;           // per-column data of pass 2: three tiles per worker warp (see k_probe_colsum)
constexpr int kTcSmem = 3 * kTile + 1024 /* alignment */ + 128 /* barriers, tmem slot */ + 4 * kSide * kM * 8;

__device__ __forceinline__ void bar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];\n" ::"r"(zc_smem_u32(bar)) : "memory");
}

__device__ __forceinline__ TcCtx tc_setup(char* raw, int a_count, int b_count) {
  TcCtx c;
  const uint32_t raw_u = zc_smem_u32(raw);
  const uint32_t base_u = (raw_u + 1023u) & ~1023u;
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

// One 128-row tile of consecutive rows (rows j0 .. j0 + 127 of tensor[b][h]: keys, or the
// gathered probe rows) by two bulk tensor copies (one per k-block); rows past the end of the
// tensor arrive as zeros.
__device__ __forceinline__ void tma_key_tile(const CUtensorMap* map, uint32_t dst, uint64_t* bar, int j0,
                                             int kv, int b) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(zc_smem_u32(bar)), "r"(kTile)
               : "memory");
#pragma unroll
  for (int kb = 0; kb < 2; ++kb)
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], "
        "[%6];\n" ::"r"(dst + kb * kKBlock),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(kb * 64), "r"(j0), "r"(kv), "r"(b), "r"(zc_smem_u32(bar))
        : "memory");
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
// A worker has issued its copies of a tile: the barrier gets this thread's arrival when they land.
__device__ __forceinline__ void copies_arrive(uint64_t* bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];\n" ::"r"(zc_smem_u32(bar)) : "memory");
}

// Worker: waits for tile cb's accumulator and fetches this thread's row of it.
__device__ __forceinline__ void worker_fetch(const TcCtx& c, int cb, int quarter, float (&v)[kM]) {
  const int buf = cb & 1;
  bar_wait(&c.mma_done[buf], (uint32_t)(cb >> 1) & 1u);
  tc_fence_after();
  tmem_ld128(v, c.tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * kM);
  tc_fence_before();
  __syncwarp();
  if ((threadIdx.x & 31) == 0) bar_arrive(&c.tmem_free[buf]);
}

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
  extern __shared__ char smem_raw[];
  // A (gathered probe rows): the 128 workers' copies; B (key tiles): bulk copies, or the workers
  TcCtx c = tc_setup(smem_raw, kM, use_tma ? 1 : kM);
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
    const int quarter = warp & 3, row = quarter * 32 + lane;
    const int wt = tid - 32, row_ld = wt >> 4, chunk = wt & 15;   // 8 rows per pass of the 128 workers
    auto load_b = [&](int cb) {   // tile cb's keys into B buffer cb & 1
#pragma unroll 4
      for (int i = 0; i < 16; ++i) {
        const int rw = row_ld + 8 * i, j = cb * kM + rw;
        load_row(c.Bs + (cb & 1) * kTile, rw, chunk, j < l ? Kb + (long long)j * ksl * 2 : nullptr);
      }
      copies_arrive(&c.b_full[cb & 1]);
    };
    // A: the block's probe rows of the Gt heads (it lands with tile 0)
#pragma unroll 4
    for (int i = 0; i < 16; ++i) {
      const int rw = row_ld + 8 * i, hl = rw / rph, r = r0 + rw % rph;
      const char* src = nullptr;
      if (r < n_probe) src = reinterpret_cast<const char*>(Q + b * qsb + (h0 + hl) * qsh) + (long long)P[r] * qsl * 2;
      load_row(c.As, rw, chunk, src);
    }
    copies_arrive(c.a_full);
    if (!use_tma) {
      load_b(0);
      if (n_cb > 1) load_b(1);
    }
    const int my_r = r0 + row % rph;
    const int my_p = my_r < n_probe ? P[my_r] : -1;
    const float scale = kLog2e * rsqrtf((float)ZC_D);
    float m_run = -INFINITY, s_run = 0.f;
    for (int cb = 0; cb < n_cb; ++cb) {
      float v[kM];
      worker_fetch(c, cb, quarter, v);
      if (!use_tma && cb + 2 < n_cb) load_b(cb + 2);   // its buffer was read by the MMA that has just completed
      const int j_base = cb * kM;
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
      if (j_base + kM - 1 <= my_p) {
#pragma unroll
        for (int e = 0; e < kM; ++e) mx4[e & 3] = fmaxf(mx4[e & 3], v[e]);
      } else {
#pragma unroll
        for (int e = 0; e < kM; ++e) {
          if (j_base + e > my_p) v[e] = -INFINITY;
          mx4[e & 3] = fmaxf(mx4[e & 3], v[e]);
        }
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
      const float mn = fmaxf(m_run, mx * scale);
      if (mn != -INFINITY) {
        float add[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int e = 0; e < kM; ++e) add[e & 3] += zc_exp2(fmaf(v[e], scale, -mn));
        s_run = s_run * zc_exp2(m_run - mn) + ((add[0] + add[1]) + (add[2] + add[3]));
        m_run = mn;
      }
    }
    if (my_r < n_probe) lse[((long long)b * h_q + h0 + row / rph) * n_probe + my_r] = m_run + log2f(s_run);
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
  extern __shared__ char smem_raw[];
  // A (the key block): one bulk copy, or the workers; B (probe rows): bulk copies from the
  // gathered copy of the probe rows when there is one (qmap), else the workers gather them
  TcCtx c = tc_setup(smem_raw, use_tma ? 1 : kM, use_qp ? 1 : kM);
  // Per-column data of a B tile (probe position and lse of each of its 128 rows): every worker
  // warp keeps its own copy, slot = tile mod 3, written two tiles ahead of its use, so the
  // warps need no barrier among themselves.
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
    const int quarter = warp & 3, row = quarter * 32 + lane;
    const int wt = tid - 32, row_ld = wt >> 4, chunk = wt & 15;   // 8 rows per pass of the 128 workers
    auto load_b = [&](int tile) {   // tile's probe rows into B buffer tile & 1, its per-column data into its slot
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
      const int slot = tile % kSide;
#pragma unroll
      for (int k = 0; k < kM / 32; ++k) {
        const int i = lane + 32 * k, r = r_start + rb * kM + i;
        Pp[slot * kM + i] = r < n_probe ? P[r] : -1;
        Ll[slot * kM + i] = r < n_probe ? lse[((long long)b * h_q + kv * G + gq) * n_probe + r] : INFINITY;
      }
    };
    if (!use_tma) {
#pragma unroll 4
      for (int i = 0; i < 16; ++i) {
        const int rw = row_ld + 8 * i, jj = j0 + rw;
        load_row(c.As, rw, chunk, jj < l ? Kb + (long long)jj * ksl * 2 : nullptr);
      }
      copies_arrive(c.a_full);
    }
    load_b(0);
    if (n_tiles > 1) load_b(1);
    __syncwarp();   // per-column data of tiles 0 and 1 is visible to the warp
    const int j = j0 + row;
    const float scale = kLog2e * rsqrtf((float)ZC_D);
    float sum4[4] = {0.f, 0.f, 0.f, 0.f};
    for (int tile = 0; tile < n_tiles; ++tile) {
      const int slot = tile % kSide;
      float v[kM];
      worker_fetch(c, tile, quarter, v);
      if (tile + 2 < n_tiles) load_b(tile + 2);   // its buffer was read by the MMA that has just completed
      __syncwarp();   // per-column data written here is read two iterations on
      const int* pp = Pp + slot * kM;
      const float* ll = Ll + slot * kM;
      if (j <= pp[0]) {   // probe rows ascend in position: every row of the tile sees column j
#pragma unroll
        for (int e = 0; e < kM; ++e) sum4[e & 3] += zc_exp2(fmaf(v[e], scale, -ll[e]));
      } else {
#pragma unroll
        for (int e = 0; e < kM; ++e) sum4[e & 3] += j <= pp[e] ? zc_exp2(fmaf(v[e], scale, -ll[e])) : 0.f;
      }
    }
    if (j < l) {
      int lo2 = r_start, hi2 = n_probe;   // rows with p_r >= j
      while (lo2 < hi2) {
        const int mid = (lo2 + hi2) >> 1;
        if (P[mid] < j) lo2 = mid + 1; else hi2 = mid;
      }
      float* scores = reinterpret_cast<float*>(cache + unit * unit_stride + off_scores);
      scores[j] = __fdiv_rn((sum4[0] + sum4[1]) + (sum4[2] + sum4[3]), (float)(G * (n_probe - lo2)));
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

// Tensor map of K as (d, l, h_kv, b) with boxes of 64 elements x 128 rows in the 128-byte
// swizzle; false when the driver entry point is missing or refuses the tensor (the kernels
// then copy the key tiles themselves).
bool make_key_map(CUtensorMap* map, const void* K, int dtype, int l, int n_kv, int batch, const int64_t* ks) {
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                               const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn encode = nullptr;
  static bool looked = false;
  if (!looked) {
    looked = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      encode = (EncodeFn)p;
    else
      cudaGetLastError();
  }
  if (!encode) return false;
  const cuuint64_t dims[4] = {(cuuint64_t)ZC_D, (cuuint64_t)l, (cuuint64_t)n_kv, (cuuint64_t)batch};
  // byte strides of dimensions 1..3; a dimension of extent 1 may come with any stride
  cuuint64_t strides[3] = {(cuuint64_t)ks[2] * 2, (cuuint64_t)ks[1] * 2, (cuuint64_t)ks[0] * 2};
  if (n_kv == 1 && strides[1] == 0) strides[1] = strides[0] * (cuuint64_t)l;
  if (batch == 1 && strides[2] == 0) strides[2] = strides[1] * (cuuint64_t)n_kv;
  for (int i = 0; i < 3; ++i)
    if (strides[i] == 0 || (strides[i] & 15) || strides[i] >= ((cuuint64_t)1 << 40)) return false;
  const cuuint32_t box[4] = {64, (cuuint32_t)kM, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult r = encode(map, dtype == ZC_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                            4, const_cast<void*>(K), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

}  // namespace

int zc_launch_probe_scores(zc_cache* c, const void* Q, const void* K, int l, const int64_t* qs,
                           const int64_t* ks, const int32_t* P_dev, int n_probe, float* lse_ws,
                           void* qp_ws, size_t qp_bytes, cudaStream_t st) {
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
    k_probe_lse<T><<<g1, kThreads, kTcSmem, st>>>((const T*)Q, (const T*)K, P_dev, n_probe, l,      \
                                                     cfg.n_q_heads, G, Gt, qs[0], qs[1], qs[2], ks[0], \
                                                     ks[1], ks[2], lse_ws, kmap, use_tma);             \
    k_probe_colsum<T><<<g2, kThreads, kTcSmem, st>>>((const T*)Q, (const T*)K, P_dev, n_probe, l,   \
                                                        cfg.n_q_heads, cfg.n_kv_heads, G, qs[0], qs[1], \
                                                        qs[2], ks[0], ks[1], ks[2], lse_ws, c->base,   \
                                                        c->lay.unit_stride, c->lay.off_scores, kmap,   \
                                                        use_tma, qmap, use_qp);                        \
  } while (0)
  if (cfg.dtype == ZC_F16) ZC_GO(__half); else ZC_GO(__nv_bfloat16);
#undef ZC_GO
  c->launches += 2 + use_qp;
  return cudaGetLastError();
}

int zc_probe_error_code(int* out) {
  return (int)cudaMemcpyFromSymbol(out, g_zc_probe_error, sizeof(int));
}
