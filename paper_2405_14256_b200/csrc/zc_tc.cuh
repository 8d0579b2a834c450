// tcgen05 / TMEM / TMA building blocks shared by the probe-score kernels and the prefill
// attention kernel: 128-row operand tiles in the 128-byte swizzle, shared-memory matrix and
// instruction descriptors, mbarrier waits with a bound, tensor-memory loads, tensor-map copies.
#pragma once
#include <cuda.h>
#include <cstring>
#include <type_traits>
#include "zc_internal.h"
#include "zc_mma.cuh"

// Set when a bounded wait ran out (one copy per translation unit that includes this header).
static __device__ int g_zc_tc_error = 0;

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
    if (spins > kSpinLimit) { atomicExch(&g_zc_tc_error, 1); break; }
    // once a wait has run out somewhere the results are void: do not add to the delay
    if ((spins & 1023) == 1023 && *reinterpret_cast<volatile int*>(&g_zc_tc_error)) break;
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

__device__ __forceinline__ void bar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];\n" ::"r"(zc_smem_u32(bar)) : "memory");
}


// A worker has issued its copies of a tile: the barrier gets this thread's arrival when they land.
__device__ __forceinline__ void copies_arrive(uint64_t* bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];\n" ::"r"(zc_smem_u32(bar)) : "memory");
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
