// Test support only (not part of the library): a producer kernel that behaves like a kernel of
// another library compiled for programmatic dependent launch.  It lets the next kernel of the
// stream start at once (griddepcontrol.launch_dependents at entry), keeps itself busy for a
// fixed number of clock cycles, and only then writes its output -- so a consumer that does not
// wait for its predecessor reads stale data.
#include <cuda_runtime.h>
#include <stdint.h>

#include "zc_quant.cuh"   // the library's device functions under test (zc_div_by)

namespace {
__global__ void k_late_copy(uint4* dst, const uint4* src, int n16, long long spin_cycles) {
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  const long long t0 = clock64();
  while (clock64() - t0 < spin_cycles) {   // bounded by time alone: nothing external is waited for
  }
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += gridDim.x * blockDim.x) dst[i] = src[i];
}
}  // namespace

// dst, src [device], 16-byte aligned, bytes a multiple of 16.  Returns the cudaError_t of the launch.
extern "C" int zct_late_copy(void* dst, const void* src, size_t bytes, long long spin_cycles, void* stream) {
  if (spin_cycles > (1ll << 31)) spin_cycles = 1ll << 31;   // about a second at most
  k_late_copy<<<8, 128, 0, (cudaStream_t)stream>>>((uint4*)dst, (const uint4*)src, (int)(bytes / 16), spin_cycles);
  return (int)cudaGetLastError();
}

// The quantiser's division by a kept reciprocal against the hardware's IEEE division:
// n pseudo-random pairs (a, b) per call, magnitudes spread over the ranges the quantiser admits
// (2^-40 .. 2^40, either sign for a), plus pairs whose quotient lies next to a rounding
// boundary (a = b * k for small odd k, nudged by an ulp).  Counts the pairs whose bits differ.
namespace {
__device__ __forceinline__ uint64_t mix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}
__global__ void k_div_check(long long n, uint64_t seed, int exp_span, unsigned long long* mismatches,
                            float* first_bad) {
  unsigned long long bad = 0;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const uint64_t r = mix64(seed + (uint64_t)i), r2 = mix64(r);
    // b: random significand, exponent in [-exp_span, exp_span]
    const int eb = (int)(r2 % (uint64_t)(2 * exp_span + 1)) - exp_span;
    const float b = __uint_as_float(((uint32_t)(127 + eb) << 23) | (uint32_t)(r & 0x7FFFFFu));
    float a;
    if ((r >> 62) == 0) {   // a quarter of the pairs: quotients at and beside small integers and halves
      const float k = (float)((r >> 40) & 0x3FF) * 0.5f + 0.5f;
      a = __fmul_rn(b, k);
      const int nudge = (int)((r >> 52) & 3) - 1;
      a = __uint_as_float(__float_as_uint(a) + nudge);
    } else {
      const int ea = (int)((r2 >> 32) % (uint64_t)(2 * exp_span + 1)) - exp_span;
      a = __uint_as_float(((uint32_t)(r2 >> 63) << 31) | ((uint32_t)(127 + ea) << 23) | (uint32_t)((r >> 23) & 0x7FFFFFu));
    }
    if (!zc_mid(a) || !zc_mid(b)) continue;
    const float want = __fdiv_rn(a, b), got = zc_div_by(a, b, __frcp_rn(b));
    if (__float_as_uint(want) != __float_as_uint(got)) {
      if (bad == 0 && atomicAdd(mismatches, 0ull) == 0) { first_bad[0] = a; first_bad[1] = b; }
      ++bad;
    }
  }
  if (bad) atomicAdd(mismatches, bad);
}
}  // namespace

// mismatches [device, one 64-bit counter, zeroed by the caller], first_bad [device, 2 floats].
extern "C" int zct_div_check(long long n, unsigned long long seed, int exp_span, void* mismatches, void* first_bad,
                             void* stream) {
  if (exp_span < 0 || exp_span > 40) return (int)cudaErrorInvalidValue;
  k_div_check<<<1184, 256, 0, (cudaStream_t)stream>>>(n, seed, exp_span, (unsigned long long*)mismatches,
                                                        (float*)first_bad);
  return (int)cudaGetLastError();
}
