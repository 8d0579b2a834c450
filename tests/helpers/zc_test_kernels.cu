// Test support only (not part of the library): a producer kernel that behaves like a kernel of
// another library compiled for programmatic dependent launch.  It lets the next kernel of the
// stream start at once (griddepcontrol.launch_dependents at entry), keeps itself busy for a
// fixed number of clock cycles, and only then writes its output -- so a consumer that does not
// wait for its predecessor reads stale data.
#include <cuda_runtime.h>
#include <stdint.h>

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
