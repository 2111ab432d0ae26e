// Test-only kernel: a producer that signals programmatic launch completion BEFORE it writes its output,
// the way library GEMMs with programmatic dependent launch enabled may do.  A consumer that does not
// wait for the producer's grid to finish would read the destination before it is written.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {
__global__ void early_trigger_copy_kernel(uint4* __restrict__ dst, const uint4* __restrict__ src, size_t n,
                                          unsigned delay_ns) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // a wait on the clock: it ends by itself after delay_ns
  unsigned long long t0, t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
  do {
    __nanosleep(500);
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  } while (t - t0 < (unsigned long long)delay_ns);
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = src[i];
}
}  // namespace

// Copies n16 16-byte vectors from src to dst on `stream`, delay_us microseconds after the kernel has
// allowed its dependents to launch (delay_us <= 1000).  Returns 0 on success.
extern "C" int st3_test_early_trigger_copy(void* dst, const void* src, size_t n16, int delay_us, void* stream) {
  if (!dst || !src || delay_us < 0 || delay_us > 1000) return 1;
  early_trigger_copy_kernel<<<8, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<uint4*>(dst), static_cast<const uint4*>(src), n16, (unsigned)delay_us * 1000u);
  return cudaGetLastError() == cudaSuccess ? 0 : 2;
}
