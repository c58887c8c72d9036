// Measurement aid of bench.py, built into a small library of its own (not part of the BlockFFN
// library, no counterpart in the paper): a read-only pass over a buffer, so that the benchmark
// can state what a plain read reaches on the device it runs on -- streaming over gigabytes, and
// in one launch the size of a call's active weights.
//
//   int benchprobe_read(const void* src, size_t bytes, int chained, void* stream)
//
// Enqueues one kernel that reads `bytes` bytes at `src` (device memory, 16-byte aligned, a
// multiple of 16 bytes) once, with 128-bit loads from four CTAs per SM, and discards them.
// chained != 0 launches it with programmatic dependent launch (it starts under the launch before
// it and waits for that launch before it ends). Returns 0, 1 for a bad argument, 4 for a CUDA
// error. Allocates nothing.
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace {

constexpr int kThreads = 256;
constexpr int kCtasPerSm = 4;   // 128-bit loads need this many resident CTAs to fill the memory system

__device__ unsigned int g_probe_sink;

__global__ void __launch_bounds__(kThreads) read_probe_kernel(const uint4* __restrict__ src,
                                                             size_t n16) {
  // The kernel may have been started under the one before it; it touches nothing that kernel
  // writes, so it needs no wait, but like every kernel of the library it waits before it ends.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const size_t stride = (size_t)gridDim.x * kThreads;
  unsigned int acc = 0;
  size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x;
  for (; i + 3 * stride < n16; i += 4 * stride) {   // four independent loads in flight
    const uint4 a = __ldcs(src + i), b = __ldcs(src + i + stride);
    const uint4 c = __ldcs(src + i + 2 * stride), e = __ldcs(src + i + 3 * stride);
    acc ^= a.x ^ a.y ^ a.z ^ a.w ^ b.x ^ b.y ^ b.z ^ b.w;
    acc ^= c.x ^ c.y ^ c.z ^ c.w ^ e.x ^ e.y ^ e.z ^ e.w;
  }
  for (; i < n16; i += stride) {
    const uint4 a = __ldcs(src + i);
    acc ^= a.x ^ a.y ^ a.z ^ a.w;
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (acc == 0x9e3779b9u) g_probe_sink = acc;   // keeps the loads alive; practically never taken
}

}  // namespace

extern "C" __attribute__((visibility("default"))) int benchprobe_read(const void* src, size_t bytes,
                                                                      int chained, void* stream) {
  if (!src || bytes == 0 || (bytes & 15u) || (reinterpret_cast<uintptr_t>(src) & 15u)) return 1;
  int device = 0, sms = 0;
  if (cudaGetDevice(&device) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
    return 4;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3(sms * kCtasPerSm);
  lc.blockDim = dim3(kThreads);
  lc.stream = static_cast<cudaStream_t>(stream);
  lc.attrs = attr;
  lc.numAttrs = chained ? 1 : 0;
  const cudaError_t e = cudaLaunchKernelEx(&lc, read_probe_kernel,
                                           static_cast<const uint4*>(src), bytes >> 4);
  return e == cudaSuccess ? 0 : 4;
}
