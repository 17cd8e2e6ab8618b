// Measurement aid for benchmarks: a kernel that does nothing but special-function operations, so
// that the rate of that pipe (the one exp2 and the square roots of the statistics run on) can be
// measured on the GPU at hand instead of being taken from a data sheet.
#include "kvs_internal.h"

namespace {

// Eight independent chains per thread, each alternating ex2.approx and sqrt.approx: 16
// special-function operations per loop trip and nothing else of weight (one add per chain keeps
// the values in range).
__global__ void __launch_bounds__(1024)
sfu_probe_kernel(int iters, float* sink) {
  float x[8];
#pragma unroll
  for (int u = 0; u < 8; ++u) x[u] = 0.25f + 0.01f * (float)((threadIdx.x + u) & 31);
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      float e, r;
      asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(x[u]));
      asm volatile("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(e));
      x[u] = r - 0.75f;
    }
  }
  float s = 0.f;
#pragma unroll
  for (int u = 0; u < 8; ++u) s += x[u];
  if (s == 12345.678f) sink[0] = s;          // keeps the loop alive; practically never true
}

}  // namespace

cudaError_t kvs_launch_sfu_probe(int blocks, int iters, float* sink, cudaStream_t st) {
  sfu_probe_kernel<<<blocks, 1024, 0, st>>>(iters, sink);
  return cudaGetLastError();
}
