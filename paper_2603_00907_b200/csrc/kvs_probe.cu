// Measurement aid for benchmarks: a kernel that does nothing but special-function operations, so
// that the rate of that pipe (the one exp2 and the square roots of the statistics run on) can be
// measured on the GPU at hand instead of being taken from a data sheet.
#include "kvs_internal.h"
#include "kvs_sm100.cuh"

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

// Second aid: what a tensor-core product costs when both operands come from shared memory.  One
// warp per CTA runs `products` back-to-back tcgen05 products D[128 x N] += A[128 x 16] B[N x 16]^T
// (bf16, zero-filled operands in the 128-byte swizzled layout the library's kernels use, four
// K slices in turn, two accumulators in turn) and reports the cycles from the first issue to the
// completion of the last.  With kReuse, consecutive products come in twos on the same A slice with
// different B slices: the first keeps A in the tensor core's collector buffer, the second takes
// it from there instead of reading shared memory again.  One elected lane issues, with
// precomputed descriptors and compile-time shapes, so that the issue itself costs as little as
// it can and the figure is the hardware's.
constexpr int kProbeA = 16384, kProbeB = 32768;    // a [128 x 64] and a [256 x 64] bf16 tile

template <int kN, bool kReuse>
__global__ void __launch_bounds__(128, 1)
mma_probe_kernel(int products, uint32_t limit_us, long long* cycles) {
  using namespace sm100;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  __shared__ uint64_t bar;
  __shared__ uint32_t tmem_base;
  __shared__ int ctl[2];
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0);
  for (int i = threadIdx.x; i < (kProbeA + kProbeB) / 16; i += 128) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
  if (threadIdx.x == 0) { mbar_init(&bar, 1); ctl[0] = 0; ctl[1] = (int)limit_us; mbar_fence_init(); }
  fence_proxy_async();
  if (warp == 0) tmem_alloc(&tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = __shfl_sync(0xffffffffu, tmem_base, 0);
  constexpr uint32_t idesc = idesc_bf16(128, kN);     // (shape and accumulator addresses are compile-time: every
                                                      //  instruction between two products shows in the figure)
  uint64_t ad[4], bd[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    ad[i] = smem_desc_sw128(smem_u32(smem) + 32 * i, 16, 1024);
    bd[i] = smem_desc_sw128(smem_u32(smem + kProbeA) + 32 * i, 16, 1024);
  }
  if (warp == 0 && elect_one()) {
    for (int i = 0; i < 8; ++i) umma_acc<0>(tmem, ad[0], bd[0], idesc);     // warm-up
    tc_commit(&bar);
    bool ok = mbar_wait(&bar, 0, ctl);
    const long long t0 = clock64();
    if (ok) {
      for (int i = 0; i < products; i += 8) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if constexpr (kReuse) {
            umma_acc<1>(tmem, ad[u], bd[u], idesc);
            umma_acc<2>(tmem + (uint32_t)kN, ad[u], bd[(u + 1) & 3], idesc);
          } else {
            umma_acc<0>(tmem, ad[u], bd[u], idesc);
            umma_acc<0>(tmem + (uint32_t)kN, ad[(u + 1) & 3], bd[(u + 1) & 3], idesc);
          }
        }
      }
      tc_commit(&bar);
      ok = mbar_wait(&bar, 1, ctl);
    }
    const long long t1 = clock64();
    cycles[blockIdx.x] = ok ? (t1 - t0) : -1;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

}  // namespace

template <int kN>
static cudaError_t launch_mma_probe_n(int blocks, int reuse_a, int products, uint32_t limit_us, long long* cycles,
                                      cudaStream_t st) {
  constexpr int kSmem = kProbeA + kProbeB + 1024;
  static KvsPerDeviceOnce configured;
  cudaError_t ce = configured.run([] {
    cudaError_t e = cudaFuncSetAttribute(mma_probe_kernel<kN, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(mma_probe_kernel<kN, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem);
  });
  if (ce != cudaSuccess) return ce;
  if (reuse_a) mma_probe_kernel<kN, true><<<blocks, 128, kSmem, st>>>(products, limit_us, cycles);
  else mma_probe_kernel<kN, false><<<blocks, 128, kSmem, st>>>(products, limit_us, cycles);
  return cudaGetLastError();
}

cudaError_t kvs_launch_mma_probe(int blocks, int n_cols, int reuse_a, int products, uint32_t limit_us,
                                 long long* cycles, cudaStream_t st) {
  switch (n_cols) {
    case 16: return launch_mma_probe_n<16>(blocks, reuse_a, products, limit_us, cycles, st);
    case 32: return launch_mma_probe_n<32>(blocks, reuse_a, products, limit_us, cycles, st);
    case 64: return launch_mma_probe_n<64>(blocks, reuse_a, products, limit_us, cycles, st);
    case 128: return launch_mma_probe_n<128>(blocks, reuse_a, products, limit_us, cycles, st);
    case 256: return launch_mma_probe_n<256>(blocks, reuse_a, products, limit_us, cycles, st);
  }
  return cudaErrorInvalidValue;
}

cudaError_t kvs_launch_sfu_probe(int blocks, int iters, float* sink, cudaStream_t st) {
  sfu_probe_kernel<<<blocks, 1024, 0, st>>>(iters, sink);
  return cudaGetLastError();
}
