// Adjacent-token cosine similarity of a bf16 tensor [B, H, Nmax, 128] along the token axis
// [Section 3.2, Eq. cosine_raw]:  cos(y_t, y_t+1) = <y_t, y_t+1> / (|y_t| |y_t+1|).
//
// A diagnostic for real caches (queries, keys and values of a layer): the paper's analysis rests
// on adjacent keys (and queries) being nearly parallel and adjacent values not.  The kernel is
// bandwidth bound: eight lanes share a row (two 16-byte loads per lane), every row is fetched once
// from HBM (its second use, as the successor of the row before, hits L1/L2), three shuffle steps
// reduce the three sums of a pair of rows.
#include "kvs_internal.h"

namespace {

struct SimArgs {
  const __nv_bfloat16* x;
  int64_t sb, sh, st;
  int32_t H, n_max;
  float* out;              // [B, H, n_max]; entry t is written for t < n - 1
};

__device__ __forceinline__ void dots8(uint4 a, uint4 b, float& aa, float& bb, float& ab) {
  const uint32_t av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float a0 = bf16lo(av[i]), a1 = bf16hi(av[i]), b0 = bf16lo(bv[i]), b1 = bf16hi(bv[i]);
    aa = fmaf(a0, a0, fmaf(a1, a1, aa));
    bb = fmaf(b0, b0, fmaf(b1, b1, bb));
    ab = fmaf(a0, b0, fmaf(a1, b1, ab));
  }
}

constexpr int kRowsPerCta = 256;     // 8 steps of 32 rows (256 threads, 8 lanes per row)

__global__ void __launch_bounds__(256)
adjacent_cosine_kernel(const SimArgs a, const RoundTable tab) {
  const SeqRound sr = tab.s[blockIdx.z];
  const int n = sr.n;
  const int h = blockIdx.y;
  const int row0 = blockIdx.x * kRowsPerCta;
  if (row0 >= n - 1) return;
  const int sub = threadIdx.x & 7;               // 16-channel part of the row
  const __nv_bfloat16* base = a.x + sr.b * a.sb + h * a.sh + sub * 16;
  float* out = a.out + ((size_t)sr.b * a.H + h) * a.n_max;
#pragma unroll 2
  for (int step = 0; step < kRowsPerCta / 32; ++step) {
    const int t = row0 + step * 32 + (threadIdx.x >> 3);
    const bool ok = t < n - 1;
    float aa = 0.f, bb = 0.f, ab = 0.f;
    if (ok) {
      const uint4* pa = reinterpret_cast<const uint4*>(base + (int64_t)t * a.st);
      const uint4* pb = reinterpret_cast<const uint4*>(base + (int64_t)(t + 1) * a.st);
      const uint4 a0 = pa[0], a1 = pa[1], b0 = pb[0], b1 = pb[1];
      dots8(a0, b0, aa, bb, ab);
      dots8(a1, b1, aa, bb, ab);
    }
#pragma unroll
    for (int k = 1; k < 8; k <<= 1) {
      aa += __shfl_xor_sync(0xffffffffu, aa, k);
      bb += __shfl_xor_sync(0xffffffffu, bb, k);
      ab += __shfl_xor_sync(0xffffffffu, ab, k);
    }
    if (ok && sub == 0) out[t] = ab / fmaxf(sqrtf(aa) * sqrtf(bb), 1e-30f);
  }
}

}  // namespace

cudaError_t kvs_launch_adjacent_cosine(const void* x, int64_t sb, int64_t sh, int64_t st, int H, int n_max,
                                       float* out, const RoundTable& t, cudaStream_t stream) {
  int nmax = 0;
  for (int i = 0; i < t.nseq; ++i) nmax = nmax > t.s[i].n ? nmax : t.s[i].n;
  if (nmax < 2) return cudaSuccess;
  SimArgs a;
  a.x = static_cast<const __nv_bfloat16*>(x);
  a.sb = sb; a.sh = sh; a.st = st; a.H = H; a.n_max = n_max; a.out = out;
  dim3 grid((nmax - 1 + kRowsPerCta - 1) / kRowsPerCta, H, t.nseq);
  adjacent_cosine_kernel<<<grid, 256, 0, stream>>>(a, t);
  return cudaGetLastError();
}
