// Appending a chunk of fresh tokens to the caches of a layer (the first half of a streaming step).
//
// Row r of the chunk of (sequence b, KV head h) goes to slot n_b + r of that unit, n_b being the
// slots in use; its count becomes 1 and its value sum is its value.  One warp per row: lanes
// 0-15 copy the 256 bytes of the key, lanes 16-31 those of the value.  Plain copies: the chunk
// is a few hundred rows per unit, far below what would need staging.
#include "kvs_internal.h"

namespace {

__global__ void __launch_bounds__(256)
append_chunk_kernel(const AppendArgs a, const RoundTable tab) {
  kvs_pdl_launch_dependents();
  kvs_pdl_wait();
  const int seq = blockIdx.z;
  const SeqRound sr = tab.s[seq];
  const int h = blockIdx.y;
  const int r = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= a.chunk_len) return;
  const int slot = sr.n + r;
  if (slot >= a.c.n_max) return;                        // (the host has checked this already)
  const size_t src = (((size_t)sr.b * a.c.Hkv + h) * a.chunk_len + r) * KVS_D;
  if (lane < 16) {
    const uint4* s = reinterpret_cast<const uint4*>(a.chunk_k + src);
    uint4* d = reinterpret_cast<uint4*>(a.c.K + (size_t)sr.b * a.c.ksb + (size_t)h * a.c.ksh + (size_t)slot * a.c.kst);
    d[lane] = s[lane];
  } else {
    const uint4* s = reinterpret_cast<const uint4*>(a.chunk_v + src);
    uint4* d = reinterpret_cast<uint4*>(a.c.V + (size_t)sr.b * a.c.vsb + (size_t)h * a.c.vsh + (size_t)slot * a.c.vst);
    d[lane - 16] = s[lane - 16];
  }
  if (lane == 0) a.c.counts[((size_t)sr.b * a.c.Hkv + h) * a.c.n_max + slot] = 1;
}

}  // namespace

cudaError_t kvs_launch_append(const AppendArgs& a, const RoundTable& t, cudaStream_t st) {
  dim3 grid((a.chunk_len + 7) / 8, a.c.Hkv, t.nseq);
  return kvs_launch_chained(append_chunk_kernel, grid, dim3(256), 0, st, a, t);
}
