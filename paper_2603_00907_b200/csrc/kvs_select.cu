// Exact selection of the R candidate pairs with the smallest (score, pair index) and the
// per-tile exclusive counts that the compaction needs.
//
// One CTA of 1024 threads per (sequence, KV head).  Scores are non-negative floats, so
// their bit patterns order like unsigned integers: a four-pass, 8-bit radix select finds
// the bit pattern of the R-th smallest score and how many pairs tied with it are still
// needed; ties are taken in index order.  A second sweep writes the mask and, for every
// compaction tile of 32 pairs, the number of merged pairs that precede it.
#include "kvs_internal.h"

namespace {

__global__ void __launch_bounds__(1024)
select_pairs_kernel(const SelectArgs a, const RoundTable tab) {
  const int seq = blockIdx.y;
  const SeqRound sr = tab.s[seq];
  const int n = sr.n;
  if (n <= 0) return;
  const int unit = sr.b * a.Hkv + blockIdx.x;
  const int P = sr.P, R = sr.R;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t* key = reinterpret_cast<const uint32_t*>(a.score) + (size_t)unit * a.pair_stride;
  uint8_t* mask = a.mask + (size_t)unit * a.pair_stride;

  __shared__ uint32_t hist[256];
  __shared__ uint32_t s_digit, s_k;
  __shared__ uint32_t s_warp_tie[32], s_warp_sel[32];
  __shared__ uint32_t s_run_tie, s_run_sel;

  uint32_t prefix = 0, pmask = 0, k = (uint32_t)R;
  if (!a.from_mask) {
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      if (tid < 256) hist[tid] = 0;
      __syncthreads();
      // four loads in flight per thread: the sweep is a chain of L2 latencies otherwise
      for (int p0 = 0; p0 < P; p0 += 4 * 1024) {
        uint32_t v4[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int p = p0 + u * 1024 + tid;
          v4[u] = (p < P) ? __ldg(key + p) : 0u;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int p = p0 + u * 1024 + tid;
          const uint32_t v = v4[u];
          const bool in = (p < P) && (v & pmask) == prefix;
          const uint32_t d = (v >> shift) & 255u;
          const uint32_t act = __ballot_sync(0xffffffffu, in);
          if (in) {
            const uint32_t same = __match_any_sync(act, d);
            if (lane == (__ffs(same) - 1)) atomicAdd(&hist[d], (uint32_t)__popc(same));
          }
        }
      }
      __syncthreads();
      if (warp == 0) {
        // lane owns bins [8 lane, 8 lane + 8)
        uint32_t loc[8], sum = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) { loc[i] = hist[8 * lane + i]; sum += loc[i]; }
        uint32_t inc = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += t;
        }
        uint32_t excl = inc - sum;
        const bool mine = excl < k && k <= inc;      // the k-th element falls in my bins
        if (mine) {
          uint32_t cum = excl;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            if (cum < k && k <= cum + loc[i]) { s_digit = 8 * lane + i; s_k = k - cum; }
            cum += loc[i];
          }
        }
      }
      __syncthreads();
      prefix |= s_digit << shift;
      pmask |= 255u << shift;
      k = s_k;
      __syncthreads();
    }
  }
  // prefix = bit pattern of the cutoff score, k = ties (in index order) still to take
  if (tid == 0) { s_run_tie = 0; s_run_sel = 0; }
  __syncthreads();
  const int ntiles = (n - tab.off + KVS_CTILE - 1) / KVS_CTILE;
  int32_t* tp = a.tile_prefix + (size_t)unit * a.tile_stride;
  const int sweep = ((ntiles * 32 + 1023) / 1024) * 1024;
  // (the value of the chunk after this one is requested before this chunk's barriers)
  uint32_t v_next = 0;
  if (tid < P) v_next = a.from_mask ? (uint32_t)mask[tid] : __ldg(key + tid);
  for (int p0 = 0; p0 < sweep; p0 += 1024) {
    const int p = p0 + tid;
    bool tie = false, less = false, sel = false;
    const uint32_t v = v_next;
    if (p + 1024 < P) v_next = a.from_mask ? (uint32_t)mask[p + 1024] : __ldg(key + p + 1024);
    if (p < P) {
      if (a.from_mask) {
        sel = v != 0;
      } else {
        less = v < prefix;
        tie = v == prefix;
      }
    }
    const uint32_t run_tie = s_run_tie, run_sel = s_run_sel;
    if (!a.from_mask) {
      const uint32_t tb = __ballot_sync(0xffffffffu, tie);
      if (lane == 0) s_warp_tie[warp] = __popc(tb);
      __syncthreads();
      uint32_t wpre = 0;
      for (int wq = 0; wq < warp; ++wq) wpre += s_warp_tie[wq];
      const uint32_t rank = run_tie + wpre + __popc(tb & ((1u << lane) - 1u));
      sel = less || (tie && rank < k);
      if (p < P) mask[p] = sel ? 1 : 0;
    }
    const uint32_t sb = __ballot_sync(0xffffffffu, sel);
    if (lane == 0) s_warp_sel[warp] = __popc(sb);
    __syncthreads();
    uint32_t spre = 0;
    for (int wq = 0; wq < warp; ++wq) spre += s_warp_sel[wq];
    const int tile = (p0 >> 5) + warp;
    if (lane == 0 && tile < ntiles) tp[tile] = (int32_t)(run_sel + spre);
    __syncthreads();
    if (tid == 1023) {
      // last warp: totals of this chunk
      uint32_t tt = 0;
      if (!a.from_mask) for (int wq = 0; wq < 32; ++wq) tt += s_warp_tie[wq];
      s_run_tie = run_tie + tt;
      s_run_sel = run_sel + spre + s_warp_sel[31];
    }
    __syncthreads();
  }
}

}  // namespace

cudaError_t kvs_launch_select(const SelectArgs& a, const RoundTable& t, cudaStream_t st) {
  dim3 grid(a.Hkv, t.nseq);
  select_pairs_kernel<<<grid, 1024, 0, st>>>(a, t);
  return cudaGetLastError();
}
