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
  kvs_pdl_launch_dependents();
  kvs_pdl_wait();
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
  __shared__ uint32_t s_cnt[128], s_pre[128];
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
  // prefix = bit pattern of the cutoff score, k = ties (in index order) still to take.
  // The sweep takes 4096 pairs per step (four per thread, 128 warp-sized groups): the groups'
  // tie counts and, after the ranks are known, their selection counts are scanned by the first
  // warp, which also gives the number of merged pairs in front of every compaction tile.
  if (tid == 0) { s_run_tie = 0; s_run_sel = 0; }
  __syncthreads();
  const int ntiles = (n - tab.off + KVS_CTILE - 1) / KVS_CTILE;
  int32_t* tp = a.tile_prefix + (size_t)unit * a.tile_stride;
  const int sweep = ((ntiles * 32 + 4095) / 4096) * 4096;
  // exclusive scan of the 128 group counts in s_cnt by warp 0 (lane i owns groups 4 i .. 4 i + 3)
  auto scan_groups = [&](uint32_t* run_total) {
    if (warp == 0) {
      uint32_t c[4], sum = 0;
#pragma unroll
      for (int i = 0; i < 4; ++i) { c[i] = s_cnt[4 * lane + i]; sum += c[i]; }
      uint32_t inc = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
      }
      uint32_t ex = *run_total + inc - sum;
#pragma unroll
      for (int i = 0; i < 4; ++i) { s_pre[4 * lane + i] = ex; ex += c[i]; }
      __syncwarp();
      if (lane == 31) *run_total = ex;
    }
  };
  uint32_t v4[4];
  auto fetch = [&](int p0) {
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int p = p0 + u * 1024 + tid;
      v4[u] = 0;
      if (p < P) v4[u] = a.from_mask ? (uint32_t)mask[p] : __ldg(key + p);
    }
  };
  fetch(0);
  for (int p0 = 0; p0 < sweep; p0 += 4096) {
    uint32_t v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = v4[u];
    if (p0 + 4096 < sweep) fetch(p0 + 4096);              // the next step's values travel meanwhile
    bool sel[4];
    if (!a.from_mask) {
      uint32_t tb[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int p = p0 + u * 1024 + tid;
        tb[u] = __ballot_sync(0xffffffffu, p < P && v[u] == prefix);
        if (lane == 0) s_cnt[u * 32 + warp] = __popc(tb[u]);
      }
      __syncthreads();
      scan_groups(&s_run_tie);
      __syncthreads();
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int p = p0 + u * 1024 + tid;
        const uint32_t rank = s_pre[u * 32 + warp] + __popc(tb[u] & ((1u << lane) - 1u));
        sel[u] = p < P && (v[u] < prefix || (v[u] == prefix && rank < k));
        if (p < P) mask[p] = sel[u] ? 1 : 0;
      }
      __syncthreads();                                    // s_pre is reused below
    } else {
#pragma unroll
      for (int u = 0; u < 4; ++u) sel[u] = (p0 + u * 1024 + tid) < P && v[u] != 0;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const uint32_t sb = __ballot_sync(0xffffffffu, sel[u]);
      if (lane == 0) s_cnt[u * 32 + warp] = __popc(sb);
    }
    __syncthreads();
    scan_groups(&s_run_sel);
    __syncthreads();
    if (lane == 0) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int tile = (p0 >> 5) + u * 32 + warp;
        if (tile < ntiles) tp[tile] = (int32_t)s_pre[u * 32 + warp];
      }
    }
    __syncthreads();
  }
}

}  // namespace

cudaError_t kvs_launch_select(const SelectArgs& a, const RoundTable& t, cudaStream_t st) {
  dim3 grid(a.Hkv, t.nseq);
  return kvs_launch_chained(select_pairs_kernel, grid, dim3(1024), 0, st, a, t);
}
