// Merge of the selected adjacent pairs and stable in-place compaction of the cache.
//
// A tile is 64 consecutive slots starting at the first candidate slot (32 candidate pairs;
// tiles past the last pair only shift the protected tail).  CTAs are persistent: within one
// (sequence, KV head) they take tiles by ticket.  A producer warp takes the ticket, streams
// the tile's K and Vsum rows into a three-stage shared-memory ring with bulk asynchronous
// copies, and stages the tile's decision (mask bits, weights, counts, merged pairs before the
// tile).  Eight consumer warps read the rows into registers, free the stage, form the merged
// rows
//   K*    = bf16( K_right + w (K_left - K_right) )        [Eq. kstar_final, weight form]
//   Vsum* = bf16( Vsum_left + Vsum_right ),  c* = c_left + c_right   [v* = v_m + v_{m+1}]
// publish "tile loaded", wait (bounded) until every earlier tile whose source rows they are
// about to overwrite has loaded too, and store the surviving rows at
//   new slot = old slot - (merged pairs before it).
// Tickets make the wait safe: a tile only waits for tiles with smaller tickets, whose owners
// are running and handle their own tiles in ticket order, so the smallest unpublished tile
// never waits.
#include "kvs_internal.h"
#include "kvs_sm100.cuh"

using namespace sm100;

namespace {

__device__ __forceinline__ uint32_t merge_k2(uint32_t l, uint32_t r, float w) {
  const float l0 = bf16lo(l), l1 = bf16hi(l), r0 = bf16lo(r), r1 = bf16hi(r);
  const float a = fmaf(w, l0 - r0, r0), b = fmaf(w, l1 - r1, r1);
  const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint32_t add_v2(uint32_t l, uint32_t r) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(bf16lo(l) + bf16lo(r), bf16hi(l) + bf16hi(r));
  return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ uint4 merge_k8(uint4 l, uint4 r, float w) {
  return make_uint4(merge_k2(l.x, r.x, w), merge_k2(l.y, r.y, w), merge_k2(l.z, r.z, w),
                    merge_k2(l.w, r.w, w));
}
__device__ __forceinline__ uint4 add_v8(uint4 l, uint4 r) {
  return make_uint4(add_v2(l.x, r.x), add_v2(l.y, r.y), add_v2(l.z, r.z), add_v2(l.w, r.w));
}

constexpr int kStages = 3;
constexpr int kRowBytes = KVS_D * 2;                       // one bf16 row
constexpr int kOperandBytes = KVS_CTILE * kRowBytes;       // 16 KB: the K (or Vsum) rows of a tile
constexpr int kStageBytes = 2 * kOperandBytes;
constexpr int kConsumers = 256;
constexpr int kThreads = kConsumers + 32;                  // + the producer warp

struct TileMeta {
  int32_t tile;                  // -1: no more tiles
  int32_t E0;                    // merged pairs before the tile
  uint32_t selbits;              // bit i: pair i of the tile is merged
  int32_t pad;
  float w[32];
  int32_t cnt[KVS_CTILE];
};
struct Shared {
  uint64_t full[kStages], meta_full[kStages], empty[kStages];
  int abort_flag, wait_us;       // (adjacent: the bounded waits read both through one pointer)
  int fail;
  TileMeta meta[kStages];
};
constexpr int kSmemBytes = kStages * kStageBytes + (int)sizeof(Shared);

__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void consumer_barrier() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Wait of all consumer warps on two mbarrier phases; either all 256 threads go on or all leave.
__device__ __forceinline__ bool consumer_wait(uint64_t* b0, uint64_t* b1, uint32_t parity, volatile int* abort_flag,
                                              volatile int* fail, int lane) {
  if (lane == 0) {
    if (!mbar_wait(b0, parity, abort_flag) || (b1 && !mbar_wait(b1, parity, abort_flag))) *fail = 1;
  }
  __syncwarp();
  consumer_barrier();
  return *fail == 0;
}

// Persistent CTAs per unit: the 2 x 148 CTAs that fit the GPU are shared out in proportion to the
// units' tile counts (a ragged batch would otherwise wait for its longest sequence, which would
// have no more CTAs than the shortest), at least one and at most one per tile.
__host__ __device__ inline int ctas_of_unit(int unit_tiles, long long all_tiles) {
  if (unit_tiles <= 0) return 0;
  long long c = all_tiles > 0 ? (2LL * 148 * unit_tiles) / all_tiles : 1;   // rounded down: all of them are resident at once
  if (c < 1) c = 1;
  if (c > unit_tiles) c = unit_tiles;
  return (int)c;
}
__host__ __device__ inline int tiles_of(int n, int off) { return n > off ? (n - off + KVS_CTILE - 1) / KVS_CTILE : 0; }

__global__ void __launch_bounds__(kThreads, 2)
merge_compact_kernel(const CompactArgs a, const RoundTable tab) {
  extern __shared__ __align__(128) uint8_t smem[];
  Shared* sh = reinterpret_cast<Shared*>(smem + kStages * kStageBytes);
  kvs_pdl_launch_dependents();
  kvs_pdl_wait();

  const int seq = blockIdx.z;
  const SeqRound sr = tab.s[seq];
  const int n = sr.n;
  if (n <= 0) return;
  const int h = blockIdx.y;
  const int unit = sr.b * a.c.Hkv + h;
  const int off = tab.off;
  const int ntiles = tiles_of(n, off);
  if (ntiles == 0) {
    // a unit that ends inside the protected prefix has nothing to move; its slot map is the identity
    if (a.new_index && blockIdx.x == 0) {
      int32_t* ni = a.new_index + (size_t)unit * a.c.n_max;
      for (int j = threadIdx.x; j < n; j += kThreads) ni[j] = j;
    }
    return;
  }
  long long all_tiles = 0;
  for (int i = 0; i < tab.nseq; ++i) all_tiles += tiles_of(tab.s[i].n, off);
  const int unit_ctas = ctas_of_unit(ntiles, all_tiles * a.c.Hkv);
  if ((int)blockIdx.x >= unit_ctas) return;                // this unit's share of the CTAs is smaller
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int P = sr.P;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->meta_full[s], 1);
      mbar_init(&sh->empty[s], kConsumers / 32);
    }
    sh->abort_flag = 0;
    sh->wait_us = (int)a.wait_us;
    sh->fail = 0;
    mbar_fence_init();
  }
  __syncthreads();
  volatile int* abort_flag = &sh->abort_flag;

  __nv_bfloat16* Kb = a.c.K + sr.b * a.c.ksb + h * a.c.ksh;
  __nv_bfloat16* Vb = a.c.V + sr.b * a.c.vsb + h * a.c.vsh;
  int32_t* Cb = a.c.counts + (size_t)unit * a.c.n_max;

  if (warp == kConsumers / 32) {
    // ================================================================ producer warp
    const uint8_t* mask = a.mask + (size_t)unit * a.pair_stride;
    const float* wl = a.w + (size_t)unit * a.pair_stride;
    uint32_t next_ticket = 0;
    if (lane == 0) next_ticket = atomicAdd(&a.tickets[unit], 1u);
    int issued = 0;                  // tiles whose copies were requested
    for (int k = 0;; ++k) {
      const int s = k % kStages;
      const uint32_t ph = (uint32_t)(k / kStages) & 1u;
      int ok = 1;
      if (lane == 0) ok = mbar_wait(&sh->empty[s], ph ^ 1u, abort_flag) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) {
        // give the copies of the last stages a bounded time to land before the CTA leaves
        if (lane == 0)
          for (int kk = max(0, issued - kStages); kk < issued; ++kk) mbar_drain(&sh->full[kk % kStages], (uint32_t)(kk / kStages) & 1u);
        break;
      }
      const int t = (int)__shfl_sync(0xffffffffu, next_ticket, 0);
      TileMeta* m = &sh->meta[s];
      if (t >= ntiles) {
        if (lane == 0) { m->tile = -1; mbar_arrive(&sh->meta_full[s]); }
        break;
      }
      if (lane == 0) next_ticket = atomicAdd(&a.tickets[unit], 1u);   // its latency hides behind this tile
      const int j0 = off + KVS_CTILE * t;
      const int rows = min(KVS_CTILE, n - j0);
      uint8_t* sk = smem + s * kStageBytes;
      uint8_t* sv = sk + kOperandBytes;
      if (lane == 0) mbar_expect_tx(&sh->full[s], (uint32_t)rows * 2u * kRowBytes);
      issued = k + 1;
      __syncwarp();
      if (a.c.kst == KVS_D && a.c.vst == KVS_D) {
        if (lane == 0) bulk_load(sk, Kb + (int64_t)j0 * KVS_D, (uint32_t)rows * kRowBytes, &sh->full[s]);
        if (lane == 1) bulk_load(sv, Vb + (int64_t)j0 * KVS_D, (uint32_t)rows * kRowBytes, &sh->full[s]);
      } else {
        for (int r = lane; r < rows; r += 32) {
          bulk_load(sk + r * kRowBytes, Kb + (int64_t)(j0 + r) * a.c.kst, kRowBytes, &sh->full[s]);
          bulk_load(sv + r * kRowBytes, Vb + (int64_t)(j0 + r) * a.c.vst, kRowBytes, &sh->full[s]);
        }
      }
      // the tile's decision
      const int pp = 32 * t + lane;
      const bool in_range = pp < P;
      const bool sel = in_range && mask[pp] != 0;
      m->w[lane] = in_range ? wl[pp] : 0.5f;
      m->cnt[lane] = (lane < rows) ? Cb[j0 + lane] : 0;
      m->cnt[lane + 32] = (lane + 32 < rows) ? Cb[j0 + lane + 32] : 0;
      const uint32_t bits = __ballot_sync(0xffffffffu, sel);
      if (lane == 0) {
        m->selbits = bits;
        m->E0 = a.tile_prefix[(size_t)unit * a.tile_stride + t];
        m->tile = t;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->meta_full[s]);
    }
  } else {
    // ================================================================ consumer warps
    const int i = tid >> 3;          // pair in tile
    const int c0 = tid & 7;          // chunks c0 and c0 + 8 (16 bytes each)
    volatile int* fail = &sh->fail;
    for (int k = 0;; ++k) {
      const int s = k % kStages;
      const uint32_t ph = (uint32_t)(k / kStages) & 1u;
      if (!consumer_wait(&sh->meta_full[s], nullptr, ph, abort_flag, fail, lane)) break;
      const TileMeta* m = &sh->meta[s];
      const int t = m->tile;
      if (t < 0) break;
      if (!consumer_wait(&sh->full[s], nullptr, ph, abort_flag, fail, lane)) break;
      const int j0 = off + KVS_CTILE * t;
      const int jl = j0 + 2 * i, jr = jl + 1;
      const bool okl = jl < n, okr = jr < n;
      const uint8_t* sk = smem + s * kStageBytes;
      const uint8_t* sv = sk + kOperandBytes;
      uint4 kl[2], kr[2], vl[2], vr[2];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const int ob = (c0 + 8 * u) * 16;
        kl[u] = *reinterpret_cast<const uint4*>(sk + (2 * i) * kRowBytes + ob);
        kr[u] = *reinterpret_cast<const uint4*>(sk + (2 * i + 1) * kRowBytes + ob);
        vl[u] = *reinterpret_cast<const uint4*>(sv + (2 * i) * kRowBytes + ob);
        vr[u] = *reinterpret_cast<const uint4*>(sv + (2 * i + 1) * kRowBytes + ob);
      }
      const uint32_t selbits = m->selbits;
      const int E0 = m->E0;
      const float w = m->w[i];
      int32_t cl = m->cnt[2 * i], cr = m->cnt[2 * i + 1];
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->empty[s]);          // the stage may be refilled

      const bool sel = (selbits >> i) & 1u;
      const int e = __popc(selbits & ((1u << i) - 1u));
      const int dl = jl - E0 - e;
      const int dr = jr - E0 - e;      // used only when !sel
      if (sel) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          kl[u] = merge_k8(kl[u], kr[u], w);
          vl[u] = add_v8(vl[u], vr[u]);
        }
        cl += cr;
      }
      // the tile's source rows are out of global memory: later tiles may overwrite them
      // (test hook: with bit 2 of debug_stall the flag stays unset, so that the waits on it run out)
      if (tid == 0 && !(a.debug_stall & 4u)) st_release_u32(&a.flags[(size_t)unit * a.tile_stride + t], a.epoch);
      const int moved = E0 + __popc(selbits);
      if (E0 > 0 && unit_ctas > 1) {
        // This tile's rows land in [j0 - E0, j0 - E0 + 64): those are source rows of at most two
        // earlier tiles (and of this tile itself), which must have been read before they are
        // overwritten; a CTA that owns the whole unit has read them itself, in order
        const int first = (j0 - E0 - off) / KVS_CTILE;
        const int last = min(t - 1, first + 1);
        for (int tt = last - tid; tt >= first; tt -= kConsumers) {
          const uint32_t* f = &a.flags[(size_t)unit * a.tile_stride + tt];
          int spins = 0;
          const uint64_t t0 = globaltimer_ns();
          while (ld_acquire_u32(f) < a.epoch) {
            const bool late = (++spins & 255) == 0 && globaltimer_ns() - t0 > (uint64_t)(uint32_t)sh->wait_us * 1000ull;
            if (late || spins > KVS_SPIN_LIMIT || *abort_flag) { *fail = 1; *abort_flag = 1; break; }
            __nanosleep(20);
          }
        }
        consumer_barrier();
        if (*fail) break;
      }
      if (moved != 0) {
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int ch = (c0 + 8 * u) * 8;
          if (okl && (sel || dl != jl)) {
            *reinterpret_cast<uint4*>(Kb + (int64_t)dl * a.c.kst + ch) = kl[u];
            *reinterpret_cast<uint4*>(Vb + (int64_t)dl * a.c.vst + ch) = vl[u];
          }
          if (okr && !sel && dr != jr) {
            *reinterpret_cast<uint4*>(Kb + (int64_t)dr * a.c.kst + ch) = kr[u];
            *reinterpret_cast<uint4*>(Vb + (int64_t)dr * a.c.vst + ch) = vr[u];
          }
        }
        if (c0 == 0) {
          if (okl) Cb[dl] = cl;
          if (okr && !sel) Cb[dr] = cr;
        }
      }
      if (a.new_index && c0 == 0) {
        int32_t* ni = a.new_index + (size_t)unit * a.c.n_max;
        if (okl) ni[jl] = dl;
        if (okr) ni[jr] = sel ? dl : dr;
      }
      if (a.new_index && t == 0) {
        int32_t* ni = a.new_index + (size_t)unit * a.c.n_max;
        for (int j = tid; j < off && j < n; j += kConsumers) ni[j] = j;
      }
    }
  }
  __syncthreads();
  if (tid == 0 && sh->abort_flag && a.status_dev) atomicExch(a.status_dev, (int)KVS_ERR_TIMEOUT);
}

}  // namespace

cudaError_t kvs_launch_compact(const CompactArgs& a, const RoundTable& t, cudaStream_t st) {
  static KvsPerDeviceOnce configured;
  cudaError_t ce = configured.run([] {
    return cudaFuncSetAttribute(merge_compact_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  });
  if (ce != cudaSuccess) return ce;
  int nmax = 0;
  for (int i = 0; i < t.nseq; ++i) nmax = nmax > t.s[i].n ? nmax : t.s[i].n;
  const int ntiles = (nmax - t.off + KVS_CTILE - 1) / KVS_CTILE;
  // (units that end inside the protected prefix still get their identity slot map)
  if (nmax <= 0 || (ntiles <= 0 && !a.new_index)) return cudaSuccess;
  // persistent CTAs: two per SM over all units of the launch, in proportion to the units' lengths;
  // the grid is as wide as the longest unit's share, the CTAs beyond a unit's share leave at once
  long long all_tiles = 0;
  for (int i = 0; i < t.nseq; ++i) all_tiles += tiles_of(t.s[i].n, t.off);
  int per_unit = 1;
  for (int i = 0; i < t.nseq; ++i) {
    const int c = ctas_of_unit(tiles_of(t.s[i].n, t.off), all_tiles * a.c.Hkv);
    if (c > per_unit) per_unit = c;
  }
  dim3 grid(per_unit, a.c.Hkv, t.nseq);
  return kvs_launch_chained(merge_compact_kernel, grid, dim3(kThreads), kSmemBytes, st, a, t);
}
