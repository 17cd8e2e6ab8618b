// Merge of the selected adjacent pairs and stable in-place compaction of the cache.
//
// A tile is 64 consecutive slots starting at the first candidate slot (32 candidate pairs;
// tiles past the last pair only shift the protected tail).  Each CTA takes a tile by ticket,
// loads its rows into registers, forms the merged rows
//   K*    = bf16( K_right + w (K_left - K_right) )        [Eq. kstar_final, weight form]
//   Vsum* = bf16( Vsum_left + Vsum_right ),  c* = c_left + c_right   [v* = v_m + v_{m+1}]
// publishes "tile loaded", waits (bounded) until every earlier tile whose source rows it is
// about to overwrite has loaded too, and stores the surviving rows at
//   new slot = old slot - (merged pairs before it).
// Tickets make the wait safe: a tile only waits for tiles that took their ticket earlier,
// and those never wait for later ones.
#include "kvs_internal.h"

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

__global__ void __launch_bounds__(256)
merge_compact_kernel(const CompactArgs a, const RoundTable tab) {
  const int seq = blockIdx.z;
  const SeqRound sr = tab.s[seq];
  const int n = sr.n;
  if (n <= 0) return;
  const int h = blockIdx.y;
  const int unit = sr.b * a.c.Hkv + h;
  const int off = tab.off;
  const int ntiles = (n - off + KVS_CTILE - 1) / KVS_CTILE;
  const int tid = threadIdx.x;

  __shared__ int s_tile;
  __shared__ uint32_t s_selbits;
  __shared__ int s_abort;
  if (tid == 0) {
    s_tile = (int)atomicAdd(&a.tickets[unit], 1u);
    s_abort = 0;
  }
  __syncthreads();
  const int t = s_tile;
  if (t >= ntiles) return;

  const int P = sr.P;
  const uint8_t* mask = a.mask + (size_t)unit * a.pair_stride;
  const float* wl = a.w + (size_t)unit * a.pair_stride;
  if (tid < 32) {
    const int p = 32 * t + tid;
    const bool sel = p < P && mask[p] != 0;
    const uint32_t bits = __ballot_sync(0xffffffffu, sel);
    if (tid == 0) s_selbits = bits;
  }
  __syncthreads();
  const uint32_t selbits = s_selbits;
  const int E0 = a.tile_prefix[(size_t)unit * a.tile_stride + t];
  const int j0 = off + KVS_CTILE * t;

  const int i = tid >> 3;          // pair in tile
  const int c0 = tid & 7;          // chunks c0 and c0 + 8 (16 bytes each)
  const int p = 32 * t + i;
  const bool sel = (selbits >> i) & 1u;
  const int e = __popc(selbits & ((1u << i) - 1u));
  const int jl = j0 + 2 * i, jr = jl + 1;
  const bool okl = jl < n, okr = jr < n;
  const int dl = jl - E0 - e;
  const int dr = jr - E0 - e;      // used only when !sel

  __nv_bfloat16* Kb = a.c.K + sr.b * a.c.ksb + h * a.c.ksh;
  __nv_bfloat16* Vb = a.c.V + sr.b * a.c.vsb + h * a.c.vsh;
  int32_t* Cb = a.c.counts + (size_t)unit * a.c.n_max;

  uint4 kl[2], kr[2], vl[2], vr[2];
  int32_t cl = 0, cr = 0;
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int ch = (c0 + 8 * u) * 8;
    kl[u] = kr[u] = vl[u] = vr[u] = make_uint4(0, 0, 0, 0);
    if (okl) {
      kl[u] = *reinterpret_cast<const uint4*>(Kb + (int64_t)jl * a.c.kst + ch);
      vl[u] = *reinterpret_cast<const uint4*>(Vb + (int64_t)jl * a.c.vst + ch);
    }
    if (okr) {
      kr[u] = *reinterpret_cast<const uint4*>(Kb + (int64_t)jr * a.c.kst + ch);
      vr[u] = *reinterpret_cast<const uint4*>(Vb + (int64_t)jr * a.c.vst + ch);
    }
  }
  if (c0 == 0) {
    if (okl) cl = Cb[jl];
    if (okr) cr = Cb[jr];
  }
  if (sel) {
    const float w = wl[p];
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      kl[u] = merge_k8(kl[u], kr[u], w);
      vl[u] = add_v8(vl[u], vr[u]);
    }
    cl += cr;
  }
  __syncthreads();   // every load of this tile has returned (its values were just used)

  const int moved = E0 + __popc(selbits);
  if (moved != 0) {
    if (tid == 0) st_release_u32(&a.flags[(size_t)unit * a.tile_stride + t], a.epoch);
    // earlier tiles whose source rows overlap [j0 - E0, j0)
    if (E0 > 0) {
      const int first = (j0 - E0 - off) / KVS_CTILE;
      for (int tt = t - 1 - tid; tt >= first; tt -= 256) {
        const uint32_t* f = &a.flags[(size_t)unit * a.tile_stride + tt];
        int spins = 0;
        while (ld_acquire_u32(f) < a.epoch) {
          if (++spins > KVS_SPIN_LIMIT) { s_abort = 1; break; }
          __nanosleep(20);
        }
      }
    }
    __syncthreads();
    if (s_abort) {
      if (tid == 0 && a.status_dev) atomicExch(a.status_dev, (int)KVS_ERR_TIMEOUT);
      return;
    }
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
  } else if (tid == 0) {
    // nothing moves, but later tiles may still wait on this flag
    st_release_u32(&a.flags[(size_t)unit * a.tile_stride + t], a.epoch);
  }
  if (a.new_index && c0 == 0) {
    int32_t* ni = a.new_index + (size_t)unit * a.c.n_max;
    if (okl) ni[jl] = dl;
    if (okr) ni[jr] = sel ? dl : dr;
  }
  if (a.new_index && t == 0) {
    int32_t* ni = a.new_index + (size_t)unit * a.c.n_max;
    for (int j = tid; j < off && j < n; j += 256) ni[j] = j;
  }
}

}  // namespace

cudaError_t kvs_launch_compact(const CompactArgs& a, const RoundTable& t, cudaStream_t st) {
  int nmax = 0;
  for (int i = 0; i < t.nseq; ++i) nmax = nmax > t.s[i].n ? nmax : t.s[i].n;
  const int ntiles = (nmax - t.off + KVS_CTILE - 1) / KVS_CTILE;
  if (ntiles <= 0) return cudaSuccess;
  dim3 grid(ntiles, a.c.Hkv, t.nseq);
  merge_compact_kernel<<<grid, 256, 0, st>>>(a, t);
  return cudaGetLastError();
}
