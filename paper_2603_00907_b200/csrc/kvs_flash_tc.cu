// Attention partials on the tensor cores (tcgen05 + TMEM + TMA), queries on TMEM lanes.
//
// One CTA owns a block of 128 query rows (Q stays in shared memory) and a contiguous range
// of 128-slot tiles.  K and V tiles travel in two separate two-stage TMA rings; per tile one
// thread issues
//   S[q, slot] = Q K_tile^T                         (fp32 in TMEM, double buffered)
// Sixteen softmax warps share the tile: the four warps of a TMEM lane quarter own the same 32
// query rows and 32 slot columns each.  A thread finds the maximum of its 32 logits; the four
// threads of a row agree on the row maximum through a shared-memory atomic maximum, keep the
// same stabiliser m (it only moves when the maximum grows by more than 2^8, in which case the
// first of the four rescales the row of O in TMEM), and each writes P' = exp(s - m), split
// into two bf16 terms, back into the tensor-memory columns the logits came from, keeping its
// part of l = sum_j c_j exp(s_j - m): the count bias ln c_j of a merged slot is just the factor
// c_j in that sum.  The issuing thread then runs
//   O[q, :] += (P'_hi + P'_lo) Vsum_tile            (P' from tensor memory, V as the MN-major operand)
// with O accumulating in TMEM across the tiles [Eq. attn_def_vec with merged slots:
// o = sum_j alpha_j Vsum_j / c_j].  At the end (stabiliser, sum, O) is written as the partial
// of this key range.  Window queries and decode queries use the same kernel.
//
// Four more warps serve the statistics pass that follows the window attention: tiles are then
// aligned with the round's candidate pairs, and for every pair they form |vbar_l|^2, |vbar_r|^2,
// |vbar_l + vbar_r|^2 and the adjacent-key cosine from the staged rows (diagonals of small
// mma.sync products), so that the statistics kernel does not have to touch the rows for it.
#include "kvs_internal.h"
#include "kvs_sm100.cuh"

using namespace sm100;

namespace {

constexpr int kTile = 128;
constexpr int kHalf = 16384;               // [128 rows x 64 bf16], 128-byte swizzle
constexpr int kOperand = 2 * kHalf;
constexpr int kStage = 2 * kOperand;       // K tile + V tile
constexpr int kSmemQ = 0, kSmemStage = kOperand;
constexpr int kSmemMisc = kSmemStage + 2 * kStage;
constexpr int kSoftmaxWarps = 16, kNormWarps = 4;
constexpr int kThreads = (2 + kSoftmaxWarps + kNormWarps) * 32;   // warp 0: TMA, 1: MMA, 2-17: softmax, 18-21: pair norms
constexpr float kRescaleGap = 8.f;         // log2 units

struct Misc {
  uint64_t kfull[2], vfull[2], kfree[2], vfree[2], sfull[2], pready[2], ofull[2], qfull;
  uint32_t tmem_base;
  int abort_flag;
  union {
    struct {
      uint32_t rowmax[3][kTile];           // per tile (mod 3) and query row: maximum logit, as an ordered integer
      alignas(16) float cnt[2][kTile];     // per tile parity: counts of the tile's slots (read as float4)
    };
    float lsum[4][kTile];                  // after the last tile: the column groups' parts of the row sums
  };
};
constexpr int kSmemBytes = kSmemMisc + (int)sizeof(Misc);
static_assert(kSmemBytes <= 232448, "shared memory of one CTA");

constexpr uint32_t kOrdNegInf = 0x007fffffu;   // ordered-integer image of -infinity
// monotone map float -> unsigned (so that an integer maximum is the float maximum) and back
__device__ __forceinline__ uint32_t f2ord(float f) {
  const uint32_t b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float ord2f(uint32_t u) {
  return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}

__device__ __forceinline__ void softmax_barrier() { asm volatile("bar.sync 1, 512;" ::: "memory"); }

// One lane polls, the warp follows.  A failed wait (time-out or abort) only makes the warp skip
// its work: it still goes through the tile loop and its one named barrier per tile, so that no
// other warp can be left waiting for it.
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int lane) {
  int ok = 1;
  if (lane == 0) ok = mbar_wait(bar, parity, abort_flag) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
__device__ __forceinline__ void warp_arrive(uint64_t* bar, int lane) {
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float* v) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])),
        "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])),
        "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
        "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15])), "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])),
        "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])), "r"(__float_as_uint(v[20])),
        "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
        "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])),
        "r"(__float_as_uint(v[27])), "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])),
        "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* v) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
               ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
               : "memory");
}
__device__ __forceinline__ void tmem_st_wait() {
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t saddr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(saddr)
               : "memory");
}
// D(16x8, fp32) += A(16x16, bf16, row major) B(16x8, bf16, column major)
__device__ __forceinline__ void mma16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// For the 8 pairs (rows 2i, 2i+1) of rows [row0, row0 + 16) of one staged operand: |x_l|^2,
// |x_r|^2 and <x_l, x_r>, delivered to lanes 0-7.  A = [x_l rows ; x_r rows] (16 x 128) against
// B = x_r and B = x_l (8 rows each): the wanted values are diagonal elements of the two
// 16 x 8 products.  All fragments are loaded first, then two accumulation chains run.
__device__ __forceinline__ void pair_dots8(const uint8_t* tile, int row0, int lane, float& ll, float& rr, float& lr) {
  const uint32_t base = smem_u32(tile);
  const int mtx = lane >> 3, rin = lane & 7;                // ldmatrix: this lane feeds row rin of matrix mtx
  const int g = lane >> 2;                                  // accumulator row held by this lane
  const int src = 4 * (lane & 7) + ((lane & 7) >> 1);       // lane that holds the diagonal of pair (lane & 7)
  const int row = row0 + 2 * rin + (mtx & 1);               // matrices 0,2: left rows; 1,3: right rows
  uint32_t fr[8][4];
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    const int chunk = 2 * (kk & 3) + (mtx >> 1);            // 16-byte chunk inside the 128-byte row
    ldmatrix_x4(fr[kk], base + (kk >> 2) * kHalf + row * 128 + ((chunk ^ (row & 7)) << 4));
  }
  float d1[4] = {0.f, 0.f, 0.f, 0.f}, d2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    mma16816(d1, fr[kk], fr[kk][1], fr[kk][3]);             // columns = right rows
    mma16816(d2, fr[kk], fr[kk][0], fr[kk][2]);             // columns = left rows
  }
  const float v_lr = (g & 1) ? d1[1] : d1[0];               // row g (left), column g (right)
  const float v_rr = (g & 1) ? d1[3] : d1[2];               // row 8 + g (right), column g (right)
  const float v_ll = (g & 1) ? d2[1] : d2[0];               // row g (left), column g (left)
  lr = __shfl_sync(0xffffffffu, v_lr, src);
  rr = __shfl_sync(0xffffffffu, v_rr, src);
  ll = __shfl_sync(0xffffffffu, v_ll, src);
}

__global__ void __launch_bounds__(kThreads, 1)
flash_partial_tc(const FlashTcArgs a, const RoundTable tab, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmQ) {
  extern __shared__ __align__(1024) uint8_t smem[];
  Misc* misc = reinterpret_cast<Misc*>(smem + kSmemMisc);

  const int seq = blockIdx.z;
  const SeqRound sr = tab.s[seq];
  const int n = sr.n;
  const int h = blockIdx.y;
  const int qblk = blockIdx.x % a.nqblk;
  const int split = blockIdx.x / a.nqblk;
  const int unit = sr.b * a.Hkv + h;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // with pair norms, tile t covers slots [128 t - shift, 128 t - shift + 128): aligned with the pairs
  const int shift = a.pair_norms ? (tab.off & 1) : 0;
  const int ntiles = (n + shift + kTile - 1) / kTile;
  const int t_begin = min(ntiles, split * a.tiles_per_split);
  const int t_end = min(ntiles, t_begin + a.tiles_per_split);
  const int my_tiles = t_end - t_begin;
  if (n <= 0) return;
  if (smem_u32(smem) & 1023u) {                        // the swizzled tiles need a 1024-byte aligned base
    if (threadIdx.x == 0 && a.status_dev) atomicExch(a.status_dev, (int)KVS_ERR_CUDA);
    return;
  }
  if (my_tiles <= 0) {
    // an empty key range still owes its (empty) partial to the combine
    if (warp >= 2 && warp < 6) {
      const int row = (warp & 3) * 32 + lane, m = qblk * 128 + row;
      if (m < a.M) a.part_ml[((size_t)unit * a.splits + split) * a.M + m] = make_float2(-INFINITY, 0.f);
    }
    return;
  }
  // the pair norms of a KV head are shared work: the first query block forms the key cosines, the
  // second one (the first again, if there is only one) the value norms
  const bool norm_k = a.pair_norms != nullptr && qblk == 0;
  const bool norm_v = a.pair_norms != nullptr && qblk == (a.nqblk > 1 ? 1 : 0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      // the K rows of a stage are free once the logits are formed, the V rows only after P V: two
      // rings, so that the next K tile is requested a whole softmax earlier than the next V tile
      mbar_init(&misc->kfull[s], 1);
      mbar_init(&misc->vfull[s], 1);
      mbar_init(&misc->kfree[s], norm_k ? 1 + kNormWarps : 1);   // MMA commit (+ the pair-norm warps)
      mbar_init(&misc->vfree[s], norm_v ? 1 + kNormWarps : 1);
      mbar_init(&misc->sfull[s], 1);
    }
    // P' is handed over in two halves (the first and the last 16 slots of every column group), so
    // that the P V products of one half run while the other half is still being written
    for (int hf = 0; hf < 2; ++hf) {
      mbar_init(&misc->pready[hf], kSoftmaxWarps);
      mbar_init(&misc->ofull[hf], 1);
    }
    mbar_init(&misc->qfull, 1);
    misc->abort_flag = 0;
    mbar_fence_init();
  }
  if (threadIdx.x < 3 * kTile) misc->rowmax[threadIdx.x / kTile][threadIdx.x % kTile] = kOrdNegInf;
  if (warp == 1) tmem_alloc(&misc->tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = misc->tmem_base;
  volatile int* abort_flag = &misc->abort_flag;

  if (warp == 0) {
    // ================================================================ TMA producer
    // one thread streams both rings: whichever of the next K tile and the next V tile has a free
    // stage is requested first
    if (lane == 0) {
      prefetch_tmap(&tmK); prefetch_tmap(&tmV); prefetch_tmap(&tmQ);
      mbar_expect_tx(&misc->qfull, kOperand);
      for (int hf = 0; hf < 2; ++hf)
        tma_load_3d(smem + kSmemQ + hf * kHalf, &tmQ, &misc->qfull, hf * 64, qblk * 128, unit);
      int kli = 0, vli = 0;
      uint64_t t0 = globaltimer_ns();
      while (kli < my_tiles || vli < my_tiles) {
        bool progress = false;
        if (kli < my_tiles && mbar_try_wait(&misc->kfree[kli & 1], ((kli >> 1) & 1) ^ 1)) {
          const int s = kli & 1;
          uint8_t* st = smem + kSmemStage + s * kStage;
          const int row = (t_begin + kli) * kTile - shift;
          mbar_expect_tx(&misc->kfull[s], kOperand);
          for (int hf = 0; hf < 2; ++hf) tma_load_4d(st + hf * kHalf, &tmK, &misc->kfull[s], hf * 64, row, h, sr.b);
          ++kli;
          progress = true;
        }
        if (vli < my_tiles && mbar_try_wait(&misc->vfree[vli & 1], ((vli >> 1) & 1) ^ 1)) {
          const int s = vli & 1;
          uint8_t* st = smem + kSmemStage + s * kStage + kOperand;
          const int row = (t_begin + vli) * kTile - shift;
          mbar_expect_tx(&misc->vfull[s], kOperand);
          for (int hf = 0; hf < 2; ++hf) tma_load_4d(st + hf * kHalf, &tmV, &misc->vfull[s], hf * 64, row, h, sr.b);
          ++vli;
          progress = true;
        }
        if (progress) {
          t0 = globaltimer_ns();
        } else {
          if (*abort_flag) break;
          if (globaltimer_ns() - t0 > 1000000000ull) { *abort_flag = 1; break; }
        }
      }
      if (*abort_flag) {
        // drain: give the copies already issued a bounded time to land before the CTA leaves
        for (int li = max(0, kli - 2); li < kli; ++li) {
          const uint64_t t1 = globaltimer_ns();
          while (!mbar_try_wait(&misc->kfull[li & 1], (li >> 1) & 1) && globaltimer_ns() - t1 < 200000000ull) {}
        }
        for (int li = max(0, vli - 2); li < vli; ++li) {
          const uint64_t t1 = globaltimer_ns();
          while (!mbar_try_wait(&misc->vfull[li & 1], (li >> 1) & 1) && globaltimer_ns() - t1 < 200000000ull) {}
        }
      }
    }
  } else if (warp == 1) {
    // ================================================================ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16(128, 128);                 // Q (K-major) x K tile (K-major)
      constexpr uint32_t idesc_o = idesc_bf16(128, 128, false, true);    // P' (K-major) x V tile (MN-major)
      const uint32_t q_addr = smem_u32(smem + kSmemQ);
      auto issue_s = [&](int li) -> bool {
        const int s = li & 1, k = li >> 1;
        // buffer s last held P' of tile li - 2, whose products were issued by this thread before
        if (!mbar_wait(&misc->kfull[s], k & 1, abort_flag)) return false;
        tc_fence_after();
        const uint32_t k_addr = smem_u32(smem + kSmemStage + s * kStage);
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t o = (kk >> 2) * kHalf + (kk & 3) * 32;
          umma_bf16(tmem + s * 128, smem_desc_sw128(q_addr + o, 16, 1024), smem_desc_sw128(k_addr + o, 16, 1024),
                    idesc_s, kk > 0);
        }
        tc_commit(&misc->sfull[s]);
        tc_commit(&misc->kfree[s]);
        return true;
      };
      bool ok = mbar_wait(&misc->qfull, 0, abort_flag);
      ok = ok && issue_s(0);
      for (int li = 0; ok && li < my_tiles; ++li) {
        if (li + 1 < my_tiles) ok = issue_s(li + 1);
        const int s = li & 1;
        const uint32_t v_addr = smem_u32(smem + kSmemStage + s * kStage + kOperand);
        if (ok && !mbar_wait(&misc->vfull[s], (li >> 1) & 1, abort_flag)) ok = false;
        const uint32_t dO = tmem + 256;
        for (int hf = 0; ok && hf < 2; ++hf) {
          if (!mbar_wait(&misc->pready[hf], li & 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int cgi = 0; cgi < 4; ++cgi) {
            const int kk = 2 * cgi + hf;                     // 16-slot step of the tile: slots [16 kk, 16 kk + 16)
#pragma unroll
            for (int hl = 0; hl < 2; ++hl) {
              // A: 16 slots = 8 columns of P'_hi (columns 0-63 of the logit buffer) or P'_lo (64-127);
              // B: 16 slots = two 8-row groups of V
              const uint32_t ap = tmem + s * 128 + hl * 64 + kk * 8;
              const uint64_t bd = smem_desc_sw128(v_addr + (kk * 16) * 128, kHalf, 1024);
              umma_bf16_ts(dO, ap, bd, idesc_o, (li > 0 || hf > 0 || cgi > 0 || hl > 0) ? 1u : 0u);
            }
          }
          tc_commit(&misc->ofull[hf]);
        }
        if (ok) tc_commit(&misc->vfree[s]);
      }
    }
  } else if (warp >= 2 + kSoftmaxWarps) {
    // ================================================================ pair-norm warps
    if (norm_k || norm_v) {
      const int nw = warp - (2 + kSoftmaxWarps);                 // rows [32 nw, 32 nw + 32) of every tile
      const int off = tab.off;
      const int32_t* Cn = a.counts + (size_t)unit * a.n_max;
      const int pl = lane & 15;                                  // lanes 0-15 own the warp's 16 pairs
      // counts of the next tile's pair travel while the current tile is processed
      float cl_next = 1.f, cr_next = 1.f;
      if (norm_v) {
        const int sl = t_begin * kTile - shift + nw * 32 + 2 * pl;
        if (sl >= off && ((sl - off) >> 1) < sr.P) { cl_next = (float)Cn[sl]; cr_next = (float)Cn[sl + 1]; }
      }
      for (int li = 0; li < my_tiles; ++li) {
        const int s = li & 1, k = li >> 1;
        const int slot_l = (t_begin + li) * kTile - shift + nw * 32 + 2 * pl;   // left slot of this lane's pair
        const int p = (slot_l - off) >> 1;
        const bool pair_ok = lane < 16 && slot_l >= off && p < sr.P;
        const float cl = cl_next, cr = cr_next;
        if (norm_v && li + 1 < my_tiles) {
          const int sl = slot_l + kTile;
          cl_next = cr_next = 1.f;
          if (sl >= off && ((sl - off) >> 1) < sr.P) { cl_next = (float)Cn[sl]; cr_next = (float)Cn[sl + 1]; }
        }
        float* out = reinterpret_cast<float*>(a.pair_norms + (size_t)unit * a.pair_stride + (pair_ok ? p : 0));
        const uint8_t* st = smem + kSmemStage + s * kStage;
        int ok = 1;
        if (norm_k) {
          if (lane == 0) ok = mbar_wait(&misc->kfull[s], k & 1, abort_flag) ? 1 : 0;
          if (!__shfl_sync(0xffffffffu, ok, 0)) break;
          float ll[2], rr[2], lr[2];
          pair_dots8(st, nw * 32, lane, ll[0], rr[0], lr[0]);
          pair_dots8(st, nw * 32 + 16, lane, ll[1], rr[1], lr[1]);
          __syncwarp();
          if (lane == 0) mbar_arrive(&misc->kfree[s]);           // the K rows are no longer needed here
          const bool b = (lane >> 3) & 1;
          const float kll = b ? ll[1] : ll[0], krr = b ? rr[1] : rr[0], klr = b ? lr[1] : lr[0];
          if (pair_ok) out[3] = klr / fmaxf(sqrtf(kll) * sqrtf(krr), 1e-30f);
        }
        if (norm_v) {
          if (lane == 0) ok = mbar_wait(&misc->vfull[s], k & 1, abort_flag) ? 1 : 0;
          if (!__shfl_sync(0xffffffffu, ok, 0)) break;
          float ll[2], rr[2], lr[2];
          pair_dots8(st + kOperand, nw * 32, lane, ll[0], rr[0], lr[0]);
          pair_dots8(st + kOperand, nw * 32 + 16, lane, ll[1], rr[1], lr[1]);
          __syncwarp();
          if (lane == 0) mbar_arrive(&misc->vfree[s]);
          const bool b = (lane >> 3) & 1;
          const float vll = b ? ll[1] : ll[0], vrr = b ? rr[1] : rr[0], vlr = b ? lr[1] : lr[0];
          if (pair_ok) {
            const float icl = 1.f / cl, icr = 1.f / cr;
            const float r2l = vll * icl * icl, r2r = vrr * icr * icr;
            out[0] = r2l; out[1] = r2r; out[2] = r2l + r2r + 2.f * vlr * icl * icr;
          }
        }
      }
    }
  } else {
    // ================================================================ softmax warps
    const int cg = (warp - 2) >> 2;                       // 32-slot column group of the tile
    const int row = (warp & 3) * 32 + lane;               // TMEM lane = query row in the block
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const int m = qblk * 128 + row;
    const int last_vis = a.causal ? (n - a.Wq + (m % a.Wq)) : (n - 1);
    const int32_t* Cb = a.counts + (size_t)unit * a.n_max;
    // stabiliser in log2 units; until a row has seen a visible slot it is 0 (keeps the arithmetic finite)
    float m_stab = 0.f, l = 0.f;
    bool have_stab = false;
    bool alive = true;
    // (first column group) the count of slot `row` of the next tile travels while the current tile is processed
    int cnt_next = 1;
    if (cg == 0) {
      const int j = t_begin * kTile - shift + row;
      if (j >= 0 && j < n) cnt_next = Cb[j];
    }
    for (int li = 0; li < my_tiles; ++li) {
      const int s = li & 1, k = li >> 1;
      const int j0 = (t_begin + li) * kTile - shift + cg * 32;    // first slot of this thread's columns
      float* cnt = misc->cnt[s];
      uint32_t* rmax = misc->rowmax[li % 3];
      if (cg == 0) {
        cnt[row] = (float)cnt_next;
        const int j = (t_begin + li + 1) * kTile - shift + row;
        cnt_next = (li + 1 < my_tiles && j >= 0 && j < n) ? Cb[j] : 1;
      }
      float x[32];
      if (alive) alive = warp_wait(&misc->sfull[s], k & 1, abort_flag, lane);
      if (alive) {
        tc_fence_after();
        tmem_ld32(tmem + lane_addr + s * 128 + cg * 32, x);
        tmem_ld_wait();
        // logits in log2 units relative to the stabiliser (one multiply-add), with mask; the stabiliser
        // ignores the counts: exp(s - m) <= 1 either way
        const bool need_mask = (j0 < 0) || (j0 + 31 > min(n - 1, a.causal ? n - a.Wq : n - 1));
        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four chains instead of one
        if (!need_mask) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            x[i] = fmaf(x[i], a.scale_log2, -m_stab);
            mx[i & 3] = fmaxf(mx[i & 3], x[i]);
          }
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float v = fmaf(x[i], a.scale_log2, -m_stab);
            x[i] = (j0 + i >= 0 && j0 + i <= last_vis) ? v : -INFINITY;
            mx[i & 3] = fmaxf(mx[i & 3], x[i]);
          }
        }
        atomicMax(&rmax[row], f2ord(fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]))));
      }
      // the one barrier of the tile: the row maxima and the staged counts are complete
      softmax_barrier();
      // the buffer of the tile after next was last read one tile ago: every thread is past that read now
      if (cg == 0) misc->rowmax[(li + 2) % 3][row] = kOrdNegInf;
      if (!alive) continue;
      // row maximum relative to the stabiliser: the stabiliser moves up by it when the row has none
      // yet or when the maximum has outgrown it by more than the gap
      const float mt = ord2f(rmax[row]);
      const bool need = mt > -INFINITY && (!have_stab || mt > kRescaleGap);
      const bool any_need = __any_sync(0xffffffffu, need && li > 0);
      // the previous tile's P V products must be done before P is overwritten: half by half, or
      // both before a rescale of O
      if (li > 0) {
        if (!(alive = warp_wait(&misc->ofull[0], (li - 1) & 1, abort_flag, lane))) continue;
        if (any_need && !(alive = warp_wait(&misc->ofull[1], (li - 1) & 1, abort_flag, lane))) continue;
        tc_fence_after();
      }
      const float f = (need && have_stab) ? fast_exp2(-mt) : 1.f;
      if (any_need) {
        if (cg == 0) {                                     // the row of O is rescaled once
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            float ov[32];
            tmem_ld32(tmem + lane_addr + 256 + c * 32, ov);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) ov[i] *= f;
            tmem_st32(tmem + lane_addr + 256 + c * 32, ov);
          }
          tmem_st_wait();
        }
        l *= f;
      }
      if (need) {
        m_stab += mt;
        have_stab = true;
#pragma unroll
        for (int i = 0; i < 32; ++i) x[i] -= mt;
      }
      // rows of the V tile outside the sequence may hold anything: each warp zeroes its share
      const int tile_row0 = (t_begin + li) * kTile - shift;
      if (tile_row0 < 0 || tile_row0 + kTile > n) {
        if (!(alive = warp_wait(&misc->vfull[s], k & 1, abort_flag, lane))) continue;
        uint8_t* vt = smem + kSmemStage + s * kStage + kOperand;
        for (int it = threadIdx.x - 64; it < kTile * 16; it += kSoftmaxWarps * 32) {
          const int r = it >> 4, ch = it & 15;
          if (tile_row0 + r < 0 || tile_row0 + r >= n)
            *reinterpret_cast<uint4*>(vt + (ch >> 3) * kHalf + r * 128 + ((ch & 7) << 4)) = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async();                               // the tensor core reads these rows
      }
      // P' = exp2(x - m) as hi + lo bf16, two slots per 32-bit column, written over the logits of
      // this buffer (every warp has read its logits: the barrier above) as the A operand of P' V:
      // hi in columns 0-63, lo in columns 64-127.  The hi term is the value cut to bf16 (a byte
      // permute, no conversion); the lo term rounds the exact remainder, so hi + lo carries 16
      // significant bits.
      float ls[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        if (hf == 1 && li > 0 && !any_need) {
          if (!(alive = warp_wait(&misc->ofull[1], (li - 1) & 1, abort_flag, lane))) break;
        }
        uint32_t hi[8], lo[8];
#pragma unroll
        for (int c = 2 * hf; c < 2 * hf + 2; ++c) {
          const float4 ca = *reinterpret_cast<const float4*>(&cnt[cg * 32 + c * 8]);
          const float4 cb = *reinterpret_cast<const float4*>(&cnt[cg * 32 + c * 8 + 4]);
          const float cc[8] = {ca.x, ca.y, ca.z, ca.w, cb.x, cb.y, cb.z, cb.w};
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int i = c * 8 + u * 2;
            const float q0 = fast_exp2(x[i]), q1 = fast_exp2(x[i + 1]);
            ls[u] = fmaf(cc[2 * u], q0, fmaf(cc[2 * u + 1], q1, ls[u]));
            const uint32_t b0 = __float_as_uint(q0), b1 = __float_as_uint(q1);
            hi[(c & 1) * 4 + u] = __byte_perm(b0, b1, 0x7632);
            lo[(c & 1) * 4 + u] = pack_bf16(q0 - __uint_as_float(b0 & 0xffff0000u), q1 - __uint_as_float(b1 & 0xffff0000u));
          }
        }
        tmem_st8(tmem + lane_addr + s * 128 + cg * 16 + hf * 8, hi);
        tmem_st8(tmem + lane_addr + s * 128 + 64 + cg * 16 + hf * 8, lo);
        tmem_st_wait();
        tc_fence_before();
        warp_arrive(&misc->pready[hf], lane);
      }
      if (!alive) continue;
      l += (ls[0] + ls[1]) + (ls[2] + ls[3]);
    }
    // ---- the partial of this key range: the four column groups of a row add their sums, then each
    //      writes 32 channels of the row of O
    softmax_barrier();                                            // row maxima and counts are dead now
    misc->lsum[cg][row] = l;
    softmax_barrier();
    if (alive && warp_wait(&misc->ofull[0], (my_tiles - 1) & 1, abort_flag, lane) &&
        warp_wait(&misc->ofull[1], (my_tiles - 1) & 1, abort_flag, lane)) {
      tc_fence_after();
      const size_t pidx = ((size_t)unit * a.splits + split) * a.M + m;
      if (cg == 0 && m < a.M)
        a.part_ml[pidx] = make_float2(have_stab ? m_stab : -INFINITY, (misc->lsum[0][row] + misc->lsum[1][row]) + (misc->lsum[2][row] + misc->lsum[3][row]));
      float ov[32];
      tmem_ld32(tmem + lane_addr + 256 + cg * 32, ov);
      tmem_ld_wait();
      if (m < a.M) {
        float4* po = reinterpret_cast<float4*>(a.part_o + pidx * KVS_D + cg * 32);
#pragma unroll
        for (int i = 0; i < 8; ++i) po[i] = make_float4(ov[4 * i], ov[4 * i + 1], ov[4 * i + 2], ov[4 * i + 3]);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
  if (threadIdx.x == 0 && misc->abort_flag && a.status_dev) atomicExch(a.status_dev, (int)KVS_ERR_TIMEOUT);
}

}  // namespace

cudaError_t kvs_launch_flash_tc(const FlashTcArgs& a, const RoundTable& t, const CUtensorMap& tmK,
                                const CUtensorMap& tmV, const CUtensorMap& tmQ, cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(flash_partial_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  dim3 grid(a.nqblk * a.splits, a.Hkv, t.nseq);
  flash_partial_tc<<<grid, kThreads, kSmemBytes, st>>>(a, t, tmK, tmV, tmQ);
  return cudaGetLastError();
}
