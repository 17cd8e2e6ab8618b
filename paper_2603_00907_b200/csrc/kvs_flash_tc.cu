// Attention partials on the tensor cores (tcgen05 + TMEM + TMA), queries on TMEM lanes.
//
// One CTA owns a block of 128 query rows (Q is staged once in shared memory) and a contiguous range
// of 128-slot tiles.  K and V tiles travel in two separate two-stage TMA rings; per tile one
// thread issues
//   S[q, slot] = Q K_tile^T                         (fp32 in TMEM, three buffers: the logits run two tiles
//                                                    ahead of the P V products, so that a softmax team that
//                                                    has finished a tile finds its next one already formed)
// Two teams of eight softmax warps take alternate tiles, so that one team's arithmetic overlaps
// the other team's waits.  Inside a team the two warps of a TMEM lane quarter own the same 32
// query rows and 64 slot columns each.  A thread reads its logits twice: once for the maximum
// (the two threads of a row show each other their maxima through shared memory),
// once to form P' = exp(s - m), split into two bf16 terms and stored back into the very columns
// the thread's logits came from (32 logits make 16 columns of hi and 16 of lo terms), keeping
// its part of l = sum_j c_j exp(s_j - m): the count bias ln c_j of a merged slot is just the
// factor c_j in that sum.  The stabiliser m of a row is one value for the whole CTA: it lives in
// shared memory, is decided tile by tile in tile order (each team waits for the other team's
// decision on the tile before) and only moves when the maximum has outgrown it by more than 2^8;
// the team that moves it rescales the row of O, and every thread brings its own part of l along
// when it next sees the new value.  The issuing thread then runs
//   O[q, :] += (P'_hi + P'_lo) Vsum_tile            (P' from tensor memory, V as the MN-major operand)
// with the one O accumulating in TMEM across all tiles [Eq. attn_def_vec with merged slots:
// o = sum_j alpha_j Vsum_j / c_j].  At the end the CTA writes (stabiliser, sum, O) as the partial
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
constexpr int kPvWarp = 2 + kSoftmaxWarps + kNormWarps;          // the warp that issues the P V products
constexpr int kThreads = (kPvWarp + 1) * 32;   // warp 0: TMA, 1: S products, 2-17: softmax, 18-21: pair norms, 22: P V products
constexpr float kRescaleGap = 8.f;         // log2 units
constexpr int kSBufs = 3;                  // logit / P' buffers in tensor memory

struct Misc {
  uint64_t kfull[2], vfull[2], kfree[2], vfree[2], sfull[kSBufs], pready[kSBufs][2], pvdone[kSBufs], ofull[2], stabdone[2], qfull;
  uint32_t tmem_base;
  int abort_flag, wait_us;                 // (adjacent: the bounded waits read both through one pointer)
  float rowmax[2][2][2][kTile];            // per team, tile parity, column half and query row: that thread's maximum logit
  alignas(16) float cnt[2][2][kTile];      // per team and tile parity: counts of the tile's slots (read as float4)
  float mstab[2][kTile];                   // per tile parity and query row: the stabiliser after that tile (-inf: none yet)
  float lsum[4][kTile];                    // the four parts of every row sum (team x column half)
};
constexpr int kSmemBytes = kSmemMisc + (int)sizeof(Misc);
static_assert(kSmemBytes <= 232448, "shared memory of one CTA");

constexpr uint32_t kColO = 384;                // TMEM columns: three logit buffers of 128, then O (128)

__device__ __forceinline__ void team_barrier(int team) { asm volatile("bar.sync %0, 256;" ::"r"(team + 1) : "memory"); }
__device__ __forceinline__ void softmax_barrier() { asm volatile("bar.sync 3, 512;" ::: "memory"); }

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
// |x_r|^2 and <x_l, x_r>, delivered to lanes 0-7 (and again to lanes 8-15).  The 16 rows are the
// A operand and, eight at a time, the B operand of small tensor-core products: the wanted values
// sit on and next to the diagonal of the 16 x 16 Gram matrix.  Every 8 x 8 fragment is eight
// consecutive rows, which the 128-byte swizzle spreads over all banks.
__device__ __forceinline__ void pair_dots8(const uint8_t* tile, int row0, int lane, float& ll, float& rr, float& lr) {
  const uint32_t base = smem_u32(tile);
  const int mtx = lane >> 3, rin = lane & 7;                // ldmatrix: this lane feeds row rin of matrix mtx
  const int row = row0 + (mtx & 1) * 8 + rin;               // matrices 0,2: rows 0-7; 1,3: rows 8-15
  uint32_t fr[8][4];
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    const int chunk = 2 * (kk & 3) + (mtx >> 1);            // 16-byte chunk inside the 128-byte row
    ldmatrix_x4(fr[kk], base + (kk >> 2) * kHalf + row * 128 + ((chunk ^ (row & 7)) << 4));
  }
  float d1[4] = {0.f, 0.f, 0.f, 0.f}, d2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    mma16816(d1, fr[kk], fr[kk][0], fr[kk][2]);             // columns = rows 0-7
    mma16816(d2, fr[kk], fr[kk][1], fr[kk][3]);             // columns = rows 8-15
  }
  // lane 4 g + t holds rows g and g + 8, columns 2 t and 2 t + 1.  Pair q < 4 (rows 2q, 2q+1, first
  // product): lane 9 q has <l,l> and <l,r>, lane 9 q + 4 has <r,r>; pair 4 + q the same lanes, in
  // the lower half of the second product.
  const int q = lane & 3, srcl = 9 * q, srcr = 9 * q + 4;
  const bool upper = (lane & 4) != 0;
  const float ll1 = __shfl_sync(0xffffffffu, d1[0], srcl), ll2 = __shfl_sync(0xffffffffu, d2[2], srcl);
  const float lr1 = __shfl_sync(0xffffffffu, d1[1], srcl), lr2 = __shfl_sync(0xffffffffu, d2[3], srcl);
  const float rr1 = __shfl_sync(0xffffffffu, d1[1], srcr), rr2 = __shfl_sync(0xffffffffu, d2[3], srcr);
  ll = upper ? ll2 : ll1;
  lr = upper ? lr2 : lr1;
  rr = upper ? rr2 : rr1;
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
  // (read from one lane, so that the compiler knows the warp index and all that follows from it
  // -- roles, TMEM and barrier addresses -- to be the same in every lane)
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  // with pair norms, tile t covers slots [128 t - shift, 128 t - shift + 128): aligned with the pairs
  const int shift = a.pair_norms ? (tab.off & 1) : 0;
  const int ntiles = (n + shift + kTile - 1) / kTile;
  const int t_begin = min(ntiles, split * a.tiles_per_split);
  const int t_end = min(ntiles, t_begin + a.tiles_per_split);
  const int my_tiles = t_end - t_begin;
  kvs_pdl_launch_dependents();
  if (n <= 0) { kvs_pdl_wait(); return; }
  if (smem_u32(smem) & 1023u) {                        // the swizzled tiles need a 1024-byte aligned base
    kvs_pdl_wait();
    if (threadIdx.x == 0 && a.status_dev) atomicExch(a.status_dev, (int)KVS_ERR_CUDA);
    return;
  }
  if (my_tiles <= 0) {
    kvs_pdl_wait();
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
      mbar_init(&misc->stabdone[s], kSoftmaxWarps / 2);
      mbar_init(&misc->ofull[s], 1);
    }
    for (int b = 0; b < kSBufs; ++b) {
      mbar_init(&misc->sfull[b], 1);
      mbar_init(&misc->pvdone[b], 1);
      // P' is handed over in two halves (the last and the first 32 slots of every thread's 64), so
      // that the P V products of one half run while the other half is still being written
      for (int hf = 0; hf < 2; ++hf) mbar_init(&misc->pready[b][hf], kSoftmaxWarps / 2);
    }
    mbar_init(&misc->qfull, 1);
    misc->abort_flag = 0;
    misc->wait_us = (int)a.wait_us;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(&misc->tmem_base, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // (everything above runs while the kernel before this one may still be draining)
  kvs_pdl_wait();
  const uint32_t tmem = __shfl_sync(0xffffffffu, misc->tmem_base, 0);   // (uniform for the compiler too)
  volatile int* abort_flag = &misc->abort_flag;
  // test hook: the producer requests no K tile, so that the waits on them run out
  const bool withhold_k = (a.debug_stall & 1u) != 0;

  if (warp == 0) {
    // ================================================================ TMA producer
    // one thread streams both rings.  Stages come free in a fixed order (the logits of tile t + 1 are
    // queued before the P V products of tile t), so the thread sleeps on one barrier at a time:
    // K(0), K(1), V(0), K(2), V(1), ...
    if (elect_one()) {
      prefetch_tmap(&tmK); prefetch_tmap(&tmV); prefetch_tmap(&tmQ);
      mbar_expect_tx(&misc->qfull, kOperand);
      for (int hf = 0; hf < 2; ++hf)
        tma_load_3d(smem + kSmemQ + hf * kHalf, &tmQ, &misc->qfull, hf * 64, qblk * 128, unit);
      int kli = 0, vli = 0;
      auto load_k = [&]() -> bool {
        const int s = kli & 1;
        if (!mbar_wait(&misc->kfree[s], ((kli >> 1) & 1) ^ 1, abort_flag)) return false;
        uint8_t* st = smem + kSmemStage + s * kStage;
        const int row = (t_begin + kli) * kTile - shift;
        if (!withhold_k) {
          mbar_expect_tx(&misc->kfull[s], kOperand);
          for (int hf = 0; hf < 2; ++hf) tma_load_4d(st + hf * kHalf, &tmK, &misc->kfull[s], hf * 64, row, h, sr.b);
        }
        ++kli;
        return true;
      };
      auto load_v = [&]() -> bool {
        const int s = vli & 1;
        if (!mbar_wait(&misc->vfree[s], ((vli >> 1) & 1) ^ 1, abort_flag)) return false;
        uint8_t* st = smem + kSmemStage + s * kStage + kOperand;
        const int row = (t_begin + vli) * kTile - shift;
        mbar_expect_tx(&misc->vfull[s], kOperand);
        for (int hf = 0; hf < 2; ++hf) tma_load_4d(st + hf * kHalf, &tmV, &misc->vfull[s], hf * 64, row, h, sr.b);
        ++vli;
        return true;
      };
      bool ok = load_k();
      while (ok && vli < my_tiles) {
        if (kli < my_tiles) ok = load_k();
        if (ok) ok = load_v();
      }
      if (*abort_flag) {
        // drain: give the copies already issued a bounded time to land before the CTA leaves
        for (int li = max(0, kli - 2); li < kli && !withhold_k; ++li) mbar_drain(&misc->kfull[li & 1], (li >> 1) & 1);
        for (int li = max(0, vli - 2); li < vli; ++li) mbar_drain(&misc->vfull[li & 1], (li >> 1) & 1);
      }
    }
  } else if (warp == 1) {
    // ================================================================ issuer of the S products
    // Two threads in two warps feed the tensor pipe, one the logits and one the P V products: a
    // single thread needed 110-125 cycles per product here (it shares its scheduler with four busy
    // softmax warps; its loop was guarded by `lane == 0` then), the pipe 64, and the softmax teams
    // waited for their logits.  Choosing the lane with elect.sync was worth another 3 %.
    if (elect_one()) {
      constexpr uint32_t idesc_s = idesc_bf16(128, 128);                 // Q (K-major) x K tile (K-major)
      const uint64_t qd0 = smem_desc_sw128(smem_u32(smem + kSmemQ), 16, 1024);
      const uint64_t kd0 = smem_desc_sw128(smem_u32(smem + kSmemStage), 16, 1024);
      const uint32_t kd_hi = (uint32_t)(kd0 >> 32), qd_lo = (uint32_t)qd0, kd_lo0 = (uint32_t)kd0;   // stage 1 is kStage / 16 further
      // The logits of tile li go to buffer li mod 3, which last held P' of tile li - 3: its P V products
      // must be complete (pvdone).  With three buffers the logits run up to three tiles ahead, so that a
      // softmax team that has finished a tile finds the logits of its next one already formed.
      bool ok = mbar_wait(&misc->qfull, 0, abort_flag);
      for (int li = 0; ok && li < my_tiles; ++li) {
        const int s = li & 1, k = li >> 1;                 // K stage and its use count
        const int b = li % kSBufs, u = li / kSBufs;        // logit buffer and its use count
        if (u > 0 && !mbar_wait(&misc->pvdone[b], (u - 1) & 1, abort_flag)) break;
        if (!mbar_wait(&misc->kfull[s], k & 1, abort_flag)) break;
        tc_fence_after();
        const uint32_t kd_lo = kd_lo0 + s * (kStage >> 4), ds = tmem + (uint32_t)b * 128;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t o = ((kk >> 2) * kHalf + (kk & 3) * 32) >> 4;
          if (kk == 0) umma_ss<false>(ds, qd_lo, kd_hi, kd_lo, kd_hi, idesc_s);
          else umma_ss<true>(ds, qd_lo + o, kd_hi, kd_lo + o, kd_hi, idesc_s);
        }
        tc_commit(&misc->sfull[b]);
        tc_commit(&misc->kfree[s]);
      }
    }
  } else if (warp == kPvWarp) {
    // ================================================================ issuer of the P V products
    if (elect_one()) {
      constexpr uint32_t idesc_o = idesc_bf16(128, 128, false, true);    // P' (K-major) x V tile (MN-major)
      const uint64_t vd0 = smem_desc_sw128(smem_u32(smem + kSmemStage + kOperand), kHalf, 1024);
      const uint32_t vd_hi = (uint32_t)(vd0 >> 32), vd_lo0 = (uint32_t)vd0;
      bool ok = true;
      for (int li = 0; ok && li < my_tiles; ++li) {
        const int s = li & 1, ph = (li >> 1) & 1;          // V stage and its phase
        const int b = li % kSBufs, bph = (li / kSBufs) & 1; // P' buffer and its phase
        if (!mbar_wait(&misc->vfull[s], ph, abort_flag)) ok = false;
        const uint32_t vd_lo = vd_lo0 + s * (kStage >> 4), ps = tmem + (uint32_t)b * 128;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          if (ok && !mbar_wait(&misc->pready[b][hf], bph, abort_flag)) ok = false;
          if (!ok) break;
          tc_fence_after();
          const int sub = 1 - hf;                            // the last 32 slots of a thread's 64 come first
#pragma unroll
          for (int c4 = 0; c4 < 4; ++c4) {
            const int ch = c4 >> 1, k2 = c4 & 1;
            const int kk = 4 * ch + 2 * sub + k2;            // 16-slot step of the tile: slots [16 kk, 16 kk + 16)
#pragma unroll
            for (int hl = 0; hl < 2; ++hl) {
              // A: 16 slots = 8 columns of hi (or, 16 columns further, lo) terms inside the owner's
              // 64 logit columns; B: 16 slots = two 8-row groups of V
              const uint32_t ap = ps + 64 * ch + 32 * sub + 16 * hl + 8 * k2;
              const uint32_t bl = vd_lo + ((kk * 16 * 128) >> 4);
              if (hf == 0 && c4 == 0 && hl == 0) umma_bf16_ts(tmem + kColO, ap, ((uint64_t)vd_hi << 32) | bl, idesc_o, li > 0 ? 1u : 0u);
              else umma_ts<true>(tmem + kColO, ap, bl, vd_hi, idesc_o);
            }
          }
        }
        if (ok) {
          tc_commit(&misc->ofull[s]);
          tc_commit(&misc->vfree[s]);
          tc_commit(&misc->pvdone[b]);
        }
      }
    }
  } else if (warp >= 2 + kSoftmaxWarps) {
    // ================================================================ pair-norm warps (18-21)
    if (norm_k || norm_v) {
      const int nw = warp - (2 + kSoftmaxWarps);                 // rows [32 nw, 32 nw + 32) of every tile
      const int off = tab.off;
      const int32_t* Cn = a.counts + (size_t)unit * a.n_max;
      const int pl = lane & 15;                                  // lanes 0-15 own the warp's 16 pairs
      // counts of the next tile's pair travel while the current tile is processed
      int cl_next = 1, cr_next = 1;
      if (norm_v) {
        const int sl = t_begin * kTile - shift + nw * 32 + 2 * pl;
        if (sl >= off && ((sl - off) >> 1) < sr.P) { cl_next = ldg_here(Cn + sl); cr_next = ldg_here(Cn + sl + 1); }
      }
      for (int li = 0; li < my_tiles; ++li) {
        const int s = li & 1, k = li >> 1;
        const int slot_l = (t_begin + li) * kTile - shift + nw * 32 + 2 * pl;   // left slot of this lane's pair
        const int p = (slot_l - off) >> 1;
        const bool pair_ok = lane < 16 && slot_l >= off && p < sr.P;
        const int cl = cl_next, cr = cr_next;
        if (norm_v && li + 1 < my_tiles) {
          const int sl = slot_l + kTile;
          cl_next = cr_next = 1;
          if (sl >= off && ((sl - off) >> 1) < sr.P) { cl_next = ldg_here(Cn + sl); cr_next = ldg_here(Cn + sl + 1); }
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
            const float icl = 1.f / (float)cl, icr = 1.f / (float)cr;
            const float r2l = vll * icl * icl, r2r = vrr * icr * icr;
            out[0] = r2l; out[1] = r2r; out[2] = r2l + r2r + 2.f * vlr * icl * icr;
          }
        }
      }
    }
  } else {
    // ================================================================ softmax warps
    const int team = (warp - 2) >> 3;                     // takes tiles li = team, team + 2, ...
    const int ch = ((warp - 2) >> 2) & 1;                 // 64-slot column half of the tile
    const int row = (warp & 3) * 32 + lane;               // TMEM lane = query row in the block
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const int m = qblk * 128 + row;
    const int last_vis = a.causal ? (n - a.Wq + (m % a.Wq)) : (n - 1);
    const int last_free = min(n - 1, a.causal ? n - a.Wq : n - 1);   // slots up to here need no mask
    const int32_t* Cb = a.counts + (size_t)unit * a.n_max;
    const int team_tiles = (my_tiles - team + 1) / 2;
    // The stabiliser (log2 units) this thread's logits and its part of l refer to.  Until the row
    // has seen a visible slot there is none (-inf in shared memory) and 0 stands in for it, which
    // keeps the arithmetic finite.
    float m_stab = 0.f, l = 0.f;
    bool have_stab = false;
    bool alive = true;
    // (first column half) the count of slot `row` of the team's next tile travels meanwhile
    int cnt_next = 1;
    if (ch == 0 && team_tiles > 0) {
      const int jj = (t_begin + team) * kTile - shift + row;
      if (jj >= 0 && jj < n) cnt_next = ldg_here(Cb + jj);
    }
    // logits of 32 columns, relative to the stabiliser (one multiply-add), masked where needed
    auto scale32 = [&](int j0, float* x) {
      if (j0 >= 0 && j0 + 31 <= last_free) {
        // (two columns per instruction: the softmax warps are bound by issue slots)
        const float2 sc2 = make_float2(a.scale_log2, a.scale_log2), nm2 = make_float2(-m_stab, -m_stab);
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float2 v = __ffma2_rn(make_float2(x[i], x[i + 1]), sc2, nm2);
          x[i] = v.x; x[i + 1] = v.y;
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i)
          x[i] = (j0 + i >= 0 && j0 + i <= last_vis) ? fmaf(x[i], a.scale_log2, -m_stab) : -INFINITY;
      }
    };
    auto load32 = [&](uint32_t col, int j0, float* x) {
      tmem_ld32(col, x);
      tmem_ld_wait();
      scale32(j0, x);
    };
    auto max32 = [&](const float* x) {
      float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four chains instead of one
#pragma unroll
      for (int i = 0; i < 32; ++i) mx[i & 3] = fmaxf(mx[i & 3], x[i]);
      return fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
    };
    // P' = exp2(x) of 32 slots as hi + lo bf16, two slots per 32-bit column, stored over the first
    // 16 (hi) and the last 16 (lo) of the 32 columns the logits were read from.  The hi term is the
    // value cut to bf16 (a byte permute, no conversion); the lo term rounds the exact remainder, so
    // hi + lo carries 16 significant bits.  Returns sum_j c_j P'_j.
    auto emit32 = [&](uint32_t col, const float* x, const float* cnt32) {
      float2 ls[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
      for (int c = 0; c < 4; c += 2) {
        uint32_t hi[8], lo[8];
#pragma unroll
        for (int c2 = c; c2 < c + 2; ++c2) {
          const float4 ca = *reinterpret_cast<const float4*>(&cnt32[c2 * 8]);
          const float4 cb = *reinterpret_cast<const float4*>(&cnt32[c2 * 8 + 4]);
          const float2 cc[4] = {make_float2(ca.x, ca.y), make_float2(ca.z, ca.w), make_float2(cb.x, cb.y), make_float2(cb.z, cb.w)};
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const int i = c2 * 8 + u * 2;
            const float2 q = make_float2(fast_exp2(x[i]), fast_exp2(x[i + 1]));
            ls[u] = __ffma2_rn(cc[u], q, ls[u]);                     // (two slots per instruction)
            const uint32_t b0 = __float_as_uint(q.x), b1 = __float_as_uint(q.y);
            hi[(c2 & 1) * 4 + u] = __byte_perm(b0, b1, 0x7632);
            const float2 r = __fadd2_rn(q, make_float2(-__uint_as_float(b0 & 0xffff0000u), -__uint_as_float(b1 & 0xffff0000u)));
            lo[(c2 & 1) * 4 + u] = pack_bf16(r.x, r.y);
          }
        }
        tmem_st8(col + (c >> 1) * 8, hi);
        tmem_st8(col + 16 + (c >> 1) * 8, lo);
      }
      tmem_st_wait();
      return ((ls[0].x + ls[0].y) + (ls[1].x + ls[1].y)) + ((ls[2].x + ls[2].y) + (ls[3].x + ls[3].y));
    };
    for (int j = 0; j < team_tiles; ++j) {
      const int li = 2 * j + team;
      const int s = li & 1, b = li % kSBufs, ph = (li / kSBufs) & 1;   // K/V stage, logit buffer and its phase
      const uint32_t scol = tmem + lane_addr + b * 128 + ch * 64;   // this thread's 64 logit columns
      const int tile_row0 = (t_begin + li) * kTile - shift;
      const int jA = tile_row0 + ch * 64, jB = jA + 32;    // first slots of this thread's two column groups
      float* cnt = misc->cnt[team][j & 1];
      float (*rmax)[kTile] = misc->rowmax[team][j & 1];   // (the other parity may still be read by a slow partner)
      if (ch == 0) {
        cnt[row] = (float)cnt_next;
        const int jj = tile_row0 + 2 * kTile + row;
        cnt_next = 1;
        if (j + 1 < team_tiles && jj >= 0 && jj < n) cnt_next = ldg_here(Cb + jj);
      }
      float x[32];
      if (alive) alive = warp_wait(&misc->sfull[b], ph, abort_flag, lane);
      if (alive) {
        tc_fence_after();
        float mx;
        {
          float xa[32];
          tmem_ld32(scol, xa);
          tmem_ld_wait();
          tmem_ld32(scol + 32, x);                         // in flight while the first 32 are reduced
          scale32(jA, xa);
          mx = max32(xa);
        }
        tmem_ld_wait();
        scale32(jB, x);                                    // these stay in registers: they are exponentiated first
        mx = fmaxf(mx, max32(x));
        rmax[ch][row] = mx;
      }
      // the one barrier of the tile: the row maxima and the staged counts of the team are complete
      team_barrier(team);
      // ---- the stabiliser after this tile, from the one after the tile before (the other team's decision)
      float m_prev = -INFINITY;
      if (li > 0) {
        if (alive) alive = warp_wait(&misc->stabdone[team ^ 1], ((li - 1) >> 1) & 1, abort_flag, lane);
        m_prev = misc->mstab[(li - 1) & 1][row];
      }
      // row maximum of the tile: it becomes the stabiliser when the row has none yet or when it
      // has outgrown the stabiliser by more than the gap
      const float mt = alive ? fmaxf(rmax[0][row], rmax[1][row]) + m_stab : -INFINITY;
      const bool need = mt > -INFINITY && (m_prev == -INFINITY || mt - m_prev > kRescaleGap);
      const float m_new = need ? mt : m_prev;
      if (ch == 0) misc->mstab[li & 1][row] = m_new;
      warp_arrive(&misc->stabdone[team], lane);            // also when this warp has given up: the other team waits for it
      if (!alive) continue;
      const bool rescale = need && m_prev > -INFINITY;
      if (__any_sync(0xffffffffu, rescale)) {
        // all earlier P V products must be done before O is touched
        if (!(alive = warp_wait(&misc->ofull[(li - 1) & 1], ((li - 1) >> 1) & 1, abort_flag, lane))) continue;
        tc_fence_after();
        if (ch == 0) {                                     // the row of O is rescaled once
          const float f = rescale ? fast_exp2(m_prev - m_new) : 1.f;
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            float ov[32];
            tmem_ld32(tmem + lane_addr + kColO + c * 32, ov);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) ov[i] *= f;
            tmem_st32(tmem + lane_addr + kColO + c * 32, ov);
          }
          tmem_st_wait();
        }
      }
      // this thread's logits and its part of l follow (the stabiliser may have moved one tile ago too)
      const float m_eff = m_new > -INFINITY ? m_new : 0.f;
      if (m_eff != m_stab) {
        const float d = m_eff - m_stab;
        if (have_stab) l *= fast_exp2(-d);                 // (without one, l is still 0 and d may be anything)
        m_stab = m_eff;
#pragma unroll
        for (int i = 0; i < 32; ++i) x[i] -= d;
      }
      have_stab = m_new > -INFINITY;
      // rows of the V tile outside the sequence may hold anything: the team zeroes them
      if (tile_row0 < 0 || tile_row0 + kTile > n) {
        if (!(alive = warp_wait(&misc->vfull[s], (li >> 1) & 1, abort_flag, lane))) continue;
        uint8_t* vt = smem + kSmemStage + s * kStage + kOperand;
        for (int it = (threadIdx.x - 64) & 255; it < kTile * 16; it += 256) {
          const int r = it >> 4, c16 = it & 15;
          if (tile_row0 + r < 0 || tile_row0 + r >= n)
            *reinterpret_cast<uint4*>(vt + (c16 >> 3) * kHalf + r * 128 + ((c16 & 7) << 4)) = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async();                               // the tensor core reads these rows
      }
      // the last 32 slots first (their logits are still in registers), then the first 32 again from TMEM
      // (one copy of the exponentiation code, run twice, keeps the four roles' code within the instruction cache)
#pragma unroll 1
      for (int hf = 0; hf < 2; ++hf) {
        const int o32 = hf == 0 ? 32 : 0;
        if (hf == 1) load32(scol, jA, x);
        l += emit32(scol + o32, x, cnt + ch * 64 + o32);
        tc_fence_before();
        warp_arrive(&misc->pready[b][hf], lane);
      }
    }
    // ---- the partial of this key range: every thread brings its part of l to the final stabiliser,
    //      the four parts of a row are added, and each thread writes 32 channels of the row of O
    softmax_barrier();                                     // the last tile's stabiliser is in place
    const float m_fin = misc->mstab[(my_tiles - 1) & 1][row];
    const int part = team * 2 + ch;
    misc->lsum[part][row] = have_stab ? l * fast_exp2(m_stab - m_fin) : 0.f;
    softmax_barrier();
    const size_t pidx = ((size_t)unit * a.splits + split) * a.M + m;
    if (alive && warp_wait(&misc->ofull[(my_tiles - 1) & 1], ((my_tiles - 1) >> 1) & 1, abort_flag, lane)) {
      tc_fence_after();
      if (part == 0 && m < a.M)
        a.part_ml[pidx] = make_float2(m_fin, (misc->lsum[0][row] + misc->lsum[1][row]) + (misc->lsum[2][row] + misc->lsum[3][row]));
      float ov[32];
      tmem_ld32(tmem + lane_addr + kColO + part * 32, ov);
      tmem_ld_wait();
      if (m < a.M) {
        float4* po = reinterpret_cast<float4*>(a.part_o + pidx * KVS_D + part * 32);
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
  static KvsPerDeviceOnce configured;
  cudaError_t ce = configured.run([] {
    return cudaFuncSetAttribute(flash_partial_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  });
  if (ce != cudaSuccess) return ce;
  dim3 grid(a.nqblk * a.splits, a.Hkv, t.nseq);
  return kvs_launch_chained(flash_partial_tc, grid, dim3(kThreads), kSmemBytes, st, a, t, tmK, tmV, tmQ);
}
