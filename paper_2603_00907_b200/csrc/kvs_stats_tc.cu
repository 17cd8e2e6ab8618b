// Hessian statistics on the tensor cores (tcgen05 + TMEM + TMA), keys on TMEM lanes.
//
// One CTA owns a block of 128 window queries (Q, and the attention output O split into two
// bf16 terms, stay in shared memory) and walks a range of 128-slot tiles of the candidate
// region.  For every tile, TMA brings the K and V rows, and one thread issues
//   S^T[slot, q] = K_tile Q^T                      (logits, fp32 in TMEM)
//   T^T[slot, q] = Vsum_tile (O_hi + O_lo)^T       (value/output inner products)
// Two groups of four warps alternate over the tiles.  Each thread owns one TMEM lane = one
// cache slot, reads its row of S and T, and reduces over the queries, in registers,
//   A_j   = sum_q alpha_qj
//   N1_j  = sum_q alpha |1 - 2 alpha| |vbar_j - o_q|                    [Eqs. c11_def, c22_def]
//   N12_p = sum_q alpha_j alpha_j+1 |vbar_j + vbar_j+1 - 2 o_q|         [Eq. c12_def]
// with |vbar_j - o_q|^2 = |vbar_j|^2 - 2 T_jq / c_j + |o_q|^2.  The probability matrix never
// leaves the SM.  The two members of a candidate pair sit in adjacent lanes and exchange
// alpha and T by shuffle.  Query blocks of one tile are summed by the last block to arrive,
// in block order, which then forms cosine, score and the merge weight of Eq. kstar_final.
#include "kvs_internal.h"
#include "kvs_sm100.cuh"

using namespace sm100;

namespace {

constexpr int kTile = 128;                 // slots per tile = TMEM lanes
constexpr int kQB = 128;                   // queries per block = accumulator columns
constexpr int kHalf = 16384;               // bytes of a [128 rows x 64 bf16] swizzled sub-tile
constexpr int kOperand = 2 * kHalf;        // a [128 x 128] bf16 operand
constexpr int kStage = 2 * kOperand;       // K tile + V tile
constexpr int kSmemQ = 0, kSmemOhi = kOperand, kSmemOlo = 2 * kOperand, kSmemStage = 3 * kOperand;
constexpr int kSmemMisc = kSmemStage + 2 * kStage;
constexpr int kThreads = 320;              // warp 0: TMA, warp 1: MMA, warps 2-9: statistics

struct Misc {
  uint64_t full[2], sfree[2], tfull[2], tfree[2], qfull;
  uint32_t tmem_base;
  int abort_flag;
  int last[2];
  int wg_fail[2];                          // sticky: a wait of this group ran out
  float2 qc[kQB];                          // per query: (max + log2 Z, |o|^2)
};
constexpr int kSmemBytes = kSmemMisc + (int)sizeof(Misc) + 1024;   // + slack to align the base

__device__ __forceinline__ void wg_barrier(int wg) {
  asm volatile("bar.sync %0, 128;" ::"r"(wg + 1) : "memory");
}

// Wait of a whole statistics group on one mbarrier phase.  One lane per warp polls; the
// four warps then agree through shared memory, so that either all 128 threads go on or all
// of them leave the tile loop (a thread that left alone would hang the others' barriers).
__device__ __forceinline__ bool wg_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                        volatile int* wg_fail, int wg, int lane) {
  int ok = 1;
  if (lane == 0) {
    ok = mbar_wait(bar, parity, abort_flag) ? 1 : 0;
    if (!ok) *wg_fail = 1;
  }
  __syncwarp();
  wg_barrier(wg);
  return *wg_fail == 0;
}

// aa, bb, ab dot products of two swizzled 128-element bf16 rows of one operand tile
__device__ __forceinline__ void row_dots(const uint8_t* tile, int ra, int rb, float& aa, float& bb, float& ab) {
  aa = bb = ab = 0.f;
#pragma unroll
  for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
    for (int c = 0; c < 8; ++c) {
      const uint4 xa = *reinterpret_cast<const uint4*>(tile + hf * kHalf + ra * 128 + ((c ^ (ra & 7)) << 4));
      const uint4 xb = *reinterpret_cast<const uint4*>(tile + hf * kHalf + rb * 128 + ((c ^ (rb & 7)) << 4));
      const uint32_t wa[4] = {xa.x, xa.y, xa.z, xa.w}, wb[4] = {xb.x, xb.y, xb.z, xb.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float a0 = bf16lo(wa[i]), a1 = bf16hi(wa[i]), b0 = bf16lo(wb[i]), b1 = bf16hi(wb[i]);
        aa = fmaf(a0, a0, aa); aa = fmaf(a1, a1, aa);
        bb = fmaf(b0, b0, bb); bb = fmaf(b1, b1, bb);
        ab = fmaf(a0, b0, ab); ab = fmaf(a1, b1, ab);
      }
    }
  }
}

__device__ __forceinline__ void finalize_pair(const StatsTcArgs& a, size_t pi, float Aj, float Ap, float N1j,
                                              float N1p, float N12, float cosv) {
  const float mass = Aj + Ap;
  const float score = (a.score_mode == 0) ? mass * fmaxf(0.f, 1.f - cosv) : mass;
  const float D = N1j - 2.f * N12 + N1p;
  float w = 0.5f;
  if (D > 1e-6f * (N1j + N1p) && D < INFINITY) w = fminf(1.f, fmaxf(0.f, (N1j - N12) / D));
  a.score[pi] = fabsf(score);
  a.w[pi] = w;
  if (a.N12) a.N12[pi] = N12;
  if (a.cosv) a.cosv[pi] = cosv;
}

__global__ void __launch_bounds__(kThreads, 1)
hessian_stats_tc(const StatsTcArgs a, const RoundTable tab, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmQ,
                 const __grid_constant__ CUtensorMap tmOhi, const __grid_constant__ CUtensorMap tmOlo) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Misc* misc = reinterpret_cast<Misc*>(smem + kSmemMisc);

  const int seq = blockIdx.z;
  const SeqRound sr = tab.s[seq];
  const int h = blockIdx.y;
  const int qblk = blockIdx.x % a.nqblk;
  const int split = blockIdx.x / a.nqblk;
  const int unit = sr.b * a.Hkv + h;
  const int off = tab.off;
  const int P = sr.P;
  const int ntiles = (2 * P + kTile - 1) / kTile;
  const int t_begin = min(ntiles, split * a.tiles_per_split);
  const int t_end = min(ntiles, t_begin + a.tiles_per_split);
  if (sr.n <= 0 || t_begin >= t_end) return;          // uniform over the CTA
  const int my_tiles = t_end - t_begin;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&misc->full[s], 1);
      mbar_init(&misc->sfree[s], 2);     // MMA commit + statistics group
      mbar_init(&misc->tfull[s], 1);
      mbar_init(&misc->tfree[s], 1);
    }
    mbar_init(&misc->qfull, 1);
    misc->abort_flag = 0;
    misc->last[0] = misc->last[1] = 0;
    misc->wg_fail[0] = misc->wg_fail[1] = 0;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(&misc->tmem_base, 512);
  // per-query constants of this block: alpha = exp2(logit2 - (max + log2 Z))
  if (threadIdx.x >= 64 && threadIdx.x < 64 + kQB) {
    const int q = threadIdx.x - 64;
    const int m = qblk * kQB + q;
    float2 v = make_float2(INFINITY, 0.f);           // rows past M contribute alpha = 0
    if (m < a.M) {
      const float4 st = a.qstat[(size_t)unit * a.M + m];
      v = make_float2(st.x + log2f(st.y), st.z);
    }
    misc->qc[q] = v;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = misc->tmem_base;
  volatile int* abort_flag = &misc->abort_flag;

  if (warp == 0) {
    // ================================================================ TMA producer
    if (lane == 0) {
      prefetch_tmap(&tmK); prefetch_tmap(&tmV); prefetch_tmap(&tmQ); prefetch_tmap(&tmOhi); prefetch_tmap(&tmOlo);
      mbar_expect_tx(&misc->qfull, 3 * kOperand);
      for (int hf = 0; hf < 2; ++hf) {
        tma_load_3d(smem + kSmemQ + hf * kHalf, &tmQ, &misc->qfull, hf * 64, qblk * kQB, unit);
        tma_load_3d(smem + kSmemOhi + hf * kHalf, &tmOhi, &misc->qfull, hf * 64, qblk * kQB, unit);
        tma_load_3d(smem + kSmemOlo + hf * kHalf, &tmOlo, &misc->qfull, hf * 64, qblk * kQB, unit);
      }
      int issued = 0;
      for (int li = 0; li < my_tiles; ++li) {
        const int s = li & 1, k = li >> 1;
        if (!mbar_wait(&misc->sfree[s], (k & 1) ^ 1, abort_flag)) break;
        uint8_t* st = smem + kSmemStage + s * kStage;
        const int row = off + (t_begin + li) * kTile;
        mbar_expect_tx(&misc->full[s], kStage);
        for (int hf = 0; hf < 2; ++hf) {
          tma_load_4d(st + hf * kHalf, &tmK, &misc->full[s], hf * 64, row, h, sr.b);
          tma_load_4d(st + kOperand + hf * kHalf, &tmV, &misc->full[s], hf * 64, row, h, sr.b);
        }
        issued = li + 1;
      }
      if (*abort_flag) {
        // drain: give the copies already issued a bounded time to land before the CTA leaves
        for (int li = max(0, issued - 2); li < issued; ++li) {
          const uint64_t t0 = globaltimer_ns();
          while (!mbar_try_wait(&misc->full[li & 1], (li >> 1) & 1) && globaltimer_ns() - t0 < 200000000ull) {}
        }
      }
    }
  } else if (warp == 1) {
    // ================================================================ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16(kTile, kQB);
      const uint32_t q_addr = smem_u32(smem + kSmemQ), ohi_addr = smem_u32(smem + kSmemOhi),
                     olo_addr = smem_u32(smem + kSmemOlo);
      bool ok = mbar_wait(&misc->qfull, 0, abort_flag);
      for (int li = 0; ok && li < my_tiles; ++li) {
        const int s = li & 1, k = li >> 1;
        if (!mbar_wait(&misc->full[s], k & 1, abort_flag)) break;
        if (!mbar_wait(&misc->tfree[s], (k & 1) ^ 1, abort_flag)) break;
        tc_fence_after();
        const uint32_t k_addr = smem_u32(smem + kSmemStage + s * kStage);
        const uint32_t v_addr = k_addr + kOperand;
        const uint32_t dS = tmem + s * 256, dT = dS + 128;
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t o = (kk >> 2) * kHalf + (kk & 3) * 32;
          umma_bf16(dS, smem_desc_sw128(k_addr + o, 16, 1024), smem_desc_sw128(q_addr + o, 16, 1024), idesc, kk > 0);
        }
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t o = (kk >> 2) * kHalf + (kk & 3) * 32;
          umma_bf16(dT, smem_desc_sw128(v_addr + o, 16, 1024), smem_desc_sw128(ohi_addr + o, 16, 1024), idesc, kk > 0);
        }
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
          const uint32_t o = (kk >> 2) * kHalf + (kk & 3) * 32;
          umma_bf16(dT, smem_desc_sw128(v_addr + o, 16, 1024), smem_desc_sw128(olo_addr + o, 16, 1024), idesc, 1);
        }
        tc_commit(&misc->tfull[s]);
        tc_commit(&misc->sfree[s]);
      }
    }
  } else {
    // ================================================================ statistics warps
    const int wg = (warp - 2) >> 2;                       // tiles li = wg, wg + 2, ...
    const int lane_t = (warp & 3) * 32 + lane;            // TMEM lane = slot within the tile
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    const bool odd = lane_t & 1;
    const int32_t* Cb = a.counts + (size_t)unit * a.n_max;
    for (int li = wg; li < my_tiles; li += 2) {
      const int s = wg, k = li >> 1;
      const int tile = t_begin + li;
      const int j = off + tile * kTile + lane_t;          // this thread's slot
      const int p = (tile * kTile + lane_t) >> 1;         // its candidate pair
      const bool slot_ok = p < P;
      float cnt = 1.f;
      if (slot_ok) cnt = (float)Cb[j];
      const float invc = 1.f / cnt, lc2 = log2f(cnt);
      if (!wg_wait(&misc->full[s], k & 1, abort_flag, &misc->wg_fail[wg], wg, lane)) break;
      // ---- per-slot norms and pair dot products from the staged rows: even lanes take the
      //      K tile, odd lanes the V tile, both on the rows of their pair
      const uint8_t* st = smem + kSmemStage + s * kStage;
      float aa, bb, ab;
      row_dots(st + (odd ? kOperand : 0), lane_t & ~1, lane_t | 1, aa, bb, ab);
      // odd lane holds (|Vsum_even|^2, |Vsum_odd|^2, <Vsum_even, Vsum_odd>); even lane the K ones
      const float o_aa = __shfl_xor_sync(0xffffffffu, aa, 1);
      const float o_bb = __shfl_xor_sync(0xffffffffu, bb, 1);
      const float o_ab = __shfl_xor_sync(0xffffffffu, ab, 1);
      const float invc_p = __shfl_xor_sync(0xffffffffu, invc, 1);
      const float v2_own = odd ? bb : o_aa, v2_par = odd ? aa : o_bb, vv = odd ? ab : o_ab;
      const float k2e = odd ? o_aa : aa, k2o = odd ? o_bb : bb, kkp = odd ? o_ab : ab;
      const float r2 = v2_own * invc * invc;                         // |vbar_j|^2
      const float r2p = v2_par * invc_p * invc_p;
      const float pair_c = r2 + r2p + 2.f * vv * invc * invc_p;      // |vbar_j + vbar_j+1|^2
      const float cosv = kkp / fmaxf(sqrtf(k2e) * sqrtf(k2o), 1e-30f);
      wg_barrier(wg);
      if (lane_t == 0) mbar_arrive(&misc->sfree[s]);                 // staged rows no longer needed here

      if (!wg_wait(&misc->tfull[s], k & 1, abort_flag, &misc->wg_fail[wg], wg, lane)) break;
      tc_fence_after();
      float accA = 0.f, accN1 = 0.f, accN12 = 0.f;
#pragma unroll 1
      for (int c = 0; c < kQB / 32; ++c) {
        float sv[32], tv[32];
        tmem_ld32(tmem + lane_addr + s * 256 + c * 32, sv);
        tmem_ld32(tmem + lane_addr + s * 256 + 128 + c * 32, tv);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          const float2 c0 = misc->qc[c * 32 + i], c1 = misc->qc[c * 32 + i + 1];
          const float al0 = fast_exp2(fmaf(sv[i], a.scale_log2, lc2) - c0.x);
          const float al1 = fast_exp2(fmaf(sv[i + 1], a.scale_log2, lc2) - c1.x);
          const float T0 = tv[i] * invc, T1 = tv[i + 1] * invc;
          const float d0 = fmaxf(r2 - 2.f * T0 + c0.y, 0.f), d1 = fmaxf(r2 - 2.f * T1 + c1.y, 0.f);
          accA += al0 + al1;
          accN1 = fmaf(al0 * fabsf(1.f - 2.f * al0), sqrtf(d0), accN1);
          accN1 = fmaf(al1 * fabsf(1.f - 2.f * al1), sqrtf(d1), accN1);
          // pair term: the even lane takes query i, the odd lane query i + 1
          const float al_send = odd ? al0 : al1, T_send = odd ? T0 : T1;
          const float al_recv = __shfl_xor_sync(0xffffffffu, al_send, 1);
          const float T_recv = __shfl_xor_sync(0xffffffffu, T_send, 1);
          const float al_own = odd ? al1 : al0, T_own = odd ? T1 : T0, on2 = odd ? c1.y : c0.y;
          const float d12 = fmaxf(pair_c - 4.f * (T_own + T_recv) + 4.f * on2, 0.f);
          accN12 = fmaf(al_own * al_recv, sqrtf(d12), accN12);
        }
      }
      tc_fence_before();
      wg_barrier(wg);
      if (lane_t == 0) mbar_arrive(&misc->tfree[s]);                 // accumulators may be overwritten
      accN12 += __shfl_xor_sync(0xffffffffu, accN12, 1);

      // ---- outputs of this tile
      const size_t pi = (size_t)unit * a.pair_stride + p;
      if (a.nqblk == 1) {
        const float A_p = __shfl_xor_sync(0xffffffffu, accA, 1);
        const float N1_p = __shfl_xor_sync(0xffffffffu, accN1, 1);
        if (slot_ok) {
          if (a.A) a.A[(size_t)unit * a.n_max + j] = accA;
          if (a.N1) a.N1[(size_t)unit * a.n_max + j] = accN1;
          if (!odd) finalize_pair(a, pi, accA, A_p, accN1, N1_p, accN12, cosv);
        }
      } else {
        // partials of this query block, then the last block of the tile sums them in order
        const size_t slot_i = ((size_t)unit * a.nqblk + qblk) * a.n_max + (slot_ok ? j : 0);
        const size_t pair_i = ((size_t)unit * a.nqblk + qblk) * a.pair_stride + p;
        if (slot_ok) {
          a.partA[slot_i] = accA;
          a.partN1[slot_i] = accN1;
          if (!odd) {
            a.partN12[pair_i] = accN12;
            if (qblk == 0) a.partCos[pi] = cosv;
          }
        }
        __threadfence();
        wg_barrier(wg);
        if (lane_t == 0) {
          const uint32_t old = atomicAdd(&a.tile_counter[(size_t)unit * a.counter_stride + tile], 1u);
          misc->last[wg] = ((old + 1) % (uint32_t)a.nqblk) == 0;
        }
        wg_barrier(wg);
        if (misc->last[wg]) {
          __threadfence();
          float sA = 0.f, sN1 = 0.f, sN12 = 0.f, cs = 0.f;
          if (slot_ok) {
            for (int qb = 0; qb < a.nqblk; ++qb) {
              const size_t si = ((size_t)unit * a.nqblk + qb) * a.n_max + j;
              sA += __ldcg(a.partA + si);
              sN1 += __ldcg(a.partN1 + si);
              if (!odd) sN12 += __ldcg(a.partN12 + ((size_t)unit * a.nqblk + qb) * a.pair_stride + p);
            }
            if (!odd) cs = __ldcg(a.partCos + pi);
          }
          const float A_p = __shfl_xor_sync(0xffffffffu, sA, 1);
          const float N1_p = __shfl_xor_sync(0xffffffffu, sN1, 1);
          if (slot_ok) {
            if (a.A) a.A[(size_t)unit * a.n_max + j] = sA;
            if (a.N1) a.N1[(size_t)unit * a.n_max + j] = sN1;
            if (!odd) finalize_pair(a, pi, sA, A_p, sN1, N1_p, sN12, cs);
          }
        }
        wg_barrier(wg);     // misc->last[wg] is rewritten by the next tile
      }
    }
  }

  // ================================================================== common exit
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

cudaError_t kvs_launch_stats_tc(const StatsTcArgs& a, const RoundTable& t, const CUtensorMap& tmK,
                                const CUtensorMap& tmV, const CUtensorMap& tmQ, const CUtensorMap& tmOhi,
                                const CUtensorMap& tmOlo, cudaStream_t st) {
  static bool configured = false;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(hessian_stats_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  dim3 grid(a.nqblk * a.splits, a.Hkv, t.nseq);
  hessian_stats_tc<<<grid, kThreads, kSmemBytes, st>>>(a, t, tmK, tmV, tmQ, tmOhi, tmOlo);
  return cudaGetLastError();
}
