// Hessian statistics on the tensor cores (tcgen05 + TMEM + TMA), candidate pairs on TMEM lanes.
//
// One CTA owns a block of 128 window queries (Q, and the attention output O split into two
// bf16 terms, stay in shared memory) and walks a range of tiles of 128 candidate pairs.
// A 5-D view of the cache, [128, parity, slot/2, head, sequence], lets TMA bring the left
// members and the right members of the 128 pairs as two separate row tiles, so that TMEM
// lane p holds everything of pair p.  For each half of 64 queries
//   S_l = K_l Q^T, S_r = K_r Q^T                    (logits, fp32 in TMEM)
//   T_l = Vsum_l (O_hi + O_lo)^T, T_r likewise      (value/output inner products)
// go into one of two TMEM buffers; while the statistics warps reduce one half, the tensor
// core fills the other.  Two threads (in two warps, each chosen with elect.sync) issue the
// products, one the chains of the left members and one those of the right members: one thread
// alone measured 2 % slower.  Each statistics thread owns one pair
// and a share of the queries and reduces, in registers and with no cross-lane traffic,
//   A_j   = sum_q alpha_qj
//   N1_j  = sum_q alpha |1 - 2 alpha| |vbar_j - o_q|                    [Eqs. c11_def, c22_def]
//   N12_p = sum_q alpha_j alpha_j+1 |vbar_j + vbar_j+1 - 2 o_q|         [Eq. c12_def]
// with |vbar_j - o_q|^2 = |vbar_j|^2 - 2 T_jq / c_j + |o_q|^2.  The probability matrix never
// leaves the SM.  The row norms |vbar|^2, |vbar_l + vbar_r|^2 and the adjacent-key cosine of
// every pair come from the attention pass that precedes this kernel (it streams the same rows).
// Every (query block, statistics group) writes its five sums per pair as a partial; a small
// kernel adds the partials in a fixed order and forms score and the merge weight of
// Eq. kstar_final (deterministic, no atomics, no hand-over between warps inside the tile loop).
// A second instantiation serves the exact weight modes: a supplied loss gradient E (one row per
// window query) takes the place of the attention output in the T products, and the statistics
// warps sum the signed scalars g_ij = E^T c_ij instead of the norms [Section 4.2, text before
// Eq. h_rank1_unified; Eq. kstar_weight_final_rewrite].
// Every synchronisation is an mbarrier with a bounded wait, so a warp that gives up can never
// leave another one stuck.
#include "kvs_internal.h"
#include "kvs_sm100.cuh"

using namespace sm100;

namespace {

constexpr int kPairs = 128;                // candidate pairs per tile = TMEM lanes
constexpr int kQB = 128;                   // queries per CTA
constexpr int kQH = 64;                    // queries per accumulator half
constexpr int kHalf = 16384;               // bytes of a [128 rows x 64 bf16] swizzled sub-tile
constexpr int kOperand = 2 * kHalf;        // a [128 x 128] bf16 operand
constexpr int kSmemQ = 0, kSmemOhi = kOperand, kSmemOlo = 2 * kOperand;
constexpr int kSmemKl = 3 * kOperand, kSmemKr = 4 * kOperand, kSmemVl = 5 * kOperand, kSmemVr = 6 * kOperand;
constexpr int kSmemMisc = 7 * kOperand;
constexpr int kGroups = KVS_STATS_GROUPS;  // statistics groups: a group reduces a share of the queries of every half
constexpr int kChunk = 8;                  // queries per round of TMEM loads
constexpr bool kDoubleBuffer = kGroups < 4;   // the next chunk's loads in flight while one chunk is reduced
constexpr int kChunks = kQH / kChunk;      // chunks of a half, dealt out to the groups as evenly as they go
constexpr int kStatWarps = 4 * kGroups;
constexpr int kIssuers = 2;
constexpr int kFirstStat = 1 + kIssuers;   // warp 0: TMA, warps 1-2: product issuers, then the statistics warps
constexpr int kThreads = (kFirstStat + kStatWarps) * 32;
static_assert(KVS_STATS_GROUPS == kGroups, "the launcher sizes the partials with KVS_STATS_GROUPS");

struct Misc {
  uint64_t kfull, vfull, kfree, vfree, tfull[2], tfree[2], qfull;
  uint32_t tmem_base;
  int abort_flag, wait_us;                 // (adjacent: the bounded waits read both through one pointer)
  // per two queries (2k, 2k+1) of the block: (c_2k, c_2k+1, h_2k, h_2k+1) with c = -(max + log2 Z) and
  // h = |o|^2 (or <E, o>): neighbours sit side by side for the packed two-float arithmetic
  alignas(16) float qconst[2 * kQB];
};
constexpr int kSmemBytes = kSmemMisc + (int)sizeof(Misc);
static_assert(kSmemBytes <= 232448, "shared memory of one CTA");

// One lane waits, the warp follows.  (Polling in a tight loop instead of letting the hardware
// suspend the lane measured the same: the statistics warps' waits, about 250 cycles per half, are
// real waits for the tensor core, not wake-up latency.)
__device__ __forceinline__ bool warp_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int lane) {
  int ok = 1;
  if (lane == 0) ok = mbar_wait(bar, parity, abort_flag) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
__device__ __forceinline__ void warp_arrive(uint64_t* bar, int lane) {
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
}

__device__ __forceinline__ float fast_sqrt(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* v) {
  uint32_t r[8];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}

// kExact: a loss gradient E (one bf16 row per window query) takes the place of the attention
// output: T = Vsum E^T needs one product chain instead of two, and the statistics warps form the
// signed sums of g_ij = E^T c_ij instead of the norms (no square roots).
template <bool kExact>
__global__ void __launch_bounds__(kThreads, 1)
hessian_stats_tc(const StatsTcArgs a, const RoundTable tab, const __grid_constant__ CUtensorMap tmKp,
                 const __grid_constant__ CUtensorMap tmVp, const __grid_constant__ CUtensorMap tmQ,
                 const __grid_constant__ CUtensorMap tmOhi, const __grid_constant__ CUtensorMap tmOlo) {
  extern __shared__ __align__(1024) uint8_t smem[];
  Misc* misc = reinterpret_cast<Misc*>(smem + kSmemMisc);

  const int seq = blockIdx.z;
  const SeqRound sr = tab.s[seq];
  const int h = blockIdx.y;
  const int qblk = blockIdx.x % a.nqblk;
  const int split = blockIdx.x / a.nqblk;
  const int unit = sr.b * a.Hkv + h;
  const int off = tab.off;
  const int P = sr.P;
  const int ntiles = (P + kPairs - 1) / kPairs;
  const int t_begin = min(ntiles, split * a.tiles_per_split);
  const int t_end = min(ntiles, t_begin + a.tiles_per_split);
  kvs_pdl_launch_dependents();
  if (sr.n <= 0 || t_begin >= t_end) { kvs_pdl_wait(); return; }   // uniform over the CTA
  if (smem_u32(smem) & 1023u) {                        // the swizzled tiles need a 1024-byte aligned base
    kvs_pdl_wait();
    if (threadIdx.x == 0 && a.status_dev) atomicExch(a.status_dev, (int)KVS_ERR_CUDA);
    return;
  }
  const int my_tiles = t_end - t_begin;
  const int nh = (min(kQB, a.M - qblk * kQB) > kQH) ? 2 : 1;   // accumulator halves in use

  // (read from one lane, so that the compiler knows the warp index and all that follows from it
  // -- roles, TMEM and barrier addresses -- to be the same in every lane)
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    // the staged K rows are free once the last logits are formed, the Vsum rows only after the last
    // T product: each operand is requested again as soon as its own buffer is free
    mbar_init(&misc->kfull, 1);
    mbar_init(&misc->vfull, 1);
    mbar_init(&misc->kfree, kIssuers);     // the issuers' commits
    mbar_init(&misc->vfree, kIssuers);
    for (int s = 0; s < 2; ++s) {
      mbar_init(&misc->tfull[s], kIssuers);
      mbar_init(&misc->tfree[s], kStatWarps);   // statistics warps
    }
    mbar_init(&misc->qfull, 1);
    misc->abort_flag = 0;
    misc->wait_us = (int)a.wait_us;
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(&misc->tmem_base, 512);
  // (everything above runs while the kernel before this one may still be draining)
  kvs_pdl_wait();
  // the per-query constants of the block (the same for every tile): read from shared memory in the loop
  if (threadIdx.x < kQB) {
    const float2 c = a.qc2[(size_t)unit * a.M_pad + qblk * kQB + threadIdx.x];
    misc->qconst[(threadIdx.x >> 1) * 4 + (threadIdx.x & 1)] = c.x;
    misc->qconst[(threadIdx.x >> 1) * 4 + 2 + (threadIdx.x & 1)] = c.y;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = __shfl_sync(0xffffffffu, misc->tmem_base, 0);   // (uniform for the compiler too)
  volatile int* abort_flag = &misc->abort_flag;
  // test hook: the producer requests no K tile, so that the waits on them run out
  const bool withhold_k = (a.debug_stall & 2u) != 0;

  // tensor-map coordinates of the pair members: slot = 2 * rho + parity
  const int par_l = off & 1, par_r = par_l ^ 1;
  const int rho_l0 = off >> 1, rho_r0 = (off + 1) >> 1;

  if (warp == 0) {
    // ================================================================ TMA producer
    if (elect_one()) {
      prefetch_tmap(&tmKp); prefetch_tmap(&tmVp); prefetch_tmap(&tmQ); prefetch_tmap(&tmOhi); prefetch_tmap(&tmOlo);
      mbar_expect_tx(&misc->qfull, (kExact ? 2 : 3) * kOperand);
      for (int hf = 0; hf < 2; ++hf) {
        tma_load_3d(smem + kSmemQ + hf * kHalf, &tmQ, &misc->qfull, hf * 64, qblk * kQB, unit);
        tma_load_3d(smem + kSmemOhi + hf * kHalf, &tmOhi, &misc->qfull, hf * 64, qblk * kQB, unit);
        if (!kExact) tma_load_3d(smem + kSmemOlo + hf * kHalf, &tmOlo, &misc->qfull, hf * 64, qblk * kQB, unit);
      }
      // one thread streams both operands; every tile is first requested into L2 one tile ahead,
      // so that the load that fills the (single) stage finds it there
      auto prefetch = [&](int li, bool v) {
        const int p0 = (t_begin + li) * kPairs;
        const CUtensorMap* tm = v ? &tmVp : &tmKp;
        for (int hf = 0; hf < 2; ++hf) {
          tma_prefetch_5d(tm, hf * 64, par_l, rho_l0 + p0, h, sr.b);
          tma_prefetch_5d(tm, hf * 64, par_r, rho_r0 + p0, h, sr.b);
        }
      };
      // K of a tile is free again before its Vsum rows are (the last logits come before the last T
      // product), and the K of the tile after that cannot be free before these Vsum rows have been
      // used: the requests go out in the fixed order K, V, K, V, ... behind blocking (bounded) waits
      int kli = 0, vli = 0;
      for (int li = 0; li < my_tiles; ++li) {
        const int p0 = (t_begin + li) * kPairs;
        if (!mbar_wait(&misc->kfree, (li & 1) ^ 1, abort_flag)) break;
        if (!withhold_k) {
          mbar_expect_tx(&misc->kfull, 2 * kOperand);
          for (int hf = 0; hf < 2; ++hf) {
            tma_load_5d(smem + kSmemKl + hf * kHalf, &tmKp, &misc->kfull, hf * 64, par_l, rho_l0 + p0, h, sr.b);
            tma_load_5d(smem + kSmemKr + hf * kHalf, &tmKp, &misc->kfull, hf * 64, par_r, rho_r0 + p0, h, sr.b);
          }
        }
        if (li + 1 < my_tiles) prefetch(li + 1, false);
        ++kli;
        if (!mbar_wait(&misc->vfree, (li & 1) ^ 1, abort_flag)) break;
        mbar_expect_tx(&misc->vfull, 2 * kOperand);
        for (int hf = 0; hf < 2; ++hf) {
          tma_load_5d(smem + kSmemVl + hf * kHalf, &tmVp, &misc->vfull, hf * 64, par_l, rho_l0 + p0, h, sr.b);
          tma_load_5d(smem + kSmemVr + hf * kHalf, &tmVp, &misc->vfull, hf * 64, par_r, rho_r0 + p0, h, sr.b);
        }
        if (li + 1 < my_tiles) prefetch(li + 1, true);
        ++vli;
      }
      if (*abort_flag) {
        // drain: give the copies already issued a bounded time to land before the CTA leaves
        if (kli > 0 && !withhold_k) mbar_drain(&misc->kfull, (kli - 1) & 1);
        if (vli > 0) mbar_drain(&misc->vfull, (vli - 1) & 1);
      }
    }
  } else if (warp < kFirstStat) {
    // ================================================================ product issuers
    // warp 1 issues the chains of the left pair members (S_l, T_l), warp 2 those of the right ones
    if (elect_one()) {
      const bool right = warp != 1;
      // descriptors are kept as a constant high word and low words that only need an addition per product
      constexpr uint32_t idesc = idesc_bf16(kPairs, kQH);
      const uint32_t dhi = (uint32_t)(smem_desc_sw128(0, 16, 1024) >> 32);
      auto dlo = [&](int off_bytes) { return (uint32_t)smem_desc_sw128(smem_u32(smem + off_bytes), 16, 1024); };
      const uint32_t q_lo = dlo(kSmemQ), ohi_lo = dlo(kSmemOhi), olo_lo = dlo(kSmemOlo);
      const uint32_t k_lo = dlo(right ? kSmemKr : kSmemKl), v_lo = dlo(right ? kSmemVr : kSmemVl);
      bool ok = mbar_wait(&misc->qfull, 0, abort_flag);
      for (int li = 0; ok && li < my_tiles; ++li) {
        if (!mbar_wait(&misc->kfull, li & 1, abort_flag)) break;
        for (int hq = 0; hq < nh; ++hq) {
          if (!mbar_wait(&misc->tfree[hq], (li & 1) ^ 1, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t d0 = tmem + hq * 256 + (right ? 64u : 0u);
          const uint32_t qrow = (uint32_t)(hq * (kQH * 128)) >> 4;   // rows 64.. of the query-side operands
          const uint32_t qh = q_lo + qrow, oh = ohi_lo + qrow, ol = olo_lo + qrow;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk) {
            const uint32_t o = ((kk >> 2) * kHalf + (kk & 3) * 32) >> 4;
            if (kk == 0) umma_ss<false>(d0, k_lo, dhi, qh, dhi, idesc);
            else umma_ss<true>(d0, k_lo + o, dhi, qh + o, dhi, idesc);
          }
          if (hq == nh - 1) tc_commit(&misc->kfree);
          if (hq == 0 && !mbar_wait(&misc->vfull, li & 1, abort_flag)) { ok = false; break; }
          constexpr int kTSteps = kExact ? 8 : 16;           // E is one bf16 term, o is two
#pragma unroll
          for (int kk = 0; kk < kTSteps; ++kk) {
            const uint32_t o = (((kk & 7) >> 2) * kHalf + (kk & 3) * 32) >> 4;
            const uint32_t ob = (kk < 8 ? oh : ol) + o;
            if (kk == 0) umma_ss<false>(d0 + 128, v_lo, dhi, ob, dhi, idesc);
            else umma_ss<true>(d0 + 128, v_lo + o, dhi, ob, dhi, idesc);
          }
          tc_commit(&misc->tfull[hq]);
        }
        if (!ok) break;
        tc_commit(&misc->vfree);
      }
    }
  } else {
    // ================================================================ statistics warps
    const int grp = (warp - kFirstStat) >> 2;             // its share of the queries of each half
    const int quarter = warp & 3;                         // TMEM lane quarter this warp may read
    const int lane_p = quarter * 32 + lane;               // pair within the tile
    const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
    const int32_t* Cb = a.counts + (size_t)unit * a.n_max;
    const float4* norms = a.pair_norms + (size_t)unit * a.norm_stride;
    // the partial sums of this (query block, group)
    const size_t sub = (size_t)unit * (a.nqblk * kGroups) + (size_t)qblk * kGroups + grp;
    float4* out4 = a.part4 + sub * a.pair_stride;
    float* out1 = a.part1 + sub * a.pair_stride;
    // norms and counts of the next tile's pair travel while the current tile is reduced
    float4 nrm_next = make_float4(1.f, 1.f, 1.f, 0.f);
    int cl_next = 1, cr_next = 1;
    {
      const int p = t_begin * kPairs + lane_p;
      if (p < P) { nrm_next = ldg_here(norms + p); cl_next = ldg_here(Cb + off + 2 * p); cr_next = ldg_here(Cb + off + 2 * p + 1); }
    }
    for (int li = 0; li < my_tiles; ++li) {
      const int tile = t_begin + li;
      const int p = tile * kPairs + lane_p;               // candidate pair of this thread
      const float4 nrm = nrm_next;
      const float cl = (float)cl_next, cr = (float)cr_next;
      if (li + 1 < my_tiles) {
        const int pn = p + kPairs;
        if (pn < P) { nrm_next = ldg_here(norms + pn); cl_next = ldg_here(Cb + off + 2 * pn); cr_next = ldg_here(Cb + off + 2 * pn + 1); }
      }
      const float icl = __fdividef(1.f, cl), icr = __fdividef(1.f, cr);   // (counts are small integers)
      const float r2l = nrm.x, r2r = nrm.y, pc = nrm.z;
      const float n2cl = -2.f * cl, n2cr = -2.f * cr, n2il = -2.f * icl, n2ir = -2.f * icr;

      // beta = alpha / c = exp2(scale * s - (max + log2 Z)); sums are scaled by the counts at the end.
      // The arithmetic runs on pairs of neighbouring queries with the packed two-float instructions
      // (fma/add/mul.f32x2): the kernel is as short of issue slots as of special-function slots, and a
      // packed instruction takes one slot for two operations.  Every sum is kept as two lanes.
      float2 sAl = make_float2(0.f, 0.f), sAr = sAl, sN1l = sAl, sN1r = sAl, sN12 = sAl;
      const float2 sc2 = make_float2(a.scale_log2, a.scale_log2), one2 = make_float2(1.f, 1.f);
      const float2 n2cl2 = make_float2(n2cl, n2cl), n2cr2 = make_float2(n2cr, n2cr);
      const float2 n2il2 = make_float2(n2il, n2il), n2ir2 = make_float2(n2ir, n2ir);
      const float2 icl2 = make_float2(icl, icl), icr2 = make_float2(icr, icr);
      const float2 r2l2 = make_float2(r2l, r2l), r2r2 = make_float2(r2r, r2r), pc2 = make_float2(pc, pc);
      const float2 four2 = make_float2(4.f, 4.f), n4il2 = make_float2(2.f * n2il, 2.f * n2il), n4ir2 = make_float2(2.f * n2ir, 2.f * n2ir);
      bool broken = false;
      for (int hq = 0; hq < nh; ++hq) {
        if (!warp_wait(&misc->tfull[hq], li & 1, abort_flag, lane)) { broken = true; break; }
        tc_fence_after();
        const uint32_t col0 = tmem + lane_addr + hq * 256;
        const float4* qc4 = reinterpret_cast<const float4*>(misc->qconst + hq * (2 * kQH));
        // chunks [c_begin, c_end) of every half (2 / 3 / 3 of the eight: letting the short share go round
        // among the groups measured slower; the group that is done early moves on to the next half
        // and the groups end up staggered, which spreads their serial phases)
        const int c_begin = (grp * kChunks) / kGroups, c_end = ((grp + 1) * kChunks) / kGroups;
        // chunks of 8 queries; the loads of the next chunk are in flight while this one is reduced
        float buf[kDoubleBuffer ? 2 : 1][4][kChunk];
        auto issue = [&](int c, int b) {
          const uint32_t col = col0 + c * kChunk;
          tmem_ld8(col, buf[b][0]);
          tmem_ld8(col + 64, buf[b][1]);
          tmem_ld8(col + 128, buf[b][2]);
          tmem_ld8(col + 192, buf[b][3]);
        };
        auto reduce = [&](int c, int b) {
#pragma unroll
          for (int i = 0; i < kChunk; i += 2) {
            const float4 cq = qc4[c * (kChunk / 2) + (i >> 1)];           // the two queries' constants (a broadcast read)
            const float2 ncq = make_float2(cq.x, cq.y), hq2 = make_float2(cq.z, cq.w);
            const float2 el = __ffma2_rn(make_float2(buf[b][0][i], buf[b][0][i + 1]), sc2, ncq);
            const float2 er = __ffma2_rn(make_float2(buf[b][1][i], buf[b][1][i + 1]), sc2, ncq);
            const float2 bl = make_float2(fast_exp2(el.x), fast_exp2(el.y));
            const float2 br = make_float2(fast_exp2(er.x), fast_exp2(er.y));
            const float2 tl = make_float2(buf[b][2][i], buf[b][2][i + 1]), tr = make_float2(buf[b][3][i], buf[b][3][i + 1]);
            sAl = __fadd2_rn(sAl, bl);
            sAr = __fadd2_rn(sAr, br);
            const float2 al = __ffma2_rn(bl, n2cl2, one2), ar = __ffma2_rn(br, n2cr2, one2);   // 1 - 2 alpha
            if constexpr (kExact) {
              // g11 = alpha (1 - 2 alpha) E^T (vbar_l - o), g12 = -alpha_l alpha_r E^T (vbar_l + vbar_r - 2 o);
              // hq2 holds <E_q, o_q> here (the sign of g12 is applied after the loop)
              const float2 nh2 = make_float2(-hq2.x, -hq2.y);
              const float2 hl = __ffma2_rn(tl, icl2, nh2), hr = __ffma2_rn(tr, icr2, nh2);     // E^T (vbar - o)
              sN1l = __ffma2_rn(__fmul2_rn(bl, al), hl, sN1l);
              sN1r = __ffma2_rn(__fmul2_rn(br, ar), hr, sN1r);
              sN12 = __ffma2_rn(__fmul2_rn(bl, br), __fadd2_rn(hl, hr), sN12);
            } else {
              const float2 gl = make_float2(bl.x * fabsf(al.x), bl.y * fabsf(al.y));          // beta |1 - 2 alpha|
              const float2 gr = make_float2(br.x * fabsf(ar.x), br.y * fabsf(ar.y));
              const float2 dl = __ffma2_rn(tl, n2il2, __fadd2_rn(r2l2, hq2));                  // |vbar_l - o|^2
              const float2 dr = __ffma2_rn(tr, n2ir2, __fadd2_rn(r2r2, hq2));
              sN1l = __ffma2_rn(gl, make_float2(fast_sqrt(fabsf(dl.x)), fast_sqrt(fabsf(dl.y))), sN1l);
              sN1r = __ffma2_rn(gr, make_float2(fast_sqrt(fabsf(dr.x)), fast_sqrt(fabsf(dr.y))), sN1r);
              // |vbar_l + vbar_r - 2 o|^2 = |vbar_l + vbar_r|^2 + 4 |o|^2 - 4 <vbar_l, o> - 4 <vbar_r, o>
              const float2 d12 = __ffma2_rn(tl, n4il2, __ffma2_rn(tr, n4ir2, __ffma2_rn(hq2, four2, pc2)));
              sN12 = __ffma2_rn(__fmul2_rn(bl, br), make_float2(fast_sqrt(fabsf(d12.x)), fast_sqrt(fabsf(d12.y))), sN12);
            }
          }
        };
        if constexpr (kDoubleBuffer) {
          issue(c_begin, 0);
          for (int c = c_begin; c < c_end; c += 2) {
            tmem_ld_wait();
            if (c + 1 < c_end) issue(c + 1, 1);
            reduce(c, 0);
            if (c + 1 < c_end) {
              tmem_ld_wait();
              if (c + 2 < c_end) issue(c + 2, 0);
              reduce(c + 1, 1);
            }
          }
        } else {
          // (with four warps per scheduler the other warps cover the latency of the loads)
          for (int c = c_begin; c < c_end; ++c) {
            issue(c, 0);
            tmem_ld_wait();
            reduce(c, 0);
          }
        }
        tc_fence_before();
        warp_arrive(&misc->tfree[hq], lane);                               // this half may be overwritten
      }
      if (broken) break;
      // the sums of this (query block, group) for the pair: a later kernel adds the partials in order
      if (p < P) {
        out4[p] = make_float4(cl * (sAl.x + sAl.y), cr * (sAr.x + sAr.y), cl * (sN1l.x + sN1l.y), cr * (sN1r.x + sN1r.y));
        out1[p] = (kExact ? -1.f : 1.f) * cl * cr * (sN12.x + sN12.y);
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

// Sum of the partials of all (query block, statistics group) pairs in a fixed order, then score and
// left-key weight of each candidate pair.  Weight modes:
//   0: the sums are norms; w = (N1_l - N12) / (N1_l - 2 N12 + N1_r)                        [Eq. kstar_final]
//   1: they are the signed sums G11, G22, G12 of g_ij = E^T c_ij; w = (G11 + G12) / (G11 + 2 G12 + G22)
//                                                                            [Eq. kstar_weight_final_rewrite]
//   2: as 1 with the coupling dropped, w = G11 / (G11 + G22)                              [Eq. simplified_k]
// A denominator that is not safely positive gives 1/2; the weight is clipped to [0, 1].
__global__ void __launch_bounds__(256)
stats_finalize_kernel(const StatsTcArgs a, const RoundTable tab) {
  kvs_pdl_launch_dependents();
  kvs_pdl_wait();
  const SeqRound sr = tab.s[blockIdx.z];
  if (sr.n <= 0) return;
  const int unit = sr.b * a.Hkv + blockIdx.y;
  const int p = blockIdx.x * 256 + threadIdx.x;
  if (p >= sr.P) return;
  const int jl = tab.off + 2 * p;
  const int nsub = a.nqblk * kGroups;
  float Al = 0.f, Ar = 0.f, N1l = 0.f, N1r = 0.f, N12 = 0.f;
  for (int sb = 0; sb < nsub; ++sb) {
    const size_t i = ((size_t)unit * nsub + sb) * a.pair_stride + p;
    const float4 v = a.part4[i];
    Al += v.x; Ar += v.y; N1l += v.z; N1r += v.w;
    N12 += a.part1[i];
  }
  const float cosv = a.pair_norms[(size_t)unit * a.norm_stride + p].w;
  const float mass = Al + Ar;
  const float score = (a.score_mode == 0) ? mass * fmaxf(0.f, 1.f - cosv) : mass;
  float w = 0.5f;
  if (a.weight_mode == 0) {
    const float D = N1l - 2.f * N12 + N1r;
    if (D > 1e-6f * (N1l + N1r) && D < INFINITY) w = fminf(1.f, fmaxf(0.f, (N1l - N12) / D));
  } else {
    const float g12 = (a.weight_mode == 2) ? 0.f : N12;
    const float gamma = N1l + 2.f * g12 + N1r;
    if (gamma > 1e-6f * (fabsf(N1l) + fabsf(N1r)) && gamma < INFINITY) w = fminf(1.f, fmaxf(0.f, (N1l + g12) / gamma));
  }
  const size_t pi = (size_t)unit * a.pair_stride + p;
  a.score[pi] = fabsf(score);
  a.w[pi] = w;
  if (a.N12) a.N12[pi] = N12;
  if (a.cosv) a.cosv[pi] = cosv;
  if (a.A) { a.A[(size_t)unit * a.n_max + jl] = Al; a.A[(size_t)unit * a.n_max + jl + 1] = Ar; }
  if (a.N1) { a.N1[(size_t)unit * a.n_max + jl] = N1l; a.N1[(size_t)unit * a.n_max + jl + 1] = N1r; }
}

}  // namespace

cudaError_t kvs_launch_stats_tc(const StatsTcArgs& a, const RoundTable& t, const CUtensorMap& tmKp,
                                const CUtensorMap& tmVp, const CUtensorMap& tmQ, const CUtensorMap& tmOhi,
                                const CUtensorMap& tmOlo, cudaStream_t st) {
  static KvsPerDeviceOnce configured;
  cudaError_t ce = configured.run([] {
    cudaError_t e = cudaFuncSetAttribute(hessian_stats_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(hessian_stats_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  });
  if (ce != cudaSuccess) return ce;
  dim3 grid(a.nqblk * a.splits, a.Hkv, t.nseq);
  cudaError_t e = (a.weight_mode == 0)
      ? kvs_launch_chained(hessian_stats_tc<false>, grid, dim3(kThreads), kSmemBytes, st, a, t, tmKp, tmVp, tmQ, tmOhi, tmOlo)
      : kvs_launch_chained(hessian_stats_tc<true>, grid, dim3(kThreads), kSmemBytes, st, a, t, tmKp, tmVp, tmQ, tmOhi, tmOlo);
  if (e != cudaSuccess) return e;
  int pmax = 0;
  for (int i = 0; i < t.nseq; ++i) pmax = pmax > t.s[i].P ? pmax : t.s[i].P;
  if (pmax <= 0) return cudaSuccess;
  dim3 fgrid((pmax + 255) / 256, a.Hkv, t.nseq);
  return kvs_launch_chained(stats_finalize_kernel, fgrid, dim3(256), 0, st, a, t);
}
