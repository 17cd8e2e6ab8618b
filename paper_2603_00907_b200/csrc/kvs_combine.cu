// Combine of the attention partials that the key ranges of a query row produce.
//
// One warp per (query row, unit): the partial maxima, sums and outputs of the row's key ranges
// are merged into the row's softmax normaliser and attention output
//   o_q = sum_j alpha_qj Vsum_j / c_j,  alpha = softmax_j(scale <q, K_j> + ln c_j)   [Eq. attn_def_vec
// with merged slots].  For the observation window the kernel writes what the statistics pass needs
// (per-query constants, o in fp32 and as two bf16 terms); for the decode check the bf16 output.
#include "kvs_internal.h"

namespace {

// One warp per (query row, unit), eight rows per CTA; a lane owns four output channels.
constexpr int kCombineRows = 8;

__global__ void __launch_bounds__(kCombineRows * 32)
combine_partials(const CombineArgs a, const RoundTable tab) {
  kvs_pdl_launch_dependents();
  kvs_pdl_wait();
  const int seq = blockIdx.z;
  const SeqRound sr = tab.s[seq];
  if (sr.n <= 0) return;
  const int unit = sr.b * a.Hkv + blockIdx.y;
  const int m = blockIdx.x * kCombineRows + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (m >= a.M) {            // padding rows of the per-query constants: alpha = exp2(-inf) = 0
    if (lane == 0 && a.qc2 && m < a.M_pad) a.qc2[(size_t)unit * a.M_pad + m] = make_float2(-INFINITY, 0.f);
    return;
  }
  const size_t base = (size_t)unit * a.splits * a.M + m;
  float mstar = -INFINITY;
  for (int s = 0; s < a.splits; ++s) mstar = fmaxf(mstar, a.part_ml[base + (size_t)s * a.M].x);
  float Z = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s = 0; s < a.splits; ++s) {
    const float2 ml = a.part_ml[base + (size_t)s * a.M];
    if (ml.x == -INFINITY) continue;
    const float f = fast_exp2(ml.x - mstar);
    Z = fmaf(ml.y, f, Z);
    const float4 po = *reinterpret_cast<const float4*>(a.part_o + (base + (size_t)s * a.M) * KVS_D + 4 * lane);
    acc.x = fmaf(po.x, f, acc.x); acc.y = fmaf(po.y, f, acc.y);
    acc.z = fmaf(po.z, f, acc.z); acc.w = fmaf(po.w, f, acc.w);
  }
  const float4 od = make_float4(acc.x / Z, acc.y / Z, acc.z / Z, acc.w / Z);
  // |o|^2 over the 128 channels
  float on2 = (od.x * od.x + od.y * od.y) + (od.z * od.z + od.w * od.w);
#pragma unroll
  for (int k = 16; k > 0; k >>= 1) on2 += __shfl_xor_sync(0xffffffffu, on2, k);
  const size_t row = (size_t)unit * a.M + m;
  const float lse = (mstar + log2f(Z)) * 0.6931471805599453f;
  // with a supplied loss gradient the statistics need <E_q, o_q> in place of |o_q|^2
  float qconst = on2;
  if (a.e) {
    const uint2 er = *reinterpret_cast<const uint2*>(a.e + row * KVS_D + 4 * lane);
    float eo = fmaf(bf16lo(er.x), od.x, bf16hi(er.x) * od.y) + fmaf(bf16lo(er.y), od.z, bf16hi(er.y) * od.w);
#pragma unroll
    for (int k = 16; k > 0; k >>= 1) eo += __shfl_xor_sync(0xffffffffu, eo, k);
    qconst = eo;
  }
  if (lane == 0) {
    if (a.qstat) a.qstat[row] = make_float4(mstar, Z, on2, lse);
    if (a.qc2) a.qc2[(size_t)unit * a.M_pad + m] = make_float2(-(mstar + log2f(Z)), qconst);
    if (a.lse_out) a.lse_out[row] = lse;
  }
  const float v[4] = {od.x, od.y, od.z, od.w};
  if (a.o) *reinterpret_cast<float4*>(a.o + row * KVS_D + 4 * lane) = od;
  if (a.o_out) *reinterpret_cast<float4*>(a.o_out + row * KVS_D + 4 * lane) = od;
  if (a.o_hi) {
    __nv_bfloat16 hi[4], lo[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      hi[i] = __float2bfloat16_rn(v[i]);
      lo[i] = __float2bfloat16_rn(v[i] - __bfloat162float(hi[i]));
    }
    *reinterpret_cast<uint2*>(a.o_hi + row * KVS_D + 4 * lane) = *reinterpret_cast<const uint2*>(hi);
    *reinterpret_cast<uint2*>(a.o_lo + row * KVS_D + 4 * lane) = *reinterpret_cast<const uint2*>(lo);
  }
  if (a.out_bf16) {
    __nv_bfloat16 ob[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) ob[i] = __float2bfloat16_rn(v[i]);
    *reinterpret_cast<uint2*>(a.out_bf16 + row * KVS_D + 4 * lane) = *reinterpret_cast<const uint2*>(ob);
  }
}

}  // namespace

cudaError_t kvs_launch_combine(const CombineArgs& a, const RoundTable& t, cudaStream_t st) {
  const int rows = a.qc2 ? a.M_pad : a.M;
  dim3 grid((rows + kCombineRows - 1) / kCombineRows, a.Hkv, t.nseq);
  return kvs_launch_chained(combine_partials, grid, dim3(kCombineRows * 32), 0, st, a, t);
}
