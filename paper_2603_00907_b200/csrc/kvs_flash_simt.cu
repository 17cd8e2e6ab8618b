// Attention partials on the CUDA cores (fp32 FMA) and their combine.
//
// flash_partial_simt: one thread per query row, one CTA per (query block of 128 rows,
// key split, KV head, sequence).  For its key range it keeps an online softmax
// (running max in log2 units, running sum, 128 output accumulators) over
//   s_qj = softmax_scale <q, K_j> + ln c_j      [Eq. attn_def_vec with merged slots]
//   o_q  = sum_j alpha_qj Vsum_j / c_j
// and writes the partial (max, sum, o).  combine_partials merges the key splits.
// The same pair of kernels serves the observation window (causal inside the last W
// slots) and the decode check (no mask).
#include "kvs_internal.h"

namespace {

constexpr int TK = 16;  // keys staged per step

__global__ void __launch_bounds__(128, 1)
flash_partial_simt(const FlashArgs a, const RoundTable tab) {
  const int seq = blockIdx.z;
  const SeqRound sr = tab.s[seq];
  const int n = sr.n;
  if (n <= 0) return;
  const int h = blockIdx.y;
  const int nqblk = (a.M + 127) / 128;
  const int split = blockIdx.x / nqblk;
  const int qblk = blockIdx.x % nqblk;
  const int tid = threadIdx.x;
  const int m = qblk * 128 + tid;
  const bool row_ok = m < a.M;
  const int unit = sr.b * a.c.Hkv + h;

  __shared__ __align__(16) float sK[TK][KVS_D];
  __shared__ __align__(16) float sV[TK][KVS_D];
  __shared__ float sLc[TK];   // log2(count)
  __shared__ float sIc[TK];   // 1 / count

  // query row as 64 packed bf16 pairs
  uint32_t qreg[64];
  {
    const __nv_bfloat16* qrow =
        a.q + ((size_t)(sr.b * a.Hq + h * a.G) * a.Wq + (row_ok ? m : 0)) * KVS_D;
    const uint4* q4 = reinterpret_cast<const uint4*>(qrow);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      uint4 v = q4[i];
      qreg[4 * i + 0] = v.x; qreg[4 * i + 1] = v.y; qreg[4 * i + 2] = v.z; qreg[4 * i + 3] = v.w;
    }
  }
  // last visible slot of this row
  const int last_vis = a.causal ? (n - a.Wq + (m % a.Wq)) : (n - 1);

  float o[KVS_D];
#pragma unroll
  for (int d = 0; d < KVS_D; ++d) o[d] = 0.f;
  float mrun = -INFINITY, l = 0.f;

  const int k0 = split * a.split_len;
  const int k1 = min(n, k0 + a.split_len);
  const __nv_bfloat16* Kb = a.c.K + sr.b * a.c.ksb + h * a.c.ksh;
  const __nv_bfloat16* Vb = a.c.V + sr.b * a.c.vsb + h * a.c.vsh;
  const int32_t* Cb = a.c.counts + (size_t)unit * a.c.n_max;

  for (int t0 = k0; t0 < k1; t0 += TK) {
    __syncthreads();
    // stage TK rows of K and V as fp32: 16 rows x 16 chunks of 8 elements = 256 chunks each
    for (int c = tid; c < TK * 16; c += 128) {
      const int r = c >> 4, ch = c & 15;
      const int j = t0 + r;
      uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
      if (j < k1) {
        kv = *reinterpret_cast<const uint4*>(Kb + (int64_t)j * a.c.kst + ch * 8);
        vv = *reinterpret_cast<const uint4*>(Vb + (int64_t)j * a.c.vst + ch * 8);
      }
      float* dk = &sK[r][ch * 8];
      float* dv = &sV[r][ch * 8];
      dk[0] = bf16lo(kv.x); dk[1] = bf16hi(kv.x); dk[2] = bf16lo(kv.y); dk[3] = bf16hi(kv.y);
      dk[4] = bf16lo(kv.z); dk[5] = bf16hi(kv.z); dk[6] = bf16lo(kv.w); dk[7] = bf16hi(kv.w);
      dv[0] = bf16lo(vv.x); dv[1] = bf16hi(vv.x); dv[2] = bf16lo(vv.y); dv[3] = bf16hi(vv.y);
      dv[4] = bf16lo(vv.z); dv[5] = bf16hi(vv.z); dv[6] = bf16lo(vv.w); dv[7] = bf16hi(vv.w);
    }
    if (tid < TK) {
      const int j = t0 + tid;
      const float cnt = (j < k1) ? (float)Cb[j] : 1.f;
      sLc[tid] = log2f(cnt);
      sIc[tid] = 1.f / cnt;
    }
    __syncthreads();

    float s[TK];
    float mt = -INFINITY;
#pragma unroll
    for (int r = 0; r < TK; ++r) {
      float acc = 0.f;
      const float4* k4 = reinterpret_cast<const float4*>(&sK[r][0]);
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float4 kk = k4[i];
        const uint32_t qa = qreg[2 * i], qb = qreg[2 * i + 1];
        acc = fmaf(bf16lo(qa), kk.x, acc);
        acc = fmaf(bf16hi(qa), kk.y, acc);
        acc = fmaf(bf16lo(qb), kk.z, acc);
        acc = fmaf(bf16hi(qb), kk.w, acc);
      }
      const int j = t0 + r;
      float v = fmaf(acc, a.scale_log2, sLc[r]);
      if (j >= k1 || j > last_vis) v = -INFINITY;
      s[r] = v;
      mt = fmaxf(mt, v);
    }
    const float mnew = fmaxf(mrun, mt);
    if (mnew == -INFINITY) continue;   // nothing visible so far (uniform per thread only)
    const float corr = fast_exp2(mrun - mnew);   // exp2(-inf) = 0
    mrun = mnew;
    l *= corr;
#pragma unroll
    for (int d = 0; d < KVS_D; ++d) o[d] *= corr;
#pragma unroll
    for (int r = 0; r < TK; ++r) {
      const float p = fast_exp2(s[r] - mnew);   // includes the count: c_j * exp(e_j - m)
      l += p;
      const float pv = p * sIc[r];
      const float4* v4 = reinterpret_cast<const float4*>(&sV[r][0]);
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float4 vv = v4[i];
        o[4 * i + 0] = fmaf(pv, vv.x, o[4 * i + 0]);
        o[4 * i + 1] = fmaf(pv, vv.y, o[4 * i + 1]);
        o[4 * i + 2] = fmaf(pv, vv.z, o[4 * i + 2]);
        o[4 * i + 3] = fmaf(pv, vv.w, o[4 * i + 3]);
      }
    }
  }
  if (row_ok) {
    const size_t pidx = ((size_t)unit * a.splits + split) * a.M + m;
    a.part_ml[pidx] = make_float2(mrun, l);
    float4* po = reinterpret_cast<float4*>(a.part_o + pidx * KVS_D);
#pragma unroll
    for (int i = 0; i < 32; ++i) po[i] = make_float4(o[4 * i], o[4 * i + 1], o[4 * i + 2], o[4 * i + 3]);
  }
}

// One warp per (query row, unit), eight rows per CTA; a lane owns four output channels.
constexpr int kCombineRows = 8;

__global__ void __launch_bounds__(kCombineRows * 32)
combine_partials(const CombineArgs a, const RoundTable tab) {
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
  if (lane == 0) {
    if (a.qstat) a.qstat[row] = make_float4(mstar, Z, on2, lse);
    if (a.qc2) a.qc2[(size_t)unit * a.M_pad + m] = make_float2(-(mstar + log2f(Z)), on2);
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

cudaError_t kvs_launch_flash_simt(const FlashArgs& a, const RoundTable& t, cudaStream_t st) {
  const int nqblk = (a.M + 127) / 128;
  dim3 grid(a.splits * nqblk, a.c.Hkv, t.nseq);
  flash_partial_simt<<<grid, 128, 0, st>>>(a, t);
  return cudaGetLastError();
}

cudaError_t kvs_launch_combine(const CombineArgs& a, const RoundTable& t, cudaStream_t st) {
  const int rows = a.qc2 ? a.M_pad : a.M;
  dim3 grid((rows + kCombineRows - 1) / kCombineRows, a.Hkv, t.nseq);
  combine_partials<<<grid, kCombineRows * 32, 0, st>>>(a, t);
  return cudaGetLastError();
}
