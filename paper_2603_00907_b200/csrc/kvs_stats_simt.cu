// Hessian statistics on the CUDA cores (fp32 FMA): one thread per cache slot.
//
// With the window softmax already normalised (max, Z and o_q per query), each thread
// recomputes the logits of its slot against every window query and reduces, over the
// queries, the forward-only norms of the closed-form Hessian terms:
//   A_j   = sum_q alpha_qj                                   (attention mass)
//   N1_j  = sum_q |c_jj^(q)| = sum_q alpha |1 - 2 alpha| |vbar_j - o_q|        [Eqs. c11_def, c22_def]
//   N12_p = sum_q |c_12^(q)| = sum_q alpha_j alpha_j+1 |vbar_j + vbar_j+1 - 2 o_q|   [Eq. c12_def]
// The distances come from T_jq = <vbar_j, o_q>:
//   |vbar_j - o_q|^2 = |vbar_j|^2 - 2 T_jq + |o_q|^2.
// Slots are laid out so that the two members of a candidate pair sit in an (even, odd)
// lane pair of one warp.  The even lane then forms the adjacent-key cosine, the pair
// score and the merge weight of Eq. kstar_final.
#include "kvs_internal.h"

namespace {

constexpr int QC = 16;  // queries staged per step

__device__ __forceinline__ float dot_packed(const uint32_t* x, const uint32_t* y) {
  float acc = 0.f;
#pragma unroll
  for (int i = 0; i < 64; ++i) {
    acc = fmaf(bf16lo(x[i]), bf16lo(y[i]), acc);
    acc = fmaf(bf16hi(x[i]), bf16hi(y[i]), acc);
  }
  return acc;
}

__global__ void __launch_bounds__(128, 2)
hessian_stats_simt(const StatsArgs a, const RoundTable tab) {
  const int seq = blockIdx.z;
  const SeqRound sr = tab.s[seq];
  const int n = sr.n;
  if (n <= 0) return;
  const int off = tab.off;
  const int shift = off & 1;
  if ((int)blockIdx.x * 128 - shift >= n) return;
  const int h = blockIdx.y;
  const int unit = sr.b * a.c.Hkv + h;
  const int tid = threadIdx.x;
  const int j = blockIdx.x * 128 + tid - shift;      // slot of this thread (may be -1 or >= n)
  const bool slot_ok = j >= 0 && j < n;
  const int jj = slot_ok ? j : 0;

  __shared__ __align__(16) float sQ[QC][KVS_D];
  __shared__ __align__(16) float sO[QC][KVS_D];
  __shared__ float4 sS[QC];

  const __nv_bfloat16* Kb = a.c.K + sr.b * a.c.ksb + h * a.c.ksh;
  const __nv_bfloat16* Vb = a.c.V + sr.b * a.c.vsb + h * a.c.vsh;
  const int32_t* Cb = a.c.counts + (size_t)unit * a.c.n_max;

  uint32_t kreg[64], vreg[64];
  {
    const uint4* k4 = reinterpret_cast<const uint4*>(Kb + (int64_t)jj * a.c.kst);
    const uint4* v4 = reinterpret_cast<const uint4*>(Vb + (int64_t)jj * a.c.vst);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      uint4 kv = k4[i], vv = v4[i];
      kreg[4 * i] = kv.x; kreg[4 * i + 1] = kv.y; kreg[4 * i + 2] = kv.z; kreg[4 * i + 3] = kv.w;
      vreg[4 * i] = vv.x; vreg[4 * i + 1] = vv.y; vreg[4 * i + 2] = vv.z; vreg[4 * i + 3] = vv.w;
    }
  }
  const float cnt = (float)Cb[jj];
  const float invc = 1.f / cnt;
  const float lc2 = log2f(cnt);
  const float r2 = dot_packed(vreg, vreg) * invc * invc;       // |vbar_j|^2
  const float k2 = dot_packed(kreg, kreg);

  // partner quantities (the odd lane's values, read by the even lane)
  float kk12 = 0.f, vv12 = 0.f;
#pragma unroll
  for (int i = 0; i < 64; ++i) {
    const uint32_t pk = __shfl_down_sync(0xffffffffu, kreg[i], 1);
    const uint32_t pv = __shfl_down_sync(0xffffffffu, vreg[i], 1);
    kk12 = fmaf(bf16lo(kreg[i]), bf16lo(pk), kk12);
    kk12 = fmaf(bf16hi(kreg[i]), bf16hi(pk), kk12);
    vv12 = fmaf(bf16lo(vreg[i]), bf16lo(pv), vv12);
    vv12 = fmaf(bf16hi(vreg[i]), bf16hi(pv), vv12);
  }
  const float invc_p = __shfl_down_sync(0xffffffffu, invc, 1);
  const float r2_p = __shfl_down_sync(0xffffffffu, r2, 1);
  const float k2_p = __shfl_down_sync(0xffffffffu, k2, 1);
  vv12 *= invc * invc_p;                                        // <vbar_j, vbar_j+1>

  const __nv_bfloat16* qbase = a.q + (size_t)(sr.b * a.Hq + h * a.G) * a.Wq * KVS_D;
  const float* obase = a.o + (size_t)unit * a.M * KVS_D;
  const float4* sbase = a.qstat + (size_t)unit * a.M;

  float accA = 0.f, accN1 = 0.f, accN12 = 0.f;
  for (int q0 = 0; q0 < a.M; q0 += QC) {
    __syncthreads();
    for (int c = tid; c < QC * 32; c += 128) {
      const int r = c >> 5, ch = c & 31;                         // 32 chunks of 4 elements
      const int m = q0 + r;
      float4 qv = make_float4(0, 0, 0, 0), ov = make_float4(0, 0, 0, 0);
      if (m < a.M) {
        const uint2 raw = *reinterpret_cast<const uint2*>(qbase + (size_t)m * KVS_D + ch * 4);
        qv = make_float4(bf16lo(raw.x), bf16hi(raw.x), bf16lo(raw.y), bf16hi(raw.y));
        ov = *reinterpret_cast<const float4*>(obase + (size_t)m * KVS_D + ch * 4);
      }
      *reinterpret_cast<float4*>(&sQ[r][ch * 4]) = qv;
      *reinterpret_cast<float4*>(&sO[r][ch * 4]) = ov;
    }
    if (tid < QC) sS[tid] = (q0 + tid < a.M) ? sbase[q0 + tid] : make_float4(0, 1, 0, 0);
    __syncthreads();
#pragma unroll 1
    for (int r = 0; r < QC; ++r) {
      const int m = q0 + r;
      if (m >= a.M) break;
      float sacc = 0.f, tacc = 0.f;
      const float4* q4 = reinterpret_cast<const float4*>(&sQ[r][0]);
      const float4* o4 = reinterpret_cast<const float4*>(&sO[r][0]);
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float4 qq = q4[i], oo = o4[i];
        const uint32_t ka = kreg[2 * i], kb = kreg[2 * i + 1];
        const uint32_t va = vreg[2 * i], vb = vreg[2 * i + 1];
        sacc = fmaf(bf16lo(ka), qq.x, sacc); sacc = fmaf(bf16hi(ka), qq.y, sacc);
        sacc = fmaf(bf16lo(kb), qq.z, sacc); sacc = fmaf(bf16hi(kb), qq.w, sacc);
        tacc = fmaf(bf16lo(va), oo.x, tacc); tacc = fmaf(bf16hi(va), oo.y, tacc);
        tacc = fmaf(bf16lo(vb), oo.z, tacc); tacc = fmaf(bf16hi(vb), oo.w, tacc);
      }
      const float4 st = sS[r];                                   // (max log2, Z, |o|^2, lse)
      const int last_vis = a.causal ? (n - a.Wq + (m % a.Wq)) : (n - 1);
      float alpha = fast_exp2(fmaf(sacc, a.scale_log2, lc2) - st.x) / st.y;
      if (!slot_ok || j > last_vis) alpha = 0.f;
      const float T = tacc * invc;
      const float d2 = fmaxf(r2 - 2.f * T + st.z, 0.f);
      accA += alpha;
      accN1 = fmaf(alpha * fabsf(1.f - 2.f * alpha), sqrtf(d2), accN1);
      const float alpha_p = __shfl_down_sync(0xffffffffu, alpha, 1);
      const float T_p = __shfl_down_sync(0xffffffffu, T, 1);
      const float d12 = fmaxf(r2 + r2_p + 2.f * vv12 - 4.f * (T + T_p) + 4.f * st.z, 0.f);
      accN12 = fmaf(alpha * alpha_p, sqrtf(d12), accN12);
    }
  }

  const float A_p = __shfl_down_sync(0xffffffffu, accA, 1);
  const float N1_p = __shfl_down_sync(0xffffffffu, accN1, 1);
  if (slot_ok) {
    if (a.A) a.A[(size_t)unit * a.c.n_max + j] = accA;
    if (a.N1) a.N1[(size_t)unit * a.c.n_max + j] = accN1;
  }
  // even lane of a candidate pair
  const int rel = j - off;
  if ((tid & 1) == 0 && rel >= 0 && (rel >> 1) < sr.P) {
    const int p = rel >> 1;
    const float cosv = kk12 / fmaxf(sqrtf(k2) * sqrtf(k2_p), 1e-30f);
    const float mass = accA + A_p;
    const float score = (a.score_mode == 0) ? mass * fmaxf(0.f, 1.f - cosv) : mass;
    const float D = accN1 - 2.f * accN12 + N1_p;
    float w = 0.5f;
    if (D > 1e-6f * (accN1 + N1_p) && D < INFINITY) w = fminf(1.f, fmaxf(0.f, (accN1 - accN12) / D));
    const size_t pi = (size_t)unit * a.pair_stride + p;
    a.score[pi] = fabsf(score);
    a.w[pi] = w;
    if (a.N12) a.N12[pi] = accN12;
    if (a.cosv) a.cosv[pi] = cosv;
  }
}

}  // namespace

cudaError_t kvs_launch_stats_simt(const StatsArgs& a, const RoundTable& t, cudaStream_t st) {
  int nmax = 0;
  for (int i = 0; i < t.nseq; ++i) nmax = nmax > t.s[i].n ? nmax : t.s[i].n;
  dim3 grid((nmax + 1 + 127) / 128, a.c.Hkv, t.nseq);
  hessian_stats_simt<<<grid, 128, 0, st>>>(a, t);
  return cudaGetLastError();
}
