// C ABI of libkvs.so: argument checks, the host round scheduler, the workspace layout and
// the launch sequence of each entry point.  No device memory is allocated here and the
// stream is never synchronised.
#include <limits.h>
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>
#include <vector>

#include "kvs_internal.h"

namespace {

thread_local char g_err[256] = "";
std::atomic<uint64_t> g_launches{0};
constexpr uint32_t kDefaultWaitUs = 1000000;       // one second per device-side wait
std::atomic<uint32_t> g_wait_us{kDefaultWaitUs};
std::atomic<uint32_t> g_debug_stall{0};

kvs_status_t fail(kvs_status_t code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}

// ------------------------------------------------------------------------------- profiling
struct ProfRec { int kind; cudaEvent_t a, b; };
struct Profiler {
  bool on = false;
  std::vector<ProfRec> recs;
  std::vector<cudaEvent_t> pool;
  size_t used = 0;
  cudaEvent_t get() {
    if (used == pool.size()) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
      pool.push_back(e);
    }
    return pool[used++];
  }
} g_prof;

template <class F>
cudaError_t launch(int kind, cudaStream_t st, F&& f) {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (!g_prof.on) return f();
  cudaEvent_t a = g_prof.get(), b = g_prof.get();
  if (!a || !b) return f();
  cudaEventRecord(a, st);
  cudaError_t e = f();
  cudaEventRecord(b, st);
  g_prof.recs.push_back({kind, a, b});
  return e;
}

// ------------------------------------------------------------------------------- tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor whose innermost dimension is the 128-wide head dimension; a box is
// [64 elements x box_rows rows] with the 128-byte swizzle that the UMMA descriptors expect.
// dims/strides are given innermost first; strides (bytes) start at dimension 1.
bool make_tmap(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
               int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t gd[5], gs[4];
  cuuint32_t box[5], es[5];
  for (int i = 0; i < rank; ++i) { gd[i] = dims[i]; box[i] = 1; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gs[i] = strides_bytes[i];
  box[0] = 64;
  box[1] = (cuuint32_t)box_rows;
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gd, gs, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 5-D pair view of a bf16 cache [B,Hkv,n_max,128]: (channel, parity, slot / 2, head, sequence),
// slot = 2 * (slot / 2) + parity.  A box is [64 channels x 128 consecutive pairs] of one parity.
bool make_tmap_pairs(CUtensorMap* m, const void* base, int n_max, int Hkv, int B, int64_t st, int64_t sh, int64_t sb) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t npairs = (cuuint64_t)(n_max / 2 > 0 ? n_max / 2 : 1);
  cuuint64_t gd[5] = {KVS_D, 2, npairs, (cuuint64_t)Hkv, (cuuint64_t)B};
  cuuint64_t gs[4] = {(cuuint64_t)st * 2, (cuuint64_t)st * 4, (cuuint64_t)sh * 2, (cuuint64_t)sb * 2};
  cuuint32_t box[5] = {64, 1, 128, 1, 1}, es[5] = {1, 1, 1, 1, 1};
  if (n_max < 2) gd[1] = 1;
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), gd, gs, box, es,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

const char* kKindNames[KVS_K_COUNT] = {"attn_partials", "combine", "hessian_stats",
                                       "select", "merge_compact", "misc"};

// ------------------------------------------------------------------------------- validation
kvs_status_t check_params(const kvs_params_t* p) {
  if (!p) return fail(KVS_ERR_INVALID_ARG, "params is NULL");
  if (p->batch <= 0 || p->n_q_heads <= 0 || p->n_kv_heads <= 0)
    return fail(KVS_ERR_INVALID_ARG, "batch and head counts must be positive");
  if (p->head_dim != KVS_D) return fail(KVS_ERR_UNSUPPORTED, "head_dim must be 128");
  if (p->n_q_heads % p->n_kv_heads) return fail(KVS_ERR_INVALID_ARG, "n_q_heads %% n_kv_heads != 0");
  if (p->window <= 0) return fail(KVS_ERR_INVALID_ARG, "window must be positive");
  if (p->sink < 0 || p->recent < 0) return fail(KVS_ERR_INVALID_ARG, "sink/recent must be >= 0");
  if (p->causal && p->recent < p->window)
    return fail(KVS_ERR_INVALID_ARG, "causal window needs recent >= window");
  if (!(p->round_frac > 0.f && p->round_frac <= 1.f))
    return fail(KVS_ERR_INVALID_ARG, "round_frac must be in (0,1]");
  if (!(p->softmax_scale > 0.f) || !isfinite(p->softmax_scale))
    return fail(KVS_ERR_INVALID_ARG, "softmax_scale must be positive and finite");
  if (p->score_mode != 0 && p->score_mode != 1) return fail(KVS_ERR_INVALID_ARG, "score_mode must be 0 or 1");
  if (p->first_round < 0) return fail(KVS_ERR_INVALID_ARG, "first_round must be >= 0");
  const int G = p->n_q_heads / p->n_kv_heads;
  if ((int64_t)G * p->window > KVS_MAX_M)
    return fail(KVS_ERR_UNSUPPORTED, "group * window must be <= %d", KVS_MAX_M);
  return KVS_OK;
}

kvs_status_t check_strides(const kvs_params_t* p) {
  const int64_t s[6] = {p->k_stride_b, p->k_stride_h, p->k_stride_t,
                        p->v_stride_b, p->v_stride_h, p->v_stride_t};
  for (int i = 0; i < 6; ++i)
    if (s[i] < 0 || (s[i] % 8)) return fail(KVS_ERR_INVALID_ARG, "strides must be non-negative multiples of 8 elements");
  if (p->k_stride_t < KVS_D || p->v_stride_t < KVS_D)
    return fail(KVS_ERR_INVALID_ARG, "slot stride must be >= 128");
  return KVS_OK;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ------------------------------------------------------------------------------- schedule
void round_plan(const kvs_params_t* p, int n, int budget, int r, int* off, int* P, int* R) {
  *off = p->sink + (r & 1);
  int cand = (n - *off - p->recent) / 2;
  if (n - *off - p->recent < 0) cand = 0;
  *P = cand > 0 ? cand : 0;
  if (*P == 0) { *R = 0; return; }
  // floor(round_frac * P) evaluated in double from the float parameter
  int want = (int)floor((double)p->round_frac * (double)*P);
  if (want < 1) want = 1;
  const int excess = n - budget;
  *R = excess < want ? excess : want;
}

// ------------------------------------------------------------------------------- workspace
size_t align_up(size_t x) { return (x + 255) & ~(size_t)255; }

struct WsLayout {
  size_t part_ml, part_o, qstat, qc2, norms, o, o_hi, o_lo, score, w, mask, tile_prefix, part4, part1, sync, total;
  int splits_max, M_max, pair_stride, tile_stride, counter_stride, nqblk_w, U;
  size_t sync_bytes;
};

// Number of key/pair ranges each (query block, KV head, sequence) item is cut into.  The CTAs run
// one per SM in waves of 148; a CTA costs its tiles plus about two tile times of set-up and
// write-back.  The cut k that minimises  waves(items * k) * (ceil(tiles / k) + 2)  is taken (the
// smaller k when two are within 1 %): 512 items of 256 tiles: k = 2 (7 half-length waves instead
// of 4 full ones); 64 items of 1024 tiles: k = 9 (576 CTAs in 4 waves of 114 tiles instead of 128
// CTAs of 512 tiles on 148 SMs); 8 items of 16 tiles: k = 16.  When the CTAs need more than one
// wave, a range is not made shorter than 16 tiles: the pipeline of a CTA (three logit buffers, two
// K/V stages) takes a few tiles to fill, which the model's constant does not cover -- 512 items of
// 20 tiles ran 2.4 % faster uncut (4 waves of 20 tiles) than cut in two (7 waves of 10), while a
// larger constant instead slowed the long ragged items of the other workloads by up to 6 %.
constexpr int kNumSMs = 148;
constexpr int kMinRangeTiles = 16;  // (see above)
constexpr int kMaxTcSplits = 16;    // per item (more only while items * k <= 148); the attention partials are sized for it

int balanced_splits(int items, int ntiles, int* tiles_per_split) {
  if (items < 1) items = 1;
  if (ntiles < 1) ntiles = 1;
  int kmax = kNumSMs / items > kMaxTcSplits ? kNumSMs / items : kMaxTcSplits;
  if (kmax > ntiles) kmax = ntiles;
  int best = 1;
  double best_cost = 1e30;
  for (int k = 1; k <= kmax; ++k) {
    const int tps = (ntiles + k - 1) / k;
    const int ctas = items * ((ntiles + tps - 1) / tps);      // ranges that are not empty
    if (k > 1 && tps < kMinRangeTiles && ctas > kNumSMs) continue;
    const double cost = (double)((ctas + kNumSMs - 1) / kNumSMs) * (tps + 2);
    if (cost < best_cost * 0.99) { best_cost = cost; best = k; }
  }
  int tps = (ntiles + best - 1) / best;
  if (tps < 1) tps = 1;
  *tiles_per_split = tps;
  const int s = (ntiles + tps - 1) / tps;
  return s > 0 ? s : 1;
}

int tc_splits(int M, int Hkv, int nseq, int ntiles, int* tiles_per_split) {
  const int nqblk = (M + 127) / 128;
  return balanced_splits(nqblk * Hkv * nseq, ntiles, tiles_per_split);
}

// upper bound of the number of attention partials per query row (workspace sizing)
int splits_bound(int M, int Hkv) {
  const int nqblk = (M + 127) / 128;
  int s = (2 * 148 + nqblk * Hkv - 1) / (nqblk * Hkv);
  if (s < 1) s = 1;
  if (s > KVS_MAX_SPLITS) s = KVS_MAX_SPLITS;
  int tc = kNumSMs / (nqblk * Hkv);
  if (tc < kMaxTcSplits) tc = kMaxTcSplits;
  return s > tc ? s : tc;
}

WsLayout make_layout(const kvs_params_t* p, int n_max, int max_new) {
  WsLayout L;
  const int G = p->n_q_heads / p->n_kv_heads;
  const int Mw = G * p->window, Md = G * max_new;
  L.M_max = Mw > Md ? Mw : Md;
  const int sw = splits_bound(Mw, p->n_kv_heads), sd = max_new > 0 ? splits_bound(Md, p->n_kv_heads) : 0;
  const size_t rows_w = (size_t)sw * Mw, rows_d = (size_t)sd * Md;
  const size_t part_rows = rows_w > rows_d ? rows_w : rows_d;
  L.splits_max = sw > sd ? sw : sd;
  L.U = p->batch * p->n_kv_heads;
  L.pair_stride = n_max / 2 + 1;
  L.tile_stride = n_max / KVS_CTILE + 2;
  size_t o = 0;
  L.part_ml = o; o += align_up((size_t)L.U * part_rows * sizeof(float2));
  L.part_o = o;  o += align_up((size_t)L.U * part_rows * KVS_D * sizeof(float));
  L.qstat = o;   o += align_up((size_t)L.U * L.M_max * sizeof(float4));
  L.qc2 = o;     o += align_up((size_t)L.U * ((Mw + 127) / 128 * 128) * sizeof(float2));
  L.o = o;       o += align_up((size_t)L.U * L.M_max * KVS_D * sizeof(float));
  L.norms = o;   o += align_up((size_t)L.U * L.pair_stride * sizeof(float4));
  L.score = o;   o += align_up((size_t)L.U * L.pair_stride * sizeof(float));
  L.w = o;       o += align_up((size_t)L.U * L.pair_stride * sizeof(float));
  L.mask = o;    o += align_up((size_t)L.U * L.pair_stride);
  L.tile_prefix = o; o += align_up((size_t)L.U * L.tile_stride * sizeof(int32_t));
  L.o_hi = o;    o += align_up((size_t)L.U * L.M_max * KVS_D * sizeof(__nv_bfloat16));
  L.o_lo = o;    o += align_up((size_t)L.U * L.M_max * KVS_D * sizeof(__nv_bfloat16));
  L.nqblk_w = (Mw + 127) / 128;
  L.counter_stride = n_max / 128 + 2;
  // partial sums of every (query block, statistics group): five floats per candidate pair
  const size_t nsub = (size_t)L.nqblk_w * KVS_STATS_GROUPS;
  L.part4 = o;   o += align_up((size_t)L.U * nsub * L.pair_stride * sizeof(float4));
  L.part1 = o;   o += align_up((size_t)L.U * nsub * L.pair_stride * sizeof(float));
  // tickets [KVS_MAX_ROUNDS][U], flags [U][tile_stride], tile counters [U][counter_stride];
  // zeroed once per call
  L.sync = o;
  L.sync_bytes = align_up(((size_t)KVS_MAX_ROUNDS * L.U + (size_t)L.U * L.tile_stride +
                           (size_t)L.U * L.counter_stride) * sizeof(uint32_t));
  o += L.sync_bytes;
  L.total = o;
  return L;
}

CacheView make_view(const kvs_params_t* p, void* K, void* V, int32_t* counts, int n_max) {
  CacheView c;
  c.K = static_cast<__nv_bfloat16*>(K);
  c.V = static_cast<__nv_bfloat16*>(V);
  c.counts = counts;
  c.ksb = p->k_stride_b; c.ksh = p->k_stride_h; c.kst = p->k_stride_t;
  c.vsb = p->v_stride_b; c.vsh = p->v_stride_h; c.vst = p->v_stride_t;
  c.n_max = n_max;
  c.Hkv = p->n_kv_heads;
  return c;
}

#define CUDA_TRY(expr)                                                                   \
  do {                                                                                   \
    cudaError_t e_ = (expr);                                                             \
    if (e_ != cudaSuccess) return fail(KVS_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e_)); \
  } while (0)

struct Common {
  const kvs_params_t* p;
  WsLayout L;
  char* ws;
  cudaStream_t st;
  int G, Mw;
  int32_t* status_dev;
  const void* e_win;         // supplied loss gradient rows [B,Hq,W,128] (exact weight modes), else NULL
  int weight_mode;           // 0: summed norms; 1: exact with E; 2: exact without the coupling
  CUtensorMap tmK, tmV, tmQ, tmOhi, tmOlo, tmKp, tmVp, tmE;
};

// Attention partials of the query rows behind `tmQ` (a [U, M, 128] view) over the caches in `view`.
// Returns the number of partials per row through *n_part.
template <class LaunchFn>
kvs_status_t enqueue_flash(const kvs_params_t* p, char* ws, const WsLayout& L, cudaStream_t st,
                           const CacheView& view, int Wq, int M, int causal,
                           const RoundTable& tab, int nmax_slots, const CUtensorMap& tmK,
                           const CUtensorMap& tmV, const CUtensorMap& tmQ, int32_t* status_dev,
                           bool pair_norms, LaunchFn&& launch_fn, int* n_part) {
  FlashTcArgs ta;
  ta.Hkv = p->n_kv_heads; ta.M = M; ta.nqblk = (M + 127) / 128;
  // with pair norms the tiles start at -(off & 1), so that candidate pairs never straddle a tile
  const int ntiles = (nmax_slots + (pair_norms ? (tab.off & 1) : 0) + 127) / 128;
  ta.pair_norms = pair_norms ? reinterpret_cast<float4*>(ws + L.norms) : nullptr;
  ta.pair_stride = L.pair_stride;
  ta.splits = tc_splits(M, p->n_kv_heads, tab.nseq, ntiles, &ta.tiles_per_split);
  ta.Wq = Wq; ta.causal = causal; ta.scale_log2 = p->softmax_scale * 1.4426950408889634f;
  ta.n_max = view.n_max; ta.counts = view.counts;
  ta.part_ml = reinterpret_cast<float2*>(ws + L.part_ml);
  ta.part_o = reinterpret_cast<float*>(ws + L.part_o);
  ta.status_dev = status_dev;
  ta.wait_us = g_wait_us.load(); ta.debug_stall = g_debug_stall.load();
  *n_part = ta.splits;
  return launch_fn([&] { return kvs_launch_flash_tc(ta, tab, tmK, tmV, tmQ, st); });
}

// Tensor maps of one call: K and V caches [B,Hkv,n_max,128] with the caller's strides, the
// window queries and the two bf16 terms of the attention output as [U, M, 128].
kvs_status_t make_call_tmaps(Common* c, const void* K, const void* V, const void* q_win, int n_max) {
  const kvs_params_t* p = c->p;
  // the pair view covers floor(n_max / 2) slot pairs: with an odd capacity and no protected suffix
  // the last slot could be the right member of a candidate pair and lie outside the view
  if ((n_max & 1) && p->recent == 0) return fail(KVS_ERR_UNSUPPORTED, "an odd n_max needs recent >= 1");
  const uint64_t kd[4] = {KVS_D, (uint64_t)n_max, (uint64_t)p->n_kv_heads, (uint64_t)p->batch};
  const uint64_t ks[3] = {(uint64_t)p->k_stride_t * 2, (uint64_t)p->k_stride_h * 2, (uint64_t)p->k_stride_b * 2};
  const uint64_t vs[3] = {(uint64_t)p->v_stride_t * 2, (uint64_t)p->v_stride_h * 2, (uint64_t)p->v_stride_b * 2};
  const uint64_t qd[3] = {KVS_D, (uint64_t)c->Mw, (uint64_t)c->L.U};
  const uint64_t qs[2] = {KVS_D * 2, (uint64_t)c->Mw * KVS_D * 2};
  bool ok = make_tmap(&c->tmK, K, 4, kd, ks, 128) && make_tmap(&c->tmV, V, 4, kd, vs, 128) &&
            make_tmap(&c->tmQ, q_win, 3, qd, qs, 128) &&
            make_tmap(&c->tmOhi, c->ws + c->L.o_hi, 3, qd, qs, 128) &&
            make_tmap(&c->tmOlo, c->ws + c->L.o_lo, 3, qd, qs, 128) &&
            make_tmap_pairs(&c->tmKp, K, n_max, p->n_kv_heads, p->batch, p->k_stride_t, p->k_stride_h, p->k_stride_b) &&
            make_tmap_pairs(&c->tmVp, V, n_max, p->n_kv_heads, p->batch, p->v_stride_t, p->v_stride_h, p->v_stride_b);
  if (ok && c->e_win) ok = make_tmap(&c->tmE, c->e_win, 3, qd, qs, 128);
  if (!ok) return fail(KVS_ERR_CUDA, "cuTensorMapEncodeTiled failed or is unavailable");
  return KVS_OK;
}

// The statistics of one round for the sequences in `tab` (window attention partials,
// combine, Hessian statistics), and optionally the selection.
kvs_status_t enqueue_round_stats(const Common& c, const CacheView& view, const void* q_win,
                                 const RoundTable& tab, int nmax_slots, bool do_select,
                                 float* A, float* N1, float* N12, float* cosv, float* score_out,
                                 float* w_out, uint8_t* mask_out, float* o_out, float* lse_out) {
  const kvs_params_t* p = c.p;
  const float scale_log2 = p->softmax_scale * 1.4426950408889634f;
  int n_part = 0;
  {
    kvs_status_t fs = enqueue_flash(p, c.ws, c.L, c.st, view, p->window, c.Mw, p->causal, tab, nmax_slots,
                                    c.tmK, c.tmV, c.tmQ, c.status_dev, true,
                                    [&](auto&& f) -> kvs_status_t {
                                      CUDA_TRY(launch(KVS_K_FLASH, c.st, f));
                                      return KVS_OK;
                                    }, &n_part);
    if (fs != KVS_OK) return fs;
  }
  CombineArgs ca;
  ca.M = c.Mw; ca.splits = n_part; ca.Hkv = p->n_kv_heads;
  ca.part_ml = reinterpret_cast<float2*>(c.ws + c.L.part_ml);
  ca.part_o = reinterpret_cast<float*>(c.ws + c.L.part_o);
  ca.qstat = reinterpret_cast<float4*>(c.ws + c.L.qstat);
  ca.o = reinterpret_cast<float*>(c.ws + c.L.o);
  ca.o_hi = reinterpret_cast<__nv_bfloat16*>(c.ws + c.L.o_hi);
  ca.o_lo = reinterpret_cast<__nv_bfloat16*>(c.ws + c.L.o_lo);
  ca.qc2 = reinterpret_cast<float2*>(c.ws + c.L.qc2);
  ca.M_pad = (c.Mw + 127) / 128 * 128;
  ca.out_bf16 = nullptr; ca.lse_out = lse_out; ca.o_out = o_out;
  ca.e = c.weight_mode ? static_cast<const __nv_bfloat16*>(c.e_win) : nullptr;
  CUDA_TRY(launch(KVS_K_COMBINE, c.st, [&] { return kvs_launch_combine(ca, tab, c.st); }));

  StatsTcArgs ta;
  ta.Hkv = p->n_kv_heads; ta.M = c.Mw; ta.nqblk = (c.Mw + 127) / 128;
  int pmax = 0;
  for (int i = 0; i < tab.nseq; ++i) pmax = pmax > tab.s[i].P ? pmax : tab.s[i].P;
  const int ntiles = (pmax + 127) / 128;               // tiles of 128 candidate pairs
  ta.splits = balanced_splits(ta.nqblk * ta.Hkv * tab.nseq, ntiles, &ta.tiles_per_split);
  ta.n_max = view.n_max; ta.pair_stride = c.L.pair_stride;
  ta.scale_log2 = scale_log2; ta.score_mode = p->score_mode; ta.weight_mode = c.weight_mode;
  ta.counts = view.counts; ta.qc2 = ca.qc2; ta.M_pad = ca.M_pad;
  ta.pair_norms = reinterpret_cast<const float4*>(c.ws + c.L.norms); ta.norm_stride = c.L.pair_stride;
  ta.score = score_out ? score_out : reinterpret_cast<float*>(c.ws + c.L.score);
  ta.w = w_out ? w_out : reinterpret_cast<float*>(c.ws + c.L.w);
  ta.A = A; ta.N1 = N1; ta.N12 = N12; ta.cosv = cosv;
  ta.part4 = reinterpret_cast<float4*>(c.ws + c.L.part4);
  ta.part1 = reinterpret_cast<float*>(c.ws + c.L.part1);
  ta.status_dev = c.status_dev;
  ta.wait_us = g_wait_us.load(); ta.debug_stall = g_debug_stall.load();
  CUDA_TRY(launch(KVS_K_STATS, c.st, [&] {
    return kvs_launch_stats_tc(ta, tab, c.tmKp, c.tmVp, c.tmQ, c.weight_mode ? c.tmE : c.tmOhi, c.tmOlo, c.st);
  }));
  g_launches.fetch_add(1, std::memory_order_relaxed);   // (two kernels behind that call: the statistics and their finalize)

  if (do_select) {
    SelectArgs se;
    se.Hkv = p->n_kv_heads;
    se.pair_stride = c.L.pair_stride; se.tile_stride = c.L.tile_stride;
    se.score = ta.score;
    se.mask = mask_out ? mask_out : reinterpret_cast<uint8_t*>(c.ws + c.L.mask);
    se.tile_prefix = reinterpret_cast<int32_t*>(c.ws + c.L.tile_prefix);
    se.from_mask = 0;
    CUDA_TRY(launch(KVS_K_SELECT, c.st, [&] { return kvs_launch_select(se, tab, c.st); }));
  }
  return KVS_OK;
}

kvs_status_t check_common(const kvs_params_t* p, const void* K, const void* V, const int32_t* counts,
                          const int32_t* seq_len, int n_max, void* ws, size_t ws_bytes, int max_new,
                          Common* c, void* stream) {
  kvs_status_t s = check_params(p);
  if (s != KVS_OK) return s;
  s = check_strides(p);
  if (s != KVS_OK) return s;
  if (!K || !V || !counts || !seq_len || !ws) return fail(KVS_ERR_INVALID_ARG, "NULL pointer argument");
  if (!aligned16(K) || !aligned16(V)) return fail(KVS_ERR_INVALID_ARG, "K and V must be 16-byte aligned");
  if ((reinterpret_cast<uintptr_t>(ws) & 255u) != 0) return fail(KVS_ERR_INVALID_ARG, "workspace must be 256-byte aligned");
  if (n_max <= 0) return fail(KVS_ERR_INVALID_ARG, "n_max must be positive");
  for (int b = 0; b < p->batch; ++b) {
    if (seq_len[b] < 0 || seq_len[b] > n_max) return fail(KVS_ERR_INVALID_ARG, "seq_len[%d] out of range", b);
  }
  c->p = p;
  c->L = make_layout(p, n_max, max_new);
  if (ws_bytes < c->L.total) return fail(KVS_ERR_WORKSPACE, "workspace too small: %zu < %zu", ws_bytes, c->L.total);
  c->ws = static_cast<char*>(ws);
  c->st = static_cast<cudaStream_t>(stream);
  c->G = p->n_q_heads / p->n_kv_heads;
  c->Mw = c->G * p->window;
  c->status_dev = nullptr;
  c->e_win = nullptr;
  c->weight_mode = 0;
  return KVS_OK;
}

// The exact weight modes take a loss gradient row per window query, laid out like q_win.
kvs_status_t check_exact(const void* e_win, int weight_mode) {
  if (weight_mode == 0) return KVS_OK;
  if (weight_mode != 1 && weight_mode != 2) return fail(KVS_ERR_INVALID_ARG, "weight_mode must be 1 or 2");
  if (!e_win) return fail(KVS_ERR_INVALID_ARG, "e_win is NULL");
  if (!aligned16(e_win)) return fail(KVS_ERR_INVALID_ARG, "e_win must be 16-byte aligned");
  return KVS_OK;
}

}  // namespace

// =================================================================================== scratch-only compaction
kvs_status_t kvs_detail_fail(kvs_status_t code, const char* msg) { return fail(code, "%s", msg); }

// Scratch layout: tile_prefix int32 [U, tile_stride] | tickets uint32 [U] | flags uint32 [U, tile_stride].
kvs_status_t kvs_detail_compact_scratch(const kvs_params_t* p, void* K, void* V, int32_t* counts,
                                        const uint8_t* merge_mask, const float* w_left,
                                        const int32_t* seq_len, const int32_t* n_merge, int32_t n_max,
                                        int32_t* new_len, int32_t* new_index, void* scratch,
                                        size_t scratch_bytes, size_t* need_bytes, int32_t* status_dev,
                                        void* cuda_stream) {
  kvs_status_t s = check_params(p);
  if (s != KVS_OK) return s;
  s = check_strides(p);
  if (s != KVS_OK) return s;
  if (!K || !V || !counts || !seq_len || !scratch || !merge_mask || !w_left || !n_merge || !new_len)
    return fail(KVS_ERR_INVALID_ARG, "NULL pointer argument");
  if (!aligned16(K) || !aligned16(V)) return fail(KVS_ERR_INVALID_ARG, "K and V must be 16-byte aligned");
  if (n_max <= 0) return fail(KVS_ERR_INVALID_ARG, "n_max must be positive");
  const int B = p->batch, U = p->batch * p->n_kv_heads;
  for (int b = 0; b < B; ++b)
    if (seq_len[b] < 0 || seq_len[b] > n_max) return fail(KVS_ERR_INVALID_ARG, "seq_len[%d] out of range", b);
  const int tile_stride = n_max / KVS_CTILE + 2;
  const size_t prefix_bytes = align_up((size_t)U * tile_stride * sizeof(int32_t));
  const size_t sync_bytes = align_up(((size_t)U + (size_t)U * tile_stride) * sizeof(uint32_t));
  if (need_bytes) *need_bytes = prefix_bytes + sync_bytes;
  if (scratch_bytes < prefix_bytes + sync_bytes)
    return fail(KVS_ERR_WORKSPACE, "scratch too small: %zu < %zu bytes", scratch_bytes, prefix_bytes + sync_bytes);
  const int off = p->sink + (p->first_round & 1);
  std::vector<SeqRound> act;
  for (int b = 0; b < B; ++b) {
    const int n = seq_len[b];
    int P = (n - off - p->recent) / 2;
    if (n - off - p->recent < 0 || P < 0) P = 0;
    if (n_merge[b] < 0 || n_merge[b] > P) return fail(KVS_ERR_INVALID_ARG, "n_merge[%d] exceeds the candidate pairs", b);
    if (n_merge[b] > 0) act.push_back({n, P, n_merge[b], b});
  }
  for (int b = 0; b < B; ++b) new_len[b] = seq_len[b] - n_merge[b];
  if (act.empty() && !new_index) return KVS_OK;
  if (new_index)
    for (int b = 0; b < B; ++b)
      if (n_merge[b] == 0 && seq_len[b] > 0) {
        int P = (seq_len[b] - off - p->recent) / 2;
        if (P < 0) P = 0;
        act.push_back({seq_len[b], P, 0, b});
      }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  char* base = static_cast<char*>(scratch);
  int32_t* tile_prefix = reinterpret_cast<int32_t*>(base);
  uint32_t* tickets = reinterpret_cast<uint32_t*>(base + prefix_bytes);
  uint32_t* flags = tickets + U;
  // tickets and flags must start at zero; the array keeps whatever the previous call left
  CUDA_TRY(cudaMemsetAsync(base + prefix_bytes, 0, sync_bytes, st));
  const CacheView view = make_view(p, K, V, counts, n_max);
  const int caller_stride = n_max / 2;
  for (size_t k = 0; k < act.size(); k += KVS_SEQ_CHUNK) {
    RoundTable tab;
    tab.nseq = 0;
    tab.off = off;
    for (size_t u = k; u < act.size() && tab.nseq < KVS_SEQ_CHUNK; ++u) tab.s[tab.nseq++] = act[u];
    SelectArgs se;
    se.Hkv = p->n_kv_heads;
    se.pair_stride = caller_stride; se.tile_stride = tile_stride;
    se.score = nullptr;
    se.mask = const_cast<uint8_t*>(merge_mask);
    se.tile_prefix = tile_prefix;
    se.from_mask = 1;
    CUDA_TRY(launch(KVS_K_MISC, st, [&] { return kvs_launch_select(se, tab, st); }));
    CompactArgs ka;
    ka.c = view;
    ka.pair_stride = caller_stride; ka.tile_stride = tile_stride;
    ka.mask = merge_mask; ka.w = w_left;
    ka.tile_prefix = tile_prefix;
    ka.tickets = tickets;
    ka.flags = flags;
    ka.epoch = 1;
    ka.new_index = new_index;
    ka.status_dev = status_dev;
    ka.wait_us = g_wait_us.load(); ka.debug_stall = g_debug_stall.load();
    CUDA_TRY(launch(KVS_K_COMPACT, st, [&] { return kvs_launch_compact(ka, tab, st); }));
  }
  return KVS_OK;
}

// =================================================================================== C ABI
extern "C" {

int kvs_version(void) { return 100; }

const char* kvs_last_error_string(void) { return g_err; }

uint64_t kvs_launch_count(void) { return g_launches.load(); }

kvs_status_t kvs_debug_set_wait(uint32_t limit_us, uint32_t withhold) {
  if (withhold > 7u) return fail(KVS_ERR_INVALID_ARG, "withhold has three bits");
  g_wait_us.store(limit_us ? limit_us : kDefaultWaitUs);
  g_debug_stall.store(withhold);
  return KVS_OK;
}

kvs_status_t kvs_round_plan(const kvs_params_t* p, int32_t n, int32_t budget, int32_t max_rounds,
                            int32_t* n_r, int32_t* off_r, int32_t* P_r, int32_t* R_r,
                            int32_t* n_rounds) {
  kvs_status_t s = check_params(p);
  if (s != KVS_OK) return s;
  if (!n_rounds) return fail(KVS_ERR_INVALID_ARG, "n_rounds is NULL");
  if (n < 0 || budget < 1) return fail(KVS_ERR_INVALID_ARG, "n must be >= 0 and budget >= 1");
  int r = p->first_round, cnt = 0;
  while (n > budget) {
    int off, P, R;
    round_plan(p, n, budget, r, &off, &P, &R);
    if (P == 0) { *n_rounds = cnt; return fail(KVS_ERR_BUDGET_UNREACHABLE, "round %d has no candidate pair (n=%d)", r, n); }
    if (cnt < max_rounds) {
      if (n_r) n_r[cnt] = n;
      if (off_r) off_r[cnt] = off;
      if (P_r) P_r[cnt] = P;
      if (R_r) R_r[cnt] = R;
    }
    n -= R; ++r; ++cnt;
  }
  *n_rounds = cnt;
  if ((n_r || off_r || P_r || R_r) && cnt > max_rounds) return fail(KVS_ERR_WORKSPACE, "plan needs %d rounds", cnt);
  return KVS_OK;
}

kvs_status_t kvs_workspace_size(const kvs_params_t* p, int32_t max_seq_len, int32_t max_new,
                                size_t* bytes) {
  kvs_status_t s = check_params(p);
  if (s != KVS_OK) return s;
  if (!bytes || max_seq_len <= 0 || max_new < 0) return fail(KVS_ERR_INVALID_ARG, "bad size argument");
  const int G = p->n_q_heads / p->n_kv_heads;
  if ((int64_t)G * max_new > KVS_MAX_M) return fail(KVS_ERR_UNSUPPORTED, "group * max_new must be <= %d", KVS_MAX_M);
  *bytes = make_layout(p, max_seq_len, max_new).total;
  return KVS_OK;
}

namespace {

// The merge pass; with `chunk_k` the rows of a chunk are appended first (seq_len then counts them
// already, `cur_len` holds the slots in use before).  Everything the host can detect is detected
// before the first launch.
kvs_status_t merge_layer_impl(const kvs_params_t* p, void* K, void* V, int32_t* counts,
                              const void* q_win, const int32_t* seq_len, const int32_t* budget,
                              int32_t n_max, int32_t* new_len, void* workspace,
                              size_t workspace_bytes, int32_t* status_dev, void* cuda_stream,
                              const void* chunk_k, const void* chunk_v, int32_t chunk_len,
                              const int32_t* cur_len, const void* e_win = nullptr, int weight_mode = 0) {
  Common c;
  kvs_status_t s = check_common(p, K, V, counts, seq_len, n_max, workspace, workspace_bytes, 0, &c, cuda_stream);
  if (s != KVS_OK) return s;
  s = check_exact(e_win, weight_mode);
  if (s != KVS_OK) return s;
  c.e_win = e_win; c.weight_mode = weight_mode;
  if (!q_win || !budget || !new_len) return fail(KVS_ERR_INVALID_ARG, "NULL pointer argument");
  if (!aligned16(q_win)) return fail(KVS_ERR_INVALID_ARG, "q_win must be 16-byte aligned");
  const int B = p->batch;
  // plan every sequence first: nothing is enqueued if any sequence cannot reach its budget
  std::vector<std::vector<SeqRound>> plan(B);
  int rounds = 0;
  for (int b = 0; b < B; ++b) {
    if (budget[b] < 1) return fail(KVS_ERR_INVALID_ARG, "budget[%d] must be >= 1", b);
    int n = seq_len[b], r = p->first_round;
    if (n > budget[b] && n < p->window) return fail(KVS_ERR_INVALID_ARG, "seq_len[%d] < window", b);
    while (n > budget[b]) {
      int off, P, R;
      round_plan(p, n, budget[b], r, &off, &P, &R);
      if (P == 0) return fail(KVS_ERR_BUDGET_UNREACHABLE, "sequence %d: no candidate pair left at n=%d", b, n);
      plan[b].push_back({n, P, R, b});
      n -= R; ++r;
    }
    if ((int)plan[b].size() > rounds) rounds = (int)plan[b].size();
  }
  if (rounds > KVS_MAX_ROUNDS) return fail(KVS_ERR_UNSUPPORTED, "more than %d rounds", KVS_MAX_ROUNDS);
  for (int b = 0; b < B; ++b) new_len[b] = seq_len[b] < budget[b] ? seq_len[b] : budget[b];
  c.status_dev = status_dev;
  if (rounds > 0) {
    s = make_call_tmaps(&c, K, V, q_win, n_max);
    if (s != KVS_OK) return s;
  }
  const CacheView view = make_view(p, K, V, counts, n_max);
  if (chunk_k && chunk_len > 0) {
    AppendArgs aa;
    aa.c = view;
    aa.chunk_k = static_cast<const __nv_bfloat16*>(chunk_k);
    aa.chunk_v = static_cast<const __nv_bfloat16*>(chunk_v);
    aa.chunk_len = chunk_len;
    for (int b0 = 0; b0 < B; b0 += KVS_SEQ_CHUNK) {
      RoundTable tab;
      tab.nseq = 0;
      tab.off = 0;
      for (int b = b0; b < B && tab.nseq < KVS_SEQ_CHUNK; ++b) tab.s[tab.nseq++] = {cur_len[b], 0, 0, b};
      CUDA_TRY(launch(KVS_K_MISC, c.st, [&] { return kvs_launch_append(aa, tab, c.st); }));
    }
  }
  if (rounds == 0) return KVS_OK;
  CUDA_TRY(cudaMemsetAsync(c.ws + c.L.sync, 0, c.L.sync_bytes, c.st));
  uint32_t* tickets = reinterpret_cast<uint32_t*>(c.ws + c.L.sync);
  uint32_t* flags = tickets + (size_t)KVS_MAX_ROUNDS * c.L.U;

  for (int i = 0; i < rounds; ++i) {
    const int r = p->first_round + i;
    // active sequences of this round, in chunks of KVS_SEQ_CHUNK
    int b = 0;
    while (b < B) {
      RoundTable tab;
      tab.nseq = 0;
      tab.off = p->sink + (r & 1);
      int nmax_slots = 0;
      for (; b < B && tab.nseq < KVS_SEQ_CHUNK; ++b) {
        if ((int)plan[b].size() > i) {
          tab.s[tab.nseq++] = plan[b][i];
          if (plan[b][i].n > nmax_slots) nmax_slots = plan[b][i].n;
        }
      }
      if (tab.nseq == 0) continue;
      s = enqueue_round_stats(c, view, q_win, tab, nmax_slots, true, nullptr, nullptr, nullptr,
                              nullptr, nullptr, nullptr, nullptr, nullptr, nullptr);
      if (s != KVS_OK) return s;
      CompactArgs ka;
      ka.c = view;
      ka.pair_stride = c.L.pair_stride; ka.tile_stride = c.L.tile_stride;
      ka.mask = reinterpret_cast<const uint8_t*>(c.ws + c.L.mask);
      ka.w = reinterpret_cast<const float*>(c.ws + c.L.w);
      ka.tile_prefix = reinterpret_cast<const int32_t*>(c.ws + c.L.tile_prefix);
      ka.tickets = tickets + (size_t)i * c.L.U;
      ka.flags = flags;
      ka.epoch = (uint32_t)(i + 1);
      ka.new_index = nullptr;
      ka.status_dev = status_dev;
      ka.wait_us = g_wait_us.load(); ka.debug_stall = g_debug_stall.load();
    ka.wait_us = g_wait_us.load(); ka.debug_stall = g_debug_stall.load();
      CUDA_TRY(launch(KVS_K_COMPACT, c.st, [&] { return kvs_launch_compact(ka, tab, c.st); }));
    }
  }
  return KVS_OK;
}

}  // namespace

kvs_status_t kvs_merge_layer(const kvs_params_t* p, void* K, void* V, int32_t* counts,
                             const void* q_win, const int32_t* seq_len, const int32_t* budget,
                             int32_t n_max, int32_t* new_len, void* workspace,
                             size_t workspace_bytes, int32_t* status_dev, void* cuda_stream) {
  return merge_layer_impl(p, K, V, counts, q_win, seq_len, budget, n_max, new_len, workspace, workspace_bytes,
                          status_dev, cuda_stream, nullptr, nullptr, 0, nullptr);
}

kvs_status_t kvs_merge_layer_exact(const kvs_params_t* p, void* K, void* V, int32_t* counts,
                                   const void* q_win, const void* e_win, int32_t weight_mode,
                                   const int32_t* seq_len, const int32_t* budget, int32_t n_max,
                                   int32_t* new_len, void* workspace, size_t workspace_bytes,
                                   int32_t* status_dev, void* cuda_stream) {
  if (weight_mode != 1 && weight_mode != 2) return fail(KVS_ERR_INVALID_ARG, "weight_mode must be 1 or 2");
  return merge_layer_impl(p, K, V, counts, q_win, seq_len, budget, n_max, new_len, workspace, workspace_bytes,
                          status_dev, cuda_stream, nullptr, nullptr, 0, nullptr, e_win, weight_mode);
}

kvs_status_t kvs_append_and_merge(const kvs_params_t* p, void* K, void* V, int32_t* counts,
                                  const void* chunk_k, const void* chunk_v, int32_t chunk_len,
                                  const void* q_win, const int32_t* cur_len, const int32_t* budget,
                                  int32_t n_max, int32_t* new_len, void* workspace,
                                  size_t workspace_bytes, int32_t* status_dev, void* cuda_stream) {
  kvs_status_t s = check_params(p);
  if (s != KVS_OK) return s;
  if (!cur_len) return fail(KVS_ERR_INVALID_ARG, "NULL pointer argument");
  if (chunk_len < 0) return fail(KVS_ERR_INVALID_ARG, "chunk_len must be >= 0");
  if (chunk_len > 0 && (!chunk_k || !chunk_v)) return fail(KVS_ERR_INVALID_ARG, "NULL pointer argument");
  if (!aligned16(chunk_k) || !aligned16(chunk_v)) return fail(KVS_ERR_INVALID_ARG, "the chunk must be 16-byte aligned");
  std::vector<int32_t> seq_len(p->batch);
  for (int b = 0; b < p->batch; ++b) {
    if (cur_len[b] < 0 || cur_len[b] > n_max - chunk_len)
      return fail(KVS_ERR_INVALID_ARG, "cur_len[%d] + chunk_len exceeds n_max", b);
    seq_len[b] = cur_len[b] + chunk_len;
  }
  return merge_layer_impl(p, K, V, counts, q_win, seq_len.data(), budget, n_max, new_len, workspace,
                          workspace_bytes, status_dev, cuda_stream, chunk_k, chunk_v, chunk_len, cur_len);
}

kvs_status_t kvs_compact(const kvs_params_t* p, void* K, void* V, int32_t* counts,
                         const uint8_t* merge_mask, const float* w_left, const int32_t* seq_len,
                         const int32_t* n_merge, int32_t n_max, int32_t* new_len,
                         int32_t* new_index, void* workspace, size_t workspace_bytes,
                         int32_t* status_dev, void* cuda_stream) {
  Common c;
  kvs_status_t s = check_common(p, K, V, counts, seq_len, n_max, workspace, workspace_bytes, 0, &c, cuda_stream);
  if (s != KVS_OK) return s;
  if (!merge_mask || !w_left || !n_merge || !new_len) return fail(KVS_ERR_INVALID_ARG, "NULL pointer argument");
  const int B = p->batch;
  const int off = p->sink + (p->first_round & 1);
  std::vector<SeqRound> act;
  for (int b = 0; b < B; ++b) {
    const int n = seq_len[b];
    int P = (n - off - p->recent) / 2;
    if (n - off - p->recent < 0 || P < 0) P = 0;
    if (n_merge[b] < 0 || n_merge[b] > P) return fail(KVS_ERR_INVALID_ARG, "n_merge[%d] exceeds the candidate pairs", b);
    if (n_merge[b] > 0) act.push_back({n, P, n_merge[b], b});
  }
  for (int b = 0; b < B; ++b) new_len[b] = seq_len[b] - n_merge[b];
  if (act.empty() && !new_index) return KVS_OK;
  if (new_index)   // sequences without a merge still need the identity map
    for (int b = 0; b < B; ++b)
      if (n_merge[b] == 0 && seq_len[b] > 0) {
        int P = (seq_len[b] - off - p->recent) / 2;
        if (P < 0) P = 0;
        act.push_back({seq_len[b], P, 0, b});
      }
  CUDA_TRY(cudaMemsetAsync(c.ws + c.L.sync, 0, c.L.sync_bytes, c.st));
  uint32_t* tickets = reinterpret_cast<uint32_t*>(c.ws + c.L.sync);
  uint32_t* flags = tickets + (size_t)KVS_MAX_ROUNDS * c.L.U;
  const CacheView view = make_view(p, K, V, counts, n_max);
  // the caller's mask is laid out [B,Hkv,n_max/2]; the kernels use pair_stride rows, so the
  // mask and weights are consumed in place with the caller's stride
  const int caller_stride = n_max / 2;
  int chunk_id = 0;
  for (size_t k = 0; k < act.size(); k += KVS_SEQ_CHUNK, ++chunk_id) {
    RoundTable tab;
    tab.nseq = 0;
    tab.off = off;
    for (size_t u = k; u < act.size() && tab.nseq < KVS_SEQ_CHUNK; ++u) tab.s[tab.nseq++] = act[u];
    SelectArgs se;
    se.Hkv = p->n_kv_heads;
    se.pair_stride = caller_stride; se.tile_stride = c.L.tile_stride;
    se.score = nullptr;
    se.mask = const_cast<uint8_t*>(merge_mask);
    se.tile_prefix = reinterpret_cast<int32_t*>(c.ws + c.L.tile_prefix);
    se.from_mask = 1;
    CUDA_TRY(launch(KVS_K_MISC, c.st, [&] { return kvs_launch_select(se, tab, c.st); }));
    CompactArgs ka;
    ka.c = view;
    ka.pair_stride = caller_stride; ka.tile_stride = c.L.tile_stride;
    ka.mask = merge_mask; ka.w = w_left;
    ka.tile_prefix = se.tile_prefix;
    ka.tickets = tickets;   // distinct sequences per chunk: one ticket row serves all chunks
    ka.flags = flags;
    ka.epoch = 1;
    ka.new_index = new_index;
    ka.status_dev = status_dev;
    ka.wait_us = g_wait_us.load(); ka.debug_stall = g_debug_stall.load();
    CUDA_TRY(launch(KVS_K_COMPACT, c.st, [&] { return kvs_launch_compact(ka, tab, c.st); }));
  }
  return KVS_OK;
}

kvs_status_t kvs_decode_attn(const kvs_params_t* p, const void* q_new, int32_t n_new, const void* K,
                             const void* V, const int32_t* counts, const int32_t* seq_len,
                             int32_t n_max, void* out, float* lse, void* workspace,
                             size_t workspace_bytes, int32_t* status_dev, void* cuda_stream) {
  if (n_new <= 0) return fail(KVS_ERR_INVALID_ARG, "n_new must be positive");
  if (p && p->n_kv_heads > 0 && (int64_t)(p->n_q_heads / p->n_kv_heads) * n_new > KVS_MAX_M)
    return fail(KVS_ERR_UNSUPPORTED, "group * n_new must be <= %d", KVS_MAX_M);
  Common c;
  kvs_status_t s = check_common(p, K, V, counts, seq_len, n_max, workspace, workspace_bytes, n_new, &c, cuda_stream);
  if (s != KVS_OK) return s;
  if (!q_new || !out) return fail(KVS_ERR_INVALID_ARG, "NULL pointer argument");
  if (!aligned16(q_new) || !aligned16(out)) return fail(KVS_ERR_INVALID_ARG, "q_new/out must be 16-byte aligned");
  const int B = p->batch;
  const int M = c.G * n_new;
  const CacheView view = make_view(p, const_cast<void*>(K), const_cast<void*>(V), const_cast<int32_t*>(counts), n_max);
  CUtensorMap tmK, tmV, tmQ;
  {
    const uint64_t kd[4] = {KVS_D, (uint64_t)n_max, (uint64_t)p->n_kv_heads, (uint64_t)p->batch};
    const uint64_t ks[3] = {(uint64_t)p->k_stride_t * 2, (uint64_t)p->k_stride_h * 2, (uint64_t)p->k_stride_b * 2};
    const uint64_t vs[3] = {(uint64_t)p->v_stride_t * 2, (uint64_t)p->v_stride_h * 2, (uint64_t)p->v_stride_b * 2};
    const uint64_t qd[3] = {KVS_D, (uint64_t)M, (uint64_t)c.L.U};
    const uint64_t qs[2] = {KVS_D * 2, (uint64_t)M * KVS_D * 2};
    if (!(make_tmap(&tmK, K, 4, kd, ks, 128) && make_tmap(&tmV, V, 4, kd, vs, 128) &&
          make_tmap(&tmQ, q_new, 3, qd, qs, 128)))
      return fail(KVS_ERR_CUDA, "cuTensorMapEncodeTiled failed or is unavailable");
  }
  for (int b0 = 0; b0 < B; b0 += KVS_SEQ_CHUNK) {
    RoundTable tab;
    tab.nseq = 0; tab.off = 0;
    int nmax_slots = 0;
    for (int b = b0; b < B && b < b0 + KVS_SEQ_CHUNK; ++b) {
      if (seq_len[b] <= 0) continue;
      tab.s[tab.nseq++] = {seq_len[b], 0, 0, b};
      if (seq_len[b] > nmax_slots) nmax_slots = seq_len[b];
    }
    if (tab.nseq == 0) continue;
    int n_part = 0;
    s = enqueue_flash(p, c.ws, c.L, c.st, view, n_new, M, 0, tab, nmax_slots, tmK, tmV, tmQ, status_dev, false,
                      [&](auto&& f) -> kvs_status_t {
                        CUDA_TRY(launch(KVS_K_FLASH, c.st, f));
                        return KVS_OK;
                      }, &n_part);
    if (s != KVS_OK) return s;
    CombineArgs ca;
    ca.M = M; ca.splits = n_part; ca.Hkv = p->n_kv_heads;
    ca.part_ml = reinterpret_cast<float2*>(c.ws + c.L.part_ml);
    ca.part_o = reinterpret_cast<float*>(c.ws + c.L.part_o);
    ca.qstat = nullptr; ca.qc2 = nullptr; ca.M_pad = 0; ca.o = nullptr; ca.o_hi = nullptr; ca.o_lo = nullptr;
    ca.out_bf16 = static_cast<__nv_bfloat16*>(out);
    ca.lse_out = lse; ca.o_out = nullptr; ca.e = nullptr;
    CUDA_TRY(launch(KVS_K_COMBINE, c.st, [&] { return kvs_launch_combine(ca, tab, c.st); }));
  }
  return KVS_OK;
}

namespace {

kvs_status_t window_stats_impl(const kvs_params_t* p, const void* K, const void* V,
                               const int32_t* counts, const void* q_win, const int32_t* seq_len,
                               const int32_t* budget, int32_t n_max, float* A, float* N1, float* N12,
                               float* cosv, float* score, float* w, uint8_t* mask, float* o_win,
                               float* lse_win, void* workspace, size_t workspace_bytes,
                               int32_t* status_dev, void* cuda_stream, const void* e_win, int weight_mode) {
  Common c;
  kvs_status_t s = check_common(p, K, V, counts, seq_len, n_max, workspace, workspace_bytes, 0, &c, cuda_stream);
  if (s != KVS_OK) return s;
  s = check_exact(e_win, weight_mode);
  if (s != KVS_OK) return s;
  c.e_win = e_win; c.weight_mode = weight_mode;
  if (!q_win || !budget) return fail(KVS_ERR_INVALID_ARG, "NULL pointer argument");
  const int B = p->batch;
  const int r = p->first_round;
  std::vector<SeqRound> act;
  for (int b = 0; b < B; ++b) {
    if (seq_len[b] <= budget[b]) continue;
    if (seq_len[b] < p->window) return fail(KVS_ERR_INVALID_ARG, "seq_len[%d] < window", b);
    int off, P, R;
    round_plan(p, seq_len[b], budget[b], r, &off, &P, &R);
    if (P == 0) return fail(KVS_ERR_BUDGET_UNREACHABLE, "sequence %d: no candidate pair at n=%d", b, seq_len[b]);
    act.push_back({seq_len[b], P, R, b});
  }
  // outputs use the caller's row lengths: per-slot n_max, per-pair n_max/2.  The internal
  // pair arrays use pair_stride, so diagnostics are written with the caller's stride by
  // running the kernels on a layout whose pair_stride is n_max/2.
  c.status_dev = status_dev;
  if (act.empty()) return KVS_OK;
  s = make_call_tmaps(&c, K, V, q_win, n_max);
  if (s != KVS_OK) return s;
  CUDA_TRY(cudaMemsetAsync(c.ws + c.L.sync, 0, c.L.sync_bytes, c.st));
  Common cc = c;
  cc.L.pair_stride = n_max / 2;
  const CacheView view = make_view(p, const_cast<void*>(K), const_cast<void*>(V), const_cast<int32_t*>(counts), n_max);
  for (size_t k = 0; k < act.size(); k += KVS_SEQ_CHUNK) {
    RoundTable tab;
    tab.nseq = 0;
    tab.off = p->sink + (r & 1);
    int nmax_slots = 0;
    for (size_t u = k; u < act.size() && tab.nseq < KVS_SEQ_CHUNK; ++u) {
      tab.s[tab.nseq++] = act[u];
      if (act[u].n > nmax_slots) nmax_slots = act[u].n;
    }
    s = enqueue_round_stats(cc, view, q_win, tab, nmax_slots, mask != nullptr, A, N1, N12, cosv,
                            score, w, mask, o_win, lse_win);
    if (s != KVS_OK) return s;
  }
  return KVS_OK;
}

}  // namespace

kvs_status_t kvs_window_stats(const kvs_params_t* p, const void* K, const void* V,
                              const int32_t* counts, const void* q_win, const int32_t* seq_len,
                              const int32_t* budget, int32_t n_max, float* A, float* N1, float* N12,
                              float* cosv, float* score, float* w, uint8_t* mask, float* o_win,
                              float* lse_win, void* workspace, size_t workspace_bytes,
                              int32_t* status_dev, void* cuda_stream) {
  return window_stats_impl(p, K, V, counts, q_win, seq_len, budget, n_max, A, N1, N12, cosv, score, w, mask, o_win,
                           lse_win, workspace, workspace_bytes, status_dev, cuda_stream, nullptr, 0);
}

kvs_status_t kvs_window_stats_exact(const kvs_params_t* p, const void* K, const void* V,
                                    const int32_t* counts, const void* q_win, const void* e_win,
                                    int32_t weight_mode, const int32_t* seq_len, const int32_t* budget,
                                    int32_t n_max, float* A, float* g_self, float* g_pair, float* cosv,
                                    float* score, float* w, uint8_t* mask, void* workspace,
                                    size_t workspace_bytes, int32_t* status_dev, void* cuda_stream) {
  if (weight_mode != 1 && weight_mode != 2) return fail(KVS_ERR_INVALID_ARG, "weight_mode must be 1 or 2");
  return window_stats_impl(p, K, V, counts, q_win, seq_len, budget, n_max, A, g_self, g_pair, cosv, score, w, mask,
                           nullptr, nullptr, workspace, workspace_bytes, status_dev, cuda_stream, e_win, weight_mode);
}

namespace {

// Per-head lengths: every (sequence, KV head) becomes a sequence of its own with one KV head and
// the G query heads of its group.  The caches, counts and queries keep their memory layout; only
// the way it is indexed changes, which needs the head stride to tile the sequence stride.
kvs_status_t remap_per_head(const kvs_params_t* p, kvs_params_t* q) {
  kvs_status_t s = check_params(p);
  if (s != KVS_OK) return s;
  if ((int64_t)p->batch * p->n_kv_heads > INT32_MAX) return fail(KVS_ERR_UNSUPPORTED, "too many (sequence, head) units");
  if (p->batch > 1 && (p->k_stride_b != p->k_stride_h * p->n_kv_heads || p->v_stride_b != p->v_stride_h * p->n_kv_heads))
    return fail(KVS_ERR_UNSUPPORTED, "per-head lengths need stride_b == n_kv_heads * stride_h");
  *q = *p;
  q->batch = p->batch * p->n_kv_heads;
  q->n_q_heads = p->n_q_heads / p->n_kv_heads;
  q->n_kv_heads = 1;
  q->k_stride_b = p->k_stride_h; q->v_stride_b = p->v_stride_h;
  return KVS_OK;
}

}  // namespace

kvs_status_t kvs_workspace_size_per_head(const kvs_params_t* p, int32_t n_max, int32_t max_new, size_t* bytes) {
  kvs_params_t q;
  kvs_status_t s = remap_per_head(p, &q);
  if (s != KVS_OK) return s;
  return kvs_workspace_size(&q, n_max, max_new, bytes);
}

kvs_status_t kvs_merge_layer_per_head(const kvs_params_t* p, void* K, void* V, int32_t* counts,
                                      const void* q_win, const int32_t* seq_len, const int32_t* budget,
                                      int32_t n_max, int32_t* new_len, void* workspace,
                                      size_t workspace_bytes, int32_t* status_dev, void* cuda_stream) {
  kvs_params_t q;
  kvs_status_t s = remap_per_head(p, &q);
  if (s != KVS_OK) return s;
  return kvs_merge_layer(&q, K, V, counts, q_win, seq_len, budget, n_max, new_len, workspace, workspace_bytes,
                         status_dev, cuda_stream);
}

kvs_status_t kvs_decode_attn_per_head(const kvs_params_t* p, const void* q_new, int32_t n_new, const void* K,
                                      const void* V, const int32_t* counts, const int32_t* seq_len,
                                      int32_t n_max, void* out, float* lse, void* workspace,
                                      size_t workspace_bytes, int32_t* status_dev, void* cuda_stream) {
  kvs_params_t q;
  kvs_status_t s = remap_per_head(p, &q);
  if (s != KVS_OK) return s;
  return kvs_decode_attn(&q, q_new, n_new, K, V, counts, seq_len, n_max, out, lse, workspace, workspace_bytes,
                         status_dev, cuda_stream);
}

kvs_status_t kvs_adjacent_cosine(const void* x, int32_t batch, int32_t n_heads, int32_t n_max,
                                 int64_t stride_b, int64_t stride_h, int64_t stride_t,
                                 const int32_t* seq_len, float* cos_out, void* cuda_stream) {
  if (!x || !seq_len || !cos_out) return fail(KVS_ERR_INVALID_ARG, "NULL pointer argument");
  if (batch <= 0 || n_heads <= 0 || n_max <= 0) return fail(KVS_ERR_INVALID_ARG, "sizes must be positive");
  if (n_heads > 65535) return fail(KVS_ERR_UNSUPPORTED, "more than 65535 heads");
  if (!aligned16(x)) return fail(KVS_ERR_INVALID_ARG, "x must be 16-byte aligned");
  const int64_t s[3] = {stride_b, stride_h, stride_t};
  for (int i = 0; i < 3; ++i)
    if (s[i] < 0 || (s[i] % 8)) return fail(KVS_ERR_INVALID_ARG, "strides must be non-negative multiples of 8 elements");
  if (stride_t < KVS_D) return fail(KVS_ERR_INVALID_ARG, "row stride must be >= 128");
  for (int b = 0; b < batch; ++b)
    if (seq_len[b] < 0 || seq_len[b] > n_max) return fail(KVS_ERR_INVALID_ARG, "seq_len[%d] out of range", b);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  for (int b0 = 0; b0 < batch; b0 += KVS_SEQ_CHUNK) {
    RoundTable tab;
    tab.nseq = 0; tab.off = 0;
    for (int b = b0; b < batch && tab.nseq < KVS_SEQ_CHUNK; ++b)
      if (seq_len[b] >= 2) tab.s[tab.nseq++] = {seq_len[b], 0, 0, b};
    if (tab.nseq == 0) continue;
    CUDA_TRY(launch(KVS_K_MISC, st, [&] {
      return kvs_launch_adjacent_cosine(x, stride_b, stride_h, stride_t, n_heads, n_max, cos_out, tab, st);
    }));
  }
  return KVS_OK;
}

kvs_status_t kvs_probe_sfu(int32_t blocks, int32_t iters, float* sink_dev, uint64_t* ops, void* cuda_stream) {
  if (blocks <= 0 || iters <= 0 || !sink_dev) return fail(KVS_ERR_INVALID_ARG, "bad probe argument");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  CUDA_TRY(launch(KVS_K_MISC, st, [&] { return kvs_launch_sfu_probe(blocks, iters, sink_dev, st); }));
  if (ops) *ops = (uint64_t)blocks * 1024ull * 16ull * (uint64_t)iters;
  return KVS_OK;
}

kvs_status_t kvs_probe_mma(int32_t blocks, int32_t n_cols, int32_t reuse_a, int32_t products, int64_t* cycles_dev,
                           void* cuda_stream) {
  const bool n_ok = n_cols == 16 || n_cols == 32 || n_cols == 64 || n_cols == 128 || n_cols == 256;
  if (blocks <= 0 || blocks > 65535 || !n_ok || products < 8 || products > (1 << 20) || (products & 7) || !cycles_dev)
    return fail(KVS_ERR_INVALID_ARG, "bad probe argument");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  CUDA_TRY(launch(KVS_K_MISC, st, [&] {
    return kvs_launch_mma_probe(blocks, n_cols, reuse_a ? 1 : 0, products, g_wait_us.load(),
                                reinterpret_cast<long long*>(cycles_dev), st);
  }));
  return KVS_OK;
}

kvs_status_t kvs_profile_begin(void) {
  g_prof.on = true;
  g_prof.recs.clear();
  g_prof.used = 0;
  return KVS_OK;
}

kvs_status_t kvs_profile_end(int32_t n_kinds, float* ms, int32_t* launches) {
  g_prof.on = false;
  if (n_kinds < 0 || (n_kinds > 0 && (!ms || !launches))) return fail(KVS_ERR_INVALID_ARG, "bad profile buffers");
  for (int k = 0; k < n_kinds; ++k) { ms[k] = 0.f; launches[k] = 0; }
  for (const ProfRec& r : g_prof.recs) {
    CUDA_TRY(cudaEventSynchronize(r.b));
    float t = 0.f;
    CUDA_TRY(cudaEventElapsedTime(&t, r.a, r.b));
    if (r.kind < n_kinds) { ms[r.kind] += t; launches[r.kind] += 1; }
  }
  g_prof.recs.clear();
  g_prof.used = 0;
  return KVS_OK;
}

const char* kvs_profile_kind_name(int32_t kind) {
  return (kind >= 0 && kind < KVS_K_COUNT) ? kKindNames[kind] : nullptr;
}

}  // extern "C"
