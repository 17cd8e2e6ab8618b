// Internal declarations shared by the translation units of libkvs.so.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "kvs.h"

#define KVS_D 128                 // head dimension
#define KVS_SEQ_CHUNK 128         // sequences handled by one launch (kernel-parameter table of 2 KB)
#define KVS_MAX_M 1024            // query rows per KV head (group * window or group * n_new)
#define KVS_MAX_SPLITS 64         // key splits of the attention partials
#define KVS_MAX_ROUNDS 64
#define KVS_CTILE 64              // slots per compaction tile (32 candidate pairs)
#define KVS_SPIN_LIMIT (1 << 22)  // iterations of any device-side wait before it gives up
#define KVS_STATS_GROUPS 3        // statistics groups per query block: each writes its own partial sums

// ----------------------------------------------------------------------------- kernel kinds
enum KvsKernelKind {
  KVS_K_FLASH = 0,     // window / decode attention partials
  KVS_K_COMBINE = 1,   // partial combine
  KVS_K_STATS = 2,     // Hessian statistics + cosine + score + weight
  KVS_K_SELECT = 3,    // exact R-smallest selection + tile prefix
  KVS_K_COMPACT = 4,   // merge + in-place compaction
  KVS_K_MISC = 5,      // mask scan for kvs_compact, chunk append, similarity diagnostics
  KVS_K_COUNT = 6
};

// ----------------------------------------------------------------------------- launch tables
struct SeqRound {
  int32_t n;   // slots in use at the start of the round (0: sequence inactive)
  int32_t P;   // candidate pairs
  int32_t R;   // pairs to merge
  int32_t b;   // sequence index in the caller's batch
};

struct RoundTable {
  int32_t nseq;  // entries used
  int32_t off;   // first candidate slot: sink + (round mod 2)
  SeqRound s[KVS_SEQ_CHUNK];
};

struct CacheView {
  __nv_bfloat16* K;
  __nv_bfloat16* V;
  int32_t* counts;
  int64_t ksb, ksh, kst, vsb, vsh, vst;
  int32_t n_max;   // slot capacity (counts row length)
  int32_t Hkv;
};

struct FlashTcArgs {
  int32_t Hkv, M, nqblk, splits, tiles_per_split;
  int32_t Wq, causal;
  float scale_log2;
  int32_t n_max;
  const int32_t* counts;   // [U, n_max]
  float2* part_ml;         // [U, splits, M]
  float* part_o;           // [U, splits, M, 128]
  float4* pair_norms;      // optional [U, pair_stride]: (|vbar_l|^2, |vbar_r|^2, |vbar_l + vbar_r|^2, cos(K_l, K_r))
  int32_t pair_stride;     //   of the round's candidate pairs; tiles are then aligned with the pairs
  int32_t* status_dev;
  uint32_t wait_us;        // time limit of one device-side wait, microseconds
  uint32_t debug_stall;    // test hook (kvs_debug_set_wait): bit 0 = the producer withholds the K tiles
};

struct CombineArgs {
  int32_t M, splits, Hkv;
  const float2* part_ml;
  const float* part_o;
  float4* qstat;           // [U, M]: (max log2, Z, |o|^2, lse natural)
  float2* qc2;             // [U, M_pad]: (-(max + log2 Z), |o|^2); rows M..M_pad-1 get (-inf, 0) (may be NULL)
  int32_t M_pad;           // M rounded up to a multiple of 128 (grid rows when qc2 is written)
  float* o;                // [U, M, 128] fp32 (may be NULL)
  __nv_bfloat16* o_hi;     // [U, M, 128]: o = o_hi + o_lo to ~2^-17 relative (may be NULL)
  __nv_bfloat16* o_lo;
  __nv_bfloat16* out_bf16; // decode: [B, Hq, n_new, 128] == [U, M, 128] (may be NULL)
  float* lse_out;          // optional [U, M]
  float* o_out;            // optional diagnostic copy [U, M, 128]
  const __nv_bfloat16* e;  // optional loss gradient rows [U, M, 128]: qc2.y then holds <E_q, o_q> instead of |o_q|^2
};

struct StatsTcArgs {
  int32_t Hkv, M, nqblk, splits, tiles_per_split;
  int32_t n_max, pair_stride;
  float scale_log2;
  int32_t score_mode;
  int32_t weight_mode;     // 0: summed norms (Eq. kstar_final); 1: exact, supplied E; 2: exact without the coupling
  const int32_t* counts;   // [U, n_max]
  const float2* qc2;       // [U, M_pad]: (-(max + log2 Z), |o|^2), or (-(max + log2 Z), <E, o>) with a supplied E
  int32_t M_pad;
  float* score;            // [U, pair_stride]
  float* w;
  float* A;                // optional diagnostics [U, n_max]
  float* N1;
  float* N12;              // optional [U, pair_stride]
  float* cosv;
  float4* part4;           // [U, nqblk * KVS_STATS_GROUPS, pair_stride]: partial (A_l, A_r, N1_l, N1_r) of a pair
  float* part1;            // [U, nqblk * KVS_STATS_GROUPS, pair_stride]: partial N12
  const float4* pair_norms; // [U, norm_stride] from the attention pass
  int32_t norm_stride;
  int32_t* status_dev;
  uint32_t wait_us;        // time limit of one device-side wait, microseconds
  uint32_t debug_stall;    // test hook: bit 1 = the producer withholds the K tiles
};

struct SelectArgs {
  int32_t Hkv;
  int32_t pair_stride;
  int32_t tile_stride;     // row length of tile_prefix
  const float* score;
  uint8_t* mask;           // [U, pair_stride]
  int32_t* tile_prefix;    // [U, tile_stride]: merged pairs before each compaction tile
  int32_t from_mask;       // 1: mask is an input (kvs_compact), only the prefix is built
};

struct CompactArgs {
  CacheView c;
  int32_t pair_stride, tile_stride;
  const uint8_t* mask;
  const float* w;
  const int32_t* tile_prefix;
  uint32_t* tickets;       // [U] zero at launch
  uint32_t* flags;         // [U, tile_stride]; value >= epoch means "tile loaded"
  uint32_t epoch;
  int32_t* new_index;      // optional [U, n_max]
  int32_t* status_dev;
  uint32_t wait_us;        // time limit of one device-side wait, microseconds
  uint32_t debug_stall;    // test hook: bit 2 = "tile loaded" flags are not published
};

// ----------------------------------------------------------------------------- launchers
// Each returns the cudaError_t of its launch.  `nseq_units` = table.nseq * Hkv.
cudaError_t kvs_launch_combine(const CombineArgs& a, const RoundTable& t, cudaStream_t st);
// tmKp / tmVp: 5-D pair views [128, parity, slot / 2, head, sequence] of the caches; with
// weight_mode != 0, tmOhi is the map of the supplied gradient rows E and tmOlo is not used
cudaError_t kvs_launch_stats_tc(const StatsTcArgs& a, const RoundTable& t, const CUtensorMap& tmKp,
                                const CUtensorMap& tmVp, const CUtensorMap& tmQ, const CUtensorMap& tmOhi,
                                const CUtensorMap& tmOlo, cudaStream_t st);
cudaError_t kvs_launch_flash_tc(const FlashTcArgs& a, const RoundTable& t, const CUtensorMap& tmK,
                                const CUtensorMap& tmV, const CUtensorMap& tmQ, cudaStream_t st);
// Chunk of fresh tokens appended after the slots in use (table entry n = slots in use).
struct AppendArgs {
  CacheView c;
  const __nv_bfloat16* chunk_k;   // [B, Hkv, chunk_len, 128] contiguous
  const __nv_bfloat16* chunk_v;
  int32_t chunk_len;
};
cudaError_t kvs_launch_append(const AppendArgs& a, const RoundTable& t, cudaStream_t st);
cudaError_t kvs_launch_select(const SelectArgs& a, const RoundTable& t, cudaStream_t st);
// Adjacent-row cosine of a bf16 tensor [B, H, n_max, 128] (element strides sb, sh, st); table entry n = rows in use.
cudaError_t kvs_launch_adjacent_cosine(const void* x, int64_t sb, int64_t sh, int64_t st, int H, int n_max,
                                       float* out, const RoundTable& t, cudaStream_t stream);
cudaError_t kvs_launch_compact(const CompactArgs& a, const RoundTable& t, cudaStream_t st);

// Runs a per-device set-up call (raising a kernel's dynamic shared-memory limit) once for every
// device ordinal that launches through it: the attribute belongs to the device's copy of the kernel.
struct KvsPerDeviceOnce {
  std::atomic<unsigned char> done[64] = {};
  template <class F>
  cudaError_t run(F&& f) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return f();      // beyond the table: set up on every launch
    if (done[dev].load(std::memory_order_acquire)) return cudaSuccess;
    e = f();
    if (e == cudaSuccess) done[dev].store(1, std::memory_order_release);
    return e;
  }
};

// Launch of a kernel of the round chain with programmatic dependent launch: the kernel may be
// scheduled while the kernel before it in the stream is still draining (its set-up then overlaps
// that kernel's last CTAs and the launch latency), and it calls kvs_pdl_wait() before it touches
// global memory -- EVERY CTA does, also one that has nothing to do, so that a kernel never completes
// before its predecessor and the chain stays ordered end to end.
#ifdef __CUDACC__
template <typename... KArgs, typename... Args>
inline cudaError_t kvs_launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                      Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
// Device side: let the next kernel of the stream be scheduled (it will wait for this grid to
// complete before it reads anything) ...
__device__ __forceinline__ void kvs_pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
// ... and wait until the kernels before this one have completed and their writes are visible.
__device__ __forceinline__ void kvs_pdl_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
#endif

// Special-function probe: `blocks` CTAs of 1024 threads, 16 * iters operations per thread.
cudaError_t kvs_launch_sfu_probe(int blocks, int iters, float* sink, cudaStream_t st);
// Operand-feed probe: `blocks` CTAs, each `products` (a multiple of 8) tcgen05 products of shape
// 128 x n_cols x 16 with both operands in shared memory; cycles[block] = elapsed cycles or -1.
cudaError_t kvs_launch_mma_probe(int blocks, int n_cols, int reuse_a, int products, uint32_t limit_us,
                                 long long* cycles, cudaStream_t st);

// ----------------------------------------------------------------------------- device helpers
#ifdef __CUDACC__
__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_u32(uint32_t* p, uint32_t v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
#endif

// ----------------------------------------------------------------------------- scratch-only compaction
// One round of merge + compaction (the operation of kvs_compact) that takes its scratch memory
// as a plain pointer instead of the general workspace.  `*need_bytes` receives the scratch size
// the arguments ask for.  Used by the entry point that allocates nothing.
kvs_status_t kvs_detail_compact_scratch(const kvs_params_t* p, void* K, void* V, int32_t* counts,
                                        const uint8_t* merge_mask, const float* w_left,
                                        const int32_t* seq_len, const int32_t* n_merge, int32_t n_max,
                                        int32_t* new_len, int32_t* new_index, void* scratch,
                                        size_t scratch_bytes, size_t* need_bytes, int32_t* status_dev,
                                        void* cuda_stream);
kvs_status_t kvs_detail_fail(kvs_status_t code, const char* msg);
