/*
 * kvs.h - C ABI of the B200 (sm_100a) KV-merge library, libkvs.so.
 *
 * The library implements the KV-merge pass of KVSlimmer: for every (sequence, KV head)
 * it computes observation-window attention, reduces the forward-only statistics that the
 * closed-form exact Hessian of an adjacent key pair needs, scores and selects adjacent
 * pairs, merges keys with the closed-form weights and values by summation, and compacts
 * the cache in place to the token budget.  A split-K attention over the merged cache
 * closes the loop.
 *
 * General conventions
 *   - Every pointer marked DEVICE is device memory owned by the caller; HOST pointers are
 *     ordinary host memory.  The library allocates no device memory, never synchronises
 *     the stream and never throws.
 *   - All compute calls are asynchronous on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL is the legacy default stream).
 *   - Errors the host can detect return a code before anything is enqueued and leave all
 *     buffers untouched.  Errors only the device can detect (a bounded wait that ran out)
 *     set *status_dev to a kvs_status_t value; the pass then finishes without touching
 *     further cache memory.  status_dev may be NULL.
 *   - bf16 tensors are passed as void* to 16-bit words; layouts are row major with the
 *     head dimension (128) innermost and contiguous.
 *   - A cache "slot" is a triple (key, value SUM, count).  A fresh token has count 1 and
 *     its value as the sum.  A merged slot stands for `count` original tokens: it enters
 *     attention with the logit bias ln(count) and the mean value sum/count.
 */
#ifndef KVS_H_
#define KVS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  KVS_OK = 0,
  KVS_ERR_INVALID_ARG = 1,        /* NULL pointer, non-positive size, bad stride ...        */
  KVS_ERR_UNSUPPORTED = 2,        /* head_dim != 128, group*window > 1024, ...              */
  KVS_ERR_WORKSPACE = 3,          /* workspace smaller than kvs_workspace_size() asks       */
  KVS_ERR_BUDGET_UNREACHABLE = 4, /* a round has no candidate pair left above the budget    */
  KVS_ERR_CUDA = 5,               /* a CUDA runtime call failed; see kvs_last_error_string  */
  KVS_ERR_TIMEOUT = 6             /* device side: a bounded wait ran out                    */
} kvs_status_t;

typedef struct {
  int32_t batch;         /* B sequences                                                      */
  int32_t n_q_heads;     /* Hq; must be a multiple of n_kv_heads                             */
  int32_t n_kv_heads;    /* Hkv                                                              */
  int32_t head_dim;      /* must be 128                                                      */
  int32_t window;        /* W: the observation queries are the last W positions              */
  int32_t sink;          /* leading slots that are never merged (the paper keeps 32)         */
  int32_t recent;        /* trailing slots never merged; >= window when causal               */
  int32_t causal;        /* 1: window query i attends to slots <= n - W + i                  */
  float   softmax_scale; /* multiplies <q,k> inside the logit (1/sqrt(128))                  */
  float   round_frac;    /* fraction of the candidate pairs merged per round, in (0,1]       */
  int32_t score_mode;    /* 0: attention mass * (1 - cosine)   1: attention mass only        */
  int32_t first_round;   /* index of the first round executed (sets the pair parity)         */
  int64_t k_stride_b, k_stride_h, k_stride_t; /* K element strides: sequence, head, slot     */
  int64_t v_stride_b, v_stride_h, v_stride_t; /* V element strides; k/v_stride_t >= 128      */
} kvs_params_t;

/* Library version (major*100 + minor). */
int kvs_version(void);

/* Text of the most recent error on the calling thread ("" if none). */
const char* kvs_last_error_string(void);

/* Number of kernels this library has launched since it was loaded (host counter). */
uint64_t kvs_launch_count(void);

/*
 * Round schedule of one sequence (host only, no CUDA call).
 * Operation: the chunk schedule of Section 3.1 ("merge chunk_size adjacent pairs in one
 * step"), repeated until the budget is met.  Round r of a cache with n slots uses the
 * aligned candidate pairs (off+2p, off+2p+1), off = sink + (r mod 2),
 * P = floor((n - off - recent)/2), and merges R = min(n - budget, max(1, floor(round_frac*P))).
 *   n, budget      current slot count and target
 *   max_rounds     capacity of the output arrays (HOST, may be NULL to count only)
 *   n_r/off_r/P_r/R_r  HOST int32[max_rounds] out
 *   n_rounds       HOST out: rounds needed
 * Returns KVS_ERR_BUDGET_UNREACHABLE if a round has P == 0, KVS_ERR_WORKSPACE if
 * max_rounds is too small (n_rounds is still set).
 */
kvs_status_t kvs_round_plan(const kvs_params_t* params, int32_t n, int32_t budget,
                            int32_t max_rounds, int32_t* n_r, int32_t* off_r, int32_t* P_r,
                            int32_t* R_r, int32_t* n_rounds);

/*
 * Bytes of DEVICE workspace that kvs_merge_layer / kvs_append_and_merge / kvs_compact /
 * kvs_window_stats need for caches whose slot capacity (the n_max argument of those calls) is
 * max_seq_len, and kvs_decode_attn for up to max_new query tokens (pass 0 if decode is not
 * used).  The workspace layout depends on the capacity, so a call with another n_max needs the
 * size asked for that n_max.  Host only.
 */
kvs_status_t kvs_workspace_size(const kvs_params_t* params, int32_t max_seq_len,
                                int32_t max_new, size_t* bytes);

/*
 * The whole merge pass of one decoder layer, in place  [Section 4: Eqs. attn_def_vec,
 * c11_def-c12_def, kstar_final; Section 3.1: v* = v_m + v_{m+1} and the chunk schedule].
 *   K, V       DEVICE bf16 [B,Hkv,Nmax,128] (strides in params); V holds value SUMS
 *   counts     DEVICE int32 [B,Hkv,Nmax] contiguous; 1 for fresh tokens
 *   q_win      DEVICE bf16 [B,Hq,W,128] contiguous: queries of the last W positions
 *   seq_len    HOST int32[B]: slots in use per sequence (<= n_max)
 *   budget     HOST int32[B]: target slot count per sequence
 *   n_max      Nmax, the slot capacity that the counts layout uses (an odd capacity needs
 *              recent >= 1: KVS_ERR_UNSUPPORTED otherwise)
 *   new_len    HOST int32[B] out: min(seq_len, budget); written before the call returns
 *   workspace  DEVICE, >= kvs_workspace_size(params, n_max, 0) (the layout follows the capacity
 *              n_max, not the longest sequence); 256-byte aligned
 * A sequence with seq_len <= budget is left untouched.  Slots at index >= new_len[b] are
 * unspecified afterwards.  Rounds run back to back on the stream with no host sync.
 */
kvs_status_t kvs_merge_layer(const kvs_params_t* params, void* K, void* V, int32_t* counts,
                             const void* q_win, const int32_t* seq_len, const int32_t* budget,
                             int32_t n_max, int32_t* new_len, void* workspace,
                             size_t workspace_bytes, int32_t* status_dev, void* cuda_stream);

/*
 * One streaming step of a decoder layer, in place  [Section 3.1: the cache is compressed each
 * time a chunk of new tokens has arrived; Section 5.1 (implementation details): budget 2048,
 * chunk 512].  The chunk's tokens are appended after the slots in use as fresh slots (count 1,
 * value sum = value), then the merge pass of kvs_merge_layer brings every sequence back to its
 * budget with q_win, the queries of the chunk's last W positions, as observation window.
 *   K, V, counts, q_win, budget, n_max, new_len, workspace: as kvs_merge_layer
 *   chunk_k, chunk_v  DEVICE bf16 [B,Hkv,chunk_len,128] contiguous, 16-byte aligned; read only
 *   chunk_len         tokens appended to every sequence (>= 0)
 *   cur_len           HOST int32[B]: slots in use before the call; cur_len[b] + chunk_len <= n_max
 *   new_len           HOST int32[B] out: min(cur_len[b] + chunk_len, budget[b])
 * The workspace must cover kvs_workspace_size(params, n_max, 0).
 * Errors that the host can detect (ranges, an unreachable budget) are returned before anything
 * is enqueued, the append included.  Asynchronous on the stream; the caller owns all buffers.
 */
kvs_status_t kvs_append_and_merge(const kvs_params_t* params, void* K, void* V, int32_t* counts,
                                  const void* chunk_k, const void* chunk_v, int32_t chunk_len,
                                  const void* q_win, const int32_t* cur_len, const int32_t* budget,
                                  int32_t n_max, int32_t* new_len, void* workspace,
                                  size_t workspace_bytes, int32_t* status_dev, void* cuda_stream);

/*
 * One round of merge + stable in-place compaction with a caller-supplied decision
 * [Eq. kstar_final for the key, v* = v_m + v_{m+1} for the value sum].
 *   merge_mask DEVICE uint8 [B,Hkv,Nmax/2]: 1 where candidate pair p is merged; pair p of
 *              sequence b covers slots (off+2p, off+2p+1), off = sink + (first_round mod 2)
 *   w_left     DEVICE fp32 [B,Hkv,Nmax/2]: weight of the left key of pair p:
 *              K* = bf16(K_right + w (K_left - K_right))
 *   seq_len    HOST int32[B]; new_len HOST int32[B] out = seq_len - (pairs merged) is NOT
 *              computed here: the caller passes n_merge HOST int32[B], the number of ones in
 *              each sequence's mask (per head, equal for all heads), and gets
 *              new_len = seq_len - n_merge
 *   new_index  optional DEVICE int32 [B,Hkv,Nmax] out: old slot -> new slot for every slot in use
 *              (the right member of a merged pair maps to its partner's new slot; a sequence
 *              without a merge gets the identity)
 * Compaction indices and counts are exact integer work: the same mask gives the same
 * result bit for bit.
 */
kvs_status_t kvs_compact(const kvs_params_t* params, void* K, void* V, int32_t* counts,
                         const uint8_t* merge_mask, const float* w_left,
                         const int32_t* seq_len, const int32_t* n_merge, int32_t n_max,
                         int32_t* new_len, int32_t* new_index, void* workspace,
                         size_t workspace_bytes, int32_t* status_dev, void* cuda_stream);

/*
 * kvs_compact without a workspace argument, for callers that must not allocate device memory.
 * The paper has no counterpart: this is a packaging variant of kvs_compact, not a step of the
 * method.
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a serving engine that
 * has handed all device memory to its own pool and forbids further allocations, inside a
 * callback or a latency-critical section where an allocation would synchronise the device, or
 * in a process whose memory budget is fixed at start-up.  kvs_compact asks such callers for a
 * workspace they cannot create; this entry point brings its own.
 *
 * The scratch memory of the compaction (per-tile merge counts, tile tickets, "tile loaded" flags)
 * lives in a fixed device array inside the library, kvs_static_scratch_bytes() = 4 MiB, which
 * every GPU that loads the library holds until the process exits.  With U = batch * n_kv_heads
 * units and T = n_max / 64 + 2 tile entries per unit the call needs
 *   round256(U * T * 4) + round256((U + U * T) * 4) bytes
 * (per-tile merge counts; then one ticket per unit and one flag per tile; round256 rounds up to a
 * multiple of 256) and returns KVS_ERR_WORKSPACE, before anything is enqueued, if that exceeds the
 * array (for example 8 KV heads x 131072 slots need 128.5 KiB; 256 units x 32768 slots need 1.005 MiB).
 * All other arguments, results and error behaviour are those of kvs_compact.
 *
 * The function calls no cudaMalloc, cudaFree or other allocating routine.  The first call on each
 * device looks up the array's device address (with that device current) and keeps it; make that
 * first call outside any stream capture.  All calls share the one array, which keeps the
 * previous call's contents: the tickets and flags are cleared on the stream at the start of each
 * call, and two calls whose kernels overlap on the GPU (different streams, or different host
 * threads on one device) race on it - serialise them.
 */
kvs_status_t kvs_compact_static(const kvs_params_t* params, void* K, void* V, int32_t* counts,
                                const uint8_t* merge_mask, const float* w_left,
                                const int32_t* seq_len, const int32_t* n_merge, int32_t n_max,
                                int32_t* new_len, int32_t* new_index, int32_t* status_dev,
                                void* cuda_stream);

/* Size in bytes of the built-in scratch array that kvs_compact_static uses. */
size_t kvs_static_scratch_bytes(void);

/*
 * Attention of new queries over a (merged) cache, split along the slots and combined
 * [Eq. attn_def_vec with merged slots: numerator uses value sums, denominator weights
 * each slot by its count]:
 *   out_q = sum_j exp(s_qj) Vsum_j / sum_j c_j exp(s_qj),  s_qj = softmax_scale <q, K_j>.
 * No causal mask.
 *   q_new      DEVICE bf16 [B,Hq,n_new,128] contiguous
 *   out        DEVICE bf16 [B,Hq,n_new,128] contiguous
 *   lse        optional DEVICE fp32 [B,Hq,n_new]: ln sum_j c_j exp(s_qj)
 *   seq_len    HOST int32[B]: slots in use
 * (n_q_heads / n_kv_heads) * n_new must be <= 1024.
 */
kvs_status_t kvs_decode_attn(const kvs_params_t* params, const void* q_new, int32_t n_new,
                             const void* K, const void* V, const int32_t* counts,
                             const int32_t* seq_len, int32_t n_max, void* out, float* lse,
                             void* workspace, size_t workspace_bytes, int32_t* status_dev,
                             void* cuda_stream);

/*
 * Diagnostic export: the statistics and the decision of ONE round (params->first_round)
 * without modifying the cache  [Eqs. attn_def_vec, c11_def-c12_def, kstar_final].
 *   A, N1      optional DEVICE fp32 [B,Hkv,Nmax]: attention mass and summed |c_jj| per slot
 *              (defined for candidate slots off <= j < off+2P; others are not written)
 *   N12, cosv, score, w   optional DEVICE fp32 [B,Hkv,Nmax/2] per candidate pair
 *   mask       optional DEVICE uint8 [B,Hkv,Nmax/2]: the R pairs with smallest (score, p)
 *   o_win      optional DEVICE fp32 [B,Hkv,G*W,128]: attention output of the window queries
 *   lse_win    optional DEVICE fp32 [B,Hkv,G*W]: ln sum_j c_j exp(s_qj) of the window queries
 */
kvs_status_t kvs_window_stats(const kvs_params_t* params, const void* K, const void* V,
                              const int32_t* counts, const void* q_win, const int32_t* seq_len,
                              const int32_t* budget, int32_t n_max, float* A, float* N1,
                              float* N12, float* cosv, float* score, float* w, uint8_t* mask,
                              float* o_win, float* lse_win, void* workspace,
                              size_t workspace_bytes, int32_t* status_dev, void* cuda_stream);

/*
 * The merge pass and its diagnostic export with EXACT merge weights from a supplied loss gradient
 * [Section 4.2: g_ij = E^T c_ij, Eqs. c11_def-c12_def, H_gamma_rank1_rewrite,
 * kstar_weight_final_rewrite].  Everything but the weight is as in kvs_merge_layer /
 * kvs_window_stats (scores and the selection do not use E).
 *   e_win        DEVICE bf16 [B,Hq,W,128] contiguous, 16-byte aligned: E = dL/do of every window
 *                query (the backward pass the gradient-free form avoids); read only
 *   weight_mode  1: w = (G11 + G12) / (G11 + 2 G12 + G22), G_ij = sum over the window queries of
 *                   E_q^T c_ij  [Eq. kstar_weight_final_rewrite]
 *                2: the same with the coupling dropped, w = G11 / (G11 + G22): the diagonal-Hessian
 *                   merge the paper starts from  [Section 3.1, Eq. simplified_k]
 *                A denominator that is not safely positive gives w = 1/2; w is clipped to [0, 1].
 *   g_self       optional DEVICE fp32 [B,Hkv,Nmax]: sum over queries of E^T c_jj per candidate slot
 *   g_pair       optional DEVICE fp32 [B,Hkv,Nmax/2]: sum over queries of E^T c_12 per candidate pair
 */
kvs_status_t kvs_merge_layer_exact(const kvs_params_t* params, void* K, void* V, int32_t* counts,
                                   const void* q_win, const void* e_win, int32_t weight_mode,
                                   const int32_t* seq_len, const int32_t* budget, int32_t n_max,
                                   int32_t* new_len, void* workspace, size_t workspace_bytes,
                                   int32_t* status_dev, void* cuda_stream);
kvs_status_t kvs_window_stats_exact(const kvs_params_t* params, const void* K, const void* V,
                                    const int32_t* counts, const void* q_win, const void* e_win,
                                    int32_t weight_mode, const int32_t* seq_len, const int32_t* budget,
                                    int32_t n_max, float* A, float* g_self, float* g_pair, float* cosv,
                                    float* score, float* w, uint8_t* mask, void* workspace,
                                    size_t workspace_bytes, int32_t* status_dev, void* cuda_stream);

/*
 * Non-uniform budgets: the merge pass and the decode check with a length and a budget per
 * (sequence, KV head) instead of per sequence  [Section 6 (discussion): one compression ratio for
 * every layer and head is the method's stated limitation; the heads of a sequence may now end at
 * different lengths].  Everything else is kvs_merge_layer / kvs_decode_attn: each (sequence, head)
 * is treated as a sequence of its own with one KV head and its n_q_heads / n_kv_heads query heads.
 *   seq_len, budget   HOST int32[B*Hkv], index b * Hkv + h
 *   new_len           HOST int32[B*Hkv] out: min(seq_len, budget) per head
 *   workspace         >= kvs_workspace_size_per_head(params, n_max, max_new)
 * The caches must have k/v_stride_b == n_kv_heads * k/v_stride_h (the usual contiguous
 * [B,Hkv,Nmax,128] layout, or any layout whose heads tile the sequence stride); otherwise
 * KVS_ERR_UNSUPPORTED.  Slots at index >= new_len[b * Hkv + h] of a head are unspecified afterwards.
 */
kvs_status_t kvs_workspace_size_per_head(const kvs_params_t* params, int32_t n_max, int32_t max_new,
                                         size_t* bytes);
kvs_status_t kvs_merge_layer_per_head(const kvs_params_t* params, void* K, void* V, int32_t* counts,
                                      const void* q_win, const int32_t* seq_len, const int32_t* budget,
                                      int32_t n_max, int32_t* new_len, void* workspace,
                                      size_t workspace_bytes, int32_t* status_dev, void* cuda_stream);
kvs_status_t kvs_decode_attn_per_head(const kvs_params_t* params, const void* q_new, int32_t n_new,
                                      const void* K, const void* V, const int32_t* counts,
                                      const int32_t* seq_len, int32_t n_max, void* out, float* lse,
                                      void* workspace, size_t workspace_bytes, int32_t* status_dev,
                                      void* cuda_stream);

/*
 * Adjacent-token cosine similarity of a bf16 tensor along its token axis  [Section 3.2,
 * Eq. cosine_raw]:  cos_out[b,h,t] = <x_t, x_t+1> / max(|x_t| |x_t+1|, 1e-30)  for t < seq_len[b] - 1.
 * A diagnostic for the queries, keys and values of a layer (the method rests on adjacent keys
 * being nearly parallel and adjacent values not); independent of the merge pass.
 *   x          DEVICE bf16 [B,H,Nmax,128], element strides stride_b / stride_h / stride_t
 *              (multiples of 8, stride_t >= 128), 16-byte aligned; read only
 *   seq_len    HOST int32[B]: rows in use per sequence (<= n_max)
 *   cos_out    DEVICE fp32 [B,H,Nmax] contiguous; entries t >= seq_len[b] - 1 are not written
 * No workspace.  Asynchronous on the stream.
 */
kvs_status_t kvs_adjacent_cosine(const void* x, int32_t batch, int32_t n_heads, int32_t n_max,
                                 int64_t stride_b, int64_t stride_h, int64_t stride_t,
                                 const int32_t* seq_len, float* cos_out, void* cuda_stream);

/*
 * Time limit of the device-side waits, and a test hook that makes one of them run out.
 * Every wait inside the kernels (on a tile that a copy engine delivers, on a tensor-core product,
 * on another CTA's "tile loaded" flag) gives up after limit_us microseconds; the kernel then sets
 * *status_dev = KVS_ERR_TIMEOUT, lets its copies in flight land, frees its tensor memory and
 * returns, and the CUDA context stays usable.  limit_us = 0 restores the default of one second.
 * `withhold` is for tests of that path and must be 0 in production: bit 0 makes the attention
 * kernel's producer request no K tiles, bit 1 does the same in the statistics kernel, bit 2 keeps
 * the compaction from publishing its "tile loaded" flags, so that the waits for them run out after
 * limit_us without any real stall.  Applies to calls made afterwards, process wide.  Host only.
 */
kvs_status_t kvs_debug_set_wait(uint32_t limit_us, uint32_t withhold);

/*
 * Measurement aid: launches a kernel that executes nothing but special-function operations
 * (ex2.approx and sqrt.approx, the operations that the softmax and the norms of Eqs. c11_def-c12_def
 * cost per (query, slot)), `blocks` CTAs of 1024 threads with 16 * iters operations per thread, and
 * returns the operation count through *ops.  Timed by the caller with CUDA events it gives the
 * special-function rate of the GPU at hand, the denominator of that roofline in the benchmark.
 *   sink_dev   DEVICE float[1] (never written in practice)
 */
kvs_status_t kvs_probe_sfu(int32_t blocks, int32_t iters, float* sink_dev, uint64_t* ops, void* cuda_stream);

/*
 * Measurement aid: what one tensor-core product costs when both of its operands are read from
 * shared memory, which is what bounds the narrow products of the statistics kernel (Eqs.
 * c11_def-c12_def need S = K Q^T and T = Vsum O^T per candidate pair; the pair members sit on the
 * 128 accumulator lanes, so every product re-reads a 128 x 16 slice of K or Vsum).  Launches
 * `blocks` CTAs; one warp of each issues `products` (a multiple of 8, at most 2^20) back-to-back
 * bf16 products of shape 128 x n_cols x 16, n_cols in {16, 32, 64, 128, 256}, on zero-filled
 * operands, and writes the cycles from the first issue to the completion of the last into
 * cycles_dev[block] (-1 if its bounded wait ran out).  With reuse_a != 0 consecutive products
 * share their A slice in twos and the second takes it from the tensor core's collector buffer.
 *   cycles_dev   DEVICE int64[blocks]
 */
kvs_status_t kvs_probe_mma(int32_t blocks, int32_t n_cols, int32_t reuse_a, int32_t products, int64_t* cycles_dev,
                           void* cuda_stream);

/*
 * Per-kernel device timing for benchmarks.  Between kvs_profile_begin() and
 * kvs_profile_end() every kernel launch of this library is bracketed by CUDA events on the
 * launching stream.  kvs_profile_end() synchronises those events and returns, for each
 * kernel kind k < n_kinds, the summed device time in milliseconds and the launch count.
 * kvs_profile_kind_name(k) names kind k (NULL past the last).  Not thread safe.
 */
kvs_status_t kvs_profile_begin(void);
kvs_status_t kvs_profile_end(int32_t n_kinds, float* ms, int32_t* launches);
const char* kvs_profile_kind_name(int32_t kind);

#ifdef __cplusplus
}
#endif
#endif /* KVS_H_ */
