// kvs_compact_static: merge + compaction for callers that cannot allocate device memory.
//
// The scratch that the compaction needs (per-tile merge counts, tile tickets and "tile loaded"
// flags) lives in a file-scope device array of fixed size instead of a caller-supplied
// workspace.  Every GPU that loads the library holds this array until the process exits.
#include <stdio.h>

#include <mutex>

#include "kvs_internal.h"

#define KVS_STATIC_SCRATCH_BYTES (4u << 20)   // the value kvs.h documents

static __device__ __align__(256) unsigned char g_static_scratch[KVS_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_setup_lock;
void* g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// In host code the array's name is only a handle: the device address has to be asked for, once
// per device and with that device current.
kvs_status_t scratch_of_current_device(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return kvs_detail_fail(KVS_ERR_CUDA, cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return kvs_detail_fail(KVS_ERR_UNSUPPORTED, "device ordinal beyond 63");
  std::lock_guard<std::mutex> guard(g_setup_lock);
  if (!g_scratch_ptr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_static_scratch);
    if (e != cudaSuccess || !ptr)
      return kvs_detail_fail(KVS_ERR_CUDA, e != cudaSuccess ? cudaGetErrorString(e)
                                                            : "cudaGetSymbolAddress returned a null address");
    g_scratch_ptr[dev] = ptr;
  }
  *out = g_scratch_ptr[dev];
  return KVS_OK;
}

}  // namespace

extern "C" {

size_t kvs_static_scratch_bytes(void) { return KVS_STATIC_SCRATCH_BYTES; }

kvs_status_t kvs_compact_static(const kvs_params_t* params, void* K, void* V, int32_t* counts,
                                const uint8_t* merge_mask, const float* w_left, const int32_t* seq_len,
                                const int32_t* n_merge, int32_t n_max, int32_t* new_len,
                                int32_t* new_index, int32_t* status_dev, void* cuda_stream) {
  void* scratch = nullptr;
  kvs_status_t s = scratch_of_current_device(&scratch);
  if (s != KVS_OK) return s;
  size_t need = 0;
  s = kvs_detail_compact_scratch(params, K, V, counts, merge_mask, w_left, seq_len, n_merge, n_max, new_len,
                                 new_index, scratch, KVS_STATIC_SCRATCH_BYTES, &need, status_dev, cuda_stream);
  if (s == KVS_ERR_WORKSPACE) {
    char msg[200];
    snprintf(msg, sizeof(msg),
             "kvs_compact_static: batch * n_kv_heads * n_max needs %zu bytes of scratch, the built-in array "
             "holds %u; use kvs_compact with a workspace",
             need, KVS_STATIC_SCRATCH_BYTES);
    return kvs_detail_fail(KVS_ERR_WORKSPACE, msg);
  }
  return s;
}

}  // extern "C"
