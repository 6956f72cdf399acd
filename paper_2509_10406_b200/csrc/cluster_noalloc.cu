// muse_cluster_noalloc: the clustering stage for callers that cannot hand the library a scratch
// buffer.  Its scratch lives in a fixed device array that is part of the loaded library image.
#include "common.cuh"

namespace {

// 32 MiB of device memory, resident on every GPU that loads the library until the process
// exits.  It holds what muse_cluster keeps in its caller-provided workspace (centre norms,
// bucket offsets, the sort permutation and counters, the bf16 hi/lo copies of the centres).
constexpr size_t kStaticScratchBytes = size_t(32) << 20;
static __device__ __align__(256) unsigned char g_cluster_scratch[kStaticScratchBytes];

// In host code `g_cluster_scratch` is only a stand-in for the symbol, not a device address.
// The address is looked up on every call, with the caller's device current: once the module is
// loaded on that device this is a cheap host-side lookup, and nothing is cached that a device
// reset or a new primary context could leave stale.  The very first lookup on a device loads the
// library's device image there, which is when the 32 MiB are actually reserved (and the one
// point where this entry can fail for lack of memory).
int scratch_address(void** out) {
  void* p = nullptr;
  if (cudaGetSymbolAddress(&p, g_cluster_scratch) != cudaSuccess || p == nullptr) {
    cudaGetLastError();                                    // leave no sticky error for the next launch check
    return MUSE_ERR_CUDA;
  }
  *out = p;
  return MUSE_OK;
}

}  // namespace

extern "C" {

size_t muse_cluster_noalloc_max_bytes(void) { return kStaticScratchBytes; }

int muse_cluster_noalloc(const muse_params_t* p, const void* Q, const void* K, const int32_t* init_q,
                         const int32_t* init_k, int32_t* assign_q, int32_t* assign_k, float* qbar, float* kcent,
                         cudaStream_t stream) {
  size_t need[6];
  int rc = muse_workspace_bytes(p, need);
  if (rc != MUSE_OK) return rc;
  if (need[0] > kStaticScratchBytes) return MUSE_ERR_WORKSPACE;    // problem too large for the built-in scratch
  void* ws = nullptr;
  rc = scratch_address(&ws);
  if (rc != MUSE_OK) return rc;
  // Same launches as muse_cluster, on the built-in scratch.  Nothing needs pre-clearing beyond
  // what the stage already clears itself (its status words and its shared-memory histograms;
  // the sort counters are fully rewritten before they are read).
  return muse_cluster(p, Q, K, init_q, init_k, assign_q, assign_k, qbar, kcent, ws, kStaticScratchBytes, stream);
}


// The status word of the last muse_cluster_noalloc call lives inside the built-in array, where the
// caller cannot point: this enqueues its 4-byte copy to `dst` (host or device memory) on `stream`.
int muse_cluster_noalloc_status_copy(int32_t* dst, cudaStream_t stream) {
  if (dst == nullptr) return MUSE_ERR_INVALID_ARG;
  void* ws = nullptr;
  int rc = scratch_address(&ws);
  if (rc != MUSE_OK) return rc;
  MUSE_CUDA_OK(cudaMemcpyAsync(dst, ws, sizeof(int32_t), cudaMemcpyDefault, stream));
  return MUSE_OK;
}

}  // extern "C"
