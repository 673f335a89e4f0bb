// slkv_score_noalloc: slkv_score for callers that cannot allocate device memory.
//
// Its scratch lives in a file-scope device array that every GPU loading the library holds until the
// process exits.  Host code may not hand the array's name to a kernel (on the host the name is only a
// stand-in): the device address is looked up once per device with cudaGetSymbolAddress and passed on as
// the workspace pointer of the ordinary score kernels.
#include <mutex>

#include "slkv_internal.cuh"

namespace {

constexpr size_t kScratchBytes = SLKV_NOALLOC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};      // device address of g_noalloc_scratch, per device ordinal

// Device address of the scratch array on the current device (looked up on the first call per device).
int scratch_of_current_device(void** out, int* cuda_err) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) { *cuda_err = (int)e; return SLKV_ERR_CUDA; }
  if (dev < 0 || dev >= kMaxDevices) return SLKV_ERR_BAD_SHAPE;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess || !p) { *cuda_err = (int)e; return SLKV_ERR_CUDA; }
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return SLKV_OK;
}

thread_local int g_noalloc_cuda_error = 0;

}  // namespace

extern "C" {

size_t slkv_noalloc_scratch_bytes(void) { return kScratchBytes; }

int slkv_noalloc_last_cuda_error(void) { return g_noalloc_cuda_error; }

int slkv_score_noalloc(const slkv_params* p, const void* q_win, const void* k, const int32_t* cu_seqlens_dev,
                       const int32_t* cu_seqlens_host, const float* lse_opt, float* pooled, int32_t* status,
                       void* stream) {
  // the argument checks of slkv_score first, so that a bad call gets the same status from either entry point
  int rc = slkv::check_score_args(p, q_win, k, cu_seqlens_dev, cu_seqlens_host, pooled);
  if (rc != SLKV_OK) return rc;
  const size_t need = slkv_workspace_bytes(p, cu_seqlens_host);
  if (need == 0 || need > kScratchBytes) return SLKV_ERR_WORKSPACE;          // shapes beyond the built-in scratch
  void* scratch = nullptr;
  g_noalloc_cuda_error = 0;
  rc = scratch_of_current_device(&scratch, &g_noalloc_cuda_error);
  if (rc != SLKV_OK) return rc;
  // Nothing in the scratch has to start at zero: every kernel writes the part it later reads.
  return slkv_score(p, q_win, k, cu_seqlens_dev, cu_seqlens_host, lse_opt, pooled, status, scratch, kScratchBytes,
                    stream);
}

}  // extern "C"
