// Tensor-core score path (tcgen05 + TMA).  Placeholder until the kernels land: reports "unsupported".
#include "slkv_internal.cuh"

namespace slkv {
bool tensor_path_supported(const slkv_params&) { return false; }
int tensor_chunk_keys(const Problem&) { return 1024; }
cudaError_t launch_score_tensor(const Problem&, cudaStream_t, int*) { return cudaErrorNotSupported; }
}  // namespace slkv
