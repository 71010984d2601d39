// placeholder until the tensor-core full-attention kernels land
#include "hs2_common.cuh"
namespace hs2 {
bool full_mma_supported(const Params &, hs2_dtype) { return false; }
cudaError_t launch_full_attn_mma(const Params &, const void *, const void *, const void *, void *, float *, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t launch_scores_mma(const Params &, const void *, const void *, const float *, float *, int64_t, int64_t, int64_t, bool, cudaStream_t) { return cudaErrorNotSupported; }
}
