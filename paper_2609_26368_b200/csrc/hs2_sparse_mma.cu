// placeholder until the tensor-core sparse kernels land
#include "hs2_common.cuh"
namespace hs2 {
bool sparse_mma_supported(const Params &, hs2_dtype) { return false; }
cudaError_t launch_sparse_mma_prefill(const Params &, const void *, const void *, const void *, const int32_t *,
                                      const float *, void *, float *, cudaStream_t) { return cudaErrorNotSupported; }
size_t sparse_mma_decode_ws_bytes(const Params &) { return 0; }
cudaError_t launch_sparse_mma_decode(const Params &, const void *, const void *, const void *, const int32_t *,
                                     const float *, void *, float *, void *, size_t, cudaStream_t) { return cudaErrorNotSupported; }
}
