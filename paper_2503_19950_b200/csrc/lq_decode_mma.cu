// placeholder until the tensor-core kernel lands
#include "lq_kernels.cuh"
namespace lq {
int decode_mma_max_splits(const CacheView&, int, int64_t, int) { return 1; }
cudaError_t launch_decode_mma(const DecodeArgs&, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace lq
