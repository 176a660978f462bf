// SGMV: tensor-core segmented GEMM for prefill-shaped segments (placeholder until the
// kernel lands: reports "unsupported" so that nothing silently falls back).
#include "plora_internal.cuh"

namespace plora {

cudaError_t sgmv_configure() { return cudaSuccess; }

cudaError_t launch_sgmv(const PoolDev&, const BucketDev&, int, const void*, float*, int32_t*, int, cudaStream_t, int*) {
    return cudaErrorNotSupported;
}

}  // namespace plora
