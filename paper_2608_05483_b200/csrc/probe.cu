// Read-only streaming probe: the denominator for kernels whose traffic is almost all reads.
// The LoRA delta at decode sizes reads adapter bytes and writes little (paper Section VI-B: the
// memory term of strategy E1 is a read term), so the bandwidth of a plain copy, half reads and
// half writes, understates what the part can deliver to it.  This kernel reads a buffer once with
// 16-byte loads and keeps a checksum so that the loads cannot be dropped; the caller times it.
#include "plora_internal.cuh"

namespace {

constexpr int kProbeThreads = 512;
constexpr int kProbeUnroll = 8;

__global__ void __launch_bounds__(kProbeThreads) stream_read_kernel(const uint4* __restrict__ src, size_t n_vec,
                                                                    uint32_t* __restrict__ sink) {
    const size_t stride = (size_t)gridDim.x * kProbeThreads;
    size_t i = (size_t)blockIdx.x * kProbeThreads + threadIdx.x;
    uint32_t acc = 0;
    for (; i + (kProbeUnroll - 1) * stride < n_vec; i += kProbeUnroll * stride) {
        uint4 v[kProbeUnroll];
#pragma unroll
        for (int u = 0; u < kProbeUnroll; ++u)
            asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                         : "=r"(v[u].x), "=r"(v[u].y), "=r"(v[u].z), "=r"(v[u].w)
                         : "l"(src + i + u * stride));
#pragma unroll
        for (int u = 0; u < kProbeUnroll; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
    }
    for (; i < n_vec; i += stride) {
        const uint4 v = src[i];
        acc ^= v.x ^ v.y ^ v.z ^ v.w;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) acc ^= __shfl_xor_sync(0xffffffffu, acc, d);
    if ((threadIdx.x & 31) == 0) atomicXor(sink + blockIdx.x, acc);
}

}  // namespace

extern "C" PLORA_API plora_status plora_stream_read(const void* buf_dev, size_t bytes, void* sink_dev, size_t sink_bytes,
                                                    void* stream) {
    if (!buf_dev || !sink_dev || ((uintptr_t)buf_dev & 15) || ((uintptr_t)sink_dev & 3) || (bytes & 15))
        return PLORA_ERR_INVALID_ARG;
    if (bytes == 0) return PLORA_OK;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return PLORA_ERR_CUDA;
    const int grid = sms * 4;   // four blocks of 512 threads fill an SM's 2048 thread slots
    if (sink_bytes < (size_t)grid * 4) return PLORA_ERR_WORKSPACE;
    stream_read_kernel<<<grid, kProbeThreads, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint4*>(buf_dev), bytes / 16, static_cast<uint32_t*>(sink_dev));
    return cudaGetLastError() == cudaSuccess ? PLORA_OK : PLORA_ERR_CUDA;
}
