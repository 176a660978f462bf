// Adapter-pool registry: repacks a pool given in the paper's logical layout
// (A_a [d_in, r_a], B_a [r_a, d_out], Section II-A) into the library's tiled slab.
// Registration is a set-up step, so this kernel favours simplicity over speed.
#include "plora_internal.cuh"

namespace plora {

namespace {

// Byte offset inside one matrix region of element (row k, column c) of the
// transposed/padded [rp][d] matrix.
__device__ __forceinline__ size_t chunk_offset(int rp, int k, int col) {
    const int tc = tile_cols(rp);
    const int tile = col / tc, ic = col - tile * tc;
    const int sub = ic >> 6, cc = (ic & 63) >> 3;
    return (size_t)tile * tile_bytes(rp) + (size_t)sub * rp * 128 + (size_t)k * 128 + (size_t)((cc ^ (k & 7)) << 4);
}

// One thread writes one 16-byte chunk (8 consecutive columns of one row).
// grid.y = adapter; grid.x strides over that adapter's chunks (A region then B region).
__global__ void __launch_bounds__(256)
repack_kernel(const AdapterEntry* __restrict__ table, const void* const* __restrict__ A_src,
              const void* const* __restrict__ B_src, int d_in, int d_out, uint8_t* __restrict__ slab) {
    const int a = blockIdx.y;
    const AdapterEntry e = table[a];
    const int rp = e.rp, r = e.r;
    const int tc = tile_cols(rp);
    const int colsA = tiles_for(d_in, rp) * tc, colsB = tiles_for(d_out, rp) * tc;
    const long long chunksA = (long long)rp * (colsA >> 3), chunksB = (long long)rp * (colsB >> 3);
    const uint16_t* A = (const uint16_t*)A_src[a];
    const uint16_t* B = (const uint16_t*)B_src[a];
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < chunksA + chunksB;
         idx += (long long)gridDim.x * blockDim.x) {
        uint16_t v[8];
        uint8_t* dst;
        if (idx < chunksA) {
            // consecutive threads take consecutive rows k of one column group: the 8 x rp block of
            // the source they read together is contiguous in A's [d_in, r] layout when rp == r
            const int k = (int)(idx % rp);
            const int col = (int)(idx / rp) << 3;
#pragma unroll
            for (int j = 0; j < 8; ++j)
                v[j] = (k < r && col + j < d_in) ? A[(size_t)(col + j) * r + k] : (uint16_t)0;
            dst = slab + e.offA + chunk_offset(rp, k, col);
        } else {
            const long long q = idx - chunksA;
            const int cg = colsB >> 3;
            const int k = (int)(q / cg);
            const int col = (int)(q % cg) << 3;
#pragma unroll
            for (int j = 0; j < 8; ++j)
                v[j] = (k < r && col + j < d_out) ? B[(size_t)k * d_out + col + j] : (uint16_t)0;
            dst = slab + e.offB + chunk_offset(rp, k, col);
        }
        uint4 o;
        o.x = v[0] | ((uint32_t)v[1] << 16);
        o.y = v[2] | ((uint32_t)v[3] << 16);
        o.z = v[4] | ((uint32_t)v[5] << 16);
        o.w = v[6] | ((uint32_t)v[7] << 16);
        *reinterpret_cast<uint4*>(dst) = o;
    }
}

}  // namespace

cudaError_t launch_repack(const AdapterEntry* table_dev, const void* const* A_dev, const void* const* B_dev,
                          int n_adapters, int d_in, int d_out, uint8_t* slab, cudaStream_t stream, int* n_launches) {
    // adapters go in grid.y, at most 65535 per launch
    for (int a0 = 0; a0 < n_adapters; a0 += 32768) {
        const int na = n_adapters - a0 < 32768 ? n_adapters - a0 : 32768;
        dim3 grid(64, na);
        repack_kernel<<<grid, 256, 0, stream>>>(table_dev + a0, A_dev + a0, B_dev + a0, d_in, d_out, slab);
        ++*n_launches;
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace plora
