// SGMV: the prefill-shaped path of the LoRA delta.  A segment (all tokens of one adapter) that
// is long enough is cut into tiles of kSgmvRows rows and each tile runs the paper's two small
// GEMMs on the tensor cores (Section V-A: shrink m = x A, then expand y = m B; large per-adapter
// batches favour computing on the GPU from resident A and B, strategy E1):
//
//     m [rows, rp]    = X [rows, d_in] * A          bf16 x bf16 -> fp32   (K = d_in)
//     y [rows, d_out] += s * m * B                  fp32 m carried as bf16 hi + lo, two products
//
// The path is bound by HBM traffic on the activations (x read once, y updated once), not by the
// tensor pipe, so the kernel is organised around keeping copies in flight: a multi-stage cp.async
// ring feeds warp-level mma.sync (m16n8k16, bf16 in, fp32 accumulate) from shared memory in the
// slab's swizzled sub-tile layout, and y is updated with one vector reduction per element.
// The intermediate m never leaves the SM: it is reduced in shared memory, scaled in fp32 and
// split into bf16 hi + lo (error ~2^-17 relative), which become the A operand of the expand.
#include "plora_internal.cuh"

namespace plora {

namespace {

constexpr int kRows = kSgmvRows;          // rows of a tile (64)
constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kStages = 4;
constexpr int kKC = kSubCols;             // K (or N) columns per stage = one slab sub-tile (64)
constexpr int kXStageBytes = kRows * kKC * 2;              // 8 KiB of x per stage
// Shared memory is sized for the pool's largest padded rank R (at least 16):
//   kStages x (x stage + one [R][64] weight sub-tile), m hi and m lo [64][R] bf16 with a padded
//   row pitch, and the tile's token indices.
__host__ __device__ inline int w_stage_bytes(int R) { return R * kKC * 2; }
__host__ __device__ inline int stage_bytes(int R) { return kXStageBytes + w_stage_bytes(R); }
__host__ __device__ inline int m_pitch(int R) { return R * 2 + 16; }
__host__ __device__ inline int m_bytes(int R) { return kRows * m_pitch(R); }
__host__ __device__ inline int smem_bytes(int R) { return kStages * stage_bytes(R) + 2 * m_bytes(R) + kRows * 4; }

struct Params {
    PoolDev pool;
    BucketDev bk;
    const uint16_t* x;
    float* y;
    int32_t* status;
    int32_t R;   // max(16, largest padded rank of the pool): sizes the shared-memory layout
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// 16-byte asynchronous copy; src_bytes = 0 writes zeros (used for columns beyond the matrix)
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t a, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t a, uint32_t (&r)[2]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(a));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t a, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void red_add_v2(float* p, float a, float b) {
    asm volatile("red.global.add.v2.f32 [%0], {%1, %2};" ::"l"(p), "f"(a), "f"(b) : "memory");
}
// fp32 -> bf16, round to nearest even, on the bit pattern
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float f) {
    const uint32_t u = __float_as_uint(f);
    return (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;
}

// One tile: up to kRows tokens of one adapter.  RP = padded rank of that adapter.
template <int RP>
__device__ void sgmv_tile(const Params& p, const WorkUnit& wu, const AdapterEntry& e, uint8_t* smem, int* tok_s) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int d_in = p.pool.d_in, d_out = p.pool.d_out;
    const int cnt = wu.cnt;
    const int kStageBytes = stage_bytes(p.R), kMPitch = m_pitch(p.R);
    uint8_t* stages = smem;
    uint8_t* m_hi = smem + kStages * kStageBytes;
    uint8_t* m_lo = m_hi + m_bytes(p.R);
    const uint32_t stages_a = smem_u32(stages);

    // token index of every row of the tile (rows beyond cnt repeat the last token: they are
    // computed and thrown away, so every address stays inside the caller's buffers)
    __syncthreads();   // the previous tile is completely done with shared memory
    if (tid < kRows) tok_s[tid] = p.bk.perm[wu.pos0 + min(tid, cnt - 1)];
    __syncthreads();

    // ------------------------------------------------------------------ shrink
    // stage = x[64 rows][64 cols] (chunk c of row r at c ^ (r & 7)) + the A^T sub-tile [RP][64] as it
    // sits in the slab.  Warp (mi, kh): rows 16*mi..+16, k16 steps {2*kh, 2*kh+1} of every stage.
    const int nK = (d_in + kKC - 1) / kKC;
    const uint8_t* a_src = p.pool.slab + e.offA;
    constexpr int NSUB = (kMaxRank / RP > kMaxSubPerTile) ? kMaxSubPerTile : kMaxRank / RP;
    auto load_shrink_stage = [&](int kc) {
        if (kc < nK) {
            const uint32_t base = stages_a + (kc % kStages) * kStageBytes;
            // x: 64 rows x 8 chunks
            for (int j = tid; j < kRows * 8; j += kThreads) {
                const int r = j >> 3, c = j & 7;
                const int col = kc * kKC + c * 8;
                const uint16_t* src = p.x + (size_t)tok_s[r] * d_in + (col < d_in ? col : 0);
                cp_async16(base + r * 128 + ((c ^ (r & 7)) << 4), src, col < d_in ? 16 : 0);
            }
            // A^T sub-tile kc: tile kc / NSUB, sub-tile kc % NSUB, RP * 128 contiguous bytes
            const uint8_t* src = a_src + (size_t)(kc / NSUB) * (RP * NSUB * 128) + (size_t)(kc % NSUB) * (RP * 128);
            for (int j = tid; j < RP * 8; j += kThreads) cp_async16(base + kXStageBytes + j * 16, src + j * 16, 16);
        }
        cp_async_commit();
    };

    constexpr int NT = RP / 8;            // n8 tiles of the shrink output
    float acc[NT][4];
#pragma unroll
    for (int n = 0; n < NT; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
    const int mi = warp & 3, kh = warp >> 2;

#pragma unroll
    for (int s = 0; s < kStages - 1; ++s) load_shrink_stage(s);
    for (int kc = 0; kc < nK; ++kc) {
        cp_async_wait<kStages - 2>();
        __syncthreads();
        load_shrink_stage(kc + kStages - 1);
        const uint32_t base = stages_a + (kc % kStages) * kStageBytes;
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {
            const int kk = (kh * 2 + ks) * 16;                 // column of this k16 step inside the stage
            uint32_t a[4];
            {
                const int r = mi * 16 + (lane & 15), c = (kk >> 3) + (lane >> 4);
                ldmatrix_x4(base + r * 128 + ((c ^ (r & 7)) << 4), a);
            }
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                uint32_t b[2];
                const int r = n * 8 + (lane & 7), c = (kk >> 3) + ((lane >> 3) & 1);
                ldmatrix_x2(base + kXStageBytes + r * 128 + ((c ^ (r & 7)) << 4), b);
                mma_bf16(acc[n], a, b[0], b[1]);
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();   // every warp is done with the stage buffers: reuse them for the reduction

    // the two K-halves meet in shared memory: red[kh][64][RP] fp32 (at most 64 KiB, inside the stages)
    float* red = reinterpret_cast<float*>(stages);
    {
        const int g = lane >> 2, q = lane & 3;
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            float* r0 = red + ((size_t)kh * kRows + mi * 16 + g) * RP + n * 8 + q * 2;
            r0[0] = acc[n][0]; r0[1] = acc[n][1];
            r0[8 * RP] = acc[n][2]; r0[8 * RP + 1] = acc[n][3];
        }
    }
    __syncthreads();
    // m = s * (half 0 + half 1), split into bf16 hi + lo, row pitch kMPitch
    for (int j = tid; j < kRows * RP; j += kThreads) {
        const int r = j / RP, k = j % RP;
        const float v = (red[(size_t)r * RP + k] + red[((size_t)kRows + r) * RP + k]) * e.scale;
        const uint32_t hi = f32_to_bf16_bits(v);
        const float rest = v - __uint_as_float(hi << 16);
        reinterpret_cast<uint16_t*>(m_hi + r * kMPitch)[k] = (uint16_t)hi;
        reinterpret_cast<uint16_t*>(m_lo + r * kMPitch)[k] = (uint16_t)f32_to_bf16_bits(rest);
    }
    if (RP < 16) {   // the expand multiplies with K = 16: columns 8..15 of m are zero
        for (int j = tid; j < kRows * 8; j += kThreads) {
            const int r = j >> 3, k = 8 + (j & 7);
            reinterpret_cast<uint16_t*>(m_hi + r * kMPitch)[k] = 0;
            reinterpret_cast<uint16_t*>(m_lo + r * kMPitch)[k] = 0;
        }
    }
    __syncthreads();

    // ------------------------------------------------------------------ expand
    // stage = the B sub-tile [RP][64 cols] as it sits in the slab.  Warp w: rows 16*(w & 3)..+16,
    // columns 32*(w >> 2)..+32 of every 64-column chunk.
    const int nN = (d_out + kKC - 1) / kKC;
    const uint8_t* b_src = p.pool.slab + e.offB;
    constexpr int KP = RP < 16 ? 16 : RP;      // K of the expand, padded to a multiple of 16
    auto load_expand_stage = [&](int nc) {
        if (nc < nN) {
            const uint32_t base = stages_a + (nc % kStages) * kStageBytes;
            const uint8_t* src = b_src + (size_t)(nc / NSUB) * (RP * NSUB * 128) + (size_t)(nc % NSUB) * (RP * 128);
            for (int j = tid; j < RP * 8; j += kThreads) cp_async16(base + j * 16, src + j * 16, 16);
            if (RP < 16)   // rows 8..15 do not exist in the slab: zeros (cp.async with no source bytes)
                for (int j = tid; j < 8 * 8; j += kThreads) cp_async16(base + (RP * 8 + j) * 16, src, 0);
        }
        cp_async_commit();
    };
    // A operands (m hi / lo) of this warp's 16 rows stay in registers for the whole expand
    uint32_t ah[KP / 16][4], al[KP / 16][4];
#pragma unroll
    for (int ks = 0; ks < KP / 16; ++ks) {
        const int r = mi * 16 + (lane & 15), cb = ks * 32 + (lane >> 4) * 16;
        ldmatrix_x4(smem_u32(m_hi) + r * kMPitch + cb, ah[ks]);
        ldmatrix_x4(smem_u32(m_lo) + r * kMPitch + cb, al[ks]);
    }
    const int nh = warp >> 2;
    const int g = lane >> 2, q = lane & 3;
    const int row0 = mi * 16 + g;
    const bool ok0 = row0 < cnt, ok1 = row0 + 8 < cnt;
    float* y0 = p.y + (size_t)tok_s[row0] * d_out;
    float* y1 = p.y + (size_t)tok_s[row0 + 8] * d_out;

#pragma unroll
    for (int s = 0; s < kStages - 1; ++s) load_expand_stage(s);
    for (int nc = 0; nc < nN; ++nc) {
        cp_async_wait<kStages - 2>();
        __syncthreads();
        load_expand_stage(nc + kStages - 1);
        const uint32_t base = stages_a + (nc % kStages) * kStageBytes;
        float c[4][4];
#pragma unroll
        for (int n = 0; n < 4; ++n) c[n][0] = c[n][1] = c[n][2] = c[n][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < KP / 16; ++ks) {
#pragma unroll
            for (int np = 0; np < 2; ++np) {
                // two n8 tiles at once: matrices (k 0-7, n), (k 8-15, n), (k 0-7, n+8), (k 8-15, n+8)
                uint32_t b[4];
                const int r = ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
                const int cch = nh * 4 + np * 2 + (lane >> 4);
                ldmatrix_x4_trans(base + r * 128 + ((cch ^ (r & 7)) << 4), b);
                mma_bf16(c[np * 2], ah[ks], b[0], b[1]);
                mma_bf16(c[np * 2], al[ks], b[0], b[1]);
                mma_bf16(c[np * 2 + 1], ah[ks], b[2], b[3]);
                mma_bf16(c[np * 2 + 1], al[ks], b[2], b[3]);
            }
        }
#pragma unroll
        for (int n = 0; n < 4; ++n) {
            const int col = nc * kKC + nh * 32 + n * 8 + q * 2;
            if (col < d_out) {
                if (ok0) red_add_v2(y0 + col, c[n][0], c[n][1]);
                if (ok1) red_add_v2(y1 + col, c[n][2], c[n][3]);
            }
        }
    }
    cp_async_wait<0>();
}

__global__ void __launch_bounds__(kThreads, 2) sgmv_kernel(const Params p) {
    extern __shared__ __align__(1024) uint8_t smem[];
    int* tok_s = reinterpret_cast<int*>(smem + kStages * stage_bytes(p.R) + 2 * m_bytes(p.R));
    const int n_tiles = *p.bk.n_sgmv_tiles;
    for (int t = blockIdx.x; t < n_tiles; t += gridDim.x) {
        const WorkUnit wu = p.bk.sgmv_tiles[t];
        const AdapterEntry e = p.pool.table[wu.adapter];
        switch (e.rp) {
            case 8: sgmv_tile<8>(p, wu, e, smem, tok_s); break;
            case 16: sgmv_tile<16>(p, wu, e, smem, tok_s); break;
            case 32: sgmv_tile<32>(p, wu, e, smem, tok_s); break;
            case 64: sgmv_tile<64>(p, wu, e, smem, tok_s); break;
            default: sgmv_tile<128>(p, wu, e, smem, tok_s); break;
        }
    }
}

}  // namespace

cudaError_t sgmv_configure() {
    return cudaFuncSetAttribute(sgmv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes(kMaxRank));
}

cudaError_t launch_sgmv(const PoolDev& pool, const BucketDev& bk, int n_tok, int sgmv_min_rows, const void* x, float* y,
                        int32_t* status, int sm_count, cudaStream_t stream, int* n_launches) {
    Params p;
    p.pool = pool;
    p.bk = bk;
    p.x = static_cast<const uint16_t*>(x);
    p.y = y;
    p.status = status;
    p.R = pool.max_rp < 16 ? 16 : pool.max_rp;
    // every tensor-core segment has at least sgmv_min_rows tokens: at most this many tiles
    const int min_rows = sgmv_min_rows < 1 ? 1 : sgmv_min_rows;
    long long max_tiles = (long long)n_tok / kRows + (long long)n_tok / min_rows + 1;
    int grid = 2 * sm_count;
    if (grid > max_tiles) grid = (int)max_tiles;
    if (grid < 1) grid = 1;
    sgmv_kernel<<<grid, kThreads, smem_bytes(p.R), stream>>>(p);
    ++*n_launches;
    return cudaGetLastError();
}

}  // namespace plora
