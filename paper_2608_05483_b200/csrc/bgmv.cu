// BGMV: the decode-shaped gather-GEMV path of the LoRA delta (paper Section V-A:
// strategy E1 computes y = x A B from matrices resident in GPU memory; strategy E4
// names the halves, shrink m = x A and expand y = m B).  One work unit is up to
// kTokChunk tokens that share an adapter.  The path is bound by HBM bandwidth on
// the adapter bytes (cost model, Section VI-B: the memory term sums D * S * R_i over
// the adapters present, once per adapter whatever its batch), so the kernel is a
// streaming pipeline:
//
//   - persistent CTAs, work units taken round-robin;
//   - one producer thread per CTA issues bulk asynchronous copies (cp.async.bulk,
//     completion counted on an mbarrier) of whole 16 KiB slab tiles, plus the
//     matching pieces of the unit's x rows, into a ring of shared-memory stages and
//     runs ahead of the consumers across tiles, phases and units;
//   - eight consumer warps split every tile by columns.  Shrink: a lane owns rank
//     rows, reads 16-byte chunks of A^T and broadcast chunks of x, accumulates in
//     fp32, and partial sums meet in shared memory in a fixed order.  Expand: a lane
//     owns two output columns, walks the rank rows, and adds its result to y with a
//     single vector reduction per element (no read of y on the SM, one addition
//     per element: bit-reproducible).
//
// The same kernel template provides the fused path (m stays in shared memory), the
// shrink-only path (m written to HBM, unscaled) and the expand-only path (m read
// from HBM).
#include "plora_internal.cuh"

namespace plora {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;   // + one producer warp
constexpr int kStages = 4;
constexpr int kXBytesPerTok = kMaxSubPerTile * kSubCols * 2;             // x piece of one token for one tile
constexpr int kSlotBytes = kTileBytesMax + kTokChunk * kXBytesPerTok;   // tile + x pieces
constexpr int kPartFloats = kConsumerWarps * kTokChunk * kMaxRank;
constexpr int kMFloats = kTokChunk * kMaxRank;
constexpr int kSmemBytes = kStages * kSlotBytes + (kPartFloats + kMFloats) * 4 + 2 * kStages * 8 + 16;
constexpr long long kWaitCycles = 4000000000ll;   // about two seconds of SM clock

struct Params {
    PoolDev pool;
    BucketDev bk;
    const uint16_t* x;
    float* y;
    float* m;
    int32_t ldm;
    int32_t n_tok;
    int32_t* status;
};

// ---- PTX wrappers -----------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  When the limit runs out the CTA-wide abort flag is raised, the
// device status word records the timeout, and every later wait returns at once:
// the kernel then finishes (with meaningless numbers) instead of hanging.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
    if (mbar_try_wait(bar, parity)) return;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return;
        if (*abort_flag) return;
        if (clock64() - t0 > kWaitCycles) break;
    }
    *abort_flag = 1;
    atomicCAS(status, 0, PLORA_ERR_TIMEOUT);
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ void red_add_v2(float* p, float a, float b) {
    asm volatile("red.global.add.v2.f32 [%0], {%1, %2};" ::"l"(p), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
    f[0] = bf_lo(v.x); f[1] = bf_hi(v.x); f[2] = bf_lo(v.y); f[3] = bf_hi(v.y);
    f[4] = bf_lo(v.z); f[5] = bf_hi(v.z); f[6] = bf_lo(v.w); f[7] = bf_hi(v.w);
}

struct Smem {
    uint32_t slots;      // shared address of stage 0
    uint32_t full;       // full[kStages] barriers
    uint32_t empty;      // empty[kStages]
    float* part;         // [kConsumerWarps][kTokChunk][kMaxRank]
    float* m_s;          // [kTokChunk][kMaxRank]
    volatile int* abort_flag;
};

// ---- one work unit, consumer side ---------------------------------------------------
template <int MODE, int RP>
__device__ __forceinline__ void consume_unit(const Params& p, const Smem& sm, const WorkUnit& wu,
                                             const AdapterEntry& e, uint32_t& it, int warp, int lane) {
    constexpr int NSUB = (kMaxRank / RP > kMaxSubPerTile) ? kMaxSubPerTile : kMaxRank / RP;
    constexpr int C = NSUB * kSubCols;                      // columns per tile
    const int cnt = wu.cnt;
    const int tid = warp * 32 + lane;
    int tok[kTokChunk];
#pragma unroll
    for (int t = 0; t < kTokChunk; ++t) tok[t] = t < cnt ? p.bk.perm[wu.pos0 + t] : 0;

    if (MODE != kExpandOnly) {
        // ---------------- shrink: m[t][k] = sum_i x[t][i] * A[i][k] ----------------
        constexpr int RPL = RP <= 32 ? 1 : RP / 32;         // rank rows per lane
        constexpr int G = RP <= 32 ? 32 / RP : 1;           // lane groups that share the rows
        constexpr int CPL = NSUB / G;                       // chunks per lane per tile
        const int row = RP <= 32 ? (lane % RP) : lane;
        const int g = RP <= 32 ? (lane / RP) : 0;
        float acc[RPL][kTokChunk];
#pragma unroll
        for (int rr = 0; rr < RPL; ++rr)
#pragma unroll
            for (int t = 0; t < kTokChunk; ++t) acc[rr][t] = 0.f;

        const int nA = (p.pool.d_in + C - 1) / C;
        for (int i = 0; i < nA; ++i, ++it) {
            const uint32_t slot = it % kStages;
            mbar_wait(sm.full + slot * 8, (it / kStages) & 1, sm.abort_flag, p.status);
            const uint32_t tile = sm.slots + slot * kSlotBytes;
            const uint32_t xs = tile + kTileBytesMax;
#pragma unroll
            for (int q = 0; q < CPL; ++q) {
                const int c = warp * NSUB + g + q * G;      // 16-byte chunk (8 columns) inside the tile
                if (i * C + c * 8 < p.pool.d_in) {
                    float af[RPL][8];
#pragma unroll
                    for (int rr = 0; rr < RPL; ++rr) {
                        const int k = row + 32 * rr;
                        unpack8(lds128(tile + (c >> 3) * (RP * 128) + k * 128 + (((c & 7) ^ (k & 7)) << 4)), af[rr]);
                    }
#pragma unroll
                    for (int t = 0; t < kTokChunk; ++t)
                        if (t < cnt) {
                            float xf[8];
                            unpack8(lds128(xs + t * kXBytesPerTok + c * 16), xf);
#pragma unroll
                            for (int rr = 0; rr < RPL; ++rr)
#pragma unroll
                                for (int j = 0; j < 8; ++j) acc[rr][t] = fmaf(xf[j], af[rr][j], acc[rr][t]);
                        }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(sm.empty + slot * 8);
        }
        // lanes of different groups hold partial sums of the same rows
#pragma unroll
        for (int d = RP; d < 32; d <<= 1)
#pragma unroll
            for (int rr = 0; rr < RPL; ++rr)
#pragma unroll
                for (int t = 0; t < kTokChunk; ++t) acc[rr][t] += __shfl_xor_sync(0xffffffffu, acc[rr][t], d);
        if (g == 0) {
#pragma unroll
            for (int rr = 0; rr < RPL; ++rr)
#pragma unroll
                for (int t = 0; t < kTokChunk; ++t)
                    if (t < cnt) sm.part[(warp * kTokChunk + t) * kMaxRank + row + 32 * rr] = acc[rr][t];
        }
        consumer_sync();
        // fixed-order sum over the warps' column slices
        for (int idx = tid; idx < cnt * RP; idx += kConsumerThreads) {
            const int t = idx / RP, k = idx % RP;
            float s = 0.f;
#pragma unroll
            for (int w = 0; w < kConsumerWarps; ++w) s += sm.part[(w * kTokChunk + t) * kMaxRank + k];
            if (MODE == kFused) {
                sm.m_s[t * kMaxRank + k] = s * e.scale;
            } else {
                p.m[(size_t)p.bk.perm[wu.pos0 + t] * p.ldm + k] = s;
            }
        }
        if (MODE == kShrinkOnly) {
            for (int idx = tid; idx < cnt * (p.ldm - RP); idx += kConsumerThreads) {
                const int t = idx / (p.ldm - RP), k = RP + idx % (p.ldm - RP);
                p.m[(size_t)p.bk.perm[wu.pos0 + t] * p.ldm + k] = 0.f;
            }
        }
        consumer_sync();
    }

    if (MODE == kExpandOnly) {
        consumer_sync();   // the previous unit's readers of m_s are done
        for (int idx = tid; idx < cnt * RP; idx += kConsumerThreads) {
            const int t = idx / RP, k = idx % RP;
            const float v = k < e.r ? p.m[(size_t)p.bk.perm[wu.pos0 + t] * p.ldm + k] : 0.f;
            sm.m_s[t * kMaxRank + k] = v * e.scale;
        }
        consumer_sync();
    }

    if (MODE != kShrinkOnly) {
        // ---------------- expand: y[t][j] += sum_k m[t][k] * B[k][j] ----------------
        constexpr int P = 4 * NSUB;                         // column pairs per warp per tile
        constexpr int RG = 32 / P;                          // lane groups that split the rank rows
        constexpr int RPG = RP / RG;                        // rows per group
        const int pair = lane % P, rg = lane / P;
        const int colw = warp * (NSUB * 8) + 2 * pair;      // column inside the tile
        const uint32_t boff = (colw >> 6) * (RP * 128) + (colw & 7) * 2;
        const int cc = (colw & 63) >> 3;
        const uint32_t m_base = smem_u32(sm.m_s) + rg * RPG * 4;
        const int nB = (p.pool.d_out + C - 1) / C;
        for (int j = 0; j < nB; ++j, ++it) {
            const uint32_t slot = it % kStages;
            mbar_wait(sm.full + slot * 8, (it / kStages) & 1, sm.abort_flag, p.status);
            const uint32_t tile = sm.slots + slot * kSlotBytes + boff;
            float acc[kTokChunk][2];
#pragma unroll
            for (int t = 0; t < kTokChunk; ++t) acc[t][0] = acc[t][1] = 0.f;
#pragma unroll 2
            for (int kk = 0; kk < RPG; kk += 4) {
                uint4 mv[kTokChunk];
#pragma unroll
                for (int t = 0; t < kTokChunk; ++t)
                    if (t < cnt) mv[t] = lds128(m_base + t * (kMaxRank * 4) + kk * 4);
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int k = rg * RPG + kk + q;
                    const uint32_t b = lds32(tile + k * 128 + ((cc ^ ((kk + q) & 7)) << 4));
                    const float b0 = bf_lo(b), b1 = bf_hi(b);
#pragma unroll
                    for (int t = 0; t < kTokChunk; ++t)
                        if (t < cnt) {
                            const float mk = __uint_as_float(q == 0 ? mv[t].x : q == 1 ? mv[t].y : q == 2 ? mv[t].z : mv[t].w);
                            acc[t][0] = fmaf(mk, b0, acc[t][0]);
                            acc[t][1] = fmaf(mk, b1, acc[t][1]);
                        }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(sm.empty + slot * 8);
#pragma unroll
            for (int d = P; d < 32; d <<= 1)
#pragma unroll
                for (int t = 0; t < kTokChunk; ++t) {
                    acc[t][0] += __shfl_xor_sync(0xffffffffu, acc[t][0], d);
                    acc[t][1] += __shfl_xor_sync(0xffffffffu, acc[t][1], d);
                }
            const int col = j * C + colw;
            if (rg == 0 && col < p.pool.d_out) {
#pragma unroll
                for (int t = 0; t < kTokChunk; ++t)
                    if (t < cnt) red_add_v2(p.y + (size_t)tok[t] * p.pool.d_out + col, acc[t][0], acc[t][1]);
            }
        }
    }
}

// RPK = the padded rank when every adapter of the pool has the same one (no dispatch
// inside the unit loop), 0 for a pool of mixed ranks.
template <int MODE, int RPK>
__global__ void __launch_bounds__(kThreads, 2) bgmv_kernel(const Params p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Smem sm;
    sm.slots = smem_u32(smem_raw);
    sm.part = reinterpret_cast<float*>(smem_raw + kStages * kSlotBytes);
    sm.m_s = sm.part + kPartFloats;
    uint8_t* bars = reinterpret_cast<uint8_t*>(sm.m_s + kMFloats);
    sm.full = smem_u32(bars);
    sm.empty = sm.full + kStages * 8;
    sm.abort_flag = reinterpret_cast<volatile int*>(bars + 2 * kStages * 8);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(sm.full + s * 8, 1);
            mbar_init(sm.empty + s * 8, kConsumerWarps);
        }
        *sm.abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();

    const int n_units = *p.bk.n_bgmv_units;

    if (MODE == kShrinkOnly) {
        // tokens without an adapter get a zero row of m
        const int n_active = *p.bk.n_active;
        const long long total = (long long)(p.n_tok - n_active) * p.ldm;
        for (long long i = (long long)blockIdx.x * kThreads + tid; i < total; i += (long long)gridDim.x * kThreads) {
            const int pos = n_active + (int)(i / p.ldm);
            p.m[(size_t)p.bk.perm[pos] * p.ldm + (int)(i % p.ldm)] = 0.f;
        }
    }

    if (warp == kConsumerWarps) {
        // ------------------------------- producer -------------------------------
        if (lane != 0) return;
        uint32_t it = 0;
        for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
            const WorkUnit wu = p.bk.bgmv_units[u];
            const AdapterEntry e = p.pool.table[wu.adapter];
            const int C = tile_cols(e.rp);
            const uint32_t tb = (uint32_t)tile_bytes(e.rp);
            if (MODE != kExpandOnly) {
                const int nA = (p.pool.d_in + C - 1) / C;
                const uint8_t* src = p.pool.slab + e.offA;
                for (int i = 0; i < nA; ++i, ++it) {
                    const uint32_t slot = it % kStages;
                    mbar_wait(sm.empty + slot * 8, ((it / kStages) & 1) ^ 1, sm.abort_flag, p.status);
                    const int cols = min(C, p.pool.d_in - i * C);
                    const uint32_t xbytes = (uint32_t)cols * 2;
                    const uint32_t dst = sm.slots + slot * kSlotBytes;
                    const uint32_t bar = sm.full + slot * 8;
                    mbar_arrive_expect_tx(bar, tb + (uint32_t)wu.cnt * xbytes);
                    bulk_g2s(dst, src + (size_t)i * tb, tb, bar);
                    for (int t = 0; t < wu.cnt; ++t) {
                        const int tk = p.bk.perm[wu.pos0 + t];
                        bulk_g2s(dst + kTileBytesMax + t * kXBytesPerTok, p.x + (size_t)tk * p.pool.d_in + (size_t)i * C,
                                 xbytes, bar);
                    }
                }
            }
            if (MODE != kShrinkOnly) {
                const int nB = (p.pool.d_out + C - 1) / C;
                const uint8_t* src = p.pool.slab + e.offB;
                for (int j = 0; j < nB; ++j, ++it) {
                    const uint32_t slot = it % kStages;
                    mbar_wait(sm.empty + slot * 8, ((it / kStages) & 1) ^ 1, sm.abort_flag, p.status);
                    const uint32_t bar = sm.full + slot * 8;
                    mbar_arrive_expect_tx(bar, tb);
                    bulk_g2s(sm.slots + slot * kSlotBytes, src + (size_t)j * tb, tb, bar);
                }
            }
        }
        return;
    }

    // ------------------------------- consumers -------------------------------
    uint32_t it = 0;
    for (int u = blockIdx.x; u < n_units; u += gridDim.x) {
        const WorkUnit wu = p.bk.bgmv_units[u];
        const AdapterEntry e = p.pool.table[wu.adapter];
        if constexpr (RPK != 0) {
            consume_unit<MODE, RPK>(p, sm, wu, e, it, warp, lane);
        } else {
            switch (e.rp) {
                case 8: consume_unit<MODE, 8>(p, sm, wu, e, it, warp, lane); break;
                case 16: consume_unit<MODE, 16>(p, sm, wu, e, it, warp, lane); break;
                case 32: consume_unit<MODE, 32>(p, sm, wu, e, it, warp, lane); break;
                case 64: consume_unit<MODE, 64>(p, sm, wu, e, it, warp, lane); break;
                default: consume_unit<MODE, 128>(p, sm, wu, e, it, warp, lane); break;
            }
        }
    }
}

}  // namespace

namespace {

using KernelFn = void (*)(const Params);

template <int MODE>
KernelFn pick_rank(int uniform_rp) {
    switch (uniform_rp) {
        case 8: return bgmv_kernel<MODE, 8>;
        case 16: return bgmv_kernel<MODE, 16>;
        case 32: return bgmv_kernel<MODE, 32>;
        case 64: return bgmv_kernel<MODE, 64>;
        case 128: return bgmv_kernel<MODE, 128>;
        default: return bgmv_kernel<MODE, 0>;
    }
}

KernelFn pick_kernel(BgmvMode mode, int uniform_rp) {
    switch (mode) {
        case kFused: return pick_rank<kFused>(uniform_rp);
        case kShrinkOnly: return pick_rank<kShrinkOnly>(uniform_rp);
        default: return pick_rank<kExpandOnly>(uniform_rp);
    }
}

}  // namespace

cudaError_t bgmv_configure() {
    const int modes[3] = {kFused, kShrinkOnly, kExpandOnly};
    const int rps[6] = {0, 8, 16, 32, 64, 128};
    for (int m : modes)
        for (int rp : rps) {
            cudaError_t e = cudaFuncSetAttribute(pick_kernel((BgmvMode)m, rp),
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
            if (e != cudaSuccess) return e;
        }
    return cudaSuccess;
}

cudaError_t launch_bgmv(BgmvMode mode, const PoolDev& pool, const BucketDev& bk, int n_tok, const void* x, float* y,
                        float* m, int ldm, int32_t* status, int sm_count, cudaStream_t stream, int* n_launches) {
    Params p;
    p.pool = pool;
    p.bk = bk;
    p.x = static_cast<const uint16_t*>(x);
    p.y = y;
    p.m = m;
    p.ldm = ldm;
    p.n_tok = n_tok;
    p.status = status;
    // persistent grid: two CTAs per SM, never more CTAs than there can be units
    int grid = 2 * sm_count;
    if (grid > n_tok) grid = n_tok;
    if (grid < 1) grid = 1;
    pick_kernel(mode, pool.uniform_rp)<<<grid, kThreads, kSmemBytes, stream>>>(p);
    ++*n_launches;
    return cudaGetLastError();
}

}  // namespace plora
