// BGMV: the decode-shaped gather-GEMV path of the LoRA delta (paper Section V-A:
// strategy E1 computes y = x A B from matrices resident in GPU memory; strategy E4
// names the halves, shrink m = x A and expand y = m B).  A work unit is up to
// kTokChunk tokens that share an adapter.  The path is bound by HBM bandwidth on
// the adapter bytes (cost model, Section VI-B: the memory term sums D * S * R_i over
// the adapters present, once per adapter whatever its batch), so the kernel is a
// streaming pipeline:
//
//   - a unit's shrink is cut into up to kMaxRuns tasks (runs of consecutive A tiles)
//     and its expand into up to kMaxRuns tasks (runs of B tiles); all shrink tasks
//     come first in the task list and persistent CTAs take tasks round-robin, so
//     the tiles of one adapter stream through many SMs at once and the load is
//     balanced at tile granularity whatever the adapter popularity;
//   - one producer warp per CTA fetches the descriptors of its next 32 tasks at once,
//     then issues bulk asynchronous copies (cp.async.bulk, completion counted on an
//     mbarrier) of whole slab tiles, plus the matching pieces of the unit's x rows,
//     into a ring of shared-memory stages, and runs ahead of the consumers across
//     tiles and tasks; each stage carries a small header that tells the consumers
//     what it holds, so they never wait on global memory for a descriptor;
//   - eight consumer warps split every tile by columns.  Shrink: a lane owns rank
//     rows, reads 16-byte chunks of A^T and broadcast chunks of x, accumulates in
//     fp32; the task's partial m goes to an L2-resident workspace as 64-bit words
//     {value, launch epoch} with plain stores and no fence.  Expand: the producer
//     warp of the CTA that owns the expand task loads the unit's partials (a word
//     whose epoch matches has arrived, otherwise it is read again), sums them in a
//     fixed order, scales them and puts m into the stage next to the B tile; a
//     consumer lane owns two output columns, walks the rank rows, and adds its
//     result to y with one vector reduction per element (no read of y on the SM;
//     one addition per element, so the result is bit-reproducible).  Consumer
//     warps therefore never wait on global memory.
//
// The same template provides the fused path, the shrink-only path (m written to
// the caller's buffer, unscaled, one task per unit) and the expand-only path.
// Every wait (mbarrier or arrival of a partial) is bounded: when it runs out the kernel records
// PLORA_ERR_TIMEOUT in the status word and runs to completion without waiting again.
#include "plora_internal.cuh"

namespace plora {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 32;   // + one producer warp
#ifndef PLORA_EXP_STAGES
#define PLORA_EXP_STAGES 4
#endif
constexpr int kStages = PLORA_EXP_STAGES;
constexpr int kXBytesPerTok = kMaxSubPerTile * kSubCols * 2;             // x piece of one token for one tile
constexpr int kHdrOffset = kTileBytesMax + kTokChunk * kXBytesPerTok;
constexpr int kSlotBytes = kHdrOffset + 128;                             // tile + x pieces + stage header
constexpr int kPartFloats = kConsumerWarps * kTokChunk * kMaxRank;       // two buffers when the rank is <= 64
constexpr int kSmemBytes = kStages * kSlotBytes + kPartFloats * 4 + (2 * kStages + 1) * 8 + 16;
constexpr int kPrefetchTasks = 8;   // tasks per CTA whose tiles are prefetched to L2 before the stream-order wait
constexpr long long kWaitCycles = 4000000000ll;   // about two seconds of SM clock

struct Params {
    PoolDev pool;
    BucketDev bk;
    const uint16_t* x;
    float* y;
    float* m;
    int32_t ldm;
    int32_t n_tok;
    int32_t runs_a, runs_b;   // tasks per unit in the shrink / expand phase
    int32_t early_tables;     // the bucket tables were complete before the previous kernel of the stream began
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
__device__ __forceinline__ void give_up(volatile int* abort_flag, int32_t* status) {
    *abort_flag = 1;
    __threadfence_block();
    atomicCAS(status, 0, PLORA_ERR_TIMEOUT);
}
// Bounded wait on an mbarrier phase.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
    if (mbar_try_wait(bar, parity)) return;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return;
        if (*abort_flag) return;
        if (clock64() - t0 > kWaitCycles) break;
    }
    give_up(abort_flag, status);
}
__device__ __forceinline__ void prefetch_l2(const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
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
__device__ __forceinline__ unsigned long long ldg_cg_u64(const unsigned long long* p) {   // L2 only: L1 may be stale
    unsigned long long v;
    asm volatile("ld.global.cg.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
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
    float* part;         // per-warp partial m of a shrink task
    volatile int* abort_flag;
    uint32_t sync_bar;   // barrier of the consumer warps (one arrival per warp)
    int32_t* status;
    uint32_t epoch;      // this launch's epoch (fused mode)
};

// Per-thread state of the consumer loop.
struct Ctl {
    int pbuf;             // which half of part[] the next shrink task uses
    uint32_t sync_phase;  // parity of the next consumer_sync
};

// Barrier over the consumer warps, built on an mbarrier so that, like every other wait
// in this kernel, it gives up after a bounded time instead of hanging.
__device__ __forceinline__ void consumer_sync(const Smem& sm, Ctl& ctl) {
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(sm.sync_bar);
    mbar_wait(sm.sync_bar, ctl.sync_phase, sm.abort_flag, sm.status);
    ctl.sync_phase ^= 1;
}

// What a stage holds (written by the producer into the stage, read by every consumer warp).
constexpr int kFlagExpand = 1, kFlagFirst = 2, kFlagLast = 4, kFlagEnd = 8;
struct StageHdr {
    int32_t flags;
    int32_t unit, run, tile;
    int32_t cnt;
    int32_t tok[kTokChunk];
    int32_t rp, r;
    float scale;
};

__device__ __forceinline__ StageHdr read_hdr(uint32_t a) {
    const uint4 q0 = lds128(a), q1 = lds128(a + 16), q2 = lds128(a + 32);
    StageHdr h;
    h.flags = (int)q0.x; h.unit = (int)q0.y; h.run = (int)q0.z; h.tile = (int)q0.w;
    h.cnt = (int)q1.x; h.tok[0] = (int)q1.y; h.tok[1] = (int)q1.z; h.tok[2] = (int)q1.w;
    h.tok[3] = (int)q2.x; h.rp = (int)q2.y; h.r = (int)q2.z; h.scale = __uint_as_float(q2.w);
    return h;
}
__device__ __forceinline__ void sts128(uint32_t a, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ int tok_at(const StageHdr& h, int t) {
    return t == 1 ? h.tok[1] : t == 2 ? h.tok[2] : t == 3 ? h.tok[3] : h.tok[0];
}

__device__ __forceinline__ size_t part_index(const Params& p, int unit, int run, int t) {
    return (((size_t)unit * p.runs_a + run) * kTokChunk + t) * p.pool.max_rp;
}
constexpr int kMaxRowsPerLane = kMaxRank / 32;

// ---- shrink: one tile of A^T against the unit's x pieces --------------------------------
// Lane mapping: for RP <= 32 a lane owns one rank row and CPL of the warp's chunks (lane
// groups that share the rows take different chunks); for RP > 32 it owns RP/32 rows and
// all of the warp's chunks.  A 16-byte chunk is 8 consecutive columns.
template <int RP>
struct ShrinkMap {
    static constexpr int NSUB = (kMaxRank / RP > kMaxSubPerTile) ? kMaxSubPerTile : kMaxRank / RP;
    static constexpr int C = NSUB * kSubCols;           // columns per tile
    static constexpr int RPL = RP <= 32 ? 1 : RP / 32;  // rank rows per lane
    static constexpr int G = RP <= 32 ? 32 / RP : 1;    // lane groups that share the rows
    static constexpr int CPL = NSUB / G;                // chunks per lane per tile
    uint32_t a_off[CPL][RPL];   // byte offset of (row, chunk) inside the tile, swizzle applied
    uint32_t x_off[CPL];        // byte offset of the chunk inside a token's x piece
    int col0;                   // first column (inside the tile) of this lane's first chunk
    __device__ __forceinline__ void init(int warp, int lane) {
        const int row = RP <= 32 ? (lane % RP) : lane;
        const int g = RP <= 32 ? (lane / RP) : 0;
#pragma unroll
        for (int q = 0; q < CPL; ++q) {
            const int c = warp * NSUB + g + q * G;
            x_off[q] = c * 16;
#pragma unroll
            for (int rr = 0; rr < RPL; ++rr) {
                const int k = row + 32 * rr;
                a_off[q][rr] = (c >> 3) * (RP * 128) + k * 128 + (((c & 7) ^ (k & 7)) << 4);
            }
        }
        col0 = (warp * NSUB + g) * 8;
    }
};

template <int RP, bool CHECKED>
__device__ __forceinline__ void shrink_chunks(const ShrinkMap<RP>& mp, int cnt, int cols_left, uint32_t tile,
                                              float (&acc)[kMaxRowsPerLane][kTokChunk]) {
    using M = ShrinkMap<RP>;
    const uint32_t xs = tile + kTileBytesMax;
#pragma unroll
    for (int q = 0; q < M::CPL; ++q) {
        if (!CHECKED || mp.col0 + q * M::G * 8 < cols_left) {
            float af[M::RPL][8];
#pragma unroll
            for (int rr = 0; rr < M::RPL; ++rr) unpack8(lds128(tile + mp.a_off[q][rr]), af[rr]);
#pragma unroll
            for (int t = 0; t < kTokChunk; ++t)
                if (t < cnt) {
                    float xf[8];
                    unpack8(lds128(xs + t * kXBytesPerTok + mp.x_off[q]), xf);
#pragma unroll
                    for (int rr = 0; rr < M::RPL; ++rr)
#pragma unroll
                        for (int j = 0; j < 8; ++j) acc[rr][t] = fmaf(xf[j], af[rr][j], acc[rr][t]);
                }
        }
    }
}

template <int RP>
__device__ __forceinline__ void shrink_tile(const Params& p, const StageHdr& h, const ShrinkMap<RP>& mp, uint32_t tile,
                                            float (&acc)[kMaxRowsPerLane][kTokChunk]) {
#ifdef PLORA_EXP_NOCOMPUTE
    return;
#endif
    const int cols_left = p.pool.d_in - h.tile * ShrinkMap<RP>::C;   // only the last tile can be ragged
    if (cols_left >= ShrinkMap<RP>::C)
        shrink_chunks<RP, false>(mp, h.cnt, cols_left, tile, acc);
    else
        shrink_chunks<RP, true>(mp, h.cnt, cols_left, tile, acc);
}

// ---- shrink: end of a task: the CTA's partial m leaves for the workspace (or the caller's m) ----
template <int MODE, int RP>
__device__ __forceinline__ void shrink_finish(const Params& p, const Smem& sm, const StageHdr& h,
                                              float (&acc)[kMaxRowsPerLane][kTokChunk], Ctl& ctl, int warp, int lane) {
    constexpr int RPL = RP <= 32 ? 1 : RP / 32;
    constexpr bool kTwoBuffers = RP <= 64;
    const int row = RP <= 32 ? (lane % RP) : lane;
    const int g = RP <= 32 ? (lane / RP) : 0;
    const int tid = warp * 32 + lane;
    // lanes of different groups hold partial sums of the same rows
#pragma unroll
    for (int d = RP; d < 32; d <<= 1)
#pragma unroll
        for (int rr = 0; rr < RPL; ++rr)
#pragma unroll
            for (int t = 0; t < kTokChunk; ++t) acc[rr][t] += __shfl_xor_sync(0xffffffffu, acc[rr][t], d);
    float* part = sm.part + (kTwoBuffers ? ctl.pbuf * (kConsumerWarps * kTokChunk * RP) : 0);
    if (g == 0) {
#pragma unroll
        for (int rr = 0; rr < RPL; ++rr)
#pragma unroll
            for (int t = 0; t < kTokChunk; ++t)
                if (t < h.cnt) part[(warp * kTokChunk + t) * RP + row + 32 * rr] = acc[rr][t];
    }
    consumer_sync(sm, ctl);
    // fixed-order sum over the warps' column slices
    const int n = h.cnt * RP;
    for (int idx = tid; idx < n; idx += kConsumerThreads) {
        const int t = idx / RP, k = idx % RP;
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) s += part[(w * kTokChunk + t) * RP + k];
        if (MODE == kFused) {
            // value and epoch leave in one 64-bit store: no fence, nobody waits for it here
            p.bk.m_part[part_index(p, h.unit, h.run, t) + k] =
                ((unsigned long long)sm.epoch << 32) | (unsigned long long)__float_as_uint(s);
        } else {
            p.m[(size_t)tok_at(h, t) * p.ldm + k] = s;
        }
    }
    if (MODE != kFused) {
        const int extra = p.ldm - RP;
        for (int idx = tid; idx < h.cnt * extra; idx += kConsumerThreads) {
            const int t = idx / extra, k = RP + idx % extra;
            p.m[(size_t)tok_at(h, t) * p.ldm + k] = 0.f;
        }
    }
    if (kTwoBuffers) ctl.pbuf ^= 1; else consumer_sync(sm, ctl);   // the next task must not overwrite what is still being summed
}

// ---- expand: one tile of B; the result goes straight to y ------------------------------------------
// Lane mapping: a lane owns two adjacent output columns; when the warp's slice has fewer
// than 32 column pairs, lane groups split the rank rows and meet by shuffles.
template <int RP>
struct ExpandMap {
    static constexpr int NSUB = (kMaxRank / RP > kMaxSubPerTile) ? kMaxSubPerTile : kMaxRank / RP;
    static constexpr int C = NSUB * kSubCols;
    static constexpr int P = 4 * NSUB;      // column pairs per warp per tile
    static constexpr int RG = 32 / P;       // lane groups that split the rank rows
    static constexpr int RPG = RP / RG;     // rows per group (8 or 16)
    uint32_t b_off;    // byte offset inside the tile of (first row of the group, this lane's pair), swizzle class 0
    uint32_t m_off;    // byte offset inside the stage of m[0][first row of the group]
    int colw;          // this lane's first column inside the tile
    int rg;
    __device__ __forceinline__ void init(int warp, int lane) {
        const int pair = lane % P;
        rg = lane / P;
        colw = warp * (NSUB * 8) + 2 * pair;
        // the chunk index sits in address bits 4..6 and everything else leaves them clear, so
        // the swizzle of row class j is one XOR with (j << 4)
        b_off = (colw >> 6) * (RP * 128) + rg * RPG * 128 + (((colw & 63) >> 3) << 4) + (colw & 7) * 2;
        m_off = kTileBytesMax + rg * RPG * 4;
    }
};

template <int MODE, int RP>
__device__ __forceinline__ void expand_tile(const Params& p, const StageHdr& h, const ExpandMap<RP>& mp, uint32_t tile,
                                            uint32_t empty_bar, int lane) {
    using M = ExpandMap<RP>;
    const uint32_t b0 = tile + mp.b_off;
    const uint32_t mb = tile + mp.m_off;
    float acc[kTokChunk][2];
#pragma unroll
    for (int t = 0; t < kTokChunk; ++t) acc[t][0] = acc[t][1] = 0.f;
#pragma unroll
    for (int kk = 0; kk < M::RPG; kk += 4) {
        uint4 mv[kTokChunk];
#pragma unroll
        for (int t = 0; t < kTokChunk; ++t)
            if (t < h.cnt) {
                mv[t] = lds128(mb + t * (RP * 4) + kk * 4);
                if (MODE == kExpandOnly && h.r < RP) {
                    // the caller's m may hold anything beyond the adapter's rank
                    const int k0 = mp.rg * M::RPG + kk;
                    if (k0 + 0 >= h.r) mv[t].x = 0u;
                    if (k0 + 1 >= h.r) mv[t].y = 0u;
                    if (k0 + 2 >= h.r) mv[t].z = 0u;
                    if (k0 + 3 >= h.r) mv[t].w = 0u;
                }
            }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int k = kk + q;   // row inside the group; its swizzle class is k & 7
            const uint32_t b = lds32((b0 ^ ((k & 7) << 4)) + k * 128);
            const float blo = bf_lo(b), bhi = bf_hi(b);
#pragma unroll
            for (int t = 0; t < kTokChunk; ++t)
                if (t < h.cnt) {
                    const float mk = __uint_as_float(q == 0 ? mv[t].x : q == 1 ? mv[t].y : q == 2 ? mv[t].z : mv[t].w);
                    acc[t][0] = fmaf(mk, blo, acc[t][0]);
                    acc[t][1] = fmaf(mk, bhi, acc[t][1]);
                }
        }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(empty_bar);
#pragma unroll
    for (int d = M::P; d < 32; d <<= 1)
#pragma unroll
        for (int t = 0; t < kTokChunk; ++t) {
            acc[t][0] += __shfl_xor_sync(0xffffffffu, acc[t][0], d);
            acc[t][1] += __shfl_xor_sync(0xffffffffu, acc[t][1], d);
        }
    const int col = h.tile * M::C + mp.colw;
    if (mp.rg == 0 && col < p.pool.d_out) {
#pragma unroll
        for (int t = 0; t < kTokChunk; ++t)
            if (t < h.cnt)
                red_add_v2(p.y + (size_t)h.tok[t] * p.pool.d_out + col, acc[t][0] * h.scale, acc[t][1] * h.scale);
    }
}

// Per-lane constants of both phases for one padded rank.
template <int RP>
struct LaneMaps {
    ShrinkMap<RP> s;
    ExpandMap<RP> e;
    __device__ __forceinline__ void init(int warp, int lane) {
        s.init(warp, lane);
        e.init(warp, lane);
    }
};

// One stage, consumer side.
template <int MODE, int RP>
__device__ __forceinline__ void consume_stage(const Params& p, const Smem& sm, const StageHdr& h,
                                              const LaneMaps<RP>& maps, uint32_t tile, uint32_t empty_bar,
                                              float (&acc)[kMaxRowsPerLane][kTokChunk], Ctl& ctl, int warp, int lane) {
    if (!(h.flags & kFlagExpand)) {
        if (MODE != kExpandOnly) {
            if (h.flags & kFlagFirst) {
#pragma unroll
                for (int rr = 0; rr < kMaxRowsPerLane; ++rr)
#pragma unroll
                    for (int t = 0; t < kTokChunk; ++t) acc[rr][t] = 0.f;
            }
            shrink_tile<RP>(p, h, maps.s, tile, acc);
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar);
            if (h.flags & kFlagLast) shrink_finish<MODE, RP>(p, sm, h, acc, ctl, warp, lane);
        }
    } else {
        if (MODE != kShrinkOnly) {
            expand_tile<MODE, RP>(p, h, maps.e, tile, empty_bar, lane);
        }
    }
}

// Pools of mixed ranks: the lane constants are rebuilt for every stage.
template <int MODE, int RP>
__device__ __noinline__ void stage_of_rank(const Params& p, const Smem& sm, const StageHdr& h, uint32_t tile,
                                           uint32_t empty_bar, float (&acc)[kMaxRowsPerLane][kTokChunk], Ctl& ctl,
                                           int warp, int lane) {
    LaneMaps<RP> maps;
    maps.init(warp, lane);
    consume_stage<MODE, RP>(p, sm, h, maps, tile, empty_bar, acc, ctl, warp, lane);
}

// ---- producer side: the m of an expand task ---------------------------------------------------
// A unit's m has cnt * rp values; lane l of the producer warp owns the values l, l + 32, ...
constexpr int kMPerLane = kTokChunk * kMaxRank / 32;

struct MVals {
    float v[kMPerLane];
    bool ok;   // every partial read so far carried this launch's epoch
};

// Read the runs_a partials of every owned value and sum them in run order.  Nothing here
// waits; `ok` tells whether every word carried this launch's epoch.
__device__ __forceinline__ void load_m(const Params& p, uint32_t epoch, int unit, int cnt, int rp, int lane, MVals& out) {
    out.ok = true;
    const int n = cnt * rp;
#pragma unroll
    for (int q = 0; q < kMPerLane; ++q) {
        const int idx = lane + 32 * q;
        float s = 0.f;
        if (idx < n) {
            const int t = idx / rp, k = idx - t * rp;
            unsigned long long w[kMaxRuns];
#pragma unroll
            for (int j = 0; j < kMaxRuns; ++j)
                w[j] = j < p.runs_a ? ldg_cg_u64(p.bk.m_part + part_index(p, unit, j, t) + k)
                                    : ((unsigned long long)epoch << 32);
#pragma unroll
            for (int j = 0; j < kMaxRuns; ++j) {
                out.ok = out.ok && (uint32_t)(w[j] >> 32) == epoch;
                s += __uint_as_float((uint32_t)w[j]);
            }
        }
        out.v[q] = s;
    }
}

// A task: one run of tiles of one unit in one phase.
struct Task {
    int unit;
    int phase;   // 0 = shrink, 1 = expand
    int run;
};

__device__ __forceinline__ Task decode_task(int t, int n_shrink_tasks, int runs_a, int runs_b) {
    Task k;
    if (t < n_shrink_tasks) {
        k.phase = 0;
        k.unit = t / runs_a;
        k.run = t - k.unit * runs_a;
    } else {
        t -= n_shrink_tasks;
        k.phase = 1;
        k.unit = t / runs_b;
        k.run = t - k.unit * runs_b;
    }
    return k;
}

// RPK = the padded rank when every adapter of the pool has the same one (no dispatch
// inside the stage loop), 0 for a pool of mixed ranks.
template <int MODE, int RPK>
__global__ void __launch_bounds__(kThreads, 2) bgmv_kernel(const Params p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Smem sm;
    sm.slots = smem_u32(smem_raw);
    sm.part = reinterpret_cast<float*>(smem_raw + kStages * kSlotBytes);
    uint8_t* bars = reinterpret_cast<uint8_t*>(sm.part + kPartFloats);
    sm.full = smem_u32(bars);
    sm.empty = sm.full + kStages * 8;
    sm.sync_bar = sm.empty + kStages * 8;
    sm.abort_flag = reinterpret_cast<volatile int*>(bars + (2 * kStages + 1) * 8);
    sm.status = p.status;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(sm.full + s * 8, 1);
            mbar_init(sm.empty + s * 8, kConsumerWarps);
            // a stage that was never filled reads as "nothing follows"
            sts128(sm.slots + s * kSlotBytes + kHdrOffset, (uint32_t)kFlagEnd, 0u, 0u, 0u);
        }
        mbar_init(sm.sync_bar, kConsumerWarps);
        *sm.abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    // Everything above may overlap the previous kernel of the stream.  Its results (x, y, m,
    // the epoch, possibly the bucket tables) are read only after grid_dependency_wait().  The
    // producer warp delays that wait: the slab is never written by a kernel, and bucket tables
    // older than the previous kernel are complete, so it fetches its first task descriptors and
    // pulls its first tiles into L2 while the previous kernel drains.
    if (warp != kConsumerWarps) {
        grid_dependency_wait();
        // Signalled only after this CTA has seen the previous kernel complete: when the next kernel
        // of the stream starts, everything older than this kernel is therefore complete.
        grid_launch_dependents();
        sm.epoch = MODE == kFused ? *p.bk.epoch : 0u;
    }

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
        // ------------------------------- producer warp -------------------------------
        // The warp fetches the descriptors of its next 32 tasks in one go (lane l owns the
        // l-th of them), then walks them: lane 0 drives the barriers, writes the stage
        // header and copies the tile; lane t < cnt copies token t's piece of x.
        bool waited = false;
        if (!p.early_tables) {
            grid_dependency_wait();
            waited = true;
        }
        const int n_units = *p.bk.n_bgmv_units;
        const int n_shrink = MODE == kExpandOnly ? 0 : n_units * p.runs_a;
        const int n_tasks = n_shrink + (MODE == kShrinkOnly ? 0 : n_units * p.runs_b);
        const int stride = gridDim.x;
        uint32_t it = 0;
        for (int base = blockIdx.x; base < n_tasks; base += 32 * stride) {
            const int my_task = base + lane * stride;
            Task mine = decode_task(my_task < n_tasks ? my_task : base, n_shrink, p.runs_a, p.runs_b);
            const WorkUnit mu = p.bk.bgmv_units[mine.unit];
            const AdapterEntry me = p.pool.table[mu.adapter];
            const int in_batch = min(32, (n_tasks - base + stride - 1) / stride);
            if (!waited) {
                // lane l pulls the tiles of this CTA's l-th task towards L2, then the warp joins the stream order
                if (my_task < n_tasks && lane < kPrefetchTasks) {
                    const int d = mine.phase ? p.pool.d_out : p.pool.d_in;
                    const int runs = mine.phase ? p.runs_b : p.runs_a;
                    const int nT = tiles_for(d, me.rp);
                    const uint32_t tb = (uint32_t)tile_bytes(me.rp);
                    const uint8_t* src = p.pool.slab + (mine.phase ? me.offB : me.offA);
                    for (int i = mine.run * nT / runs; i < (mine.run + 1) * nT / runs; ++i)
                        prefetch_l2(src + (size_t)i * tb, tb);
                }
                grid_dependency_wait();
                waited = true;
            }
            if (base == (int)blockIdx.x) sm.epoch = MODE == kFused ? *p.bk.epoch : 0u;
            for (int b = 0; b < in_batch; ++b) {
                const unsigned full = 0xffffffffu;
                const int phase = __shfl_sync(full, mine.phase, b), unit = __shfl_sync(full, mine.unit, b);
                const int run = __shfl_sync(full, mine.run, b), cnt = __shfl_sync(full, mu.cnt, b);
                const int tok0 = __shfl_sync(full, mu.tok[0], b), tok1 = __shfl_sync(full, mu.tok[1], b);
                const int tok2 = __shfl_sync(full, mu.tok[2], b), tok3 = __shfl_sync(full, mu.tok[3], b);
                const int rp = __shfl_sync(full, me.rp, b), r = __shfl_sync(full, me.r, b);
                const uint32_t scale_bits = __shfl_sync(full, __float_as_uint(me.scale), b);
                const unsigned long long off = __shfl_sync(full, phase ? me.offB : me.offA, b);
                const int C = tile_cols(rp);
                const uint32_t tb = (uint32_t)tile_bytes(rp);
                const int d = phase ? p.pool.d_out : p.pool.d_in;
                const int runs = phase ? p.runs_b : p.runs_a;
                const int nT = tiles_for(d, rp);
                const int lo = run * nT / runs, hi = (run + 1) * nT / runs;
                const uint8_t* src = p.pool.slab + off;
                const int my_tok = lane == 1 ? tok1 : lane == 2 ? tok2 : lane == 3 ? tok3 : tok0;
                const uint16_t* xrow = p.x + (size_t)my_tok * p.pool.d_in;
                const uint16_t* mrow = reinterpret_cast<const uint16_t*>(p.m + (size_t)my_tok * p.ldm);
                MVals mv;
                if (MODE == kFused && phase) {
                    load_m(p, sm.epoch, unit, cnt, rp, lane, mv);
                    if (!__all_sync(full, mv.ok)) {
                        // some shrink task of this unit has not delivered yet: read again, for a bounded time
                        const long long t0 = clock64();
                        for (;;) {
                            __nanosleep(100);
                            load_m(p, sm.epoch, unit, cnt, rp, lane, mv);
                            if (__all_sync(full, mv.ok) || *sm.abort_flag) break;
                            if (clock64() - t0 > kWaitCycles) {
                                if (lane == 0) give_up(sm.abort_flag, p.status);
                                break;
                            }
                        }
                    }
                }
                // bytes a token adds to the stage besides the tile: its x piece (shrink) or its m row (expand-only)
                const uint32_t mbytes = (MODE == kExpandOnly) ? (uint32_t)rp * 4u : 0u;
                for (int i = lo; i < hi; ++i, ++it) {
                    const uint32_t slot = it % kStages;
                    const uint32_t dst = sm.slots + slot * kSlotBytes;
                    const uint32_t bar = sm.full + slot * 8;
                    const uint32_t tbytes = phase ? mbytes : (uint32_t)min(C, d - i * C) * 2u;
                    if (lane == 0) {
                        mbar_wait(sm.empty + slot * 8, ((it / kStages) & 1) ^ 1, sm.abort_flag, p.status);
                        const int flags = (phase ? kFlagExpand : 0) | (i == lo ? kFlagFirst : 0) | (i == hi - 1 ? kFlagLast : 0);
                        sts128(dst + kHdrOffset, (uint32_t)flags, (uint32_t)unit, (uint32_t)run, (uint32_t)i);
                        sts128(dst + kHdrOffset + 16, (uint32_t)cnt, (uint32_t)tok0, (uint32_t)tok1, (uint32_t)tok2);
                        sts128(dst + kHdrOffset + 32, (uint32_t)tok3, (uint32_t)rp, (uint32_t)r, scale_bits);
                    }
                    __syncwarp();   // the stage is free before anyone writes into it
                    if (MODE == kFused && phase) {
                        // m[t][k] of the unit (unscaled) rides in the stage's x area
#pragma unroll
                        for (int q = 0; q < kMPerLane; ++q)
                            if (lane + 32 * q < cnt * rp)
                                asm volatile("st.shared.f32 [%0], %1;" ::"r"(dst + kTileBytesMax + (lane + 32 * q) * 4),
                                             "f"(mv.v[q]) : "memory");
                        __syncwarp();
                    }
                    if (lane == 0) {
                        mbar_arrive_expect_tx(bar, tb + (uint32_t)cnt * tbytes);
                        bulk_g2s(dst, src + (size_t)i * tb, tb, bar);
                    }
                    if (lane < cnt) {
                        if (!phase)
                            bulk_g2s(dst + kTileBytesMax + lane * kXBytesPerTok, xrow + (size_t)i * C, tbytes, bar);
                        else if (MODE == kExpandOnly)   // the caller's m row, rp floats, lands as m[t][0..rp)
                            bulk_g2s(dst + kTileBytesMax + lane * mbytes, mrow, mbytes, bar);
                    }
                }
            }
        }
        if (!waited) grid_dependency_wait();
        if (lane == 0) {   // tell the consumers that nothing follows
            const uint32_t slot = it % kStages;
            mbar_wait(sm.empty + slot * 8, ((it / kStages) & 1) ^ 1, sm.abort_flag, p.status);
            sts128(sm.slots + slot * kSlotBytes + kHdrOffset, (uint32_t)kFlagEnd, 0u, 0u, 0u);
            mbar_arrive(sm.full + slot * 8);
        }
        return;
    }

    // ------------------------------- consumer warps -------------------------------
    float acc[kMaxRowsPerLane][kTokChunk];
    Ctl ctl;
    ctl.pbuf = 0;
    ctl.sync_phase = 0;
    LaneMaps<RPK == 0 ? 8 : RPK> maps;   // per-lane constants, computed once when the rank is uniform
    if constexpr (RPK != 0) maps.init(warp, lane);
    for (uint32_t it = 0;; ++it) {
        const uint32_t slot = it % kStages;
        mbar_wait(sm.full + slot * 8, (it / kStages) & 1, sm.abort_flag, p.status);
        const uint32_t tile = sm.slots + slot * kSlotBytes;
        const StageHdr h = read_hdr(tile + kHdrOffset);
        if ((h.flags & kFlagEnd) || *sm.abort_flag) break;
        const uint32_t empty_bar = sm.empty + slot * 8;
        if constexpr (RPK != 0) {
            consume_stage<MODE, RPK>(p, sm, h, maps, tile, empty_bar, acc, ctl, warp, lane);
        } else {
            switch (h.rp) {
                case 8: stage_of_rank<MODE, 8>(p, sm, h, tile, empty_bar, acc, ctl, warp, lane); break;
                case 16: stage_of_rank<MODE, 16>(p, sm, h, tile, empty_bar, acc, ctl, warp, lane); break;
                case 32: stage_of_rank<MODE, 32>(p, sm, h, tile, empty_bar, acc, ctl, warp, lane); break;
                case 64: stage_of_rank<MODE, 64>(p, sm, h, tile, empty_bar, acc, ctl, warp, lane); break;
                default: stage_of_rank<MODE, 128>(p, sm, h, tile, empty_bar, acc, ctl, warp, lane); break;
            }
        }
    }
    if (MODE == kFused && tid == 0) {
        // the last CTA to finish opens the next epoch: words written by this launch can never
        // be mistaken for the next one's
        if (atomicAdd(p.bk.exit_count, 1u) == gridDim.x - 1) {
            *p.bk.exit_count = 0u;
            *p.bk.epoch = sm.epoch + 1u;
        }
    }
}

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

int clamp_runs(int tiles) { return tiles < 1 ? 1 : (tiles > kMaxRuns ? kMaxRuns : tiles); }

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
                        float* m, int ldm, int32_t* status, int sm_count, bool early_tables, cudaStream_t stream,
                        int* n_launches) {
    Params p;
    p.pool = pool;
    p.bk = bk;
    p.x = static_cast<const uint16_t*>(x);
    p.y = y;
    p.m = m;
    p.ldm = ldm;
    p.n_tok = n_tok;
    p.status = status;
    p.early_tables = early_tables ? 1 : 0;
    // Every adapter has at least tiles_for(d, min_rp) tiles, so each unit can be cut into that many runs.
    p.runs_a = mode == kShrinkOnly ? 1 : clamp_runs(tiles_for(pool.d_in, pool.min_rp));
    // an expand task pays one round trip for its m before its first tile: give it at least two tiles
    p.runs_b = clamp_runs(tiles_for(pool.d_out, pool.min_rp) / (mode == kFused ? 2 : 1));
    if (mode == kFused) {
        // the partial-m workspace holds n_units * runs_a * kTokChunk * max_rp words, n_units <= n_tok
        const size_t per_run = (size_t)n_tok * kTokChunk * pool.max_rp * sizeof(unsigned long long);
        while (p.runs_a > 1 && per_run * p.runs_a > bk.m_part_bytes) --p.runs_a;
        if (per_run * p.runs_a > bk.m_part_bytes) return cudaErrorMemoryAllocation;
    }
    // persistent grid: two CTAs per SM, never more CTAs than there can be tasks
    const long long max_tasks = (long long)n_tok * (p.runs_a + p.runs_b);
    int grid = 2 * sm_count;
    if (grid > max_tasks) grid = (int)max_tasks;
    if (grid < 1) grid = 1;

    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, pick_kernel(mode, pool.uniform_rp), p);
    ++*n_launches;
    return e;
}

}  // namespace plora
