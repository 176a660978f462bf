// BGMV: the decode-shaped gather-GEMV path of the LoRA delta (paper Section V-A:
// strategy E1 computes y = x A B from matrices resident in GPU memory; strategy E4
// names the halves, shrink m = x A and expand y = m B).  A work unit is up to
// kTokChunk tokens that share an adapter.  The path is bound by HBM bandwidth on
// the adapter bytes (cost model, Section VI-B: the memory term sums D * S * R_i over
// the adapters present, once per adapter whatever its batch), so the kernel is a
// streaming pipeline:
//
//   - a unit's shrink is cut into up to kMaxRunsA tasks (runs of consecutive A tiles; a launch with
//     few units of padded rank 64 or 128 also cuts along the rank, see "Row slices") and its expand
//     into runs of B tiles; all shrink tasks come first in the task list and persistent CTAs take
//     tasks round-robin, so the tiles of one adapter stream through many SMs at once and the load
//     is balanced at tile granularity whatever the adapter popularity.  A launch serves one padded
//     rank (its loops are compiled for that rank) or, for a small batch on a pool of mixed ranks,
//     all ranks at once, with the classes cut to tasks of equal size (see "the task list of a launch");
//   - one producer warp per CTA fetches the descriptors of its next 32 tasks at once,
//     then issues bulk asynchronous copies (cp.async.bulk, completion counted on an
//     mbarrier) of whole slab tiles, plus the matching pieces of the unit's x rows,
//     into a ring of shared-memory stages, and runs ahead of the consumers across
//     tiles and tasks; each stage carries a small header that tells the consumers
//     what it holds, so they never wait on global memory for a descriptor;
//   - eight consumer warps work on every tile.  Shrink: the warps split the rank rows,
//     the lanes of a warp split the tile's columns (16-byte chunks of A^T against the
//     matching chunks of x, fp32 accumulation) and meet by shuffles at the end of the
//     task, so a warp owns complete sums of its rows and no warp waits for another;
//     the task's partial m goes to an L2-resident workspace as 64-bit words
//     {value, launch epoch} with plain stores and no fence.  Expand: a gather warp of the CTA
//     that owns the expand task loads the unit's partials (a word whose epoch matches has
//     arrived, otherwise it is read again), sums them in a fixed order and puts m into a small
//     ring next to the stages; a consumer lane owns two output columns, walks the rank rows, and
//     adds its result to y with one vector reduction per element (no read of y on the SM;
//     one addition per element, so the result is bit-reproducible).  Consumer warps therefore
//     never wait on global memory.  Both inner loops use the packed fp32 multiply-add of sm_100
//     (two FMAs per instruction): the kernel is bound by instruction issue where HBM does not
//     bound it.  The shrink of a unit with several tokens at padded rank 64 or 128 runs on the
//     tensor cores (mma.sync) in one-rank launches.
//
// The same template provides the fused path, the shrink-only path (m written to
// the caller's buffer, unscaled, one task per unit) and the expand-only path.
// Every wait (mbarrier or arrival of a partial) is bounded: when it runs out the kernel records
// PLORA_ERR_TIMEOUT in the status word and runs to completion without waiting again.
#include <cuda_fp16.h>

#include "plora_internal.cuh"

namespace plora {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kProducerWarp = kConsumerWarps;       // issues the copies
constexpr int kGatherWarp = kConsumerWarps + 1;     // fused mode: assembles the m of the expand tasks
constexpr int kThreads = kConsumerThreads + 64;
constexpr int kCtasPerSm = 2;   // persistent CTAs per SM
constexpr int kStages = 5;
// x piece of one token for one tile, plus 32 bytes: the pieces of a unit's (up to four) tokens then start in
// different banks, and the tensor-core shrink reads one word of each at a time
constexpr int kXBytesPerTok = kMaxSubPerTile * kSubCols * 2 + 32;
constexpr int kHdrOffset = kTileBytesMax + kTokChunk * kXBytesPerTok;
constexpr int kSlotBytes = kHdrOffset + 128;                             // tile + x pieces + stage header
// m of the expand tasks in flight (fused mode): a ring filled by the gather warp and drained by
// the consumers, with a full / empty barrier pair per entry.
constexpr int kMRing = 4;
constexpr int kMRingBytes = kTokChunk * kMaxRank * 4;
constexpr int kNumBarriers = 2 * kStages + 2 * kMRing;
constexpr int kSmemBytes = kStages * kSlotBytes + kMRing * kMRingBytes + kNumBarriers * 8 + 16;
constexpr uint32_t kSuspendHintNs = 20000;   // a waiting thread may sleep this long inside one try_wait
constexpr long long kWaitCycles = 4000000000ll;   // default limit of a wait: about two seconds of SM clock

// Projections that do not depend on one another (q, k and v of a layer; up and gate) can share a
// launch: the task list simply runs over "virtual units" (group, unit).  The pools of a group have
// the same shape.
constexpr int kMaxGroup = kMaxGroupPools;

struct Params {
    PoolDev pool;                                // shape (d_in, d_out, max_rp) shared by the group
    BucketDev bk;
    int32_t n_groups;
    const uint8_t* slab_g[kMaxGroup];
    uint64_t slab_bytes_g[kMaxGroup];   // (read by the debug build's address checks only)
    const AdapterEntry* table_g[kMaxGroup];
    const uint16_t* x_g[kMaxGroup];
    float* y_g[kMaxGroup];
    float* m;                 // shrink-only / expand-only: the caller's m, fp32 or (m16) bf16, ldm values per token
    int32_t ldm;
    int32_t m16;              // m holds 2-byte values (the paper's strategy E4 ships m at S = 2 bytes)
    int32_t n_tok;
    int32_t runs_a, runs_b;   // tasks per unit in the shrink / expand phase
    int32_t runs_a_sliced;    // column runs per unit when the launch cuts its units into row slices
    int32_t early_tables;     // the bucket tables were complete before the previous kernel of the stream began
    int32_t maybe_empty;      // the batch may have sent every segment to the tensor-core path: look before setting up
    int32_t by_class;         // the launch walks its class's part of bk.cls_list (pools of mixed ranks)
    // The class launches of one call work on different units: a later one need not wait for the
    // one before it.  It joins the stream order only when its CTAs are done (so that its completion
    // still implies the completion of everything before it) and leaves the epoch to the last of them.
    int32_t defer_wait;
    int32_t bump_epoch;

    int32_t* status;
    long long wait_cycles;    // limit of every bounded wait, in SM clock cycles
    int32_t test_hook;        // PLORA_HOOK_*: tests make a wait run out with it
    // The caller states that x was complete before the previous kernel of the stream began
    // (plora_set_inputs_resident): the launch uses the kernels that stream and multiply x before they join
    // the stream order, and join when they first have something to write (host side only).
    int32_t inputs_resident;
    int32_t sort_by_cnt;      // classify pass: order the units of a class by token count (the launch for all classes follows)
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
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void give_up(volatile int* abort_flag, int32_t* status) {
    *abort_flag = 1;
    __threadfence_block();
    atomicCAS(status, 0, PLORA_ERR_TIMEOUT);
}
// Bounded wait on an mbarrier phase.  True: the phase is complete.  False: the wait ran out, here
// (then the status word says so) or in another role of this CTA (the abort flag).  What the caller
// does with a false: a consumer lane leaves the kernel at once, executing no warp-level operation on
// its way out (the lanes of a warp may get different answers in the instant a give-up happens, and
// the shuffles and warp barriers further on are defined over the lanes that have not exited); the
// copy warp and the gather warp let one lane decide and broadcast it, and stop issuing.
struct WaitCtl {
    volatile int* abort_flag;
    int32_t* status;
    long long limit;
};
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtl& w) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*w.abort_flag) return false;
        if (clock64() - t0 > w.limit) break;
    }
    give_up(w.abort_flag, w.status);
    return false;
}
// The copy warp's last look at a stage before it leaves: has everything it asked for arrived?  Waits
// whatever the abort flag says, for at most the limit (a CTA must not retire with a bulk copy still on
// its way into its shared memory).
// (Inlined on purpose, like every wait here: a real call anywhere in the kernel made the whole kernel slower, 1.6 % on
// the 7B decode step for this one, 4 % for a called slow path of mbar_wait.)
__device__ __forceinline__ bool mbar_drain(uint32_t bar, uint32_t parity, long long limit) {
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity))
        if (clock64() - t0 > limit) return false;
    return true;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
// Source of a bulk copy, [ptr, ptr + bytes) inside [base, base + size).  Debug build: a source outside its buffer is
// recorded and replaced by the start of the buffer (the copy still runs, so the stage's barrier completes and the
// pipeline keeps moving; the result is wrong and the status word says why).  Ordinary build: the pointer as it is.
__device__ __forceinline__ const void* checked_src(const void* ptr, uint32_t bytes, const void* base, uint64_t size,
                                                   int32_t* status) {
#ifdef PLORA_DEBUG
    const uint64_t off = (uint64_t)(static_cast<const uint8_t*>(ptr) - static_cast<const uint8_t*>(base));
    if (ptr < base || off + bytes > size) {
        atomicCAS(status, 0, PLORA_ERR_DEBUG_CHECK);
        return base;
    }
#endif
    return ptr;
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
// The two 16-bit values of a word as fp32: bf16 (H = false) or IEEE half (H = true) inputs.
template <bool H>
__device__ __forceinline__ float in_lo(uint32_t w) {
    return H ? __half2float(__ushort_as_half((unsigned short)(w & 0xffffu))) : bf_lo(w);
}
template <bool H>
__device__ __forceinline__ float in_hi(uint32_t w) {
    return H ? __half2float(__ushort_as_half((unsigned short)(w >> 16))) : bf_hi(w);
}
template <bool H>
__device__ __forceinline__ void unpack8(const uint4& v, float* f) {
    f[0] = in_lo<H>(v.x); f[1] = in_hi<H>(v.x); f[2] = in_lo<H>(v.y); f[3] = in_hi<H>(v.y);
    f[4] = in_lo<H>(v.z); f[5] = in_hi<H>(v.z); f[6] = in_lo<H>(v.w); f[7] = in_hi<H>(v.w);
}

// The four words of a 16-byte chunk as four (even column, odd column) pairs.
template <bool H>
__device__ __forceinline__ void unpack4x2(const uint4& v, float2* f) {
    f[0] = make_float2(in_lo<H>(v.x), in_hi<H>(v.x));
    f[1] = make_float2(in_lo<H>(v.y), in_hi<H>(v.y));
    f[2] = make_float2(in_lo<H>(v.z), in_hi<H>(v.z));
    f[3] = make_float2(in_lo<H>(v.w), in_hi<H>(v.w));
}

struct Smem {
    uint32_t slots;      // shared address of stage 0
    uint32_t full;       // full[kStages] barriers
    uint32_t empty;      // empty[kStages]
    WaitCtl wait;        // abort flag of the CTA, status word, limit of a wait
    uint32_t m_ring;     // shared address of the m ring (fused mode): kMRing entries of kMRingBytes
    uint32_t m_full;     // m_full[kMRing]: the gather warp has written the entry
    uint32_t m_empty;    // m_empty[kMRing]: every consumer warp is done with the entry
    mutable uint32_t epoch;   // this launch's epoch (fused mode); mutable: a thread that joins late learns it then
    bool withhold;       // test hook: this warp never hands a stage back
    mutable bool joined;      // lazy launches: this thread has joined the stream order and knows the epoch
};
// A consumer warp is done with a stage.
__device__ __forceinline__ void release_stage(const Smem& sm, uint32_t empty_bar, int lane) {
    if (lane == 0 && !sm.withhold) mbar_arrive(empty_bar);
}

// A consumer thread that put off joining the stream order does so now: from here on it may write
// (partial words, y), and it knows the launch's epoch.
__device__ __forceinline__ void join_stream(const Params& p, const Smem& sm) {
    if (!sm.joined) {
        grid_dependency_wait();
        grid_launch_dependents();
        sm.epoch = *p.bk.epoch;
        sm.joined = true;
    }
}

// What a stage holds (written by the producer into the stage, read by every consumer warp).
constexpr int kFlagExpand = 1, kFlagFirst = 2, kFlagLast = 4, kFlagEnd = 8, kFlagSlice = 16;
struct StageHdr {
    int32_t flags;
    int32_t unit, run, tile;
    int32_t cnt;
    int32_t tok[kTokChunk];
    int32_t rp, r;
    float scale;
    int32_t m_seq;    // fused expand stages: running number of the expand task in this CTA (m-ring entry = m_seq % kMRing)
    int32_t group;    // which projection of the launch's group (unit = group * n_units + bucket unit)
    int32_t k0;       // shrink stages of a row slice: first rank row of the slice (otherwise 0)
    // (the word after k0 holds the stage's running number, for the copy warp's own use: kStampOffset)
};
constexpr int kStampOffset = 60;            // byte offset inside the header
constexpr uint32_t kNoStamp = 0xffffffffu;  // the stage was never armed

__device__ __forceinline__ StageHdr read_hdr(uint32_t a) {
    const uint4 q0 = lds128(a), q1 = lds128(a + 16), q2 = lds128(a + 32);
    const uint32_t q3 = lds32(a + 48), q4 = lds32(a + 52), q5 = lds32(a + 56);
    StageHdr h;
    h.flags = (int)q0.x; h.unit = (int)q0.y; h.run = (int)q0.z; h.tile = (int)q0.w;
    h.cnt = (int)q1.x; h.tok[0] = (int)q1.y; h.tok[1] = (int)q1.z; h.tok[2] = (int)q1.w;
    h.tok[3] = (int)q2.x; h.rp = (int)q2.y; h.r = (int)q2.z; h.scale = __uint_as_float(q2.w);
    h.m_seq = (int)q3;
    h.group = (int)q4;
    h.k0 = (int)q5;
    return h;
}
__device__ __forceinline__ void sts128(uint32_t a, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ int tok_at(const StageHdr& h, int t) {
    return t == 1 ? h.tok[1] : t == 2 ? h.tok[2] : t == 3 ? h.tok[3] : h.tok[0];
}

// Where the partial m of (run, token) lives: a token is named by its projection and its position in
// the sorted order (row0 = projection * n_tok + position of the unit's first token).  The layout does
// not depend on a launch's own number of runs or on its rank class: the class launches of one call
// share an epoch, so their units must not meet in the workspace.
// One value of the caller's m (shrink-only mode): fp32, or bf16 rounded to nearest even.
__device__ __forceinline__ void store_m(const Params& p, size_t idx, float v) {
    PLORA_CHECKED(idx < (size_t)p.n_tok * p.ldm, p.status)
    if (p.m16) {
        const uint32_t u = __float_as_uint(v);
        reinterpret_cast<uint16_t*>(p.m)[idx] = (uint16_t)((u + 0x7fffu + ((u >> 16) & 1u)) >> 16);
    } else {
        p.m[idx] = v;
    }
}
__device__ __forceinline__ size_t part_index(const Params& p, int row0, int run, int t) {
    return (((size_t)row0 + t) * kMaxRunsA + run) * p.pool.max_rp;
}
constexpr int kMaxRowsPerLane = kMaxRank / 32;

// ---- shrink: one tile of A^T against the unit's x pieces --------------------------------
// Work split: warp w owns the rank rows [w * RP/8, (w + 1) * RP/8).  Inside the warp the lanes
// split the tile's 16-byte chunks (8 columns each); when the tile has fewer than 32 chunks
// (RP >= 64) lane groups also split the warp's rows.  Every lane ends up with 32 products per
// token and tile (16 for RP = 8, whose tile is half as large).
template <int RP>
struct ShrinkMap {
    static constexpr int NSUB = (kMaxRank / RP > kMaxSubPerTile) ? kMaxSubPerTile : kMaxRank / RP;
    static constexpr int C = NSUB * kSubCols;            // columns per tile
    static constexpr int CH = 8 * NSUB;                  // chunks per tile
    static constexpr int CHL = CH < 32 ? CH : 32;        // lanes that split the chunks
    static constexpr int LG = 32 / CHL;                  // lane groups that split the warp's rows
    static constexpr int CPL = CH / CHL;                 // chunks per lane
    static constexpr int RW = RP / 8;                    // rows per warp
    static constexpr int RPL = RW / LG;                  // rows per lane
    static_assert(RPL >= 1 && RPL <= kMaxRowsPerLane, "row split");
    uint32_t a_off[CPL][RPL];   // byte offset of (row, chunk) inside the tile, swizzle applied
    uint32_t x_off[CPL];        // byte offset of the chunk inside a token's x piece
    int col0;                   // first column (inside the tile) of this lane's first chunk
    int row0;                   // first rank row of this lane
    __device__ __forceinline__ void init(int warp, int lane) {
        const int cl = lane % CHL, rg = lane / CHL;
        row0 = warp * RW + rg * RPL;
#pragma unroll
        for (int q = 0; q < CPL; ++q) {
            const int c = cl + q * CHL;
            x_off[q] = c * 16;
#pragma unroll
            for (int rr = 0; rr < RPL; ++rr) {
                const int k = row0 + rr;
                a_off[q][rr] = (c >> 3) * (RP * 128) + k * 128 + (((c & 7) ^ (k & 7)) << 4);
            }
        }
        col0 = cl * 8;
    }
};

// CNT (tokens of the unit) is a template parameter: the loops unroll without branches, every
// load of the tile is issued before the first use, and each (row, token, chunk) product
// runs as two short chains (even / odd columns) instead of one long one.
template <int RP, int CNT, bool CHECKED, bool H>
__device__ __forceinline__ void shrink_chunks(const ShrinkMap<RP>& mp, int cols_left, uint32_t tile,
                                              float (&acc)[kMaxRowsPerLane][kTokChunk]) {
    using M = ShrinkMap<RP>;
    const uint32_t xs = tile + kTileBytesMax;
    uint4 araw[M::CPL][M::RPL], xraw[M::CPL][CNT];
#pragma unroll
    for (int q = 0; q < M::CPL; ++q) {
#pragma unroll
        for (int rr = 0; rr < M::RPL; ++rr) araw[q][rr] = lds128(tile + mp.a_off[q][rr]);
#pragma unroll
        for (int t = 0; t < CNT; ++t) xraw[q][t] = lds128(xs + t * kXBytesPerTok + mp.x_off[q]);
    }
#pragma unroll
    for (int q = 0; q < M::CPL; ++q) {
        if (!CHECKED || mp.col0 + q * M::CHL * 8 < cols_left) {
            // The two values of a 32-bit word (even / odd column) stay together as a pair and every
            // multiply-add is the packed one (two fp32 FMAs per instruction on sm_100): the even and the
            // odd chain of a product advance in one issue slot.
            float2 xp[CNT][4];
#pragma unroll
            for (int t = 0; t < CNT; ++t) unpack4x2<H>(xraw[q][t], xp[t]);
#pragma unroll
            for (int rr = 0; rr < M::RPL; ++rr) {
                float2 ap[4];
                unpack4x2<H>(araw[q][rr], ap);
#pragma unroll
                for (int t = 0; t < CNT; ++t) {
                    float2 eo = __fmul2_rn(xp[t][0], ap[0]);
                    eo = __ffma2_rn(xp[t][1], ap[1], eo);
                    eo = __ffma2_rn(xp[t][2], ap[2], eo);
                    eo = __ffma2_rn(xp[t][3], ap[3], eo);
                    acc[rr][t] += eo.x + eo.y;
                }
            }
        }
    }
}

template <int RP, int CNT, bool H>
__device__ __forceinline__ void shrink_tile_cnt(const Params& p, const StageHdr& h, const ShrinkMap<RP>& mp,
                                                uint32_t tile, float (&acc)[kMaxRowsPerLane][kTokChunk]) {
    const int cols_left = p.pool.d_in - h.tile * ShrinkMap<RP>::C;   // only the last tile can be ragged
    if (cols_left >= ShrinkMap<RP>::C)
        shrink_chunks<RP, CNT, false, H>(mp, cols_left, tile, acc);
    else
        shrink_chunks<RP, CNT, true, H>(mp, cols_left, tile, acc);
}

template <int RP, bool H>
__device__ __forceinline__ void shrink_tile(const Params& p, const StageHdr& h, const ShrinkMap<RP>& mp, uint32_t tile,
                                            float (&acc)[kMaxRowsPerLane][kTokChunk]) {
    switch (h.cnt) {
        case 1: shrink_tile_cnt<RP, 1, H>(p, h, mp, tile, acc); break;
        case 2: shrink_tile_cnt<RP, 2, H>(p, h, mp, tile, acc); break;
        case 3: shrink_tile_cnt<RP, 3, H>(p, h, mp, tile, acc); break;
        default: shrink_tile_cnt<RP, 4, H>(p, h, mp, tile, acc); break;
    }
}

// ---- shrink: end of a task ---------------------------------------------------------------
// The lanes that split the chunks meet by shuffles; every (row, token) sum of the warp's rows
// is then complete and one lane per value sends it off: to the workspace as a {value, epoch}
// word (fused) or to the caller's m (shrink-only).  No warp waits for another.
//
// CNT is the token count rounded up to a power of two (tokens beyond the unit's count hold
// zeros and are not written).  The butterfly runs over the CHL lanes that split the chunks;
// while a lane holds more than one value each step also halves them (partners swap halves),
// so a step costs one shuffle per surviving value instead of one per value.
template <int MODE, int RP, int CNT>
__device__ __forceinline__ void shrink_finish_cnt(const Params& p, const Smem& sm, const StageHdr& h,
                                                  const ShrinkMap<RP>& mp, float (&acc)[kMaxRowsPerLane][kTokChunk],
                                                  int lane) {
    using M = ShrinkMap<RP>;
    constexpr int V = M::RPL * CNT;   // values per lane; value v = (row v / CNT, token v % CNT)
    constexpr int kLog2V = V >= 16 ? 4 : V >= 8 ? 3 : V >= 4 ? 2 : V >= 2 ? 1 : 0;
    constexpr int kLog2L = M::CHL >= 32 ? 5 : M::CHL >= 16 ? 4 : 3;
    constexpr int kHalvings = kLog2V < kLog2L ? kLog2V : kLog2L;
    constexpr int kLeft = V >> kHalvings;                 // values per lane at the end
    constexpr int kLanesPerValue = M::CHL >> kHalvings;   // lanes that end up with the same values
    float val[V];
#pragma unroll
    for (int v = 0; v < V; ++v) val[v] = acc[v / CNT][v % CNT];
    const int cl = lane % M::CHL;
    int idx = 0;   // first value this lane holds
#pragma unroll
    for (int s = 0; s < kLog2L; ++s) {
        const int d = M::CHL >> (s + 1);
        if (s < kHalvings) {
            const int n = V >> s;                 // values held before this step
            const bool upper = (cl & d) != 0;     // lower lanes keep the first half, upper lanes the second
#pragma unroll
            for (int v = 0; v < V / 2; ++v) {
                if (v < n / 2) {
                    const float keep = upper ? val[v + n / 2] : val[v];
                    const float give = upper ? val[v] : val[v + n / 2];
                    val[v] = keep + __shfl_xor_sync(0xffffffffu, give, d);
                }
            }
            if (upper) idx += n / 2;
        } else {
#pragma unroll
            for (int v = 0; v < kLeft; ++v) val[v] += __shfl_xor_sync(0xffffffffu, val[v], d);
        }
    }
    // the lane holds the values idx .. idx + kLeft - 1, complete; one lane of each group of equals writes
    if ((cl & (kLanesPerValue - 1)) == 0) {
#pragma unroll
        for (int j = 0; j < kLeft; ++j) {
            const int rr = (idx + j) / CNT, t = (idx + j) % CNT;
            if (t < h.cnt) {
                const int k = h.k0 + mp.row0 + rr;
                if (MODE == kFused) {
                    // value and epoch leave in one 64-bit store: no fence, nobody waits for it here
                    PLORA_CHECKED((part_index(p, h.unit, h.run, t) + k + 1) * 8 <= p.bk.m_part_bytes, p.status)
                    p.bk.m_part[part_index(p, h.unit, h.run, t) + k] =
                        ((unsigned long long)sm.epoch << 32) | (unsigned long long)__float_as_uint(val[j]);
                } else {
                    store_m(p, (size_t)tok_at(h, t) * p.ldm + k, val[j]);
                }
            }
        }
    }
}

template <int MODE, int RP>
__device__ __forceinline__ void shrink_finish(const Params& p, const Smem& sm, const StageHdr& h,
                                              const ShrinkMap<RP>& mp, float (&acc)[kMaxRowsPerLane][kTokChunk],
                                              int warp, int lane) {
    switch (h.cnt) {
        case 1: shrink_finish_cnt<MODE, RP, 1>(p, sm, h, mp, acc, lane); break;
        case 2: shrink_finish_cnt<MODE, RP, 2>(p, sm, h, mp, acc, lane); break;
        default: shrink_finish_cnt<MODE, RP, 4>(p, sm, h, mp, acc, lane); break;
    }
    if (MODE != kFused) {
        // columns beyond this adapter's padded rank are zeros
        const int extra = p.ldm - RP;
        for (int idx = warp * 32 + lane; idx < h.cnt * extra; idx += kConsumerThreads) {
            const int t = idx / extra, k = RP + idx % extra;
            store_m(p, (size_t)tok_at(h, t) * p.ldm + k, 0.f);
        }
    }
}

// ---- shrink on the tensor cores: units of several tokens (padded rank >= 16) ----------------------------
// A unit of 2..4 tokens costs the CUDA-core loop 2..2.6 times the instructions of a one-token unit.  Here
// m^T[16 rank rows x 8] += A^T[16 x 16 columns] x^T[16 x 8] by mma.sync.m16n8k16: warp w takes the rank
// rows [16 w, 16 w + 16) of every sub-tile of the stage (warps beyond RP / 16 have nothing to do and only
// release the stage), A fragments by ldmatrix from the swizzled sub-tile (conflict-free), x fragments as
// one word per lane from the unit's x pieces (tokens beyond the unit's count read some other token's
// piece: their columns of the result are never stored).  The accumulator fragment holds complete sums of
// the warp's rows for the task's columns, so the end of a task is one store per value: no shuffles.
__device__ __forceinline__ void ldmatrix_x4(uint32_t a, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
template <bool H>
__device__ __forceinline__ void mma_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    if (H)
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
    else
        asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
template <int RP, bool H>
__device__ __forceinline__ void shrink_tile_mma(const Params& p, const StageHdr& h, uint32_t tile, float (&d)[4], int warp, int lane) {
    constexpr int NSUB = (kMaxRank / RP > kMaxSubPerTile) ? kMaxSubPerTile : kMaxRank / RP;
    if (warp >= RP / 16) return;
    const int g = lane >> 2, q = lane & 3;
    const int cols_left = p.pool.d_in - h.tile * (NSUB * kSubCols);   // only the last tile can be ragged
    const int arow = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;  // the lane's row of the 8 x 8 blocks it addresses
    const uint32_t xrow = tile + kTileBytesMax + (g & (kTokChunk - 1)) * kXBytesPerTok;
#pragma unroll
    for (int sb = 0; sb < NSUB; ++sb) {
        if (sb * kSubCols >= cols_left) break;   // nothing was copied for these columns
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            uint32_t a[4];
            const int ch = 2 * ks + (lane >> 4);
            ldmatrix_x4(tile + sb * (RP * 128) + arow * 128 + ((ch ^ (arow & 7)) << 4), a);
            const int col = sb * kSubCols + ks * 16 + 2 * q;
            // columns beyond d_in: the slab holds zeros there, the x piece holds whatever was in the stage
            const uint32_t b0 = col < cols_left ? lds32(xrow + col * 2) : 0u;
            const uint32_t b1 = col + 8 < cols_left ? lds32(xrow + col * 2 + 16) : 0u;
            mma_16816<H>(d, a, b0, b1);
        }
    }
}
template <int MODE, int RP>
__device__ __forceinline__ void shrink_finish_mma(const Params& p, const Smem& sm, const StageHdr& h, const float (&d)[4],
                                                  int warp, int lane) {
    if (warp < RP / 16) {
        const int g = lane >> 2, q = lane & 3;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int t = 2 * q + (j & 1), k = h.k0 + warp * 16 + g + (j >> 1) * 8;
            if (t < h.cnt) {
                if (MODE == kFused) {
                    PLORA_CHECKED((part_index(p, h.unit, h.run, t) + k + 1) * 8 <= p.bk.m_part_bytes, p.status)
                    p.bk.m_part[part_index(p, h.unit, h.run, t) + k] =
                        ((unsigned long long)sm.epoch << 32) | (unsigned long long)__float_as_uint(d[j]);
                } else
                    store_m(p, (size_t)tok_at(h, t) * p.ldm + k, d[j]);
            }
        }
    }
    if (MODE != kFused) {
        // columns beyond this adapter's padded rank are zeros
        const int extra = p.ldm - RP;
        for (int idx = warp * 32 + lane; idx < h.cnt * extra; idx += kConsumerThreads) {
            const int t = idx / extra, k = RP + idx % extra;
            store_m(p, (size_t)tok_at(h, t) * p.ldm + k, 0.f);
        }
    }
}

// ---- expand: one tile of B; the result goes straight to y ------------------------------------------
// Lane mapping: a lane owns two adjacent output columns; when the warp's slice has fewer
// than 32 column pairs, RG lane groups split the rank rows and meet by shuffles.
//
// Which rows a group takes decides the bank conflicts of the B loads.  All rows of a sub-tile
// start at the same bank (a row is 128 bytes) and only the swizzle, by the row's number mod 8,
// moves a column's chunk.  Groups that took blocks of consecutive rows would read rows of the same
// swizzle class at the same time, the same 16 bytes' banks RG times over (8-way at rank 128).
// Group g therefore takes the rows g, g + RG, g + 2 RG, ...: at every step the RG groups read RG
// different classes, that is RG different chunks of the 128-byte bank window.  In the fused kernel
// the gather warp stores m so that a group's rows are consecutive (m_slot_of); the expand-only
// kernel gets m from the caller in natural order and reads it value by value.
template <int RP>
struct ExpandMap {
    static constexpr int NSUB = (kMaxRank / RP > kMaxSubPerTile) ? kMaxSubPerTile : kMaxRank / RP;
    static constexpr int C = NSUB * kSubCols;
    static constexpr int P = 4 * NSUB;      // column pairs per warp per tile
    static constexpr int RG = 32 / P;       // lane groups that split the rank rows
    static constexpr int RPG = RP / RG;     // rows per group (8 or 16)
    static_assert(RG == (RP >= 32 ? RP / 16 : 1), "the gather warp computes the row groups from the rank");
    uint32_t b_col;    // byte offset inside the tile of (row 0, this lane's pair), swizzle class 0
    int colw;          // this lane's first column inside the tile
    int rg;
    __device__ __forceinline__ void init(int warp, int lane) {
        const int pair = lane % P;
        rg = lane / P;
        colw = warp * (NSUB * 8) + 2 * pair;
        // the chunk index sits in address bits 4..6 and everything else leaves them clear, so
        // the swizzle of row class j is one XOR with (j << 4)
        b_col = (colw >> 6) * (RP * 128) + (((colw & 63) >> 3) << 4) + (colw & 7) * 2;
    }
    // where the gather warp puts m[k] of a token (fused kernel): group-major
    __device__ static __forceinline__ int m_slot_of(int k) { return (k % RG) * RPG + k / RG; }
};

template <int MODE, int RP, int CNT, bool H>
__device__ __forceinline__ bool expand_tile_cnt(const Params& p, const Smem& sm, const StageHdr& h,
                                                const ExpandMap<RP>& mp, uint32_t tile, uint32_t empty_bar, int lane) {
    using M = ExpandMap<RP>;
    // Interleaved: group g takes the rows g + RG * j, and the address of this lane's pair in row j is
    // base ^ (class(j) << 4) + row(j) * 128.  The expand-only kernel with RG <= 2 keeps blocks of rows
    // (g * RPG + j): it would pay more for fetching its m value by value than the two-way conflict costs.
    constexpr bool kInterleaved = MODE == kFused || M::RG >= 4;
    const uint32_t b0 = kInterleaved ? ((tile + mp.b_col) ^ ((uint32_t)mp.rg << 4)) + mp.rg * 128
                                     : tile + mp.b_col + mp.rg * M::RPG * 128;
    const int m_slot = h.m_seq % kMRing;
    if (MODE == kFused && (h.flags & kFlagFirst))   // the gather warp has assembled this task's m
        if (!mbar_wait(sm.m_full + m_slot * 8, (h.m_seq / kMRing) & 1, sm.wait)) return false;   // gave up: nothing of this tile reaches y
    // fused: m in the m ring, group-major, so the group's rows are RPG consecutive floats per token;
    // expand-only: the caller's m next to the tile, in natural order
    const uint32_t mb = MODE == kFused ? sm.m_ring + m_slot * kMRingBytes + mp.rg * M::RPG * 4 : tile + kTileBytesMax;
    // accumulators: per token and column a pair (sum over the even rows, sum over the odd rows), so
    // that two rows advance per packed multiply-add
    float2 acc[CNT][2];
#pragma unroll
    for (int t = 0; t < CNT; ++t) acc[t][0] = acc[t][1] = make_float2(0.f, 0.f);
#pragma unroll
    for (int kk = 0; kk < M::RPG; kk += 4) {
        uint32_t mv[CNT][4];
        uint32_t braw[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int j = kk + q;
            braw[q] = kInterleaved ? lds32((b0 ^ (((j * M::RG) & 7) << 4)) + j * (M::RG * 128))
                                   : lds32((b0 ^ ((j & 7) << 4)) + j * 128);
        }
#pragma unroll
        for (int t = 0; t < CNT; ++t) {
            if (MODE == kFused) {
                const uint4 v = lds128(mb + t * (RP * 4) + kk * 4);
                mv[t][0] = v.x; mv[t][1] = v.y; mv[t][2] = v.z; mv[t][3] = v.w;
            } else if (!kInterleaved && !p.m16) {
                const int row = mp.rg * M::RPG + kk;   // four consecutive fp32 values
                const uint4 v = lds128(mb + t * (RP * 4) + row * 4);
                mv[t][0] = row + 0 < h.r ? v.x : 0u;
                mv[t][1] = row + 1 < h.r ? v.y : 0u;
                mv[t][2] = row + 2 < h.r ? v.z : 0u;
                mv[t][3] = row + 3 < h.r ? v.w : 0u;
            } else {
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int row = kInterleaved ? mp.rg + (kk + q) * M::RG : mp.rg * M::RPG + kk + q;
                    uint32_t v;
                    if (p.m16) {   // 2-byte m: a bf16 value, widened (exactly) to fp32
                        const uint32_t w = lds32(mb + t * (RP * 2) + (row & ~1) * 2);
                        v = (row & 1) ? (w & 0xffff0000u) : (w << 16);
                    } else {
                        v = lds32(mb + t * (RP * 4) + row * 4);
                    }
                    mv[t][q] = row < h.r ? v : 0u;   // the caller's m may hold anything beyond the adapter's rank
                }
            }
        }
#pragma unroll
        for (int q = 0; q < 4; q += 2) {
            // rows q and q + 1 of this step: (row q, row q + 1) pairs of the first and of the second column
            const float2 b0 = make_float2(in_lo<H>(braw[q]), in_lo<H>(braw[q + 1]));
            const float2 b1 = make_float2(in_hi<H>(braw[q]), in_hi<H>(braw[q + 1]));
#pragma unroll
            for (int t = 0; t < CNT; ++t) {
                const float2 mk = make_float2(__uint_as_float(mv[t][q]), __uint_as_float(mv[t][q + 1]));
                acc[t][0] = __ffma2_rn(mk, b0, acc[t][0]);
                acc[t][1] = __ffma2_rn(mk, b1, acc[t][1]);
            }
        }
    }
    __syncwarp();
    release_stage(sm, empty_bar, lane);
    if (lane == 0 && MODE == kFused && (h.flags & kFlagLast)) mbar_arrive(sm.m_empty + m_slot * 8);
    float out[CNT][2];
#pragma unroll
    for (int t = 0; t < CNT; ++t) {
        out[t][0] = acc[t][0].x + acc[t][0].y;
        out[t][1] = acc[t][1].x + acc[t][1].y;
    }
#pragma unroll
    for (int d = M::P; d < 32; d <<= 1)
#pragma unroll
        for (int t = 0; t < CNT; ++t) {
            out[t][0] += __shfl_xor_sync(0xffffffffu, out[t][0], d);
            out[t][1] += __shfl_xor_sync(0xffffffffu, out[t][1], d);
        }
    const int col = h.tile * M::C + mp.colw;
    if (mp.rg == 0 && col < p.pool.d_out) {
#pragma unroll
        for (int t = 0; t < CNT; ++t) {
            PLORA_CHECKED((unsigned)h.tok[t] < (unsigned)p.n_tok && col + 1 < p.pool.d_out, p.status)
            red_add_v2(p.y_g[h.group] + (size_t)h.tok[t] * p.pool.d_out + col, out[t][0] * h.scale, out[t][1] * h.scale);
        }
    }
    return true;
}

template <int MODE, int RP, bool H>
__device__ __forceinline__ bool expand_tile(const Params& p, const Smem& sm, const StageHdr& h, const ExpandMap<RP>& mp,
                                            uint32_t tile, uint32_t empty_bar, int lane) {
    switch (h.cnt) {
        case 1: return expand_tile_cnt<MODE, RP, 1, H>(p, sm, h, mp, tile, empty_bar, lane);
        case 2: return expand_tile_cnt<MODE, RP, 2, H>(p, sm, h, mp, tile, empty_bar, lane);
        case 3: return expand_tile_cnt<MODE, RP, 3, H>(p, sm, h, mp, tile, empty_bar, lane);
        default: return expand_tile_cnt<MODE, RP, 4, H>(p, sm, h, mp, tile, empty_bar, lane);
    }
}

// Row slices.  A unit of padded rank 64 or 128 has few, large tiles (16 KiB for 64 columns at rank
// 128): cut into at most kMaxRunsA column runs, its shrink keeps only a few CTAs busy when the
// launch has few units (a rank class of a mixed pool, a small batch).  A fused launch that finds
// fewer shrink tasks than CTAs therefore also cuts along the rank: a task takes kSliceRows rank
// rows of a column run.  The rows [k0, k0 + 32) of a sub-tile are contiguous (32 rows of 128 bytes)
// and keep their swizzle (k0 is a multiple of 8), so four of them, from four consecutive sub-tiles,
// put side by side in a stage are exactly a tile of a rank-32 adapter over 256 columns: the
// consumers run the rank-32 code on it and add k0 to the row number when they hand the sums over.
// The partial words of the slices of one column run fill disjoint rows of the same run, so the
// workspace and the gather are as without slices; x pieces are fetched once per slice (from L2
// after the first).  With many units the slices only add copies and hand-overs (measured: 0.86 of
// the roofline instead of 0.98 on the 13B decode shapes at rank 64), hence the choice per launch.
constexpr int kSliceRows = 32;
template <int MODE, int RPK>
struct SliceCfg {
    static constexpr bool kCan = MODE == kFused && RPK > kSliceRows;
    static constexpr int kSlices = kCan ? RPK / kSliceRows : 1;   // when the launch slices
    static constexpr int kSliceRp = kCan ? kSliceRows : RPK;      // geometry of a slice stage
};
// How a launch cuts the shrink of its units.  Every CTA computes the same plan from the same counts.
struct ShrinkPlan {
    int runs;     // column runs per unit
    int slices;   // row slices per column run
};
template <int MODE, int RPK>
__device__ __forceinline__ ShrinkPlan shrink_plan(const Params& p, int n_vunits) {
    ShrinkPlan pl;
    pl.runs = p.runs_a;
    pl.slices = 1;
    if (SliceCfg<MODE, RPK>::kCan && n_vunits * p.runs_a < (int)gridDim.x) {
        pl.runs = p.runs_a_sliced;
        pl.slices = SliceCfg<MODE, RPK>::kSlices;
    }
    return pl;
}

// Per-lane constants of both phases: shrink stages have the geometry of padded rank RP or, for
// slice stages, RPS; expand stages that of RP.
template <int RP, int RPS>
struct LaneMaps {
    ShrinkMap<RP> s;
    ShrinkMap<RPS> s2;
    ExpandMap<RP> e;
    __device__ __forceinline__ void init(int warp, int lane) {
        s.init(warp, lane);
        if (RPS != RP) s2.init(warp, lane);
        e.init(warp, lane);
    }
};

// One stage, consumer side.
// (false: this lane gave up inside the stage)
template <int MODE, int RP, bool H, bool TC, bool LAZY>
__device__ __forceinline__ bool consume_stage(const Params& p, const Smem& sm, const StageHdr& h,
                                              const LaneMaps<RP, SliceCfg<MODE, RP>::kSliceRp>& maps, uint32_t tile, uint32_t empty_bar,
                                              float (&acc)[kMaxRowsPerLane][kTokChunk], int warp, int lane) {
    if (!(h.flags & kFlagExpand)) {
        if (MODE != kExpandOnly) {
            if (h.flags & kFlagFirst) {
#pragma unroll
                for (int rr = 0; rr < kMaxRowsPerLane; ++rr)
#pragma unroll
                    for (int t = 0; t < kTokChunk; ++t) acc[rr][t] = 0.f;
            }
            constexpr int RPS = SliceCfg<MODE, RP>::kSliceRp;
            // several tokens: the tensor-core loop (its accumulator fragment lives in acc[0]) where it has at least
            // four warps to run on (padded rank 64 and 128); with two warps (rank 32, row slices) or one (rank 16)
            // it loses against the CUDA-core loop on all eight (measured)
            const bool tc4 = TC && h.cnt >= 2;   // (not in the launch for all classes, which cuts these ranks into slices)
            if (RPS != RP && (h.flags & kFlagSlice)) {
                const bool tc = RPS >= 64 && tc4;
                if (tc) shrink_tile_mma<RPS < 16 ? 16 : RPS, H>(p, h, tile, acc[0], warp, lane);
                else shrink_tile<RPS, H>(p, h, maps.s2, tile, acc);
                __syncwarp();
                release_stage(sm, empty_bar, lane);
                if (h.flags & kFlagLast) {
                    if (LAZY) join_stream(p, sm);
                    if (tc) shrink_finish_mma<MODE, RPS < 16 ? 16 : RPS>(p, sm, h, acc[0], warp, lane);
                    else shrink_finish<MODE, RPS>(p, sm, h, maps.s2, acc, warp, lane);
                }
            } else if (RP >= 64 && tc4) {
                shrink_tile_mma<RP < 16 ? 16 : RP, H>(p, h, tile, acc[0], warp, lane);
                __syncwarp();
                release_stage(sm, empty_bar, lane);
                if (h.flags & kFlagLast) {
                    if (LAZY) join_stream(p, sm);
                    shrink_finish_mma<MODE, RP < 16 ? 16 : RP>(p, sm, h, acc[0], warp, lane);
                }
            } else {
                shrink_tile<RP, H>(p, h, maps.s, tile, acc);
                __syncwarp();
                release_stage(sm, empty_bar, lane);
                if (h.flags & kFlagLast) {
                    if (LAZY) join_stream(p, sm);
                    shrink_finish<MODE, RP>(p, sm, h, maps.s, acc, warp, lane);
                }
            }
        }
    } else {
        // (a lazy launch needs no join here: the m this tile waits for is published by the gather warp, which
        // joined the stream order before it read the first partial word, and the expand does not use the epoch)
        if (MODE != kShrinkOnly) return expand_tile<MODE, RP, H>(p, sm, h, maps.e, tile, empty_bar, lane);
    }
    return true;
}

// Consumes stages from stage `it` on for as long as they belong to padded rank RP (a one-class
// launch: to the end).  Returns true when stage `it` is another class's (it has not been touched),
// false when nothing follows or this lane gave up (gave_up: it must leave the kernel now).
template <int MODE, int RP, bool H, bool ONLY, bool LAZY>
__device__ __forceinline__ bool consume_class(const Params& p, const Smem& sm, uint32_t& it, bool& gave_up,
                                              float (&acc)[kMaxRowsPerLane][kTokChunk], int warp, int lane) {
    LaneMaps<RP, SliceCfg<MODE, RP>::kSliceRp> maps;   // per-lane constants of both phases
    maps.init(warp, lane);
    for (;; ++it) {
        const uint32_t slot = it % kStages;
        if (!mbar_wait(sm.full + slot * 8, (it / kStages) & 1, sm.wait)) {
            gave_up = true;
            return false;
        }
        const uint32_t tile = sm.slots + slot * kSlotBytes;
        const StageHdr h = read_hdr(tile + kHdrOffset);
        if (h.flags & kFlagEnd) return false;
        if (!ONLY && h.rp != RP) return true;
        if (!consume_stage<MODE, RP, H, ONLY, LAZY>(p, sm, h, maps, tile, sm.empty + slot * 8, acc, warp, lane)) {
            gave_up = true;
            return false;
        }
    }
}

// ---- producer side: the m of an expand task ---------------------------------------------------
// A unit's m has cnt * rp values; lane l of the producer warp owns the values l, l + 32, ...
// For every owned value the runs_a partial words are read, checked for this launch's epoch,
// summed in run order and the sum stored into the m-ring entry.  Nothing here waits: the
// return value tells whether every word had arrived (if not, the next attempt rewrites the
// entry).  rp is a power of two.
__device__ __forceinline__ const unsigned long long* partial_src(const Params& p, int unit, int idx, int rp) {
    const int sh = __ffs(rp) - 1;
    const int t = idx >> sh, k = idx & (rp - 1);
    return p.bk.m_part + part_index(p, unit, 0, t) + k;
}
__device__ __forceinline__ void partial_load(const Params& p, int runs_a, uint32_t epoch, const unsigned long long* src,
                                             unsigned long long (&w)[kMaxRunsA]) {
    const size_t run_stride = (size_t)p.pool.max_rp;
#pragma unroll
    for (int j = 0; j < kMaxRunsA; ++j)
    {
        w[j] = (unsigned long long)epoch << 32;
        if (j < runs_a) {
            PLORA_CHECKED((size_t)(src + j * run_stride + 1 - p.bk.m_part) * 8 <= p.bk.m_part_bytes, p.status)
            w[j] = ldg_cg_u64(src + j * run_stride);
        }
    }
}
__device__ __forceinline__ bool partial_sum(uint32_t epoch, const unsigned long long (&w)[kMaxRunsA], uint32_t dst) {
    bool ok = true;
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < kMaxRunsA; ++j) {
        ok = ok && (uint32_t)(w[j] >> 32) == epoch;
        s += __uint_as_float((uint32_t)w[j]);
    }
    asm volatile("st.shared.f32 [%0], %1;" ::"r"(dst), "f"(s) : "memory");
    return ok;
}
// The words of up to kGatherDepth values per lane are requested before the first of them is
// used: a unit's m costs one round trip to L2 per 32 * kGatherDepth values, not one per 32.
constexpr int kGatherDepth = 2;
// rp is a power of two (a compile-time constant in a one-class launch).
__device__ __forceinline__ bool gather_m(const Params& p, int rp, int runs_a, uint32_t epoch, int unit, int cnt, int lane,
                                         uint32_t mdst) {
    bool ok = true;
    const int n = cnt * rp;
    // the expand lanes' row groups (ExpandMap): rg groups of rpg rows; value k goes to (k % rg) * rpg + k / rg
    const int rg = rp >= 32 ? rp / 16 : 1, rpg = rp / rg;
    for (int i0 = lane; i0 < n; i0 += 32 * kGatherDepth) {
        unsigned long long w[kGatherDepth][kMaxRunsA];
#pragma unroll
        for (int q = 0; q < kGatherDepth; ++q)
            if (i0 + q * 32 < n) partial_load(p, runs_a, epoch, partial_src(p, unit, i0 + q * 32, rp), w[q]);
#pragma unroll
        for (int q = 0; q < kGatherDepth; ++q) {
            const int i = i0 + q * 32;
            const int k = i & (rp - 1);
            // value k of token t goes where the expand lanes of its row group look for it
            if (i < n) ok = partial_sum(epoch, w[q], mdst + ((i - k) + (k & (rg - 1)) * rpg + k / rg) * 4) && ok;
        }
    }
    return ok;
}

// ---- the task list of a launch -------------------------------------------------------------------
// A task is one run of tiles of one unit in one phase.  A launch serves one rank class (RPK != 0:
// a pool of one rank, or the unfused halves of a mixed pool, one launch per class) or, fused, all
// classes of a mixed pool at once (RPK == 0).  Either way the list is: the shrink tasks of every
// class, largest rank first, then the expand tasks in the same order; CTAs take tasks round-robin.
//
// Mixed launch: tasks of very different sizes under a static round-robin leave the CTAs that drew
// the large ones far behind (measured 2x slower than one launch per class), so the classes are cut to
// tasks of about the same size, chosen so that a CTA gets a few tasks per phase (TaskPlanCfg): between
// kTaskBytesMin and kTaskBytesMax of adapter bytes.  A unit of padded rank 128 then makes up to 16
// shrink tasks (4 column runs x 4 row slices) and 16 expand tasks, one of rank 8 at least one and one.
// (Between 32 and 256 KiB: with tasks of 16 to 32 KiB, one or two stages each, the hand-over of a partial m per task
// and the gather before every expand task weighed more than the finer balance gained; the paper's skewed decode mix
// on 8 layers took 0.906 ms per step with those, 0.857 ms with these, and no more with a ceiling of 512 KiB or 1 MiB.
// Two tasks per CTA and phase: since consecutive launches overlap (a launch's CTAs start on their inputs under the
// previous launch's tail), an uneven end costs less than the hand-overs of finer tasks; the same mix with four, three,
// two, one task per CTA: 0.820, 0.817, 0.795, 0.869 ms, and two with a ceiling of 512 KiB loses 7 % on uniform ids.)
// The expand phase does with one task per CTA (an expand task has no hand-over at its end, but a gather at its start):
// 0.779 -> 0.768 ms on the same mix, better on six of seven other small mixed-rank batches.
// These coarse tasks are for the kernels that join the stream order late, whose launches overlap; a launch that waits
// at its start for the one before it keeps four tasks per CTA and phase and slices from twice the target size on
// (without the hint the same mix takes 0.854 ms per step with those, about 0.905 ms with the coarse plan).
constexpr int kTaskBytesMin = 32 * 1024, kTaskBytesMax = 256 * 1024;
template <bool LAZY>
struct TaskPlanCfg {
    static constexpr int kShrinkTasksPerCta = LAZY ? 2 : 4;
    static constexpr int kExpandTasksPerCta = LAZY ? 1 : 4;
    static constexpr int kSliceFactor = LAZY ? 4 : 2;   // row slices when a column run exceeds this many targets
};
// The one launch pays off for small batches, where the per-class launches are mostly fixed cost
// (256 tokens, ranks 8..128, q/k/v grouped: 1.10 -> 1.00 ms for 8 layers); with many units per
// class the per-class launches, each with loops compiled for its rank, are faster (2048 tokens,
// ranks 8..64: 0.34 ms against 0.39 ms, whatever the task size), so the host picks by batch size.
constexpr int kMixedLaunchMaxRows = 1024;   // tokens x projections of the call
struct Task {
    int slot;    // class slot of the plan
    int unit;    // index into the slot's list of (group, unit) pairs
    int phase;   // 0 = shrink, 1 = expand
    int run;
    int slice;   // shrink: which row slice of the column run (0 when the unit is not sliced)
};

template <int NC>
struct Plan {
    int rp[NC];                  // padded rank of the slot's class
    const int32_t* list[NC];     // the slot's units, sorted out by the classify pass; nullptr: all units, in order
    int per_group[NC];           // how many units the slot has (in each projection of the group)
    int n[NC];                   // (projection, unit) pairs of the slot: per_group * n_groups, projection-major
    int n_units;                 // units of the bucket
    int s_runs[NC], s_slices[NC], e_runs[NC];
    int s_start[NC + 1], e_start[NC + 1];   // first task of the slot in each phase (expand counted from n_shrink)
    int n_shrink, n_tasks;
    // pair i of a slot as group * n_units + unit
    __device__ __forceinline__ int unit_at(int slot, int i) const {
        if (!list[slot]) return i;
        const int g = i / max(per_group[slot], 1);
        return g * n_units + list[slot][i - g * per_group[slot]];
    }
    __device__ __forceinline__ Task decode(int t) const {
        Task k;
        k.phase = t >= n_shrink ? 1 : 0;
        if (k.phase) t -= n_shrink;
        k.slot = 0;
        int first = 0;
#pragma unroll
        for (int i = 1; i < NC; ++i) {
            const int st = k.phase ? e_start[i] : s_start[i];
            if (t >= st) {
                k.slot = i;
                first = st;
            }
        }
        t -= first;
        if (k.phase) {
            const int runs = e_runs[k.slot];
            k.unit = t / runs;
            k.run = t - k.unit * runs;
            k.slice = 0;
        } else {
            // run-major, the slices of one column run next to one another (their x pieces are the same bytes)
            const int runs = s_runs[k.slot], slices = s_slices[k.slot];
            k.unit = t / (runs * slices);
            const int rem = t - k.unit * (runs * slices);
            k.run = rem / slices;
            k.slice = rem - k.run * slices;
        }
        return k;
    }
};

__device__ __forceinline__ int clamp_int(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }

// Expand tasks per unit of a one-class launch.  The host proposes a number from the shapes alone; a
// launch that turns out to have few units (the CTAs see the count, the host does not) cuts its units
// finer, down to two tiles per task, until there are about two tasks per CTA.  Every CTA computes
// the same number.
template <int MODE, int RPK>
__device__ __forceinline__ int expand_runs(const Params& p, int n_vunits) {
    int runs = p.runs_b;
    if (MODE == kFused) {
        const int cap = max(runs, tiles_for(p.pool.d_out, RPK) / 2);
        const int want = (2 * (int)gridDim.x + n_vunits - 1) / max(n_vunits, 1);
        runs = min(cap, max(runs, want));
    }
    return runs;
}

template <int MODE, int RPK, bool LAZY>
__device__ __forceinline__ Plan<RPK ? 1 : kRankClasses> make_plan(const Params& p, int n_units) {
    constexpr int NC = RPK ? 1 : kRankClasses;
    Plan<NC> pl;
    pl.n_units = n_units;
    if (RPK) {
        constexpr int kClass = RPK == 8 ? 0 : RPK == 16 ? 1 : RPK == 32 ? 2 : RPK == 64 ? 3 : 4;
        if (p.by_class) {
            const int lo = p.bk.cls_start[kClass], hi = p.bk.cls_start[kClass + 1];
            pl.list[0] = p.bk.cls_list + lo;
            pl.per_group[0] = hi - lo;
        } else {
            pl.list[0] = nullptr;
            pl.per_group[0] = n_units;
        }
        pl.n[0] = pl.per_group[0] * p.n_groups;
        pl.rp[0] = RPK;
        const ShrinkPlan sp = shrink_plan<MODE, RPK ? RPK : 8>(p, pl.n[0]);
        pl.s_runs[0] = sp.runs;
        pl.s_slices[0] = sp.slices;
        pl.e_runs[0] = expand_runs<MODE, RPK ? RPK : 8>(p, pl.n[0]);
    } else {
        long long tot_a = 0, tot_b = 0;   // bytes of A and of B the launch streams
#pragma unroll
        for (int i = 0; i < NC; ++i) {
            const int c = kRankClasses - 1 - i, rp = 8 << c;   // largest rank first
            const int lo = p.bk.cls_start[c], hi = p.bk.cls_start[c + 1];
            pl.list[i] = p.bk.cls_list + lo;
            pl.per_group[i] = hi - lo;
            pl.n[i] = (hi - lo) * p.n_groups;
            pl.rp[i] = rp;
            tot_a += (long long)pl.n[i] * p.pool.d_in * rp * 2;
            tot_b += (long long)pl.n[i] * p.pool.d_out * rp * 2;
        }
        // task size: a few shrink and expand tasks per CTA (TaskPlanCfg), within the bounds above
        using Cfg = TaskPlanCfg<LAZY>;
        const int tgt_a = clamp_int((int)(tot_a / (Cfg::kShrinkTasksPerCta * (long long)gridDim.x)), kTaskBytesMin, kTaskBytesMax);
        const int tgt_b = clamp_int((int)(tot_b / (Cfg::kExpandTasksPerCta * (long long)gridDim.x)), kTaskBytesMin, kTaskBytesMax);
#pragma unroll
        for (int i = 0; i < NC; ++i) {
            const int rp = pl.rp[i];
            const int half_a = p.pool.d_in * rp * 2, half_b = p.pool.d_out * rp * 2;   // bytes of a unit's A and B
            int s_runs = clamp_int((half_a + tgt_a / 2) / tgt_a, 1, min(kMaxRunsA, tiles_for(p.pool.d_in, rp)));
            int slices = 1;
            if (rp > kSliceRows && half_a / s_runs > Cfg::kSliceFactor * tgt_a) {
                // the column runs alone leave the tasks far too large (a handful of units in a small batch): cut
                // along the rank too.  (Only then: slice stages cost four copies each and run the rank-32 loops;
                // with the threshold at twice the target the skewed decode mix took 0.795 ms per step, at four
                // times, eight times or without slices 0.779.)
                slices = rp / kSliceRows;
                s_runs = clamp_int((half_a / slices + tgt_a / 2) / tgt_a, 1, min(kMaxRunsA, tiles_for(p.pool.d_in, kSliceRows)));
            }
            pl.s_slices[i] = slices;
            pl.s_runs[i] = s_runs;
            const int tiles_b = tiles_for(p.pool.d_out, rp);
            pl.e_runs[i] = clamp_int((half_b + tgt_b / 2) / tgt_b, 1, min(2 * kMaxRuns, max(1, tiles_b / 2)));
        }
    }
    int s = 0, e = 0;
#pragma unroll
    for (int i = 0; i < NC; ++i) {
        pl.s_start[i] = s;
        pl.e_start[i] = e;
        s += MODE == kExpandOnly ? 0 : pl.n[i] * pl.s_runs[i] * pl.s_slices[i];
        e += MODE == kShrinkOnly ? 0 : pl.n[i] * pl.e_runs[i];
    }
    pl.s_start[NC] = s;
    pl.e_start[NC] = e;
    pl.n_shrink = s;
    pl.n_tasks = s + e;
    return pl;
}

#ifndef PLORA_BGMV_LAZY_UNIT
// Classify pass (pools of mixed ranks): sorts the bucket's units by the padded rank of the unit's
// adapter, keeping their order inside a class, so that every class gets a dense list.  The ranks
// are those of the call's first pool; the pools of a group, and every later call that reuses the
// sort, have the same ranks (rank_sig).  One CTA.
constexpr int kClassifyThreads = 1024;
// For the launch that serves all classes at once the units of a class are also ordered by their number of
// tokens, fewest first (then as the bucket has them): stages of one kind follow one another in every CTA's
// task sequence.  Measured on the paper's skewed decode mix: 0.840 ms per step in bucket order, 0.828 with the
// units of most tokens first, 0.821 with the fewest first.  The launches per class lose by either order
// (2048 tokens, ranks 8..64: 0.266 -> 0.272 / 0.268 ms), so their lists stay in bucket order.
constexpr int kSubKeys = kTokChunk;
constexpr int kKeys = kRankClasses * kSubKeys;
__device__ __forceinline__ int key_of(const Params& p, int u) {
    const WorkUnit w = p.bk.bgmv_units[u];
    const int rp = p.table_g[0][w.adapter].rp;
    const int cnt = w.cnt < 1 ? 1 : (w.cnt > kTokChunk ? kTokChunk : w.cnt);
    return (__ffs(rp) - 4) * kSubKeys + (p.sort_by_cnt ? cnt - 1 : 0);   // class: 8 -> 0, 16 -> 1, ...
}
__global__ void __launch_bounds__(kClassifyThreads) classify_kernel(const Params p) {
    __shared__ int total[kKeys], base[kKeys];
    __shared__ int warp_cnt[kClassifyThreads / 32][kKeys];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    grid_dependency_wait();
    grid_launch_dependents();
    const int n_v = *p.bk.n_bgmv_units;
    if (tid < kKeys) total[tid] = 0;
    __syncthreads();
    for (int v0 = 0; v0 < n_v; v0 += kClassifyThreads) {
        const int v = v0 + tid;
        const int c = v < n_v ? key_of(p, v) : -1;
        for (int cc = 0; cc < kKeys; ++cc) {
            const unsigned mask = __ballot_sync(0xffffffffu, c == cc);
            if (lane == 0 && mask) atomicAdd(&total[cc], __popc(mask));
        }
    }
    __syncthreads();
    if (tid == 0) {
        int run = 0;
        for (int cc = 0; cc < kKeys; ++cc) {
            base[cc] = run;
            if (cc % kSubKeys == 0) p.bk.cls_start[cc / kSubKeys] = run;
            run += total[cc];
        }
        p.bk.cls_start[kRankClasses] = run;
    }
    __syncthreads();
    for (int v0 = 0; v0 < n_v; v0 += kClassifyThreads) {
        const int v = v0 + tid;
        const int c = v < n_v ? key_of(p, v) : -1;
        int rank = 0;
        for (int cc = 0; cc < kKeys; ++cc) {
            const unsigned mask = __ballot_sync(0xffffffffu, c == cc);
            if (lane == 0) warp_cnt[warp][cc] = __popc(mask);
            if (c == cc) rank = __popc(mask & ((1u << lane) - 1u));
        }
        __syncthreads();
        if (c >= 0) {
            int before = 0;
            for (int w = 0; w < warp; ++w) before += warp_cnt[w][c];
            p.bk.cls_list[base[c] + before + rank] = v;
        }
        __syncthreads();
        if (tid < kKeys) {
            int add = 0;
            for (int w = 0; w < kClassifyThreads / 32; ++w) add += warp_cnt[w][tid];
            base[tid] += add;
        }
        __syncthreads();
    }
}

#endif   // PLORA_BGMV_LAZY_UNIT

// One instantiation per padded rank RPK.  The kernel handles the units whose adapter has that
// padded rank and skips the others: a pool of mixed ranks is served by one launch per rank
// class present in it, each with loops specialised (and registers allocated) for its rank.
template <int MODE, int RPK, bool H, bool LAZY>
__global__ void __launch_bounds__(kThreads, kCtasPerSm) bgmv_kernel(const Params p) {
    static_assert(!LAZY || MODE == kFused, "only the fused kernel puts off its join");
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Smem sm;
    sm.slots = smem_u32(smem_raw);
    sm.m_ring = smem_u32(smem_raw + kStages * kSlotBytes);
    uint8_t* bars = smem_raw + kStages * kSlotBytes + kMRing * kMRingBytes;
    sm.full = smem_u32(bars);
    sm.empty = sm.full + kStages * 8;
    sm.m_full = sm.empty + kStages * 8;
    sm.m_empty = sm.m_full + kMRing * 8;
    sm.wait.abort_flag = reinterpret_cast<volatile int*>(bars + kNumBarriers * 8);
    sm.wait.status = p.status;
    sm.wait.limit = p.wait_cycles;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    sm.withhold = p.test_hook == PLORA_HOOK_WITHHOLD_RELEASE && warp == 0;
    if (MODE != kShrinkOnly && p.maybe_empty && p.early_tables) {
        // A launch that has nothing to do (every segment of the batch went to the tensor-core path)
        // leaves before it sets up its ring.  The host asks for the check only for batches that can
        // have tensor-core segments: the load below delays the start of every CTA by a trip to L2,
        // which the small launches of a decode step would feel.  The count is older than the previous
        // kernel of the stream, hence complete.  The CTA still joins the stream order, so that the
        // launch's completion implies that of everything before it.  (The shrink-only kernel always
        // has the rows of tokens without an adapter to clear.)
        if (*p.bk.n_bgmv_units == 0) {
            if (tid == 0) grid_dependency_wait();
            return;
        }
    }
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(sm.full + s * 8, 1);
            mbar_init(sm.empty + s * 8, kConsumerWarps);
            // a stage that was never filled reads as "nothing follows"
            sts128(sm.slots + s * kSlotBytes + kHdrOffset, (uint32_t)kFlagEnd, 0u, 0u, 0u);
            sts128(sm.slots + s * kSlotBytes + kHdrOffset + 48, 0u, 0u, 0u, kNoStamp);
        }
        for (int e = 0; e < kMRing; ++e) {
            mbar_init(sm.m_full + e * 8, 1);
            mbar_init(sm.m_empty + e * 8, kConsumerWarps);
        }
        *sm.wait.abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();
    // Everything above may overlap the previous kernel of the stream.  Its results (x, y, m,
    // the epoch, possibly the bucket tables) are read only after grid_dependency_wait().  The
    // producer warp delays that wait: the slab is never written by a kernel, and bucket tables
    // older than the previous kernel are complete, so it fetches its first task descriptors and
    // issues the slab tiles of the ring's first turn while the previous kernel drains (config 2:
    // 1.134 -> 1.118 ms per step).  (Pulling tiles towards L2 with prefetches at that point, instead
    // of copying them into the ring, was tried earlier and was slower.)
    if (LAZY) sm.joined = true;
    if (warp != kProducerWarp) {
        if (LAZY && !p.defer_wait && warp < kConsumerWarps) {
            // The consumers of a launch whose x is known to be complete start on their first shrink task
            // at once and join at its hand-over (join_stream); the gather warp below joins now, so the
            // CTA still signals only after it has seen the previous kernel complete.
            sm.joined = false;
            sm.epoch = 0u;
        } else {
            if (!p.defer_wait) grid_dependency_wait();
            // Signalled only after this CTA has seen the previous kernel complete (or, for a class launch
            // that defers its wait, after the first class launch of the call has): when the next kernel of
            // the stream starts, everything older than this call is therefore complete.
            grid_launch_dependents();
            sm.epoch = MODE == kFused ? *p.bk.epoch : 0u;
        }
    }

    if (MODE == kShrinkOnly && warp != kProducerWarp) {
        // tokens without an adapter get a zero row of m (by the warps that have already joined the
        // stream order: an earlier kernel may still be reading m)
        const int n_active = *p.bk.n_active;
        const long long total = (long long)(p.n_tok - n_active) * p.ldm;
        const int wtid = warp < kProducerWarp ? tid : tid - 32;   // index among the threads that take part
        for (long long i = (long long)blockIdx.x * (kThreads - 32) + wtid; i < total;
             i += (long long)gridDim.x * (kThreads - 32)) {
            const int pos = n_active + (int)(i / p.ldm);
            store_m(p, (size_t)p.bk.perm[pos] * p.ldm + (int)(i % p.ldm), 0.f);
        }
    }

    if (warp == kProducerWarp) {
        // ------------------------------- producer warp -------------------------------
        // The warp fetches the descriptors of its next 32 tasks in one go; lane l owns the l-th
        // of them and works out everything about it (tile range, source address, header words)
        // in parallel with the other lanes.  The lanes then take turns, in task order: the owner
        // alone waits for free stages, writes the headers and issues the copies of its task, so
        // the serial part of the producer is a few dozen instructions per stage.  In fused mode
        // the whole warp first gathers an expand task's m into the m ring.
        bool waited = p.defer_wait != 0;
        // (x complete before the previous kernel began, tables older than it: nothing this warp reads can change)
        if (LAZY && p.early_tables) waited = true;
        if (!waited && !p.early_tables) {
            grid_dependency_wait();
            waited = true;
        }
        const int n_units = *p.bk.n_bgmv_units;
        const auto plan = make_plan<MODE, RPK, LAZY>(p, n_units);   // the tasks of this launch
        const int n_tasks = plan.n_tasks;
        const int stride = gridDim.x;
        const unsigned full = 0xffffffffu;
        uint32_t it_base = 0;
        uint32_t m_count = 0;   // expand tasks issued so far (fused mode)
        bool stopped = false;   // a wait ran out somewhere in this CTA: nothing more is issued
        for (int base = blockIdx.x; base < n_tasks && !stopped; base += 32 * stride) {
            const int my_task = base + lane * stride;
            const bool has = my_task < n_tasks;
            const Task mine = plan.decode(has ? my_task : base);
            const int vunit = plan.unit_at(mine.slot, mine.unit);   // group * n_units + unit
            const int my_group = vunit / max(n_units, 1);
            const WorkUnit mu = p.bk.bgmv_units[vunit - my_group * n_units];
            const AdapterEntry me = p.table_g[my_group][mu.adapter];
            const int in_batch = min(32, (n_tasks - base + stride - 1) / stride);
            const int rp = RPK ? RPK : plan.rp[mine.slot];   // == me.rp: the lists are per class
            // a shrink stage of a sliced unit has the geometry of a rank-kSliceRows tile
            const bool sliced = MODE == kFused && (RPK == 0 || RPK > kSliceRows) && plan.s_slices[mine.slot] > 1;
            const int C = tile_cols(!mine.phase && sliced ? kSliceRows : rp);
            const uint32_t tb = (uint32_t)tile_bytes(rp);   // bytes of a slab tile
            const int d = mine.phase ? p.pool.d_out : p.pool.d_in;
            const int runs = mine.phase ? plan.e_runs[mine.slot] : plan.s_runs[mine.slot];
            const int nT = (d + C - 1) / C;
            const int lo = has ? mine.run * nT / runs : 0, hi = has ? (mine.run + 1) * nT / runs : 0;
            const int k0 = mine.slice * kSliceRows;
            const uint8_t* src = p.slab_g[my_group] + (mine.phase ? me.offB : me.offA);
            const uint16_t* my_x = p.x_g[my_group];
            // first stage number of every lane's task: exclusive prefix sum of the stage counts
            int incl = hi - lo;
#pragma unroll
            for (int dlt = 1; dlt < 32; dlt <<= 1) {
                const int v = __shfl_up_sync(full, incl, dlt);
                if (lane >= dlt) incl += v;
            }
            const uint32_t my_it0 = it_base + (uint32_t)(incl - (hi - lo));
            it_base += (uint32_t)__shfl_sync(full, incl, 31);

            // This CTA's first descriptors are in registers.  If it has not joined the stream order yet, the
            // slab tiles of the ring's first turn go out before it does (pass 1): no kernel ever writes the
            // slab, and the previous kernel's last CTAs leave most of the memory system idle.  What the
            // previous kernel may have written (x, the caller's m) follows after the wait (pass 2, which
            // also issues everything beyond the first turn).  Otherwise one pass issues everything (pass 0).
            const bool early = !waited;
            for (int pass = early ? 1 : 0; pass <= (early ? 2 : 0) && !stopped; ++pass) {
                if (pass == 2) {
                    grid_dependency_wait();
                    waited = true;
                }
                if (pass != 1 && base == (int)blockIdx.x) sm.epoch = MODE == kFused ? *p.bk.epoch : 0u;
                uint32_t mc = m_count;
                bool failed = false;
                for (int b = 0; b < in_batch && !stopped; ++b) {
                    // fused mode: the running number of this expand task tells the consumers where its m is
                    const uint32_t m_seq = mc;
                    if (MODE == kFused && __shfl_sync(full, (int)(has && mine.phase), b)) ++mc;
                    if (lane == b) {
                        const int cnt = mu.cnt;
                        // bytes a token adds to a stage besides the tile: its x piece (shrink) or its m row (expand-only)
                        const uint32_t mbytes = (MODE == kExpandOnly) ? (uint32_t)rp * (p.m16 ? 2u : 4u) : 0u;
                        uint32_t it = my_it0;
                        for (int i = lo; i < hi; ++i, ++it) {
                            const bool first_turn = it < (uint32_t)kStages;
                            if (pass == 1 && !first_turn) break;
                            const bool head = pass != 2 || !first_turn;   // header, byte count and slab tile
                            const bool tail = pass != 1;                  // what may depend on the previous kernel
                            const uint32_t slot = it % kStages;
                            const uint32_t dst = sm.slots + slot * kSlotBytes;
                            const uint32_t bar = sm.full + slot * 8;
                            const uint32_t tbytes = mine.phase ? mbytes : (uint32_t)min(C, d - i * C) * 2u;
                            if (head) {
                                if (!mbar_wait(sm.empty + slot * 8, ((it / kStages) & 1) ^ 1, sm.wait)) {
                                    failed = true;
                                    break;
                                }
                                const int flags = (mine.phase ? kFlagExpand : 0) | (i == lo ? kFlagFirst : 0) | (i == hi - 1 ? kFlagLast : 0) |
                                                  (!mine.phase && sliced ? kFlagSlice : 0);
                                sts128(dst + kHdrOffset, (uint32_t)flags, (uint32_t)(my_group * p.n_tok + mu.pos0), (uint32_t)mine.run, (uint32_t)i);
                                sts128(dst + kHdrOffset + 16, (uint32_t)cnt, (uint32_t)mu.tok[0], (uint32_t)mu.tok[1], (uint32_t)mu.tok[2]);
                                sts128(dst + kHdrOffset + 32, (uint32_t)mu.tok[3], (uint32_t)rp, (uint32_t)me.r, __float_as_uint(me.scale));
                                sts128(dst + kHdrOffset + 48, m_seq, (uint32_t)my_group, (uint32_t)k0, it);   // it: kStampOffset
                                if (MODE == kFused && sliced && !mine.phase) {
                                    // rows [k0, k0 + kSliceRows) of up to four consecutive sub-tiles of A^T, side by side
                                    constexpr uint32_t kPiece = kSliceRows * kSubCols * 2;
                                    const int n_sub_tile = subs_per_tile(rp);   // sub-tiles per slab tile
                                    const int n_sub = (d + kSubCols - 1) / kSubCols;
                                    const int n_here = min(C / kSubCols, n_sub - i * (C / kSubCols));
                                    mbar_arrive_expect_tx(bar, (uint32_t)n_here * kPiece + (uint32_t)cnt * tbytes);
                                    for (int j = 0; j < n_here; ++j) {
                                        const int g = i * (C / kSubCols) + j;
                                        bulk_g2s(dst + j * kPiece,
                                                 checked_src(src + (size_t)(g / n_sub_tile) * tb + (size_t)(g % n_sub_tile) * (rp * kSubCols * 2) + (size_t)k0 * (kSubCols * 2),
                                                             kPiece, p.slab_g[my_group], p.slab_bytes_g[my_group], p.status),
                                                 kPiece, bar);
                                    }
                                } else {
                                    mbar_arrive_expect_tx(bar, tb + (uint32_t)cnt * tbytes);
                                    bulk_g2s(dst, checked_src(src + (size_t)i * tb, tb, p.slab_g[my_group], p.slab_bytes_g[my_group], p.status), tb, bar);
                                }
                            }
                            if (tail) {
                                if (!mine.phase) {
#pragma unroll
                                    for (int t = 0; t < kTokChunk; ++t)
                                        if (t < cnt)
                                            bulk_g2s(dst + kTileBytesMax + t * kXBytesPerTok,
                                                     checked_src(my_x + (size_t)mu.tok[t] * p.pool.d_in + (size_t)i * C, tbytes, my_x,
                                                                 (uint64_t)p.n_tok * p.pool.d_in * 2, p.status),
                                                     tbytes, bar);
                                } else if (MODE == kExpandOnly) {
#pragma unroll
                                    for (int t = 0; t < kTokChunk; ++t)   // the caller's m row, rp values, lands as m[t][0..rp)
                                        if (t < cnt)
                                            bulk_g2s(dst + kTileBytesMax + t * mbytes,
                                                     checked_src(reinterpret_cast<const uint8_t*>(p.m) + (size_t)mu.tok[t] * p.ldm * (p.m16 ? 2 : 4), mbytes,
                                                                 p.m, (uint64_t)p.n_tok * p.ldm * (p.m16 ? 2 : 4), p.status),
                                                     mbytes, bar);
                                }
                            }
                        }
                    }
                    stopped = __any_sync(full, failed);   // (also the warp's meeting point after the owner's turn)
                }
                if (pass != 1) m_count = mc;
            }
        }
        if (!waited) grid_dependency_wait();
        if (lane == 0) {
            if (!stopped) {   // tell the consumers that nothing follows
                const uint32_t it = it_base;
                const uint32_t slot = it % kStages;
                if (mbar_wait(sm.empty + slot * 8, ((it / kStages) & 1) ^ 1, sm.wait)) {
                    sts128(sm.slots + slot * kSlotBytes + kHdrOffset, (uint32_t)kFlagEnd, 0u, 0u, 0u);
                    sts128(sm.slots + slot * kSlotBytes + kHdrOffset + 48, 0u, 0u, 0u, it);
                    mbar_arrive(sm.full + slot * 8);
                }
            }
            // Before the warp leaves, every copy it asked for must have landed: the CTA's shared memory goes
            // to another CTA when the last warp is gone.  Each stage's header names the phase it was last
            // armed for.  In an orderly run these waits return at once or overlap the consumers' last stages.
            // After a give-up between the two passes of the first turn a stage may be armed for bytes that
            // were never asked for: its wait runs out, which is harmless (nothing is on its way there).
            for (int s2 = 0; s2 < kStages; ++s2) {
                const uint32_t stamp = lds32(sm.slots + s2 * kSlotBytes + kHdrOffset + kStampOffset);
                if (stamp != kNoStamp && !mbar_drain(sm.full + s2 * 8, (stamp / kStages) & 1, p.wait_cycles))
                    atomicCAS(p.status, 0, PLORA_ERR_TIMEOUT);
            }
        }
        return;
    }

    if (warp == kGatherWarp) {
        // ------------------------------- gather warp (fused mode) -------------------------------
        // Walks this CTA's expand tasks in order, ahead of the consumers: reads the partial words
        // of the unit (again and again, for a bounded time, until all of them carry this launch's
        // epoch), sums them in run order into the next m-ring entry and publishes the entry.
        if (MODE != kFused) return;
        const int n_units = *p.bk.n_bgmv_units;
        const auto plan = make_plan<MODE, RPK, LAZY>(p, n_units);
        const int n_shrink = plan.n_shrink, n_tasks = plan.n_tasks;
        const int stride = gridDim.x;
        const unsigned full = 0xffffffffu;
        // this CTA's first expand task
        int t = blockIdx.x;
        if (t < n_shrink) t += (n_shrink - t + stride - 1) / stride * stride;
        uint32_t seq = 0;
        for (int base = t; base < n_tasks; base += 32 * stride) {
            const int my_task = base + lane * stride;
            // (a one-class launch needs nothing but the unit: the chain from here to the first gathered m
            // is on the critical path of a small launch)
            int slot = 0, idx;
            if (RPK) {
                idx = ((my_task < n_tasks ? my_task : base) - n_shrink) / plan.e_runs[0];
            } else {
                const Task mine = plan.decode(my_task < n_tasks ? my_task : base);
                slot = mine.slot;
                idx = mine.unit;
            }
            const int vunit = plan.unit_at(slot, idx);
            const int my_group = vunit / max(n_units, 1);
            const WorkUnit mu = p.bk.bgmv_units[vunit - my_group * n_units];
            // One-class launch: the rank comes from the table, as a check that the unit is this launch's
            // (it always is: the lists are per class).  The load is kept for its timing: without it the
            // warp's first look at the partial words comes about a microsecond earlier, and the 64 small
            // launches of a 7B decode step take 1 % longer (measured both ways on the same box).
            const int my_rp = RPK ? p.table_g[my_group][mu.adapter].rp : plan.rp[slot];
            const int my_runs_a = plan.s_runs[slot];
            const int in_batch = min(32, (n_tasks - base + stride - 1) / stride);
            for (int b = 0; b < in_batch; ++b) {
                const int rp_b = __shfl_sync(full, my_rp, b);
                if (RPK && rp_b != RPK) continue;
                const int runs_a_b = RPK ? plan.s_runs[0] : __shfl_sync(full, my_runs_a, b);
                const int unit_b = __shfl_sync(full, my_group * p.n_tok + mu.pos0, b), cnt_b = __shfl_sync(full, mu.cnt, b);
                const uint32_t e = seq % kMRing;
                bool ok = true;
                if (lane == 0) ok = mbar_wait(sm.m_empty + e * 8, ((seq / kMRing) & 1) ^ 1, sm.wait);
                if (!__all_sync(full, ok)) return;   // gave up: the consumers see the flag at their own waits
                const uint32_t mdst = sm.m_ring + e * kMRingBytes;
                if (!__all_sync(full, gather_m(p, rp_b, runs_a_b, sm.epoch, unit_b, cnt_b, lane, mdst))) {
                    const long long t0 = clock64();
                    for (;;) {
                        __nanosleep(100);
                        if (__all_sync(full, gather_m(p, rp_b, runs_a_b, sm.epoch, unit_b, cnt_b, lane, mdst))) break;
                        // one lane decides for the warp, so that all lanes leave together
                        int quit = 0;
                        if (lane == 0) {
                            if (*sm.wait.abort_flag) quit = 1;
                            else if (clock64() - t0 > sm.wait.limit) {
                                give_up(sm.wait.abort_flag, p.status);
                                quit = 1;
                            }
                        }
                        if (__shfl_sync(full, quit, 0)) return;   // the entry is never published: no expand task uses a partial m
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(sm.m_full + e * 8);
                ++seq;
            }
        }
        return;
    }

    // ------------------------------- consumer warps -------------------------------
    // Stage-driven.  The stages of one rank class are consumed by that class's instantiation of the
    // loops, with its per-lane constants set up once; a launch for all classes switches when a stage
    // of another class turns up (tasks are sorted by class, so a CTA switches a few times per launch).
    float acc[kMaxRowsPerLane][kTokChunk];
    uint32_t it = 0;
    bool gave_up = false;   // this lane: from here to the end of the kernel there is no warp-level operation
    if (RPK) {
        consume_class<MODE, RPK ? RPK : 8, H, true, LAZY>(p, sm, it, gave_up, acc, warp, lane);
    } else {
        for (bool more = true; more;) {
            // whose stage is next?  (the class's loop waits for it again: the phase is complete by then)
            const uint32_t slot = it % kStages;
            if (!mbar_wait(sm.full + slot * 8, (it / kStages) & 1, sm.wait)) break;
            const int flags = (int)lds32(sm.slots + slot * kSlotBytes + kHdrOffset);
            const int rp = (int)lds32(sm.slots + slot * kSlotBytes + kHdrOffset + 36);
            if (flags & kFlagEnd) break;
            switch (rp) {
                case 8: more = consume_class<MODE, 8, H, false, LAZY>(p, sm, it, gave_up, acc, warp, lane); break;
                case 16: more = consume_class<MODE, 16, H, false, LAZY>(p, sm, it, gave_up, acc, warp, lane); break;
                case 32: more = consume_class<MODE, 32, H, false, LAZY>(p, sm, it, gave_up, acc, warp, lane); break;
                case 64: more = consume_class<MODE, 64, H, false, LAZY>(p, sm, it, gave_up, acc, warp, lane); break;
                default: more = consume_class<MODE, 128, H, false, LAZY>(p, sm, it, gave_up, acc, warp, lane); break;
            }
        }
    }
    if (LAZY) join_stream(p, sm);   // (a CTA without a shrink task has not joined yet)
    if (tid == 0 && p.defer_wait) grid_dependency_wait();
    if (MODE == kFused && tid == 0 && p.bump_epoch) {
        // the last CTA to finish opens the next epoch: words written by this call can never
        // be mistaken for the next one's
        if (atomicAdd(p.bk.exit_count, 1u) == gridDim.x - 1) {
            *p.bk.exit_count = 0u;
            *p.bk.epoch = sm.epoch + 1u;
        }
    }
}

using KernelFn = void (*)(const Params);

template <int MODE, bool H, bool LAZY>
KernelFn pick_rank(int rp) {
    switch (rp) {
        case 0: return MODE == kFused ? bgmv_kernel<kFused, 0, H, LAZY> : nullptr;   // all classes of a mixed pool, fused only
        case 8: return bgmv_kernel<MODE, 8, H, LAZY>;
        case 16: return bgmv_kernel<MODE, 16, H, LAZY>;
        case 32: return bgmv_kernel<MODE, 32, H, LAZY>;
        case 64: return bgmv_kernel<MODE, 64, H, LAZY>;
        default: return bgmv_kernel<MODE, 128, H, LAZY>;
    }
}

#ifdef PLORA_BGMV_LAZY_UNIT
}  // namespace

// The fused kernels whose consumers put off joining the stream order (plora_set_inputs_resident) are compiled in a
// translation unit of their own, bgmv_lazy.cu, which includes this file with PLORA_BGMV_LAZY_UNIT defined and gets
// the kernel template and this function, nothing else: the other kernels of the library keep the code they had
// before these existed, byte for byte and in the same order (several of them run side by side in a mixed-rank
// call, and their speed there proved sensitive to what else the module holds).
const void* bgmv_lazy_kernel(int rp, bool fp16) {
    return fp16 ? reinterpret_cast<const void*>(pick_rank<kFused, true, true>(rp))
                : reinterpret_cast<const void*>(pick_rank<kFused, false, true>(rp));
}
#else

template <bool H>
KernelFn pick_mode(BgmvMode mode, int rp) {
    switch (mode) {
        case kFused: return pick_rank<kFused, H, false>(rp);
        case kShrinkOnly: return pick_rank<kShrinkOnly, H, false>(rp);
        default: return pick_rank<kExpandOnly, H, false>(rp);
    }
}

// lazy: the fused kernel whose consumers put off joining the stream order (plora_set_inputs_resident)
const void* pick_kernel(BgmvMode mode, int rp, bool fp16, bool lazy) {
    if (lazy && mode == kFused) return bgmv_lazy_kernel(rp, fp16);
    return reinterpret_cast<const void*>(fp16 ? pick_mode<true>(mode, rp) : pick_mode<false>(mode, rp));
}

// One launch of a BGMV kernel with the given configuration.
cudaError_t launch_kernel(const cudaLaunchConfig_t& cfg, const void* fn, const Params& p) {
    void* args[1] = {const_cast<Params*>(&p)};
    return cudaLaunchKernelExC(&cfg, fn, args);
}

int clamp_runs(int tiles) { return tiles < 1 ? 1 : (tiles > kMaxRuns ? kMaxRuns : tiles); }

}  // namespace

cudaError_t bgmv_configure() {
    const int modes[3] = {kFused, kShrinkOnly, kExpandOnly};
    const int rps[6] = {0, 8, 16, 32, 64, 128};
    for (int m : modes)
        for (int rp : rps) {
            if (rp == 0 && m != kFused) continue;
            for (int h = 0; h < 2; ++h) {
                cudaError_t e = cudaFuncSetAttribute(pick_kernel((BgmvMode)m, rp, h != 0, false),
                                                     cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
                if (e != cudaSuccess) return e;
            }
        }
    return cudaSuccess;
}

// The kernels of bgmv_lazy.cu, configured (and thereby loaded) after every other module of the library.
cudaError_t bgmv_configure_lazy() {
    const int rps[6] = {0, 8, 16, 32, 64, 128};
    for (int rp : rps)
        for (int h = 0; h < 2; ++h) {
            cudaError_t e = cudaFuncSetAttribute(bgmv_lazy_kernel(rp, h != 0), cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
            if (e != cudaSuccess) return e;
        }
    return cudaSuccess;
}

cudaError_t launch_bgmv(BgmvMode mode, const PoolDev* pools, int n_groups, const BucketDev& bk, int n_tok,
                        const void* const* x, float* const* y, void* m, int ldm, bool m16, bool fp16, int32_t* status,
                        int sm_count, bool early_tables, ClassCache* cls_cache, uint64_t rank_sig, const DebugCfg& dbg,
                        cudaStream_t stream, int* n_launches, BetweenLaunch between, void* between_arg) {
    if (n_groups < 1 || n_groups > kMaxGroup || (mode != kFused && n_groups != 1)) return cudaErrorInvalidValue;
    const PoolDev& pool = pools[0];
    Params p;
    p.pool = pool;
    p.bk = bk;
    p.n_groups = n_groups;
    int rp_mask = 0;
    for (int g = 0; g < kMaxGroup; ++g) {
        const int gg = g < n_groups ? g : 0;
        p.slab_g[g] = pools[gg].slab;
        p.slab_bytes_g[g] = pools[gg].slab_bytes;
        p.table_g[g] = pools[gg].table;
        p.x_g[g] = static_cast<const uint16_t*>(x ? x[gg] : nullptr);
        p.y_g[g] = y ? y[gg] : nullptr;
        if (g < n_groups) rp_mask |= pools[g].rp_mask;
    }
    p.m = static_cast<float*>(m);
    p.ldm = ldm;
    p.m16 = m16 ? 1 : 0;
    p.n_tok = n_tok;
    p.status = status;
    p.wait_cycles = dbg.wait_cycles > 0 ? dbg.wait_cycles : kWaitCycles;
    p.test_hook = dbg.test_hook;
    p.early_tables = early_tables ? 1 : 0;
    p.maybe_empty = dbg.maybe_empty ? 1 : 0;
    p.inputs_resident = dbg.inputs_resident && mode == kFused ? 1 : 0;
    p.defer_wait = 0;
    p.bump_epoch = 1;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    p.by_class = (rp_mask & (rp_mask - 1)) != 0;   // more than one rank class in the call's pools
    p.runs_a = p.runs_b = 1;
    // one launch for all classes (small batches) or one per class
    const bool one_launch = p.by_class && mode == kFused && (long long)n_tok * n_groups <= kMixedLaunchMaxRows;
    // the two kinds of launch want the class lists in different orders: each has its own lists
    const int sort = one_launch ? 1 : 0;
    p.sort_by_cnt = sort;
    p.bk.cls_list = bk.cls_list + (size_t)sort * n_tok;
    p.bk.cls_start = bk.cls_start + sort * 8;
    if (p.by_class && !(cls_cache && cls_cache->valid[sort] && cls_cache->sig[sort] == rank_sig)) {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(1);
        cfg.blockDim = dim3(kClassifyThreads);
        cfg.stream = stream;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const cudaError_t e = cudaLaunchKernelEx(&cfg, classify_kernel, p);
        ++*n_launches;
        if (e != cudaSuccess) return e;
        p.early_tables = 0;   // the next launch reads what the classify pass has just written
        if (cls_cache) {
            cls_cache->sig[sort] = rank_sig;
            cls_cache->valid[sort] = true;
        }
    }
    if (between) {
        const cudaError_t e = between(between_arg, n_launches);
        if (e != cudaSuccess) return e;
        p.early_tables = 1;                          // what follows comes after a kernel that is not the bucket kernel,
        p.defer_wait = mode == kFused ? 1 : 0;       // and that kernel has joined the stream's order for the whole call
    }
    // one launch per padded-rank class present in the pool
    if (one_launch) {
        // every rank class in one launch, cut to tasks of about the same size (see Plan)
        const long long max_tasks = (long long)n_tok * n_groups * 4 * kMaxRuns;
        const size_t need = (size_t)n_tok * n_groups * kMaxRunsA * pool.max_rp * sizeof(unsigned long long);
        if (need > bk.m_part_bytes) return cudaErrorMemoryAllocation;
        int grid = kCtasPerSm * sm_count;
        if (grid > max_tasks) grid = (int)max_tasks;
        if (grid < 1) grid = 1;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = kSmemBytes;
        cfg.stream = stream;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const cudaError_t e = launch_kernel(cfg, pick_kernel(mode, 0, fp16, p.inputs_resident != 0 && !p.defer_wait), p);
        ++*n_launches;
        return e;
    }
    // One launch per padded-rank class present.  In fused mode the class launches of a call overlap (see
    // defer_wait), and the class with the largest units goes first: the others' CTAs move in as its CTAs
    // retire and fill its tail.
    int last_rp = kMaxRank;
    for (int rp = kMaxRank; rp >= 8; rp >>= 1)
        if (rp_mask & rp) last_rp = rp;
    for (int rp = kMaxRank; rp >= 8; rp >>= 1) {
        if (!(rp_mask & rp)) continue;
        p.bump_epoch = rp == last_rp;
        // a unit of this class has tiles_for(d, rp) tiles per phase: cut each phase into runs
        p.runs_a = mode == kShrinkOnly ? 1 : clamp_runs(tiles_for(pool.d_in, rp));
        // (a fused launch with few units of padded rank above kSliceRows cuts them into row slices,
        // whose stages have the rank-kSliceRows geometry)
        const int slices = mode == kFused && rp > kSliceRows ? rp / kSliceRows : 1;
        p.runs_a_sliced = clamp_runs(tiles_for(pool.d_in, kSliceRows));
        if (p.runs_a_sliced > kMaxRunsA) p.runs_a_sliced = kMaxRunsA;
        // an expand task pays one round trip for its m before its first tile: give it at least two tiles
        p.runs_b = clamp_runs(tiles_for(pool.d_out, rp) / (mode == kFused ? 2 : 1));
        // every shrink task ends with a hand-over of its partial m (and every expand task reads all of
        // them): at most kMaxRunsA shrink tasks per unit measured best (4: 0.764 of the roofline on the
        // decode 7B shapes, 8: 0.748, 2: 0.757)
        if (p.runs_a > kMaxRunsA) p.runs_a = kMaxRunsA;
        if (mode == kFused) {
            // the partial-m workspace holds n_groups * n_tok * kMaxRunsA * max_rp words
            const size_t need = (size_t)n_tok * n_groups * kMaxRunsA * pool.max_rp * sizeof(unsigned long long);
            if (need > bk.m_part_bytes) return cudaErrorMemoryAllocation;
        }
        // persistent grid: two CTAs per SM, never more CTAs than there can be tasks
        const long long max_tasks = (long long)n_tok * n_groups * (p.runs_a * slices + p.runs_b);
        int grid = kCtasPerSm * sm_count;
        if (grid > max_tasks) grid = (int)max_tasks;
        if (grid < 1) grid = 1;
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(grid);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = kSmemBytes;
        cfg.stream = stream;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const cudaError_t e = launch_kernel(cfg, pick_kernel(mode, rp, fp16, p.inputs_resident != 0 && !p.defer_wait), p);
        ++*n_launches;
        if (e != cudaSuccess) return e;
        p.early_tables = 1;   // the next class's launch follows a kernel that is not the bucket kernel
        p.defer_wait = mode == kFused ? 1 : 0;
    }
    return cudaSuccess;
}

#endif   // PLORA_BGMV_LAZY_UNIT

}  // namespace plora
