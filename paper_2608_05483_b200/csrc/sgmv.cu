// SGMV: the prefill-shaped path of the LoRA delta.  A segment (all tokens of one adapter) that
// is long enough is cut into tiles of kSgmvRows rows and each tile runs the paper's two small
// GEMMs on the tensor cores (Section V-A: shrink m = x A, then expand y = m B; large per-adapter
// batches favour computing on the GPU from resident A and B, strategy E1):
//
//     m [rows, rp]    = X [rows, d_in] * A          bf16 x bf16 -> fp32   (K = d_in)
//     y [rows, d_out] += s * m * B                  fp32 m carried as bf16 hi + lo, two products
//
// Both GEMMs are issued as tcgen05.mma (M = 64, accumulators in tensor memory) by one thread
// of the CTA; the operands reach shared memory without passing through registers:
//
//   - the x rows of a tile are gathered by token index with the tensor-map copy in gather mode
//     (four rows of 64 columns per instruction) straight into the 128-byte-swizzled K-major
//     operand layout; the matching [rp][64] sub-tile of A^T, stored in the slab in that very
//     layout, arrives with one bulk copy;
//   - in the expand the [rp][64] sub-tiles of B are the MN-major operand, again as they sit in
//     the slab;
//   - four epilogue warps read the shrink result from tensor memory, scale it, split it into
//     bf16 hi + lo (error ~2^-17 relative) and store it as the K-major operand of the expand;
//     they then drain every 64-column block of the expand result: transposed through a small
//     per-warp staging buffer so that a warp adds whole 256-byte row pieces to y with vector
//     reductions (one addition per element of y, so the result is bit-reproducible).
//
// Roles: the first warps issue the copies (stage i belongs to copy warp i mod their number), the
// next warp owns the tensor memory and issues the MMAs, the last four are the epilogue.  Stages (x block + weight sub-tile) cycle through a ring guarded by
// full / empty mbarriers; the MMA thread releases a stage with tcgen05.commit.  The path is
// bound by HBM traffic on the activations (x read once, y updated once), not by the tensor
// pipe.  Every wait is bounded: when one runs out the kernel records PLORA_ERR_TIMEOUT, every
// role leaves its loop, and the tensor memory is freed before the CTA exits.
//
// Two launch shapes share the code.  Wide: persistent CTAs, a CTA runs whole tiles (a batch with
// enough tiles to occupy the GPU, prefill).  Split: a batch with only a handful of long segments
// (the paper's per-adapter batches go up to 256 requests, Section V-A, also inside an otherwise
// decode-shaped step) gives too few tiles for that, and a tile is a long serial job.  There a
// thread-block cluster of kClusterSize CTAs takes one tile: CTA c shrinks over its eighth of d_in,
// the partial m of the cluster meet through distributed shared memory (each CTA sums eight of the
// 64 rows in a fixed order, scales, splits into hi + lo and stores the finished rows into every
// CTA's operand buffers), and CTA c expands its eighth of d_out.  Every CTA fetches its own
// operands: no copy is shared between the CTAs of a cluster.
#include <cuda.h>
#include <cuda_fp16.h>

#include "plora_internal.cuh"

namespace plora {

namespace {

constexpr int kRows = kSgmvRows;          // rows of a tile = M of the MMAs (64)
constexpr int kRowsPerWarp = kRows / 4;   // M = 64: row r of the accumulator sits in tensor-memory lane 32 (r / 16) + r % 16
static_assert(kRows == 64, "the epilogue's lane mapping is the one of M = 64");
constexpr int kKC = kSubCols;             // K (or N) columns per stage = one slab sub-tile (64)
constexpr int kXStageBytes = kRows * kKC * 2;              // 8 KiB of x per stage
constexpr int kEpiGroups = 1;   // groups of four epilogue warps; with more than one they take the expand blocks in turn
// The gather copy moves four rows per instruction and is paced by the copy engine's rate of
// instructions; where 32 rows of a tile are consecutive tokens (a prefill request is a
// contiguous run) one ordinary box copy brings all of them.
constexpr int kBoxRows = 32;
constexpr int kBoxLanes = kBoxRows / 4;   // lanes of the copy warp whose rows one box covers
// A thread gets a copy instruction out about every 45 ns and a stage takes up to five of them:
// the stages are dealt out to two copy warps.  (The copy engine itself moves about 50 GB/s per
// SM in boxes of this shape, which is what bounds the shrink phase.)
constexpr int kProducerWarps = 2;
constexpr int kMmaWarp = kProducerWarps, kFirstEpiWarp = kProducerWarps + 1, kEpiWarps = 4 * kEpiGroups;
constexpr int kThreads = (kFirstEpiWarp + kEpiWarps) * 32;
constexpr int kMaxStages = 8;
constexpr int kD2Bufs = 2;                // expand accumulators in flight (64 columns each)
constexpr int kTmemCols = 256;            // columns [0, 128): shrink result; [128, 256): expand blocks; two CTAs share an SM's 512
constexpr int kTmemD2 = 128;
constexpr int kStagePitch = kKC * 4 + 16;                  // row pitch of the epilogue staging buffer
constexpr int kStagingBytes = kEpiWarps * kRowsPerWarp * kStagePitch;
constexpr int kSmemBudget = 227 * 1024;                    // of an SM
constexpr int kSmemPerCta = kSmemBudget / 2 - 1024;        // two CTAs per SM, so that one tile's shrink overlaps another's expand
constexpr long long kWaitCycles = 4000000000ll;            // default limit of a wait: about two seconds of SM clock
constexpr int kClusterSize = 8;                            // split shape: CTAs per tile
constexpr int kRedRows = kRows / kClusterSize;             // rows of the tile a CTA of the cluster sums

// Shared memory, sized for R = max(16, largest padded rank of the pool):
//   ring of n_stages x (x block 8 KiB + weight sub-tile R x 128 B)       1024-byte aligned
//   m hi, m lo: (R / 8) column chunks x 64 rows x 16 B each              no-swizzle K-major operand
//   staging buffer of the epilogue, token indices of the tile, barriers
__host__ __device__ inline int w_stage_bytes(int R) { return R * 128; }
__host__ __device__ inline int stage_bytes(int R) { return kXStageBytes + w_stage_bytes(R); }
__host__ __device__ inline int m_bytes(int R) { return (R / 8) * kRows * 16; }
constexpr int kTailBytes = kStagingBytes + kRows * 4 + 256;
// split shape: where the cluster's partial sums of this CTA's kRedRows rows arrive, [source CTA][row][R] floats
__host__ __device__ inline int red_bytes(int R, bool split) { return split ? kClusterSize * kRedRows * R * 4 : 0; }
__host__ __device__ inline int stages_for(int R, bool split) {
    const int fixed = 1024 + kTailBytes + 2 * m_bytes(R) + red_bytes(R, split);
    int n = (kSmemPerCta - fixed) / stage_bytes(R);
    if (n < 3) n = (kSmemBudget - fixed) / stage_bytes(R);   // rank 128: one CTA per SM
    return n > kMaxStages ? kMaxStages : n;
}
__host__ __device__ inline int smem_bytes(int R, bool split) {
    return 1024 + stages_for(R, split) * stage_bytes(R) + 2 * m_bytes(R) + red_bytes(R, split) + kTailBytes;
}

struct Params {
    PoolDev pool;
    BucketDev bk;
    float* y;
    int32_t* status;
    int32_t R;          // max(16, largest padded rank of the pool): sizes the shared-memory layout
    int32_t n_stages;
    // The launch follows the BGMV launches of the same call, which work on other tokens: it need not
    // wait for them.  It joins the stream order only when its CTAs are done, so that its completion
    // still implies the completion of everything before it.
    int32_t defer_wait;
    int32_t fp16;       // x, A and B hold IEEE half values instead of bf16 (m is then split into half hi + lo)
    int32_t n_tok;      // rows of x and y (read by the debug build's address checks only)
    long long wait_cycles;   // limit of every bounded wait, in SM clock cycles
    int32_t test_hook;       // PLORA_HOOK_*: tests make a wait run out with it
};

// ---- PTX wrappers -----------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
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
// Bounded wait on an mbarrier phase; false when the CTA has given up (here or elsewhere).
struct WaitCtl {
    volatile int* abort_flag;
    int32_t* status;
    long long limit;
};
__device__ __forceinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, const WaitCtl& w) {
    const long long t0 = clock64();
    for (;;) {
        if (*w.abort_flag) return false;
        for (int i = 0; i < 16; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (clock64() - t0 > w.limit) break;
    }
    *w.abort_flag = 1;
    __threadfence_block();
    atomicCAS(w.status, 0, PLORA_ERR_TIMEOUT);
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtl& w) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, w);
}
// Winding down after a give-up: wait for a phase whatever the abort flag says, for at most the limit.
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
// Rows r0..r3 of the 2-D tensor, 64 columns from `col`, land as four consecutive 128-byte rows.
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap* tm, int col, int r0, int r1, int r2, int r3,
                                            uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3, %4, %5, %6}], [%7];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tm)), "r"(col), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(bar)
        : "memory");
}
// A box of kBoxRows consecutive rows x 64 columns of the 2-D tensor lands as 128-byte rows, swizzled.
__device__ __forceinline__ void tma_box(uint32_t dst, const CUtensorMap* tm, int col, int row, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tm)), "r"(col), "r"(row), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, %0;" ::"n"(kEpiWarps * 32) : "memory"); }

// Shared-memory matrix descriptor of tcgen05.mma: start address, leading and stride byte
// offsets (all in 16-byte units), descriptor version 1, layout type (0 none, 2 128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout) {
    return (uint64_t)((saddr >> 4) & 0x3fffu) | ((uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16) |
           ((uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32) | ((uint64_t)1 << 46) | ((uint64_t)layout << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 (format 1) or half (format 0) operands, A K-major,
// B K- or MN-major, M = kRows.
__device__ __forceinline__ uint32_t instr_desc(int n, bool b_mn_major, bool fp16) {
    const uint32_t fmt = fp16 ? 0u : 1u;
    return (1u << 4) | (fmt << 7) | (fmt << 10) | (b_mn_major ? (1u << 16) : 0u) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(kRows >> 4) << 24);
}
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate)
        : "memory");
}
// The mbarrier gets one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive columns of this thread's lane of tensor memory.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void red_add_v4(float* p, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
// fp32 -> bf16, round to nearest even, on the bit pattern
__device__ __forceinline__ uint32_t f32_to_bf16_bits(float f) {
    const uint32_t u = __float_as_uint(f);
    return (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;
}

// ---- thread-block cluster pieces of the split shape ---------------------------------------------------
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// The address, in the cluster's shared window, of `addr` (an address in this CTA's shared memory) in CTA `rank`.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared::cluster.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// One arrival on a barrier of another CTA of the cluster; everything this thread has observed or written before
// (its own stores, and those of the threads it has met at a CTA barrier) is visible to whoever acquires the phase.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void fence_cluster() { asm volatile("fence.acq_rel.cluster;" ::: "memory"); }
// All threads of all CTAs of the cluster (the hardware's own barrier; used at the two ends of the kernel only, where
// every thread is certain to arrive: after the barriers are set up, and before any CTA gives up its shared memory).
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// What a CTA does of which tiles: the wide shape walks whole tiles, the split shape takes one tile and an
// eighth of each of its two loops.
struct Span {
    int t0, t_step;      // tiles t0, t0 + t_step, ... below the tile count
    int kc0, kc1;        // shrink stages (64 columns of d_in each)
    int nc0, nc1;        // expand blocks (64 columns of d_out each)
};
template <bool SPLIT>
__device__ __forceinline__ Span make_span(int nK, int nN) {
    Span sp;
    if (SPLIT) {
        const int c = (int)cluster_rank();
        sp.t0 = blockIdx.x / kClusterSize;
        sp.t_step = 1 << 30;
        sp.kc0 = c * nK / kClusterSize;
        sp.kc1 = (c + 1) * nK / kClusterSize;
        sp.nc0 = c * nN / kClusterSize;
        sp.nc1 = (c + 1) * nN / kClusterSize;
    } else {
        sp.t0 = blockIdx.x;
        sp.t_step = gridDim.x;
        sp.kc0 = 0; sp.kc1 = nK;
        sp.nc0 = 0; sp.nc1 = nN;
    }
    return sp;
}

struct Smem {
    uint32_t ring;        // stage 0 (1024-byte aligned); stage = x block, then the weight sub-tile
    uint32_t m_hi, m_lo;  // K-major operand of the expand, chunk kc (8 columns) of row r at kc * 2048 + r * 16
    uint32_t staging;     // epilogue staging, one 32-row block per epilogue warp
    int* tok;             // token index of every row of the tile
    uint32_t full, empty; // [kMaxStages] each
    uint32_t d_full;      // the shrink accumulator is complete
    uint32_t m_ready;     // the epilogue has stored m hi / lo (and is done with the shrink accumulator)
    uint32_t d2_full, d2_empty;   // [kD2Bufs] each
    uint32_t wind_down;   // after a give-up: the MMAs issued so far have completed
    uint32_t red;         // split shape: partial sums from the cluster (see red_bytes)
    uint32_t part_in;     // split shape: every CTA of the cluster has delivered its partial rows (kClusterSize arrivals)
    uint32_t m_in;        // split shape: every CTA of the cluster has delivered its finished rows of m
    WaitCtl wait;         // abort flag of the CTA, status word, limit of a wait
    uint32_t* tmem_slot;
    uint32_t* armed;      // [kMaxStages]: 1 + the running number of the stage a slot was last armed for (0: never)
};

__device__ __forceinline__ Smem carve(uint8_t* raw, const Params& p, bool split) {
    uint8_t* base = raw + ((1024u - (smem_u32(raw) & 1023u)) & 1023u);
    uint8_t* m = base + p.n_stages * stage_bytes(p.R);
    uint8_t* red = m + 2 * m_bytes(p.R);
    uint8_t* staging = red + red_bytes(p.R, split);
    uint8_t* tok = staging + kStagingBytes;
    uint8_t* bars = tok + kRows * 4;
    Smem s;
    s.ring = smem_u32(base);
    s.m_hi = smem_u32(m);
    s.m_lo = s.m_hi + m_bytes(p.R);
    s.staging = smem_u32(staging);
    s.tok = reinterpret_cast<int*>(tok);
    s.full = smem_u32(bars);
    s.empty = s.full + kMaxStages * 8;
    s.d_full = s.empty + kMaxStages * 8;
    s.m_ready = s.d_full + 8;
    s.d2_full = s.m_ready + 8;
    s.d2_empty = s.d2_full + kD2Bufs * 8;
    s.wind_down = s.d2_empty + kD2Bufs * 8;
    s.part_in = s.wind_down + 8;
    s.m_in = s.part_in + 8;
    s.red = smem_u32(red);
    uint8_t* words = bars + (2 * kMaxStages + 5 + 2 * kD2Bufs) * 8;
    s.wait.abort_flag = reinterpret_cast<volatile int*>(words);
    s.wait.status = p.status;
    s.wait.limit = p.wait_cycles;
    s.tmem_slot = reinterpret_cast<uint32_t*>(words + 8);
    s.armed = reinterpret_cast<uint32_t*>(words + 16);
    return s;
}

// ---- copy warps ----------------------------------------------------------------------------
// Lane g owns rows 4g .. 4g + 3 of every tile: one gather instruction per lane and stage.  Rows
// beyond the tile's count repeat its last token (their results are never written); groups that
// lie entirely beyond it are not copied at all.
template <bool SPLIT>
__device__ __forceinline__ void producer_warp(const Params& p, const Smem& sm, const CUtensorMap* tm_x,
                                              const CUtensorMap* tm_box, int n_tiles, int warp, int lane) {
    const int nK = (p.pool.d_in + kKC - 1) / kKC, nN = (p.pool.d_out + kKC - 1) / kKC;
    const Span sp = make_span<SPLIT>(nK, nN);
    const int stage = stage_bytes(p.R);
    uint32_t it = 0;
    for (int t = sp.t0; t < n_tiles; t += sp.t_step) {
        const WorkUnit wu = p.bk.sgmv_tiles[t];
        const AdapterEntry e = p.pool.table[wu.adapter];
        const int cnt = wu.cnt;
        int r[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) r[j] = p.bk.perm[wu.pos0 + min(4 * lane + j, cnt - 1)];
        const bool active = 4 * lane < cnt;
        // lanes 8j .. 8j + 7 hold rows 32j .. 32j + 31: one box copy if those are consecutive tokens
        const int lead = lane & ~(kBoxLanes - 1);
        const int first = __shfl_sync(0xffffffffu, r[0], lead);
        const bool in_run = 4 * lane + 3 < cnt && r[0] == first + 4 * (lane - lead) && r[1] == r[0] + 1 &&
                            r[2] == r[0] + 2 && r[3] == r[0] + 3;
        constexpr unsigned kBoxMask = kBoxLanes >= 32 ? 0xffffffffu : ((1u << kBoxLanes) - 1u);
        const bool boxed = ((__ballot_sync(0xffffffffu, in_run) >> lead) & kBoxMask) == kBoxMask;
        const uint32_t xbytes = (uint32_t)((cnt + 3) / 4) * 512u, wbytes = (uint32_t)e.rp * 128u;
        const uint8_t* a_src = p.pool.slab + e.offA;
        const uint8_t* b_src = p.pool.slab + e.offB;
        const int n_shrink = sp.kc1 - sp.kc0, n_all = n_shrink + sp.nc1 - sp.nc0;
        for (int j = 0; j < n_all; ++j, ++it) {
            if ((int)(it % kProducerWarps) != warp) continue;   // another copy warp's stage
            const uint32_t slot = it % p.n_stages;
            const uint32_t dst = sm.ring + slot * stage, bar = sm.full + slot * 8;
            const bool shrink = j < n_shrink;
            const int c = shrink ? sp.kc0 + j : nK + sp.nc0 + (j - n_shrink);   // stage number in the tile's whole sequence
            int ok = 1;
            if (lane == 0) {
                ok = mbar_wait(sm.empty + slot * 8, ((it / p.n_stages) & 1) ^ 1, sm.wait);
                if (ok) {
                    sm.armed[slot] = it + 1;
                    mbar_arrive_expect_tx(bar, wbytes + (shrink ? xbytes : 0u));
                    const uint8_t* w_src = shrink ? a_src + (size_t)c * wbytes : b_src + (size_t)(c - nK) * wbytes;
#ifdef PLORA_DEBUG
                    if (w_src < p.pool.slab || (uint64_t)(w_src - p.pool.slab) + wbytes > p.pool.slab_bytes) {
                        atomicCAS(p.status, 0, PLORA_ERR_DEBUG_CHECK);
                        w_src = p.pool.slab;   // the copy still runs, so that the stage's barrier completes
                    }
#endif
                    bulk_g2s(dst + kXStageBytes, w_src, wbytes, bar);
                }
            }
            if (!__shfl_sync(0xffffffffu, ok, 0)) return;
            if (shrink && active) {
                if (!boxed)
                    tma_gather4(dst + lane * 512, tm_x, c * kKC, r[0], r[1], r[2], r[3], bar);
                else if (lane == lead)
                    tma_box(dst + lane * 512, tm_box, c * kKC, first, bar);
            }
        }
    }
}

// ---- MMA warp, one lane --------------------------------------------------------------------
template <bool SPLIT>
__device__ __forceinline__ void mma_thread(const Params& p, const Smem& sm, uint32_t tmem, int n_tiles) {
    const int nK = (p.pool.d_in + kKC - 1) / kKC, nN = (p.pool.d_out + kKC - 1) / kKC;
    const Span sp = make_span<SPLIT>(nK, nN);
    const int stage = stage_bytes(p.R);
    uint32_t it = 0, d2 = 0, tile_idx = 0;
    const bool withhold = p.test_hook == PLORA_HOOK_WITHHOLD_RELEASE;   // test hook: shrink stages are never handed back
    for (int t = sp.t0; t < n_tiles; t += sp.t_step, ++tile_idx) {
        const WorkUnit wu = p.bk.sgmv_tiles[t];
        const int rp = p.pool.table[wu.adapter].rp;
        const int KP = rp < 16 ? 16 : rp;      // N of the shrink, K of the expand
        // shrink: D[128, KP] (tensor-memory columns [0, KP)) = sum over stages of X[128, 64] * W[KP, 64]^T
        const uint32_t idesc_s = instr_desc(KP, false, p.fp16 != 0);
        for (int kc = sp.kc0; kc < sp.kc1; ++kc, ++it) {
            const uint32_t slot = it % p.n_stages;
            if (!mbar_wait(sm.full + slot * 8, (it / p.n_stages) & 1, sm.wait)) return;
            tc_fence_after();
            const uint32_t xa = sm.ring + slot * stage, wa = xa + kXStageBytes;
#pragma unroll
            for (int k = 0; k < kKC / 16; ++k)   // 16 columns = 32 bytes further along the swizzled rows
                umma(tmem, smem_desc(xa + k * 32, 16, 1024, 2), smem_desc(wa + k * 32, 16, 1024, 2), idesc_s, kc > sp.kc0 || k > 0);
            if (!withhold) umma_commit(sm.empty + slot * 8);
        }
        umma_commit(sm.d_full);
        // expand: for every 64-column block, D2[128, 64] = (m_hi + m_lo)[128, KP] * B[KP, 64]
        if (!mbar_wait(sm.m_ready, tile_idx & 1, sm.wait)) return;
        tc_fence_after();
        const uint32_t idesc_e = instr_desc(kKC, true, p.fp16 != 0);
        for (int nc = sp.nc0; nc < sp.nc1; ++nc, ++it, ++d2) {
            const uint32_t slot = it % p.n_stages, b = d2 % kD2Bufs;
            if (!mbar_wait(sm.full + slot * 8, (it / p.n_stages) & 1, sm.wait)) return;
            if (!mbar_wait(sm.d2_empty + b * 8, ((d2 / kD2Bufs) & 1) ^ 1, sm.wait)) return;
            tc_fence_after();
            const uint32_t wa = sm.ring + slot * stage + kXStageBytes;
            const uint32_t dst = tmem + kTmemD2 + b * kKC;
            for (int k = 0; k < KP / 16; ++k) {
                // 16 rank rows of the sub-tile = two 8-row groups of 1024 bytes; 16 columns of m = two chunks of kRows * 16 bytes
                const uint64_t bd = smem_desc(wa + k * 2048, 1024, 1024, 2);
                umma(dst, smem_desc(sm.m_hi + k * (2 * kRows * 16), kRows * 16, 128, 0), bd, idesc_e, k > 0);
                umma(dst, smem_desc(sm.m_lo + k * (2 * kRows * 16), kRows * 16, 128, 0), bd, idesc_e, true);
            }
            umma_commit(sm.empty + slot * 8);
            umma_commit(sm.d2_full + b * 8);
        }
    }
}

// fp32 -> 16-bit hi + lo halves of the expand's left operand (bf16, or IEEE half when the inputs are)
__device__ __forceinline__ void split_hi_lo(float v, bool fp16, uint32_t& hi, uint32_t& lo) {
    if (fp16) {
        const __half hv = __float2half_rn(v);
        hi = __half_as_ushort(hv);
        lo = __half_as_ushort(__float2half_rn(v - __half2float(hv)));
    } else {
        hi = f32_to_bf16_bits(v);
        lo = f32_to_bf16_bits(v - __uint_as_float(hi << 16));
    }
}

// Bounded wait of the epilogue warps for a barrier other CTAs of the cluster arrive on (acquires what they wrote).
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, const WaitCtl& w) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait_cluster(bar, parity)) return true;
        if (*w.abort_flag) return false;
        if (clock64() - t0 > w.limit) break;
    }
    *w.abort_flag = 1;
    __threadfence_block();
    atomicCAS(w.status, 0, PLORA_ERR_TIMEOUT);
    return false;
}

// Split shape, between the two GEMMs: the cluster's eight partial m (one per slice of d_in) become one m in every CTA.
//   1. every CTA sends row r of its partial (fp32, from its tensor memory) to CTA r / kRedRows, which owns that row;
//   2. the owner adds the eight partials of each of its rows in the order of the CTAs' ranks (a fixed order: the result
//      is bit-reproducible), scales, splits into hi + lo and stores the 16-byte operand chunks into the m buffers of
//      all eight CTAs (its own among them, through the same path);
//   3. when all eight owners have delivered, m is complete here and the expand can start.
// Hand-overs are counted on two barriers per CTA, one arrival per CTA of the cluster each, made by one thread after the
// CTA's epilogue threads have met (their stores come before the meeting, the arrival after it, with release at cluster
// scope; the waiters acquire).  Returns false if a wait ran out (uniform over the warp).
__device__ __forceinline__ bool split_exchange(const Params& p, const Smem& sm, uint32_t lane_addr, const AdapterEntry& e,
                                               int KP, bool has_partial, int row, bool owner, int warp, int lane) {
    const unsigned full = 0xffffffffu;
    const uint32_t me = cluster_rank();
    const int e_tid = (warp - kFirstEpiWarp) * 32 + lane;   // 0 .. 127 among the epilogue threads
    // 1. partial rows to their owners
    const uint32_t dst_row = map_to_cta(sm.red + (uint32_t)((me * kRedRows + (row % kRedRows)) * p.R) * 4u, (uint32_t)(row / kRedRows));
    for (int c0 = 0; c0 < KP; c0 += 32) {
        uint32_t r[32];
        tmem_ld32(lane_addr + c0, r);
        tmem_ld_wait();
        if (owner) {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (c0 + 4 * j < KP) {
                    if (has_partial) st_cluster_v4(dst_row + (c0 + 4 * j) * 4, r[4 * j], r[4 * j + 1], r[4 * j + 2], r[4 * j + 3]);
                    else st_cluster_v4(dst_row + (c0 + 4 * j) * 4, 0u, 0u, 0u, 0u);   // this CTA had no columns of d_in
                }
            }
        }
    }
    tc_fence_before();
    fence_cluster();
    epi_barrier();
    if (e_tid < kClusterSize) mbar_arrive_remote(map_to_cta(sm.part_in, (uint32_t)e_tid));
    // 2. the rows this CTA owns.  (A warp whose wait ran out skips the work but still takes part in the meeting and in
    // the arrivals below: the four warps must reach the same CTA barriers, and the peers get their count.)
    const bool ok1 = __all_sync(full, mbar_wait_cluster(sm.part_in, 0, sm.wait));
    const int chunks_per_row = KP / 8;
    for (int ch = e_tid; ok1 && ch < kRedRows * chunks_per_row; ch += kEpiWarps * 32) {
        const int rl = ch / chunks_per_row, kc = ch - rl * chunks_per_row;
        float acc[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) acc[u] = 0.f;
#pragma unroll
        for (int src = 0; src < kClusterSize; ++src) {
            const uint32_t a = sm.red + (uint32_t)((src * kRedRows + rl) * p.R + kc * 8) * 4u;
            float4 v0, v1;
            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v0.x), "=f"(v0.y), "=f"(v0.z), "=f"(v0.w) : "r"(a));
            asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v1.x), "=f"(v1.y), "=f"(v1.z), "=f"(v1.w) : "r"(a + 16));
            acc[0] += v0.x; acc[1] += v0.y; acc[2] += v0.z; acc[3] += v0.w;
            acc[4] += v1.x; acc[5] += v1.y; acc[6] += v1.z; acc[7] += v1.w;
        }
        uint32_t hi[4], lo[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            uint32_t h2[2], l2[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int k = kc * 8 + 2 * j + u;
                split_hi_lo(k < e.rp ? acc[2 * j + u] * e.scale : 0.f, p.fp16 != 0, h2[u], l2[u]);
            }
            hi[j] = h2[0] | (h2[1] << 16);
            lo[j] = l2[0] | (l2[1] << 16);
        }
        const uint32_t off = (uint32_t)kc * (kRows * 16) + (uint32_t)(me * kRedRows + rl) * 16;
#pragma unroll
        for (int dst = 0; dst < kClusterSize; ++dst) {
            st_cluster_v4(map_to_cta(sm.m_hi + off, (uint32_t)dst), hi[0], hi[1], hi[2], hi[3]);
            st_cluster_v4(map_to_cta(sm.m_lo + off, (uint32_t)dst), lo[0], lo[1], lo[2], lo[3]);
        }
    }
    fence_cluster();
    epi_barrier();
    if (e_tid < kClusterSize) mbar_arrive_remote(map_to_cta(sm.m_in, (uint32_t)e_tid));
    // 3. everybody's rows are here
    const bool ok2 = __all_sync(full, mbar_wait_cluster(sm.m_in, 0, sm.wait));
    return ok1 && ok2;
}

// ---- the last four warps: epilogue -----------------------------------------------------------------------
// Thread (q, lane < 16) owns row 16 q + lane of the tile, q = warp % 4 being the quarter of the
// tensor memory lanes its warp may read (with M = 64 a quarter holds 16 rows in its first 16
// lanes; the other lanes of the warp take part in the loads and help in the write-out).  `alive` is kept uniform over the warp, and the two
// barriers per tile are executed whatever happens, so a wait that ran out cannot strand a thread.
template <bool SPLIT>
__device__ __forceinline__ void epilogue_warp(const Params& p, const Smem& sm, uint32_t tmem, int n_tiles, int warp,
                                              int lane) {
    const int nK = (p.pool.d_in + kKC - 1) / kKC, nN = (p.pool.d_out + kKC - 1) / kKC;
    const Span sp = make_span<SPLIT>(nK, nN);
    const int q = warp & 3, row = q * kRowsPerWarp + (lane & (kRowsPerWarp - 1));
    const bool owner = lane < kRowsPerWarp;
    const int grp = (warp - kFirstEpiWarp) >> 2;   // which group of four warps
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    const uint32_t stg = sm.staging + (warp - kFirstEpiWarp) * kRowsPerWarp * kStagePitch;
    const unsigned full = 0xffffffffu;
    uint32_t d2 = 0, tile_idx = 0;
    bool alive = true;
    for (int t = sp.t0; t < n_tiles; t += sp.t_step, ++tile_idx) {
        const WorkUnit wu = p.bk.sgmv_tiles[t];
        const AdapterEntry e = p.pool.table[wu.adapter];
        const int cnt = wu.cnt, KP = e.rp < 16 ? 16 : e.rp;
        epi_barrier();   // every epilogue thread is done with the previous tile's token indices
        if (owner) {
            sm.tok[row] = 0;
            PLORA_CHECKED((unsigned)(wu.pos0 + min(row, cnt - 1)) < (unsigned)p.n_tok, p.status)
            sm.tok[row] = p.bk.perm[wu.pos0 + min(row, cnt - 1)];
        }
        epi_barrier();
        if (alive) alive = __all_sync(full, mbar_wait(sm.d_full, tile_idx & 1, sm.wait));
        if (!alive) continue;
        tc_fence_after();
        if (SPLIT) {
            if (!split_exchange(p, sm, lane_addr, e, KP, sp.kc1 > sp.kc0, row, owner, warp, lane)) {
                alive = false;
                continue;
            }
        }
        // m = s * (x A), split into bf16 hi + lo; columns beyond the padded rank (rank 8 only) are zeros
        for (int c0 = 0; !SPLIT && c0 < KP; c0 += 32) {
            uint32_t r[32];
            tmem_ld32(lane_addr + c0, r);
            tmem_ld_wait();
#pragma unroll
            for (int kc = 0; kc < 4; ++kc) {
                if (owner && c0 + kc * 8 < KP && (kc % kEpiGroups) == grp) {   // the groups share the 8-column chunks
                    uint32_t hi[4], lo[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint32_t h2[2], l2[2];
#pragma unroll
                        for (int u = 0; u < 2; ++u) {
                            const int k = c0 + kc * 8 + 2 * j + u;
                            const float v = k < e.rp ? __uint_as_float(r[kc * 8 + 2 * j + u]) * e.scale : 0.f;
                            if (p.fp16) {
                                const __half hv = __float2half_rn(v);
                                h2[u] = __half_as_ushort(hv);
                                l2[u] = __half_as_ushort(__float2half_rn(v - __half2float(hv)));
                            } else {
                                h2[u] = f32_to_bf16_bits(v);
                                l2[u] = f32_to_bf16_bits(v - __uint_as_float(h2[u] << 16));
                            }
                        }
                        hi[j] = h2[0] | (h2[1] << 16);
                        lo[j] = l2[0] | (l2[1] << 16);
                    }
                    const uint32_t off = (uint32_t)(c0 / 8 + kc) * (kRows * 16) + row * 16;
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(sm.m_hi + off), "r"(hi[0]), "r"(hi[1]), "r"(hi[2]), "r"(hi[3]) : "memory");
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(sm.m_lo + off), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]), "r"(lo[3]) : "memory");
                }
            }
        }
        fence_async_smem();   // the MMAs read m through the asynchronous proxy
        tc_fence_before();
        mbar_arrive(sm.m_ready);
        // y += every 64-column block of the expand result
        for (int nc = sp.nc0; nc < sp.nc1; ++nc, ++d2) {
            const uint32_t b = d2 % kD2Bufs;
            if ((int)(d2 % kEpiGroups) != grp) continue;   // the other group's block
            // lane (h, c) handles the 16-byte piece c of rows 2i + h of its warp's 32 rows
            const int c = lane & 15, col = nc * kKC + c * 4;
            alive = __all_sync(full, mbar_wait(sm.d2_full + b * 8, (d2 / kD2Bufs) & 1, sm.wait));
            if (!alive) break;
            tc_fence_after();
            uint32_t r0[32], r1[32];
            tmem_ld32(lane_addr + kTmemD2 + b * kKC, r0);
            tmem_ld32(lane_addr + kTmemD2 + b * kKC + 32, r1);
            tmem_ld_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(sm.d2_empty + b * 8);
            // this thread's row goes to the staging buffer ...
            if (owner) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(stg + lane * kStagePitch + j * 16), "r"(r0[4 * j]), "r"(r0[4 * j + 1]), "r"(r0[4 * j + 2]), "r"(r0[4 * j + 3]) : "memory");
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(stg + lane * kStagePitch + 128 + j * 16), "r"(r1[4 * j]), "r"(r1[4 * j + 1]), "r"(r1[4 * j + 2]), "r"(r1[4 * j + 3]) : "memory");
                }
            }
            __syncwarp();
            // ... and leaves it two rows per instruction: 16 lanes cover the 256 bytes of a row piece
#pragma unroll
            for (int i = 0; i < kRowsPerWarp / 2; ++i) {
                const int rr = 2 * i + (lane >> 4), grow = q * kRowsPerWarp + rr;
                float4 v;
                asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(stg + rr * kStagePitch + c * 16));
                if (grow < cnt && col < p.pool.d_out) {
                    float* dst = p.y + (size_t)sm.tok[grow] * p.pool.d_out + col;
                    PLORA_CHECKED((unsigned)sm.tok[grow] < (unsigned)p.n_tok && col + 3 < p.pool.d_out, p.status)
                    red_add_v4(dst, v.x, v.y, v.z, v.w);
                }
            }
            __syncwarp();
        }
    }
}

template <bool SPLIT>
__global__ void __launch_bounds__(kThreads, 2)
sgmv_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_box, const Params p) {
    extern __shared__ uint8_t smem_raw[];
    // Launched with programmatic stream serialisation: nothing of the stream's earlier work is read
    // before this wait, unless the launch defers it (then the kernels it overlaps are those of its own
    // call, and everything older is complete because the first of them has waited).
    if (!p.defer_wait) asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // the bucket kernel says which launch shape its tiles are for; the other shape's launch finds none
    const int n_tiles = (*p.bk.sgmv_split != 0) == SPLIT ? *p.bk.n_sgmv_tiles : 0;
    // nothing for this CTA (often: no tensor-core segment in the batch); in the split shape a whole cluster leaves together
    if ((int)(SPLIT ? blockIdx.x / kClusterSize : blockIdx.x) >= n_tiles) {
        if (p.defer_wait && threadIdx.x == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
        return;
    }
    const Smem sm = carve(smem_raw, p, SPLIT);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(sm.full + s * 8, 1);
            mbar_init(sm.empty + s * 8, 1);
        }
        mbar_init(sm.d_full, 1);
        mbar_init(sm.m_ready, kEpiWarps * 32);
        for (int b = 0; b < kD2Bufs; ++b) {
            mbar_init(sm.d2_full + b * 8, 1);
            mbar_init(sm.d2_empty + b * 8, 4);   // one arrival per warp of the group that drains the block
        }
        mbar_init(sm.wind_down, 1);
        mbar_init(sm.part_in, kClusterSize);
        mbar_init(sm.m_in, kClusterSize);
        for (int s = 0; s < kMaxStages; ++s) sm.armed[s] = 0;
        *sm.wait.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // The weight area of every stage starts as zeros: a rank-8 sub-tile fills 8 of the 16 rows
    // the MMAs read, the others must hold finite values (zeros now, older weights later).
    for (int s = 0; s < p.n_stages; ++s)
        for (int i = tid * 16; i < w_stage_bytes(p.R); i += kThreads * 16)
            asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(sm.ring + s * stage_bytes(p.R) + kXStageBytes + i), "r"(0u) : "memory");
    fence_async_smem();
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(sm.tmem_slot)), "r"((uint32_t)kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *sm.tmem_slot;
    if (SPLIT) cluster_sync_all();   // every CTA's barriers are ready before a peer can arrive on them

    if (warp < kProducerWarps) {
        producer_warp<SPLIT>(p, sm, &tm_x, &tm_box, n_tiles, warp, lane);
    } else if (warp == kMmaWarp) {
        if (lane == 0) mma_thread<SPLIT>(p, sm, tmem, n_tiles);
    } else {
        epilogue_warp<SPLIT>(p, sm, tmem, n_tiles, warp, lane);
    }
    tc_fence_before();
    __syncthreads();
    if (*sm.wait.abort_flag) {
        // A wait ran out and every role has left its loop.  Before the tensor memory is freed and the CTA's
        // shared memory goes to another CTA, the MMAs issued so far must have completed and every copy asked
        // for must have landed (bounded waits again; they return at once unless something is truly stuck).
        if (warp == kMmaWarp && lane == 0) {
            umma_commit(sm.wind_down);
            if (!mbar_drain(sm.wind_down, 0, p.wait_cycles)) atomicCAS(p.status, 0, PLORA_ERR_TIMEOUT);
        }
        if (tid == 0)
            for (int s = 0; s < p.n_stages; ++s) {
                const uint32_t a = sm.armed[s];
                if (a && !mbar_drain(sm.full + s * 8, ((a - 1) / p.n_stages) & 1, p.wait_cycles))
                    atomicCAS(p.status, 0, PLORA_ERR_TIMEOUT);
            }
        __syncthreads();
    }
    // no CTA of the cluster gives up its shared memory while a peer may still store into it or arrive on its barriers
    if (SPLIT) cluster_sync_all();
    if (warp == kMmaWarp)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((uint32_t)kTmemCols) : "memory");
    if (p.defer_wait && tid == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess) f = nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

}  // namespace

cudaError_t sgmv_configure() {
    if (!encode_tiled()) return cudaErrorNotSupported;
    cudaError_t e = cudaFuncSetAttribute(sgmv_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(sgmv_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
}

cudaError_t launch_sgmv(const PoolDev& pool, const BucketDev& bk, int n_tok, int sgmv_min_rows, const void* x, float* y,
                        bool fp16, int32_t* status, int sm_count, bool after_bgmv_of_same_call, bool split,
                        int split_max_tiles, const DebugCfg& dbg, cudaStream_t stream, int* n_launches) {
    Params p;
    p.pool = pool;
    p.bk = bk;
    p.y = y;
    p.status = status;
    p.R = pool.max_rp < 16 ? 16 : pool.max_rp;
    p.n_stages = stages_for(p.R, split);
    p.defer_wait = after_bgmv_of_same_call ? 1 : 0;
    p.fp16 = fp16 ? 1 : 0;
    p.n_tok = n_tok;
    p.wait_cycles = dbg.wait_cycles > 0 ? dbg.wait_cycles : kWaitCycles;
    p.test_hook = dbg.test_hook;
    // x as a 2-D tensor [n_tok][d_in] of bf16; a gather instruction copies 64 columns of four rows,
    // 128-byte swizzled (columns beyond d_in read as zeros)
    CUtensorMap tm, tm_box;
    const cuuint64_t dims[2] = {(cuuint64_t)pool.d_in, (cuuint64_t)n_tok};
    const cuuint64_t strides[1] = {(cuuint64_t)pool.d_in * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kKC, 1};
    const cuuint32_t elem_strides[2] = {1, 1};
    if (encode_tiled()(&tm, (fp16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16), 2, const_cast<void*>(x), dims, strides, box, elem_strides,
                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    const cuuint32_t box_rows[2] = {(cuuint32_t)kKC, (cuuint32_t)kBoxRows};
    if (encode_tiled()(&tm_box, (fp16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16), 2, const_cast<void*>(x), dims, strides, box_rows,
                       elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                       CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return cudaErrorInvalidValue;
    // every tensor-core segment has at least sgmv_min_rows tokens: at most this many tiles
    const int min_rows = sgmv_min_rows < 1 ? 1 : sgmv_min_rows;
    long long max_tiles = (long long)n_tok / kRows + (long long)n_tok / min_rows + 1;
    int grid = 2 * sm_count;   // two CTAs per SM, half of its tensor memory each
    if (grid > max_tiles) grid = (int)max_tiles;
    if (grid < 1) grid = 1;
    // split shape: one cluster per tile the batch can have at most (the host does not know the count; clusters
    // beyond it leave at once)
    // (split_max_tiles: the bucket kernel sends at most that many tiles to this shape)
    if (split) {
        if (max_tiles > split_max_tiles) max_tiles = split_max_tiles;
        grid = (int)(max_tiles < 1 ? 1 : max_tiles) * kClusterSize;
    }
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = kClusterSize;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem_bytes(p.R, split);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = split ? 2 : 1;
    const cudaError_t e = split ? cudaLaunchKernelEx(&cfg, sgmv_kernel<true>, tm, tm_box, p)
                                : cudaLaunchKernelEx(&cfg, sgmv_kernel<false>, tm, tm_box, p);
    ++*n_launches;
    return e;
}

}  // namespace plora
