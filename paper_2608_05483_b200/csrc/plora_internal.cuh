// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "plora.h"

namespace plora {

// ---------------------------------------------------------------------------------
// Slab layout (private).  Per adapter, A is stored transposed as rp rows (one per
// rank index k, rp = rank padded to a power of two >= 8, zero rows beyond r) of d_in
// values; B as rp rows of d_out values.  Each is cut along the long dimension into
// tiles of TILE_COLS(rp) columns; a tile is nsub sub-tiles of [rp rows][64 columns]
// (128-byte rows), sub-tiles back to back, and inside a sub-tile the 16-byte chunk c
// of row k sits at chunk position c ^ (k & 7).  A tile is therefore one contiguous
// block of rp * TILE_COLS * 2 bytes (16 KiB, 8 KiB for rp = 8): one bulk copy brings
// it into shared memory, lanes that read one chunk per row at consecutive rows, or
// consecutive chunks of one row, touch distinct banks, and a [rp][64] sub-tile has
// the row pitch and chunk permutation of the tensor core's 128-byte-swizzled operand.
// Columns beyond d_in / d_out in the last tile are zero.
// ---------------------------------------------------------------------------------
constexpr int kMaxRank = 128;
constexpr int kSubCols = 64;                 // columns of one sub-tile (128 bytes of bf16)
constexpr int kMaxSubPerTile = 8;            // at most 512 columns per tile
constexpr int kTileBytesMax = 16384;

__host__ __device__ inline int pad_rank(int r) {
    int rp = 8;
    while (rp < r) rp <<= 1;
    return rp;
}
__host__ __device__ inline int subs_per_tile(int rp) {
    int n = kMaxRank / rp;
    return n > kMaxSubPerTile ? kMaxSubPerTile : n;
}
__host__ __device__ inline int tile_cols(int rp) { return subs_per_tile(rp) * kSubCols; }
__host__ __device__ inline int tile_bytes(int rp) { return rp * tile_cols(rp) * 2; }
__host__ __device__ inline int tiles_for(int d, int rp) { return (d + tile_cols(rp) - 1) / tile_cols(rp); }

// One row of the per-pool offset table (device resident).
struct AdapterEntry {
    uint64_t offA;   // byte offset of the adapter's A tiles in the slab
    uint64_t offB;   // byte offset of its B tiles
    int32_t r;       // rank
    int32_t rp;      // padded rank
    float scale;     // s_a
    int32_t pad_;
};
static_assert(sizeof(AdapterEntry) == 32, "table row is 32 bytes");

// Debug build (-DPLORA_DEBUG): every address a kernel forms from a table, a work unit or a token index is
// checked against the buffer it belongs to before it is used; a failed check records PLORA_ERR_DEBUG_CHECK in
// the status word and skips the access (nothing traps, the kernel runs on).  The checks stand in for a memory
// checker on machines where none can be run.  In the ordinary build the macro disappears.
//   PLORA_CHECKED(cond, status) statement;
#ifdef PLORA_DEBUG
#define PLORA_CHECKED(cond, status) \
    if (!(cond)) atomicCAS((status), 0, PLORA_ERR_DEBUG_CHECK); \
    else
#else
#define PLORA_CHECKED(cond, status)
#endif

struct PoolDev {
    const uint8_t* slab;
    uint64_t slab_bytes;  // size of the slab (the debug build checks tile addresses against it)
    const AdapterEntry* table;
    int32_t d_in, d_out, n_adapters, max_rp;
    int32_t rp_mask;      // OR of the padded ranks present in the pool (each a power of two, 8..128)
    int32_t min_rp;
};

// ---------------------------------------------------------------------------------
// Bucket (device resident, owned by the context).
// ---------------------------------------------------------------------------------
constexpr int kTokChunk = 4;      // tokens of one segment a BGMV work unit handles
constexpr int kSgmvRows = 64;     // rows of one SGMV tile (M of the tensor-core instruction)

struct WorkUnit {   // 32 bytes
    int32_t adapter;
    int32_t pos0;   // first position in perm
    int32_t cnt;    // tokens (<= kTokChunk for BGMV, <= kSgmvRows for SGMV)
    int32_t seg;
    int32_t tok[kTokChunk];   // the first min(cnt, kTokChunk) token indices, perm[pos0 ...]
};
static_assert(sizeof(WorkUnit) == 32 && kTokChunk == 4, "work unit is two 16-byte words");

constexpr int kMaxRuns = 8;       // a unit's expand is cut into at most this many tasks
constexpr int kMaxRunsA = 4;      // ... and its shrink into at most this many

struct BucketDev {
    int32_t* perm;
    int32_t* seg_adapter;
    int32_t* seg_start;
    int32_t* n_seg;
    int32_t* n_active;
    WorkUnit* bgmv_units;
    int32_t* n_bgmv_units;
    WorkUnit* sgmv_tiles;
    int32_t* n_sgmv_tiles;
    int32_t* sgmv_split;    // 1: the tiles are few and go to the split launch shape (a cluster per tile), 0: to the wide one
    // cross-CTA hand-over of the fused BGMV kernel: every partial m value travels as one
    // 64-bit word {value, launch epoch}, so a reader can tell on its own whether it has arrived
    unsigned long long* m_part;
    size_t m_part_bytes;
    uint32_t* epoch;        // launch epoch, advanced by the last CTA of every fused launch (starts at 1)
    uint32_t* exit_count;   // CTAs of the running launch that have finished
    // pools of mixed ranks: the (projection, unit) pairs of a call sorted by padded-rank class, so
    // that the launch of a class walks only its own units (written by the classify pass)
    int32_t* cls_list;      // room for kMaxGroupPools * max_tokens entries; a sort fills n_units of them (unit numbers), the second sort starts n_tok entries in
    int32_t* cls_start;     // kRankClasses + 1 offsets into cls_list (the second sort's: 8 words further on)
};
constexpr int kRankClasses = 5;   // padded ranks 8, 16, 32, 64, 128

// Launchers (each returns the cudaError_t of its launch).
// sgmv_min_tiles: from this many tensor-core tiles on they go to the wide launch shape; fewer go to the split
// shape if split_ok, else their segments stay with BGMV
cudaError_t launch_bucket(const int32_t* ids, int n_tok, int n_adapters, int sgmv_min_rows, int sgmv_min_tiles,
                          bool split_ok, BucketDev bk, int32_t* status, cudaStream_t stream, int* n_launches);
cudaError_t launch_repack(const AdapterEntry* table_dev, const void* const* A_dev, const void* const* B_dev,
                          int n_adapters, int d_in, int d_out, uint8_t* slab, cudaStream_t stream, int* n_launches);

enum BgmvMode { kFused = 0, kShrinkOnly = 1, kExpandOnly = 2 };
// x: bf16 [n_tok, d_in]; y: fp32 [n_tok, d_out] (accumulated); m: fp32 [n_tok, ldm]
// pools[0 .. n_groups): projections of one launch (same shape; more than one only in fused mode);
// x / y: per-projection pointers (x unused by the expand-only mode, y by the shrink-only mode)
constexpr int kMaxGroupPools = 4;
// m / ldm / m16: the caller's m of the shrink-only and expand-only modes, fp32 or (m16) bf16 values
// fp16: x, A and B hold IEEE half values instead of bf16
// cls_cache: which pools' ranks the bucket's units are currently sorted by (pools of mixed ranks).  The
// sort is a kernel of its own; an adapter usually has one rank in every layer and projection, so the
// calls of a step share one sort.  The owner resets it whenever the bucket is rebuilt.  The pools of a
// group must have the same ranks if they hold more than one rank class.  rank_sig: a hash of the
// padded ranks of the call's pools (host side only).
// Two sorts are kept side by side: [0] the class lists in bucket order (one launch per class), [1] ordered by token
// count inside a class as well (one launch for all classes); a step whose calls use both kinds sorts twice, not per call.
struct ClassCache {
    uint64_t sig[2] = {0, 0};
    bool valid[2] = {false, false};
    void reset() { valid[0] = valid[1] = false; }
};
// Per-launch settings that come from the context: the diagnostics of the bounded waits
// (plora_set_wait_limit, plora_set_test_hook) and what the host knows about the batch.
struct DebugCfg {
    long long wait_cycles = 0;   // 0: the kernels' default
    int32_t test_hook = 0;       // PLORA_HOOK_*
    bool maybe_empty = false;    // the bucket may hold tensor-core segments only (BGMV launches look before they set up)
    bool inputs_resident = false;   // plora_set_inputs_resident: x of a call was complete before the previous kernel of the stream began
};
// between: a launch the caller wants between the classify pass (if one is needed) and the BGMV launches, nullptr for
// none: the split tensor-core launch of the same call, which works on other tokens.  It joins the stream's order (the
// BGMV launches behind it then need not), and its CTAs, one per SM for a few tens of microseconds, overlap the BGMV
// launches instead of trailing them.  It gets its argument and the launch counter and returns its launch's error.
typedef cudaError_t (*BetweenLaunch)(void* arg, int* n_launches);
cudaError_t launch_bgmv(BgmvMode mode, const PoolDev* pools, int n_groups, const BucketDev& bk, int n_tok,
                        const void* const* x, float* const* y, void* m, int ldm, bool m16, bool fp16, int32_t* status,
                        int sm_count, bool early_tables, ClassCache* cls_cache, uint64_t rank_sig, const DebugCfg& dbg,
                        cudaStream_t stream, int* n_launches, BetweenLaunch between = nullptr, void* between_arg = nullptr);
// The fused BGMV kernel of padded rank rp (0: all classes) whose consumers put off joining the stream order.
const void* bgmv_lazy_kernel(int rp, bool fp16);
// after_bgmv_of_same_call: the launch follows fused BGMV launches of the same call (other tokens of the
// same batch) and may overlap them
cudaError_t launch_sgmv(const PoolDev& pool, const BucketDev& bk, int n_tok, int sgmv_min_rows, const void* x, float* y,
                        bool fp16, int32_t* status, int sm_count, bool after_bgmv_of_same_call, bool split,
                        int split_max_tiles, const DebugCfg& dbg, cudaStream_t stream, int* n_launches);
// per-device function attributes (dynamic shared memory); called by plora_create
cudaError_t bucket_configure();
cudaError_t bgmv_configure();
cudaError_t sgmv_configure();
cudaError_t bgmv_configure_lazy();   // after the others: see bgmv_lazy_kernel
int bucket_max_adapters();      // largest pool the single-CTA bucketing kernel handles

}  // namespace plora
