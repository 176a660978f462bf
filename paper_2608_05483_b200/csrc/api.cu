// C ABI of the library (declared in plora.h): context, adapter-pool registry,
// bucketing and the delta entry points.  Host code only; the kernels live in
// bucket.cu, registry.cu, bgmv.cu and sgmv.cu.
#include <climits>
#include <cstdlib>
#include <cstring>
#include <new>
#include <unordered_map>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "plora_internal.cuh"

using namespace plora;

namespace {
// A named range around every entry point that enqueues work, for timelines (Nsight Systems and the like).  Off
// unless the environment has PLORA_NVTX=1 when the library is first used; without a tool attached a range is a
// call into a stub.
struct ApiRange {
    bool on;
    static bool enabled() {
        static const bool v = [] {
            const char* e = std::getenv("PLORA_NVTX");
            return e && e[0] == '1';
        }();
        return v;
    }
    explicit ApiRange(const char* name) : on(enabled()) {
        if (on) nvtxRangePushA(name);
    }
    ~ApiRange() {
        if (on) nvtxRangePop();
    }
};
}  // namespace

namespace {

struct PoolRec {
    int32_t layer, proj;
    PoolDev dev;
    AdapterEntry* table_dev;
    uint64_t rank_sig;   // hash of the adapters' padded ranks: pools with the same value sort a batch's units alike
};

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
        if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
        if (prev == dev) prev = -1;
    }
    ~DeviceGuard() {
        if (prev >= 0) cudaSetDevice(prev);
    }
};

constexpr int kDefaultSgmvMinRows = 32;   // AUTO: segments at least this long take the tensor-core path ...
// ... in batches at least this large (a decode batch stays one launch).  The host cannot know whether a batch has such
// a segment, and a tensor-core launch that finds none still takes its place in the stream's chain of launches (2 to
// 4 us each): measured on 512 uniformly tagged tokens (the 13B decode workload) it cost 2.5 % of the step.
constexpr int kSgmvMinBatch = 1024;
// ... and only if they make at least this many 64-row tiles together: a tile is one CTA's serial chain
// over the whole width (with 8 tiles allowed, the mixed batch of config 5 took 0.52 ms instead of 0.34)
constexpr int kSgmvMinTiles = 128;

}  // namespace

struct plora_ctx {
    int device = 0;
    int32_t max_tokens = 0, max_adapters = 0;
    int sm_count = 0;
    // bucket
    void* bucket_block = nullptr;
    BucketDev bk{};
    int32_t* status_dev = nullptr;
    const int32_t* cur_ids = nullptr;
    int32_t cur_ntok = -1, cur_nadapters = -1;
    bool bucket_valid = false;
    // Who made the current bucket.  plora_bucket makes an explicit one: the caller vouches that the ids
    // buffer keeps its contents until the next plora_bucket, so every later call with that buffer reuses
    // it.  A delta call that finds no such bucket makes an implicit one, good for that call alone: the
    // library cannot know whether the caller rewrote the buffer (or the allocator handed the address to
    // a new tensor) before the next call.
    bool bucket_explicit = false;
    uint64_t call_gen = 0;     // one per entry into the library through a delta entry point
    uint64_t bucket_gen = 0;   // the call that made the implicit bucket
    int32_t path = PLORA_PATH_AUTO;
    int32_t sgmv_min_rows = kDefaultSgmvMinRows;
    int32_t bucket_sgmv_min = INT_MAX;   // threshold the current bucket was built with
    // workspace for the unfused path's m
    float* m_ws = nullptr;
    // staging for the host-buffer entry points: a ring of sets, so that one call's copy back to the
    // host, the next call's kernels and the call after that's copy to the device run at the same time
    struct HostStage {
        void* x = nullptr;
        int32_t* ids = nullptr;
        float* y[kMaxGroupPools] = {};
        size_t x_bytes = 0, y_bytes[kMaxGroupPools] = {};
        cudaEvent_t up = nullptr, done = nullptr, freed = nullptr;
        bool in_flight = false;
    };
    static constexpr int kHostStages = 4;
    HostStage stage[kHostStages];
    cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
    int next_stage = 0;
    std::vector<PoolRec> pools;
    std::unordered_map<uint64_t, size_t> pool_index;   // (layer, proj) -> position in pools
    int64_t launches = 0;
    // kernels launched through this context since the bucket kernel: from the second one on, the
    // bucket tables were complete before the kernel preceding it in the stream started
    int32_t launches_since_bucket = 0;
    ClassCache cls_cache;   // the bucket's units are sorted by the rank classes of pools with this signature
    bool fp16 = false;   // x, A and B are IEEE half instead of bf16
    DebugCfg dbg;        // wait limit and test hook of the kernels' bounded waits
};

namespace {

inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }

inline uint64_t pool_key(int32_t layer, int32_t proj) { return ((uint64_t)(uint32_t)layer << 32) | (uint32_t)proj; }

PoolRec* find_pool(plora_ctx* ctx, int32_t layer, int32_t proj) {
    const auto it = ctx->pool_index.find(pool_key(layer, proj));
    return it == ctx->pool_index.end() ? nullptr : &ctx->pools[it->second];
}

bool desc_shape_ok(const plora_pool_desc* d, plora_status* why) {
    if (!d || !d->ranks || d->n_adapters < 1 || d->d_in < 1 || d->d_out < 1) { *why = PLORA_ERR_INVALID_ARG; return false; }
    if ((d->d_in & 7) || (d->d_out & 7)) { *why = PLORA_ERR_UNSUPPORTED; return false; }
    for (int a = 0; a < d->n_adapters; ++a) {
        if (d->ranks[a] < 1) { *why = PLORA_ERR_INVALID_ARG; return false; }
        if (d->ranks[a] > kMaxRank) { *why = PLORA_ERR_UNSUPPORTED; return false; }
    }
    return true;
}

// Fills the offset table (host copy) and returns the slab size.
size_t layout_pool(const plora_pool_desc* d, std::vector<AdapterEntry>* table, int* max_rp, int* rp_mask = nullptr,
                   int* min_rp = nullptr) {
    size_t off = 0;
    int mrp = 0, mask = 0, lrp = kMaxRank;
    if (table) table->resize(d->n_adapters);
    for (int a = 0; a < d->n_adapters; ++a) {
        const int rp = pad_rank(d->ranks[a]);
        const size_t tb = (size_t)tile_bytes(rp);
        AdapterEntry e{};
        e.offA = off;
        off += tb * tiles_for(d->d_in, rp);
        e.offB = off;
        off += tb * tiles_for(d->d_out, rp);
        e.r = d->ranks[a];
        e.rp = rp;
        e.scale = d->scales ? d->scales[a] : 1.0f;
        if (table) (*table)[a] = e;
        if (rp > mrp) mrp = rp;
        if (rp < lrp) lrp = rp;
        mask |= rp;
    }
    if (max_rp) *max_rp = mrp;
    if (rp_mask) *rp_mask = mask;
    if (min_rp) *min_rp = lrp;
    return off;
}

int32_t effective_sgmv_min(const plora_ctx* ctx, int32_t n_tok) {
    switch (ctx->path) {
        case PLORA_PATH_SGMV:
        case PLORA_PATH_SGMV_SPLIT: return 1;
        case PLORA_PATH_AUTO: return n_tok >= kSgmvMinBatch ? ctx->sgmv_min_rows : INT_MAX;
        default: return INT_MAX;
    }
}

// Which tensor-core launches a call makes.  The wide shape needs kSgmvMinTiles tiles, which hold at least
// kSgmvMinTiles * sgmv_min_rows tokens: a smaller batch cannot reach it and is spared the launch that would find
// no tile.  The host does not know how many tiles a batch has; of the two launches of a large batch one finds none.
bool wide_launch(const plora_ctx* ctx, int32_t n_tok) {
    if (ctx->path == PLORA_PATH_SGMV) return true;
    return ctx->path == PLORA_PATH_AUTO && ctx->bucket_sgmv_min != INT_MAX &&
           (long long)n_tok >= (long long)kSgmvMinTiles * ctx->bucket_sgmv_min;
}
// under AUTO the bucket kernel sends kSgmvMinTiles tiles or more to the wide shape
int split_max_tiles(const plora_ctx* ctx) { return ctx->path == PLORA_PATH_AUTO ? kSgmvMinTiles - 1 : INT_MAX; }
// AUTO: the split shape serves the batches that are too small for the wide one.  (Launching both for a large batch
// and letting the bucket kernel's tile count decide cost the prefill step 5 %: a launch of up to 127 clusters that
// all find nothing still takes 6 us.  A large batch whose long segments make fewer than kSgmvMinTiles tiles keeps
// them on BGMV.)
bool split_launch(const plora_ctx* ctx, int32_t n_tok) {
    return ctx->path == PLORA_PATH_SGMV_SPLIT ||
           (ctx->path == PLORA_PATH_AUTO && ctx->bucket_sgmv_min != INT_MAX && !wide_launch(ctx, n_tok));
}

plora_status do_bucket(plora_ctx* ctx, const int32_t* ids, int32_t n_tok, int32_t n_adapters, cudaStream_t st,
                       bool is_explicit) {
    const int32_t thr = effective_sgmv_min(ctx, n_tok);
    int nl = 0;
    const int min_tiles = ctx->path == PLORA_PATH_AUTO ? kSgmvMinTiles : ctx->path == PLORA_PATH_SGMV_SPLIT ? INT_MAX : 0;
    const bool split_ok = ctx->path == PLORA_PATH_SGMV_SPLIT ||
                          (ctx->path == PLORA_PATH_AUTO && thr != INT_MAX && (long long)n_tok < (long long)kSgmvMinTiles * thr);
    cudaError_t e = launch_bucket(ids, n_tok, n_adapters, thr, min_tiles, split_ok, ctx->bk, ctx->status_dev, st, &nl);
    ctx->launches += nl;
    if (e != cudaSuccess) { ctx->bucket_valid = false; return PLORA_ERR_CUDA; }
    ctx->cur_ids = ids;
    ctx->cur_ntok = n_tok;
    ctx->cur_nadapters = n_adapters;
    ctx->bucket_sgmv_min = thr;
    // every segment may have gone to the tensor-core path (a prefill batch): the BGMV launches then look before they
    // set up; a smaller batch always keeps short segments, and is spared the look
    ctx->dbg.maybe_empty = thr != INT_MAX && (long long)n_tok >= (long long)kSgmvMinTiles * thr;
    ctx->bucket_valid = true;
    ctx->bucket_explicit = is_explicit;
    ctx->bucket_gen = ctx->call_gen;
    ctx->launches_since_bucket = 0;
    ctx->cls_cache.reset();
    return PLORA_OK;
}

plora_status ensure_bucket(plora_ctx* ctx, const int32_t* ids, int32_t n_tok, int32_t n_adapters, cudaStream_t st) {
    // an explicit bucket serves every call that names its ids; an implicit one only the call that made it
    if (ctx->bucket_valid && (ctx->bucket_explicit || ctx->bucket_gen == ctx->call_gen) && ctx->cur_ids == ids &&
        ctx->cur_ntok == n_tok && ctx->cur_nadapters == n_adapters && ctx->bucket_sgmv_min == effective_sgmv_min(ctx, n_tok))
        return PLORA_OK;
    return do_bucket(ctx, ids, n_tok, n_adapters, st, false);
}

cudaError_t launch_bgmv_one(BgmvMode mode, const PoolDev& pool, const BucketDev& bk, int n_tok, const void* x, float* y,
                            void* m, int ldm, int32_t* status, int sm_count, bool early_tables, ClassCache* cls_cache,
                            uint64_t rank_sig, cudaStream_t stream, int* n_launches, bool m16, bool fp16,
                            const DebugCfg& dbg) {
    const void* xs[1] = {x};
    float* ys[1] = {y};
    return launch_bgmv(mode, &pool, 1, bk, n_tok, xs, ys, m, ldm, m16, fp16, status, sm_count, early_tables, cls_cache,
                       rank_sig, dbg, stream, n_launches);
}

plora_status check_call(plora_ctx* ctx, const void* a, const void* ids, int32_t n_tok, const void* b) {
    if (!ctx || n_tok < 0 || n_tok > ctx->max_tokens) return PLORA_ERR_INVALID_ARG;
    if (n_tok > 0 && (!a || !ids || !b)) return PLORA_ERR_INVALID_ARG;
    if (((uintptr_t)a & 15) || ((uintptr_t)b & 15) || ((uintptr_t)ids & 3)) return PLORA_ERR_INVALID_ARG;
    return PLORA_OK;
}

}  // namespace

extern "C" {

PLORA_API const char* plora_status_string(plora_status s) {
    switch (s) {
        case PLORA_OK: return "ok";
        case PLORA_ERR_INVALID_ARG: return "invalid argument";
        case PLORA_ERR_NOT_REGISTERED: return "no pool registered for (layer, proj)";
        case PLORA_ERR_BAD_ADAPTER_ID: return "adapter id out of range";
        case PLORA_ERR_WORKSPACE: return "slab or workspace too small";
        case PLORA_ERR_CUDA: return "CUDA runtime error";
        case PLORA_ERR_TIMEOUT: return "bounded device wait ran out";
        case PLORA_ERR_UNSUPPORTED: return "unsupported shape";
        case PLORA_ERR_DEBUG_CHECK: return "debug build: an out-of-bounds access was caught and skipped";
        default: return "unknown status";
    }
}

PLORA_API plora_status plora_create(plora_ctx** out, int device, int32_t max_tokens, int32_t max_adapters) {
    if (!out || max_tokens < 1 || max_adapters < 1) return PLORA_ERR_INVALID_ARG;
    if (max_adapters > bucket_max_adapters()) return PLORA_ERR_UNSUPPORTED;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess) return PLORA_ERR_CUDA;
    if (device < 0 || device >= n_dev) return PLORA_ERR_INVALID_ARG;
    DeviceGuard g(device);
    if (!g.ok) return PLORA_ERR_CUDA;
    plora_ctx* ctx = new (std::nothrow) plora_ctx();
    if (!ctx) return PLORA_ERR_WORKSPACE;
    ctx->device = device;
    ctx->max_tokens = max_tokens;
    ctx->max_adapters = max_adapters;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) { delete ctx; return PLORA_ERR_CUDA; }
    ctx->sm_count = prop.multiProcessorCount;
    if (prop.major < 10) { delete ctx; return PLORA_ERR_UNSUPPORTED; }

    const size_t T = (size_t)max_tokens;
    const size_t cap = T < (size_t)max_adapters ? T : (size_t)max_adapters;
    auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
    const size_t o_perm = 0;
    const size_t o_sega = o_perm + up(T * 4);
    const size_t o_segs = o_sega + up((cap + 1) * 4);
    const size_t o_scal = o_segs + up((cap + 2) * 4);
    const size_t o_bg = o_scal + 256;
    const size_t o_sg = o_bg + up(T * sizeof(WorkUnit));
    const size_t o_m = o_sg + up(T * sizeof(WorkUnit));
    const size_t o_part = o_m + up(T * kMaxRank * 4);
    // partial-m hand-over of the fused kernel: one 64-bit word per (projection of a grouped call, token,
    // shrink run, rank row)
    const size_t part_need = T * kMaxGroupPools * kMaxRunsA * kMaxRank * sizeof(unsigned long long);
    const size_t part_bytes = up(part_need > ((size_t)16 << 20) ? part_need : ((size_t)16 << 20));
    const size_t o_cls = o_part + part_bytes;
    const size_t total = o_cls + up(T * kMaxGroupPools * 4);
    uint8_t* blk = nullptr;
    if (cudaMalloc(&blk, total) != cudaSuccess) { delete ctx; return PLORA_ERR_WORKSPACE; }
    if (cudaMemset(blk, 0, total) != cudaSuccess) { cudaFree(blk); delete ctx; return PLORA_ERR_CUDA; }
    ctx->bucket_block = blk;
    ctx->bk.perm = (int32_t*)(blk + o_perm);
    ctx->bk.seg_adapter = (int32_t*)(blk + o_sega);
    ctx->bk.seg_start = (int32_t*)(blk + o_segs);
    int32_t* scal = (int32_t*)(blk + o_scal);
    ctx->bk.n_seg = scal + 0;
    ctx->bk.n_active = scal + 1;
    ctx->bk.n_bgmv_units = scal + 2;
    ctx->bk.n_sgmv_tiles = scal + 3;
    ctx->bk.sgmv_split = scal + 4;
    ctx->status_dev = scal + 8;
    ctx->bk.bgmv_units = (WorkUnit*)(blk + o_bg);
    ctx->bk.sgmv_tiles = (WorkUnit*)(blk + o_sg);
    ctx->m_ws = (float*)(blk + o_m);
    ctx->bk.m_part = (unsigned long long*)(blk + o_part);
    ctx->bk.m_part_bytes = part_bytes;
    ctx->bk.epoch = (uint32_t*)(scal + 16);
    ctx->bk.exit_count = (uint32_t*)(scal + 17);
    ctx->bk.cls_start = scal + 24;
    ctx->bk.cls_list = (int32_t*)(blk + o_cls);
    {
        const uint32_t one = 1;
        if (cudaMemcpy(ctx->bk.epoch, &one, 4, cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaFree(blk);
            delete ctx;
            return PLORA_ERR_CUDA;
        }
    }
    if (bucket_configure() != cudaSuccess || bgmv_configure() != cudaSuccess || sgmv_configure() != cudaSuccess || bgmv_configure_lazy() != cudaSuccess ||
        cudaDeviceSynchronize() != cudaSuccess) {
        cudaFree(blk);
        delete ctx;
        return PLORA_ERR_CUDA;
    }
    *out = ctx;
    return PLORA_OK;
}

PLORA_API plora_status plora_destroy(plora_ctx* ctx) {
    if (!ctx) return PLORA_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    cudaDeviceSynchronize();
    for (auto& p : ctx->pools) cudaFree(p.table_dev);
    cudaFree(ctx->bucket_block);
    for (auto& hs : ctx->stage) {
        cudaFree(hs.x);
        cudaFree(hs.ids);
        for (float* y : hs.y) cudaFree(y);
        if (hs.up) cudaEventDestroy(hs.up);
        if (hs.done) cudaEventDestroy(hs.done);
        if (hs.freed) cudaEventDestroy(hs.freed);
    }
    if (ctx->h2d_stream) cudaStreamDestroy(ctx->h2d_stream);
    if (ctx->d2h_stream) cudaStreamDestroy(ctx->d2h_stream);
    delete ctx;
    return PLORA_OK;
}

PLORA_API size_t plora_pool_slab_bytes(const plora_pool_desc* desc) {
    plora_status why;
    if (!desc_shape_ok(desc, &why)) return 0;
    return layout_pool(desc, nullptr, nullptr);
}

PLORA_API plora_status plora_register_pool(plora_ctx* ctx, const plora_pool_desc* d, void* slab_dev, size_t slab_bytes,
                                 void* stream) {
    ApiRange nvtx_range("plora_register_pool");
    if (!ctx || !d || !slab_dev || !d->A || !d->B) return PLORA_ERR_INVALID_ARG;
    plora_status why;
    if (!desc_shape_ok(d, &why)) return why;
    if (d->n_adapters > ctx->max_adapters) return PLORA_ERR_WORKSPACE;
    if ((uintptr_t)slab_dev & 255) return PLORA_ERR_INVALID_ARG;
    for (int a = 0; a < d->n_adapters; ++a)
        if (!d->A[a] || !d->B[a]) return PLORA_ERR_INVALID_ARG;
    std::vector<AdapterEntry> table;
    int max_rp = 0, rp_mask = 0, min_rp = 0;
    const size_t need = layout_pool(d, &table, &max_rp, &rp_mask, &min_rp);
    if (slab_bytes < need) return PLORA_ERR_WORKSPACE;

    DeviceGuard g(ctx->device);
    if (!g.ok) return PLORA_ERR_CUDA;
    cudaStream_t st = as_stream(stream);
    const int N = d->n_adapters;
    AdapterEntry* table_dev = nullptr;
    const void** ptrs_dev = nullptr;   // [2N]: A pointers then B pointers
    uint8_t* staging = nullptr;
    plora_status rc = PLORA_OK;
    std::vector<const void*> ptrs(2 * (size_t)N);
    do {
        if (cudaMalloc(&table_dev, sizeof(AdapterEntry) * N) != cudaSuccess ||
            cudaMalloc(&ptrs_dev, sizeof(void*) * 2 * N) != cudaSuccess) { rc = PLORA_ERR_WORKSPACE; break; }
        if (d->ab_on_device) {
            for (int a = 0; a < N; ++a) { ptrs[a] = d->A[a]; ptrs[N + a] = d->B[a]; }
        } else {
            // stage the logical matrices on the device, then repack from there
            size_t bytes = 0;
            for (int a = 0; a < N; ++a) bytes += ((size_t)d->ranks[a] * (d->d_in + d->d_out) * 2 + 15) & ~(size_t)15;
            if (cudaMalloc(&staging, bytes) != cudaSuccess) { rc = PLORA_ERR_WORKSPACE; break; }
            size_t off = 0;
            bool bad = false;
            for (int a = 0; a < N && !bad; ++a) {
                const size_t ba = (size_t)d->ranks[a] * d->d_in * 2, bb = (size_t)d->ranks[a] * d->d_out * 2;
                bad |= cudaMemcpyAsync(staging + off, d->A[a], ba, cudaMemcpyHostToDevice, st) != cudaSuccess;
                ptrs[a] = staging + off;
                bad |= cudaMemcpyAsync(staging + off + ba, d->B[a], bb, cudaMemcpyHostToDevice, st) != cudaSuccess;
                ptrs[N + a] = staging + off + ba;
                off += (ba + bb + 15) & ~(size_t)15;
            }
            if (bad) { rc = PLORA_ERR_CUDA; break; }
        }
        if (cudaMemcpyAsync(table_dev, table.data(), sizeof(AdapterEntry) * N, cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(ptrs_dev, ptrs.data(), sizeof(void*) * 2 * N, cudaMemcpyHostToDevice, st) != cudaSuccess) {
            rc = PLORA_ERR_CUDA;
            break;
        }
        int nl = 0;
        cudaError_t e = launch_repack(table_dev, ptrs_dev, ptrs_dev + N, N, d->d_in, d->d_out, (uint8_t*)slab_dev, st, &nl);
        ctx->launches += nl;
        if (e != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) { rc = PLORA_ERR_CUDA; break; }
    } while (0);
    cudaFree(staging);
    cudaFree(ptrs_dev);
    if (rc != PLORA_OK) {
        cudaFree(table_dev);
        cudaGetLastError();
        return rc;
    }
    PoolRec rec{};
    rec.layer = d->layer;
    rec.proj = d->proj;
    rec.table_dev = table_dev;
    rec.dev.slab = (const uint8_t*)slab_dev;
    rec.dev.slab_bytes = need;
    rec.dev.table = table_dev;
    rec.dev.d_in = d->d_in;
    rec.dev.d_out = d->d_out;
    rec.dev.n_adapters = N;
    rec.dev.max_rp = max_rp;
    rec.dev.rp_mask = rp_mask;
    rec.dev.min_rp = min_rp;
    {
        uint64_t hsh = 1469598103934665603ull;   // FNV-1a over the padded ranks
        for (int a = 0; a < N; ++a) hsh = (hsh ^ (uint64_t)table[a].rp) * 1099511628211ull;
        rec.rank_sig = hsh ^ (uint64_t)N;
    }
    if (PoolRec* old = find_pool(ctx, d->layer, d->proj)) {
        cudaStreamSynchronize(st);
        cudaFree(old->table_dev);
        *old = rec;
    } else {
        ctx->pool_index[pool_key(d->layer, d->proj)] = ctx->pools.size();
        ctx->pools.push_back(rec);
    }
    return PLORA_OK;
}

PLORA_API int32_t plora_pool_max_rank(plora_ctx* ctx, int32_t layer, int32_t proj) {
    if (!ctx) return PLORA_ERR_INVALID_ARG;
    PoolRec* p = find_pool(ctx, layer, proj);
    return p ? p->dev.max_rp : PLORA_ERR_NOT_REGISTERED;
}

PLORA_API plora_status plora_bucket(plora_ctx* ctx, const int32_t* ids, int32_t n_tok, int32_t n_adapters, void* stream) {
    ApiRange nvtx_range("plora_bucket");
    if (!ctx || n_tok < 0 || n_tok > ctx->max_tokens || n_adapters < 1 || n_adapters > ctx->max_adapters)
        return PLORA_ERR_INVALID_ARG;
    if (n_tok > 0 && !ids) return PLORA_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return PLORA_ERR_CUDA;
    return do_bucket(ctx, ids, n_tok, n_adapters, as_stream(stream), true);
}

PLORA_API plora_status plora_bucket_view(plora_ctx* ctx, const int32_t** perm, const int32_t** seg_adapter,
                               const int32_t** seg_start, const int32_t** n_seg, const int32_t** n_active) {
    if (!ctx || !ctx->bucket_valid) return PLORA_ERR_INVALID_ARG;
    if (perm) *perm = ctx->bk.perm;
    if (seg_adapter) *seg_adapter = ctx->bk.seg_adapter;
    if (seg_start) *seg_start = ctx->bk.seg_start;
    if (n_seg) *n_seg = ctx->bk.n_seg;
    if (n_active) *n_active = ctx->bk.n_active;
    return PLORA_OK;
}

PLORA_API plora_status plora_set_path(plora_ctx* ctx, int32_t path, int32_t sgmv_min_rows) {
    if (!ctx || path < PLORA_PATH_AUTO || path > PLORA_PATH_SGMV_SPLIT || sgmv_min_rows < 0) return PLORA_ERR_INVALID_ARG;
    ctx->path = path;
    ctx->sgmv_min_rows = sgmv_min_rows > 0 ? sgmv_min_rows : kDefaultSgmvMinRows;
    return PLORA_OK;
}

PLORA_API plora_status plora_set_wait_limit(plora_ctx* ctx, int64_t cycles) {
    if (!ctx || cycles < 0) return PLORA_ERR_INVALID_ARG;
    ctx->dbg.wait_cycles = cycles;
    if (cycles == 0 || cycles > PLORA_HOOK_MAX_CYCLES) ctx->dbg.test_hook = PLORA_HOOK_NONE;   // a hook needs a short limit
    return PLORA_OK;
}

PLORA_API plora_status plora_set_test_hook(plora_ctx* ctx, int32_t hook) {
    if (!ctx || (hook != PLORA_HOOK_NONE && hook != PLORA_HOOK_WITHHOLD_RELEASE)) return PLORA_ERR_INVALID_ARG;
    if (hook != PLORA_HOOK_NONE && (ctx->dbg.wait_cycles < 1 || ctx->dbg.wait_cycles > PLORA_HOOK_MAX_CYCLES))
        return PLORA_ERR_INVALID_ARG;
    ctx->dbg.test_hook = hook;
    return PLORA_OK;
}

PLORA_API plora_status plora_set_inputs_resident(plora_ctx* ctx, int32_t resident) {
    if (!ctx || (resident != 0 && resident != 1)) return PLORA_ERR_INVALID_ARG;
    ctx->dbg.inputs_resident = resident != 0;
    return PLORA_OK;
}

PLORA_API plora_status plora_set_input_type(plora_ctx* ctx, int32_t type) {
    if (!ctx || (type != PLORA_INPUT_BF16 && type != PLORA_INPUT_FP16)) return PLORA_ERR_INVALID_ARG;
    ctx->fp16 = type == PLORA_INPUT_FP16;
    return PLORA_OK;
}

}  // extern "C"

namespace {
// One projection's delta; the caller has opened the call (call_gen).
plora_status delta_one(plora_ctx* ctx, const void* x, const int32_t* ids, int32_t n_tok, int32_t layer, int32_t proj,
                       float* y, void* stream) {
    plora_status rc = check_call(ctx, x, ids, n_tok, y);
    if (rc != PLORA_OK) return rc;
    PoolRec* pool = find_pool(ctx, layer, proj);
    if (!pool) return PLORA_ERR_NOT_REGISTERED;
    if (n_tok == 0) return PLORA_OK;
    DeviceGuard g(ctx->device);
    if (!g.ok) return PLORA_ERR_CUDA;
    cudaStream_t st = as_stream(stream);
    rc = ensure_bucket(ctx, ids, n_tok, pool->dev.n_adapters, st);
    if (rc != PLORA_OK) return rc;
    int nl = 0;
    cudaError_t e = cudaSuccess;
    if (ctx->path == PLORA_PATH_UNFUSED) {
        e = launch_bgmv_one(kShrinkOnly, pool->dev, ctx->bk, n_tok, x, nullptr, ctx->m_ws, pool->dev.max_rp, ctx->status_dev,
                        ctx->sm_count, ctx->launches_since_bucket++ > 0, &ctx->cls_cache, pool->rank_sig, st, &nl, false, ctx->fp16, ctx->dbg);
        if (e == cudaSuccess)
            e = launch_bgmv_one(kExpandOnly, pool->dev, ctx->bk, n_tok, nullptr, y, ctx->m_ws, pool->dev.max_rp,
                            ctx->status_dev, ctx->sm_count, ctx->launches_since_bucket++ > 0, &ctx->cls_cache, pool->rank_sig, st, &nl, false, ctx->fp16, ctx->dbg);
    } else {
        // a batch shorter than the threshold cannot hold a segment for the tensor-core path
        const bool may_bgmv = ctx->path != PLORA_PATH_SGMV && ctx->path != PLORA_PATH_SGMV_SPLIT;
        // The split tensor-core launch goes between the classify pass and the BGMV launches of the call: its CTAs (one
        // per SM) then run beside the BGMV launches' instead of after them (mixed-rank workload: 0.277 -> 0.27 ms per step).
        struct SplitArgs {
            plora_ctx* ctx; PoolRec* pool; int32_t n_tok; const void* x; float* y; cudaStream_t st;
        } sa{ctx, pool, n_tok, x, y, st};
        const bool split = split_launch(ctx, n_tok);
        const BetweenLaunch split_between = [](void* a, int* n_launches) -> cudaError_t {
            SplitArgs* s = static_cast<SplitArgs*>(a);
            s->ctx->launches_since_bucket++;
            return launch_sgmv(s->pool->dev, s->ctx->bk, s->n_tok, s->ctx->bucket_sgmv_min, s->x, s->y, s->ctx->fp16,
                               s->ctx->status_dev, s->ctx->sm_count, false, true, split_max_tiles(s->ctx), s->ctx->dbg, s->st,
                               n_launches);
        };
        if (may_bgmv) {
            const void* xs[1] = {x};
            float* ys[1] = {y};
            e = launch_bgmv(kFused, &pool->dev, 1, ctx->bk, n_tok, xs, ys, nullptr, 0, false, ctx->fp16, ctx->status_dev,
                            ctx->sm_count, ctx->launches_since_bucket++ > 0, &ctx->cls_cache, pool->rank_sig, ctx->dbg, st, &nl,
                            split ? split_between : nullptr, &sa);
        }
        if (e == cudaSuccess && wide_launch(ctx, n_tok))
            e = launch_sgmv(pool->dev, ctx->bk, n_tok, ctx->bucket_sgmv_min, x, y, ctx->fp16, ctx->status_dev, ctx->sm_count, may_bgmv, false, 0, ctx->dbg, st, &nl);
        if (e == cudaSuccess && split && !may_bgmv)
            e = launch_sgmv(pool->dev, ctx->bk, n_tok, ctx->bucket_sgmv_min, x, y, ctx->fp16, ctx->status_dev, ctx->sm_count, false, true, split_max_tiles(ctx), ctx->dbg, st, &nl);
    }
    ctx->launches += nl;
    return e == cudaSuccess ? PLORA_OK : PLORA_ERR_CUDA;
}
}  // namespace

extern "C" {

PLORA_API plora_status plora_lora_delta(plora_ctx* ctx, const void* x, const int32_t* ids, int32_t n_tok, int32_t layer,
                                        int32_t proj, float* y, void* stream) {
    ApiRange nvtx_range("plora_lora_delta");
    if (ctx) ++ctx->call_gen;
    return delta_one(ctx, x, ids, n_tok, layer, proj, y, stream);
}

PLORA_API plora_status plora_lora_delta_group(plora_ctx* ctx, int32_t n, const void* const* x, const int32_t* ids,
                                              int32_t n_tok, const int32_t* layers, const int32_t* projs, float* const* y,
                                              void* stream) {
    ApiRange nvtx_range("plora_lora_delta_group");
    if (!ctx || n < 1 || n > kMaxGroupPools || !x || !y || !layers || !projs) return PLORA_ERR_INVALID_ARG;
    ++ctx->call_gen;
    PoolRec* recs[kMaxGroupPools];
    for (int g = 0; g < n; ++g) {
        plora_status rc = check_call(ctx, x[g], ids, n_tok, y[g]);
        if (rc != PLORA_OK) return rc;
        recs[g] = find_pool(ctx, layers[g], projs[g]);
        if (!recs[g]) return PLORA_ERR_NOT_REGISTERED;
    }
    if (n_tok == 0) return PLORA_OK;
    bool same = true;
    for (int g = 1; g < n; ++g)
        same = same && recs[g]->dev.d_in == recs[0]->dev.d_in && recs[g]->dev.d_out == recs[0]->dev.d_out &&
               recs[g]->dev.n_adapters == recs[0]->dev.n_adapters && recs[g]->dev.max_rp == recs[0]->dev.max_rp &&
               recs[g]->dev.rp_mask == recs[0]->dev.rp_mask &&
               (recs[g]->rank_sig == recs[0]->rank_sig || (recs[0]->dev.rp_mask & (recs[0]->dev.rp_mask - 1)) == 0);
    if (!same || ctx->path == PLORA_PATH_UNFUSED || ctx->path == PLORA_PATH_SGMV || ctx->path == PLORA_PATH_SGMV_SPLIT) {
        // pools of different shape, or a path without a grouped kernel: one projection after the other
        for (int g = 0; g < n; ++g) {
            plora_status rc = delta_one(ctx, x[g], ids, n_tok, layers[g], projs[g], y[g], stream);
            if (rc != PLORA_OK) return rc;
        }
        return PLORA_OK;
    }
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return PLORA_ERR_CUDA;
    cudaStream_t st = as_stream(stream);
    plora_status rc = ensure_bucket(ctx, ids, n_tok, recs[0]->dev.n_adapters, st);
    if (rc != PLORA_OK) return rc;
    PoolDev pools[kMaxGroupPools];
    for (int g = 0; g < n; ++g) pools[g] = recs[g]->dev;
    int nl = 0;
    // (the split tensor-core launches of the projections go between the classify pass and the BGMV launch, as in
    // plora_lora_delta: the first of them joins the stream's order, the others and the BGMV launch follow it freely)
    struct GroupSplitArgs {
        plora_ctx* ctx; const PoolDev* pools; int n; int32_t n_tok; const void* const* x; float* const* y; cudaStream_t st;
    } ga{ctx, pools, n, n_tok, x, y, st};
    const bool split = split_launch(ctx, n_tok);
    const BetweenLaunch split_between = [](void* a, int* n_launches) -> cudaError_t {
        GroupSplitArgs* s = static_cast<GroupSplitArgs*>(a);
        cudaError_t err = cudaSuccess;
        for (int g = 0; g < s->n && err == cudaSuccess; ++g) {
            s->ctx->launches_since_bucket++;
            err = launch_sgmv(s->pools[g], s->ctx->bk, s->n_tok, s->ctx->bucket_sgmv_min, s->x[g], s->y[g], s->ctx->fp16,
                              s->ctx->status_dev, s->ctx->sm_count, g > 0, true, split_max_tiles(s->ctx), s->ctx->dbg, s->st,
                              n_launches);
        }
        return err;
    };
    cudaError_t e = launch_bgmv(kFused, pools, n, ctx->bk, n_tok, x, y, nullptr, 0, false, ctx->fp16, ctx->status_dev, ctx->sm_count,
                                ctx->launches_since_bucket++ > 0, &ctx->cls_cache, recs[0]->rank_sig, ctx->dbg, st, &nl,
                                split ? split_between : nullptr, &ga);
    for (int g = 0; g < n && e == cudaSuccess && wide_launch(ctx, n_tok); ++g)
        e = launch_sgmv(pools[g], ctx->bk, n_tok, ctx->bucket_sgmv_min, x[g], y[g], ctx->fp16, ctx->status_dev, ctx->sm_count, true, false, 0, ctx->dbg, st, &nl);
    ctx->launches += nl;
    return e == cudaSuccess ? PLORA_OK : PLORA_ERR_CUDA;
}

namespace {
// The split entry points always take the BGMV kernels: bucket with no tensor-core segments.
plora_status split_call(plora_ctx* ctx, BgmvMode mode, const void* x, void* m, int32_t ldm, bool m16, const int32_t* ids,
                        int32_t n_tok, int32_t layer, int32_t proj, float* y, void* stream) {
    plora_status rc = check_call(ctx, mode == kShrinkOnly ? x : m, ids, n_tok, mode == kShrinkOnly ? m : (void*)y);
    if (rc != PLORA_OK) return rc;
    ++ctx->call_gen;
    PoolRec* pool = find_pool(ctx, layer, proj);
    if (!pool) return PLORA_ERR_NOT_REGISTERED;
    // rows of m start on 16-byte boundaries (the expand copies them in bulk)
    if (ldm < pool->dev.max_rp || (ldm & (m16 ? 7 : 3))) return PLORA_ERR_INVALID_ARG;
    if (n_tok == 0) return PLORA_OK;
    DeviceGuard g(ctx->device);
    if (!g.ok) return PLORA_ERR_CUDA;
    cudaStream_t st = as_stream(stream);
    const int32_t saved = ctx->path;
    ctx->path = PLORA_PATH_UNFUSED;
    rc = ensure_bucket(ctx, ids, n_tok, pool->dev.n_adapters, st);
    ctx->path = saved;
    if (rc != PLORA_OK) return rc;
    int nl = 0;
    cudaError_t e = launch_bgmv_one(mode, pool->dev, ctx->bk, n_tok, x, y, m, ldm, ctx->status_dev, ctx->sm_count,
                                    ctx->launches_since_bucket++ > 0, &ctx->cls_cache, pool->rank_sig, st, &nl, m16, ctx->fp16, ctx->dbg);
    ctx->launches += nl;
    return e == cudaSuccess ? PLORA_OK : PLORA_ERR_CUDA;
}
}  // namespace

PLORA_API plora_status plora_shrink(plora_ctx* ctx, const void* x, const int32_t* ids, int32_t n_tok, int32_t layer, int32_t proj,
                          float* m, int32_t ldm, void* stream) {
    ApiRange nvtx_range("plora_shrink");
    return split_call(ctx, kShrinkOnly, x, m, ldm, false, ids, n_tok, layer, proj, nullptr, stream);
}

PLORA_API plora_status plora_expand(plora_ctx* ctx, const float* m, int32_t ldm, const int32_t* ids, int32_t n_tok,
                          int32_t layer, int32_t proj, float* y, void* stream) {
    ApiRange nvtx_range("plora_expand");
    return split_call(ctx, kExpandOnly, nullptr, const_cast<float*>(m), ldm, false, ids, n_tok, layer, proj, y, stream);
}

PLORA_API plora_status plora_shrink_m16(plora_ctx* ctx, const void* x, const int32_t* ids, int32_t n_tok, int32_t layer,
                                        int32_t proj, void* m_bf16, int32_t ldm, void* stream) {
    ApiRange nvtx_range("plora_shrink_m16");
    return split_call(ctx, kShrinkOnly, x, m_bf16, ldm, true, ids, n_tok, layer, proj, nullptr, stream);
}

PLORA_API plora_status plora_expand_m16(plora_ctx* ctx, const void* m_bf16, int32_t ldm, const int32_t* ids, int32_t n_tok,
                                        int32_t layer, int32_t proj, float* y, void* stream) {
    ApiRange nvtx_range("plora_expand_m16");
    return split_call(ctx, kExpandOnly, nullptr, const_cast<void*>(m_bf16), ldm, true, ids, n_tok, layer, proj, y, stream);
}

namespace {

bool grow(void** p, size_t* have, size_t want) {
    if (*have >= want) return true;
    cudaFree(*p);
    *p = nullptr;
    *have = 0;
    if (cudaMalloc(p, want) != cudaSuccess) return false;
    *have = want;
    return true;
}

}  // namespace

PLORA_API plora_status plora_host_sync(plora_ctx* ctx) {
    ApiRange nvtx_range("plora_host_sync");
    if (!ctx) return PLORA_ERR_INVALID_ARG;
    if (!ctx->d2h_stream) return PLORA_OK;   // nothing was ever queued
    DeviceGuard g(ctx->device);
    if (!g.ok) return PLORA_ERR_CUDA;
    // the copy-back stream is last in every call's chain, and in order across calls
    if (cudaStreamSynchronize(ctx->d2h_stream) != cudaSuccess) return PLORA_ERR_CUDA;
    for (auto& hs : ctx->stage) hs.in_flight = false;
    return PLORA_OK;
}

PLORA_API plora_status plora_lora_delta_host_async(plora_ctx* ctx, int32_t n, const void* x_host, const int32_t* ids_host,
                                                   int32_t n_tok, const int32_t* layers, const int32_t* projs,
                                                   float* const* y_host, void* stream) {
    ApiRange nvtx_range("plora_lora_delta_host_async");
    if (!ctx || n < 1 || n > kMaxGroupPools || !layers || !projs || !y_host) return PLORA_ERR_INVALID_ARG;
    if (n_tok < 0 || n_tok > ctx->max_tokens) return PLORA_ERR_INVALID_ARG;
    if (n_tok > 0 && (!x_host || !ids_host)) return PLORA_ERR_INVALID_ARG;
    PoolRec* recs[kMaxGroupPools];
    for (int g = 0; g < n; ++g) {
        if (n_tok > 0 && !y_host[g]) return PLORA_ERR_INVALID_ARG;
        recs[g] = find_pool(ctx, layers[g], projs[g]);
        if (!recs[g]) return PLORA_ERR_NOT_REGISTERED;
        if (recs[g]->dev.d_in != recs[0]->dev.d_in) return PLORA_ERR_INVALID_ARG;   // one x serves the whole group
    }
    if (n_tok == 0) return PLORA_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return PLORA_ERR_CUDA;
    cudaStream_t st = as_stream(stream);
    if (!ctx->h2d_stream) {
        if (cudaStreamCreateWithFlags(&ctx->h2d_stream, cudaStreamNonBlocking) != cudaSuccess ||
            cudaStreamCreateWithFlags(&ctx->d2h_stream, cudaStreamNonBlocking) != cudaSuccess)
            return PLORA_ERR_CUDA;
    }
    plora_ctx::HostStage& hs = ctx->stage[ctx->next_stage];
    ctx->next_stage = (ctx->next_stage + 1) % plora_ctx::kHostStages;
    if (!hs.up) {
        if (cudaEventCreateWithFlags(&hs.up, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&hs.done, cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&hs.freed, cudaEventDisableTiming) != cudaSuccess)
            return PLORA_ERR_CUDA;
    }
    // buffers sized for the context's largest batch, so they are allocated once per shape
    const size_t want_x = (size_t)ctx->max_tokens * recs[0]->dev.d_in * 2;
    bool fits = hs.x_bytes >= want_x && hs.ids != nullptr;
    for (int g = 0; g < n; ++g) fits = fits && hs.y_bytes[g] >= (size_t)ctx->max_tokens * recs[g]->dev.d_out * 4;
    if (!fits) {
        plora_status rc = plora_host_sync(ctx);   // nothing may still be using what is freed here
        if (rc != PLORA_OK) return rc;
        if (cudaStreamSynchronize(st) != cudaSuccess) return PLORA_ERR_CUDA;
        if (!grow(&hs.x, &hs.x_bytes, want_x)) return PLORA_ERR_WORKSPACE;
        if (!hs.ids && cudaMalloc(&hs.ids, (size_t)ctx->max_tokens * 4) != cudaSuccess) return PLORA_ERR_WORKSPACE;
        for (int g = 0; g < n; ++g)
            if (!grow((void**)&hs.y[g], &hs.y_bytes[g], (size_t)ctx->max_tokens * recs[g]->dev.d_out * 4))
                return PLORA_ERR_WORKSPACE;
    }
    // to the device, once the set's previous user has copied its result out
    if (hs.in_flight && cudaStreamWaitEvent(ctx->h2d_stream, hs.freed, 0) != cudaSuccess) return PLORA_ERR_CUDA;
    hs.in_flight = true;
    const size_t nx = (size_t)n_tok * recs[0]->dev.d_in * 2;
    if (cudaMemcpyAsync(hs.ids, ids_host, (size_t)n_tok * 4, cudaMemcpyHostToDevice, ctx->h2d_stream) != cudaSuccess ||
        cudaMemcpyAsync(hs.x, x_host, nx, cudaMemcpyHostToDevice, ctx->h2d_stream) != cudaSuccess)
        return PLORA_ERR_CUDA;
    for (int g = 0; g < n; ++g)
        if (cudaMemcpyAsync(hs.y[g], y_host[g], (size_t)n_tok * recs[g]->dev.d_out * 4, cudaMemcpyHostToDevice,
                            ctx->h2d_stream) != cudaSuccess)
            return PLORA_ERR_CUDA;
    if (cudaEventRecord(hs.up, ctx->h2d_stream) != cudaSuccess || cudaStreamWaitEvent(st, hs.up, 0) != cudaSuccess)
        return PLORA_ERR_CUDA;
    // the delta, on the caller's stream
    ctx->bucket_valid = false;   // another set's ids, or new ids under the same pointer
    const void* xs[kMaxGroupPools];
    float* ys[kMaxGroupPools];
    for (int g = 0; g < n; ++g) {
        xs[g] = hs.x;
        ys[g] = hs.y[g];
    }
    plora_status rc = n == 1 ? plora_lora_delta(ctx, hs.x, hs.ids, n_tok, layers[0], projs[0], hs.y[0], stream)
                             : plora_lora_delta_group(ctx, n, xs, hs.ids, n_tok, layers, projs, ys, stream);
    ctx->bucket_valid = false;
    if (rc != PLORA_OK) return rc;
    if (cudaEventRecord(hs.done, st) != cudaSuccess || cudaStreamWaitEvent(ctx->d2h_stream, hs.done, 0) != cudaSuccess)
        return PLORA_ERR_CUDA;
    // back to the host
    for (int g = 0; g < n; ++g)
        if (cudaMemcpyAsync(y_host[g], hs.y[g], (size_t)n_tok * recs[g]->dev.d_out * 4, cudaMemcpyDeviceToHost,
                            ctx->d2h_stream) != cudaSuccess)
            return PLORA_ERR_CUDA;
    if (cudaEventRecord(hs.freed, ctx->d2h_stream) != cudaSuccess) return PLORA_ERR_CUDA;
    return PLORA_OK;
}

PLORA_API plora_status plora_lora_delta_host(plora_ctx* ctx, const void* x_host, const int32_t* ids_host, int32_t n_tok,
                                   int32_t layer, int32_t proj, float* y_host, void* stream) {
    plora_status rc = plora_lora_delta_host_async(ctx, 1, x_host, ids_host, n_tok, &layer, &proj, &y_host, stream);
    if (rc != PLORA_OK) return rc;
    return plora_host_sync(ctx);
}

PLORA_API plora_status plora_device_status(plora_ctx* ctx, void* stream, int32_t* host_out) {
    if (!ctx || !host_out) return PLORA_ERR_INVALID_ARG;
    DeviceGuard g(ctx->device);
    if (!g.ok) return PLORA_ERR_CUDA;
    cudaStream_t st = as_stream(stream);
    int32_t v = 0;
    if (cudaMemcpyAsync(&v, ctx->status_dev, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return PLORA_ERR_CUDA;
    if (v != 0 && (cudaMemsetAsync(ctx->status_dev, 0, 4, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess))
        return PLORA_ERR_CUDA;
    *host_out = v;
    return PLORA_OK;
}

PLORA_API int64_t plora_launch_count(plora_ctx* ctx) { return ctx ? ctx->launches : -1; }

}  // extern "C"

// ---------------------------------------------------------------------------------
// The delta without any allocation: m = x A lives in an array of the library image.
// ---------------------------------------------------------------------------------
namespace {

// Part of the library image on every device that loads it.  In host code this name is only
// a handle for cudaGetSymbolAddress: it is NOT a device address and must never be passed to
// a kernel as it is.
static __device__ __align__(256) float g_noalloc_scratch[PLORA_NOALLOC_SCRATCH_FLOATS];

constexpr int kMaxDevicesTracked = 64;
float* g_noalloc_scratch_addr[kMaxDevicesTracked] = {};   // per device, filled on first use

// Device address of the scratch array on `device`, which must be the current device.
cudaError_t noalloc_scratch_address(int device, float** out) {
    if (device < 0 || device >= kMaxDevicesTracked) return cudaErrorInvalidDevice;
    if (!g_noalloc_scratch_addr[device]) {
        void* addr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&addr, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        g_noalloc_scratch_addr[device] = static_cast<float*>(addr);
    }
    *out = g_noalloc_scratch_addr[device];
    return cudaSuccess;
}

}  // namespace

extern "C" {

PLORA_API plora_status plora_lora_delta_noalloc(plora_ctx* ctx, const void* x, const int32_t* ids, int32_t n_tok,
                                                int32_t layer, int32_t proj, float* y, void* stream) {
    ApiRange nvtx_range("plora_lora_delta_noalloc");
    plora_status rc = check_call(ctx, x, ids, n_tok, y);
    if (rc != PLORA_OK) return rc;
    ++ctx->call_gen;
    PoolRec* pool = find_pool(ctx, layer, proj);
    if (!pool) return PLORA_ERR_NOT_REGISTERED;
    if (n_tok == 0) return PLORA_OK;
    const int32_t ldm = pool->dev.max_rp;
    if ((size_t)n_tok * (size_t)ldm > (size_t)PLORA_NOALLOC_SCRATCH_FLOATS) return PLORA_ERR_WORKSPACE;
    DeviceGuard g(ctx->device);
    if (!g.ok) return PLORA_ERR_CUDA;
    float* m = nullptr;
    if (noalloc_scratch_address(ctx->device, &m) != cudaSuccess) return PLORA_ERR_CUDA;
    cudaStream_t st = as_stream(stream);
    // the two BGMV kernels take every segment: bucket with no tensor-core segments
    const int32_t saved = ctx->path;
    ctx->path = PLORA_PATH_UNFUSED;
    rc = ensure_bucket(ctx, ids, n_tok, pool->dev.n_adapters, st);
    ctx->path = saved;
    if (rc != PLORA_OK) return rc;
    int nl = 0;
    cudaError_t e = launch_bgmv_one(kShrinkOnly, pool->dev, ctx->bk, n_tok, x, nullptr, m, ldm, ctx->status_dev,
                                ctx->sm_count, ctx->launches_since_bucket++ > 0, &ctx->cls_cache, pool->rank_sig, st, &nl, false, ctx->fp16, ctx->dbg);
    if (e == cudaSuccess)
        e = launch_bgmv_one(kExpandOnly, pool->dev, ctx->bk, n_tok, nullptr, y, m, ldm, ctx->status_dev, ctx->sm_count,
                        ctx->launches_since_bucket++ > 0, &ctx->cls_cache, pool->rank_sig, st, &nl, false, ctx->fp16, ctx->dbg);
    ctx->launches += nl;
    return e == cudaSuccess ? PLORA_OK : PLORA_ERR_CUDA;
}

}  // extern "C"
