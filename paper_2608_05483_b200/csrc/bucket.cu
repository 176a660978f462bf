// Token bucketing: a stable counting sort of token indices by adapter id, the list
// of segments (one per adapter present; its length is the per-adapter request
// count B_i of the paper's cost model, Section VI-B), and the work lists the
// delta kernels walk.  One CTA, no global atomics on the outputs: the result is
// unique and deterministic.
#include "plora_internal.cuh"

namespace plora {

namespace {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;

// In-place exclusive scan of a[0..n) in shared memory by the whole block.
// Returns the total in every thread.  wsum: 33 ints of shared scratch.
__device__ int block_exclusive_scan(int* a, int n, int* wsum) {
    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    const int per = (n + kThreads - 1) / kThreads;
    const int lo = min(n, tid * per), hi = min(n, lo + per);
    int s = 0;
    for (int i = lo; i < hi; ++i) s += a[i];
    int incl = s;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        int v = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += v;
    }
    __syncthreads();   // wsum may still be read from an earlier call
    if (lane == 31) wsum[w] = incl;
    __syncthreads();
    if (w == 0) {
        int v = wsum[lane], iv = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            int u = __shfl_up_sync(0xffffffffu, iv, d);
            if (lane >= d) iv += u;
        }
        wsum[lane] = iv - v;
        if (lane == 31) wsum[32] = iv;
    }
    __syncthreads();
    int run = incl - s + wsum[w];
    for (int i = lo; i < hi; ++i) {
        int v = a[i];
        a[i] = run;
        run += v;
    }
    const int total = wsum[32];
    __syncthreads();
    return total;
}

__device__ __forceinline__ int units_of(int cnt, int per) { return (cnt + per - 1) / per; }

// Fill one work list: unit u belongs to the last bin b with ustart[b] <= u.
__device__ void write_units(WorkUnit* out, int n_units, const int* ustart, const int* start, const int* total,
                            const int* segidx, int n_bins, int per, const int32_t* perm) {
    for (int u = threadIdx.x; u < n_units; u += kThreads) {
        int lo = 0, hi = n_bins;   // find first b with ustart[b] > u
        while (lo < hi) {
            int mid = (lo + hi) >> 1;
            if (ustart[mid] <= u) lo = mid + 1; else hi = mid;
        }
        const int b = lo - 1;
        const int k = u - ustart[b];
        WorkUnit wu;
        wu.adapter = b;
        wu.pos0 = start[b] + k * per;
        wu.cnt = min(per, total[b] - k * per);
        wu.seg = segidx[b];
#pragma unroll
        for (int t = 0; t < kTokChunk; ++t) wu.tok[t] = t < wu.cnt ? perm[wu.pos0 + t] : 0;
        out[u] = wu;
    }
}

__global__ void __launch_bounds__(kThreads, 1)
bucket_kernel(const int32_t* __restrict__ ids, int T, int N, int nch, int sgmv_min_rows, int sgmv_min_tiles,
              int split_ok, BucketDev bk, int32_t* status) {
    extern __shared__ int smem[];
    const int nb = N + 1;                 // bins: ids 0..N-1, then "no adapter"
    int* cnt = smem;                      // [nch][nb]   per-chunk counts, later per-chunk cursors
    int* total = cnt + nch * nb;          // [nb]
    int* start = total + nb;              // [nb + 1]    exclusive scan of total
    int* segidx = start + nb + 1;         // [nb]
    int* ubg = segidx + nb;               // [nb]
    int* usg = ubg + nb;                  // [nb]
    int* wsum = usg + nb;                 // [33]

    const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
    for (int i = tid; i < nch * nb; i += kThreads) cnt[i] = 0;
    __syncthreads();

    // tokens are cut into nch contiguous chunks, chunk c handled by warp c
    const int per = ((T + nch - 1) / nch + 31) & ~31;
    const int c_lo = min(T, w * per), c_hi = min(T, c_lo + per);
    if (w < nch) {
        for (int t = c_lo + lane; t < c_hi; t += 32) {
            int id = ids[t];
            if (id < -1 || id >= N) {
                atomicCAS(status, 0, PLORA_ERR_BAD_ADAPTER_ID);
                id = -1;
            }
            atomicAdd(&cnt[w * nb + (id < 0 ? N : id)], 1);
        }
    }
    __syncthreads();

    // per bin: counts -> exclusive prefix over chunks, and the bin total
    for (int b = tid; b < nb; b += kThreads) {
        int run = 0;
        for (int c = 0; c < nch; ++c) {
            int v = cnt[c * nb + b];
            cnt[c * nb + b] = run;
            run += v;
        }
        total[b] = run;
        start[b] = run;
        segidx[b] = (b < N && run > 0) ? 1 : 0;
        usg[b] = (b < N && run > 0 && run >= sgmv_min_rows) ? units_of(run, kSgmvRows) : 0;
    }
    __syncthreads();
    block_exclusive_scan(start, nb, wsum);
    if (tid == 0) start[nb] = T;
    const int n_seg = block_exclusive_scan(segidx, nb, wsum);
    // Long segments go to the tensor-core path.  If together they make enough tiles to occupy the
    // GPU, a CTA takes whole tiles (wide shape); a handful of tiles would each be one long serial
    // job, so they go to the split shape (a cluster of CTAs per tile) where the caller has it, and
    // stay with BGMV otherwise.
    const int n_sg_cand = block_exclusive_scan(usg, nb, wsum);
    const bool wide = n_sg_cand >= sgmv_min_tiles;
    const bool use_sg = wide || (split_ok && n_sg_cand > 0);
    const int n_sg = use_sg ? n_sg_cand : 0;
    for (int b = tid; b < nb; b += kThreads) {
        const int run = total[b];
        const bool sg = use_sg && run >= sgmv_min_rows;
        ubg[b] = (b < N && run > 0 && !sg) ? units_of(run, kTokChunk) : 0;
    }
    __syncthreads();
    const int n_bg = block_exclusive_scan(ubg, nb, wsum);
    const int n_active = start[N];

    // stable scatter: each warp walks its chunk in order, 32 tokens at a time
    if (w < nch) {
        for (int base = c_lo; base < c_hi; base += 32) {
            const int t = base + lane;
            const bool valid = t < c_hi;
            int key = nb + lane;   // distinct dummy keys keep idle lanes out of every group
            if (valid) {
                int id = ids[t];
                key = (id < 0 || id >= N) ? N : id;
            }
            const unsigned peers = __match_any_sync(0xffffffffu, key);
            const int rank = __popc(peers & ((1u << lane) - 1u));
            int cur = 0;
            if (valid) cur = cnt[w * nb + key];
            __syncwarp();
            if (valid && rank == 0) cnt[w * nb + key] = cur + __popc(peers);
            __syncwarp();
            if (valid) {
                PLORA_CHECKED((unsigned)(start[key] + cur + rank) < (unsigned)T, status)
                bk.perm[start[key] + cur + rank] = t;
            }
        }
    }

    // segment list with its tails
    const int cap = min(T, N);
    for (int b = tid; b < N; b += kThreads) {
        if (total[b] > 0) {
            bk.seg_adapter[segidx[b]] = b;
            bk.seg_start[segidx[b]] = start[b];
        }
    }
    for (int k = n_seg + tid; k <= cap; k += kThreads) {
        if (k < cap) bk.seg_adapter[k] = -1;
        bk.seg_start[k] = n_active;
    }
    if (tid == 0) {
        *bk.n_seg = n_seg;
        *bk.n_active = n_active;
        *bk.n_bgmv_units = n_bg;
        *bk.n_sgmv_tiles = n_sg;
        *bk.sgmv_split = (use_sg && !wide) ? 1 : 0;
    }
    __syncthreads();   // perm is complete (written by this block) before the units quote it
    write_units(bk.bgmv_units, n_bg, ubg, start, total, segidx, N, kTokChunk, bk.perm);
    write_units(bk.sgmv_tiles, n_sg, usg, start, total, segidx, N, kSgmvRows, bk.perm);
}

constexpr size_t kBucketSmemLimit = 200 * 1024;
size_t bucket_smem_bytes(int N, int nch) { return sizeof(int) * ((size_t)nch * (N + 1) + 5 * (size_t)(N + 2) + 40); }

}  // namespace

cudaError_t bucket_configure() {
    return cudaFuncSetAttribute(bucket_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kBucketSmemLimit);
}

int bucket_max_adapters() {
    int n = 1;
    while (bucket_smem_bytes(n * 2, 1) <= kBucketSmemLimit) n *= 2;
    while (bucket_smem_bytes(n + 256, 1) <= kBucketSmemLimit) n += 256;
    return n;
}

cudaError_t launch_bucket(const int32_t* ids, int n_tok, int n_adapters, int sgmv_min_rows, int sgmv_min_tiles,
                          bool split_ok, BucketDev bk, int32_t* status, cudaStream_t stream, int* n_launches) {
    int nch = kWarps;
    while (nch > 1 && bucket_smem_bytes(n_adapters, nch) > kBucketSmemLimit) nch >>= 1;
    const size_t smem = bucket_smem_bytes(n_adapters, nch);
    if (smem > kBucketSmemLimit) return cudaErrorInvalidValue;
    bucket_kernel<<<1, kThreads, smem, stream>>>(ids, n_tok, n_adapters, nch, sgmv_min_rows, sgmv_min_tiles, split_ok ? 1 : 0, bk, status);
    ++*n_launches;
    return cudaGetLastError();
}

}  // namespace plora
