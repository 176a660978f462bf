// Decode attention (paper Section V-B): per request and head P = q K^T, S = softmax(P), O = S V over
// the request's KV cache, one query token per request.  Steps 1 and 3 are memory-bound GEMVs, so the
// path is bound by HBM bandwidth on the KV bytes (the cost model's memory term 2 D S sum_k l_k).  The
// paper's integral execution strategy deals a request's cache out to partitions, lets every partition
// run all three steps on its share with a partial softmax that keeps an anchor (its maximum), and
// rescales the partial outputs into the exact global output.  Here a partition is a chunk of
// kChunkTokens consecutive tokens of one (request, KV head): chunks stream through persistent CTAs,
// a second small kernel does the anchor merge.
//
//   prep kernel     kv_len -> list of (request, chunk) units, so that long and short requests spread
//                   evenly over the CTAs;
//   partial kernel  work item = (unit, KV head).  A producer warp brings 64-token tiles of K and V
//                   (tensor-map box copies into 128-byte-swizzled shared memory; the query rows of the
//                   item ride along with a bulk copy) through a ring of stages; eight consumer warps
//                   take 8 tokens of every tile each: scores with 4 lanes per token, an online softmax
//                   per warp (anchor m, sum l, output o, in the base-2 domain), the weighted sum of V
//                   with a lane per 4 dimensions; with several query heads per KV head both products
//                   run on the tensor cores instead (mma.sync, the query heads as rows of the 16-row
//                   operand); at the end of an item the warps' triples meet in shared memory and the
//                   item's (m, l, o) goes to the workspace;
//   merge kernel    one warp per (request, query head) rescales the chunks' partial outputs by their
//                   anchors: O = sum 2^(m_c - m) o_c / sum 2^(m_c - m) l_c.
//
// Every wait is bounded; when one runs out the kernels record PLORA_ERR_TIMEOUT in the workspace's
// status word and run to completion.
#include <cuda.h>

#include "plora.h"

namespace plora {
namespace attn {

constexpr int kHeadDim = 128;
constexpr int kTileTokens = 64;                       // tokens per stage
constexpr int kChunkTokens = 256;                     // tokens per partition (4 tiles)
constexpr int kConsumerWarps = 8;
constexpr int kThreads = (kConsumerWarps + 1) * 32;   // + producer warp
constexpr int kStages = 3;
constexpr int kMaxQPerKv = 8;
constexpr int kKBytes = kTileTokens * kHeadDim * 2;   // 16 KiB: two sub-tiles [64 tokens][64 dims], 128-byte rows, swizzled
constexpr int kQOffset = 2 * kKBytes;
constexpr int kQBytes = kMaxQPerKv * kHeadDim * 2;
constexpr int kHdrOffset = kQOffset + kQBytes;
constexpr int kSlotBytes = (kHdrOffset + 128 + 1023) / 1024 * 1024;   // the swizzled tiles need 1024-byte aligned slots
constexpr int kMergeStride = kHeadDim + 4;            // floats per warp in the meeting buffer: o[128], m, l (16-byte aligned rows)
constexpr int kMergeFloats = kConsumerWarps * kMergeStride;
constexpr int kSmemBytes = 1024 + kStages * kSlotBytes + kMergeFloats * 4 + (2 * kStages + 1) * 8 + 16;
constexpr int kPartFloats = kHeadDim + 4;             // per (unit, query head): o[128], m, l, pad
constexpr long long kWaitCycles = 4000000000ll;   // default limit of a wait: about two seconds of SM clock
// Words of the workspace header (its first 256 bytes; word 0 is the status word, word 1 the unit count):
constexpr int kHookWord = 8;     // PLORA_HOOK_*: tests make a wait run out with it
constexpr int kLimitWord = 10;   // 64-bit: limit of a wait in SM clock cycles, 0 = the default
constexpr int kFlagFirst = 1, kFlagLast = 2, kFlagEnd = 4;

struct Work {
    int32_t* status;       // sticky status word
    int32_t* n_units;
    int32_t* unit_req;
    int32_t* unit_chunk;
    int32_t* unit_start;   // [n_req + 1]: first unit of every request
    float* partials;       // [units][n_q_heads][kPartFloats]
};

struct Params {
    Work w;
    const uint16_t* q;     // bf16 [n_req][n_q_heads][128]
    const int32_t* kv_len;
    float* out;            // fp32 [n_req][n_q_heads][128]
    int32_t n_req, max_kv_len, n_kv_heads, q_per_kv;
    float scale_log2e;     // softmax scale times log2(e): scores live in the base-2 domain
};

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
__device__ __forceinline__ long long wait_limit(const int32_t* status) {
    const long long v = *reinterpret_cast<const volatile long long*>(status + kLimitWord);
    return v > 0 ? v : kWaitCycles;
}
// Bounded wait on an mbarrier phase; false when the CTA has given up (here or elsewhere).
// (The slow path is a real call here: inlined, its timing variables raised the register pressure of the grouped-query
// variants, which sit at their register limit, and doubled their spills; the call costs those kernels nothing measurable.
// The BGMV kernel is the opposite case: there a called slow path cost 4 %, see bgmv.cu.)
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
    const long long t0 = clock64();
    long long limit = 0;
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (limit == 0) limit = wait_limit(status);
        if (clock64() - t0 > limit) break;
    }
    *abort_flag = 1;
    __threadfence_block();
    atomicCAS(status, 0, PLORA_ERR_TIMEOUT);
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, status);
}
// The copy thread's last look at a stage before it leaves: waits whatever the abort flag says, for at
// most the limit (a CTA must not retire with a copy still on its way into its shared memory).
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
// Box of the 4-D cache tensor [request][KV head][token][dim]: 64 dims x 64 tokens of one head, swizzled.
__device__ __forceinline__ void tma_box4(uint32_t dst, const CUtensorMap* tm, int dim, int tok, int head, int req,
                                         uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%2, %3, %4, %5}], [%6];" ::"r"(dst),
        "l"(reinterpret_cast<uint64_t>(tm)), "r"(dim), "r"(tok), "r"(head), "r"(req), "r"(bar)
        : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t a, uint32_t x, uint32_t y, uint32_t z, uint32_t w) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(x), "r"(y), "r"(z), "r"(w) : "memory");
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// ---- tensor-core pieces of the grouped-query path -----------------------------------------------------
__device__ __forceinline__ void ldmatrix_x4(uint32_t a, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t a, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
// D[16 x 8] += A[16 x 16] B[16 x 8], bf16 in, fp32 out; rows 8..15 of A are zero (registers a1, a3)
__device__ __forceinline__ void mma_16816(float (&d)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    const uint32_t z = 0u;
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a0), "r"(z), "r"(a2), "r"(z), "r"(b0), "r"(b1));
}
// D[16 x 8] += A[16 x 8] B[8 x 8]; a0 holds rows 0..7 of A, a1 rows 8..15
__device__ __forceinline__ void mma_1688(float& d0, float& d1, float& d2, float& d3, uint32_t a0, uint32_t a1, uint32_t b0) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
                 : "+f"(d0), "+f"(d1), "+f"(d2), "+f"(d3) : "r"(a0), "r"(a1), "r"(b0));
}
__device__ __forceinline__ uint32_t bf16_rn_bits(float v) {
    const uint32_t u = __float_as_uint(v);
    return (u + 0x7fffu + ((u >> 16) & 1u)) >> 16;   // finite, non-negative inputs only
}

// ---- prep: the list of (request, chunk) units -------------------------------------------------------
__global__ void __launch_bounds__(1024) prep_kernel(const Params p) {
    __shared__ int warp_sum[32];
    __shared__ int carry;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) carry = 0;
    __syncthreads();
    for (int r0 = 0; r0 < p.n_req; r0 += 1024) {
        const int r = r0 + tid;
        int len = r < p.n_req ? p.kv_len[r] : 0;
        len = len < 0 ? 0 : (len > p.max_kv_len ? p.max_kv_len : len);
        const int n = (len + kChunkTokens - 1) / kChunkTokens;
        int incl = n;
        for (int d = 1; d < 32; d <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += v;
        }
        if (lane == 31) warp_sum[warp] = incl;
        __syncthreads();
        int before = carry;
        for (int w = 0; w < warp; ++w) before += warp_sum[w];
        const int start = before + incl - n;
        if (r < p.n_req) {
            p.w.unit_start[r] = start;
            for (int c = 0; c < n; ++c) {
                p.w.unit_req[start + c] = r;
                p.w.unit_chunk[start + c] = c;
            }
        }
        __syncthreads();
        if (tid == 1023) carry = before + incl;
        __syncthreads();
    }
    if (tid == 0) {
        p.w.unit_start[p.n_req] = carry;
        *p.w.n_units = carry;
    }
}

// ---- partial kernel -----------------------------------------------------------------------------------
struct StageHdr {
    int32_t flags, unit, head, n_tok;   // n_tok: valid tokens of this tile (1..64)
};

template <int G>
__global__ void __launch_bounds__(kThreads, 2)
partial_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, const Params p) {
    extern __shared__ uint8_t raw[];
    uint8_t* base = raw + ((1024u - (smem_u32(raw) & 1023u)) & 1023u);
    const uint32_t slots = smem_u32(base);
    float* merge = reinterpret_cast<float*>(base + kStages * kSlotBytes);
    uint8_t* bars = base + kStages * kSlotBytes + kMergeFloats * 4;
    const uint32_t full = smem_u32(bars), empty = full + kStages * 8, meet = empty + kStages * 8;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bars + (2 * kStages + 1) * 8);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full + s * 8, 1);
            mbar_init(empty + s * 8, kConsumerWarps);
        }
        mbar_init(meet, kConsumerWarps);   // where the consumer warps meet at the end of an item (a bounded wait, like all others)
        *abort_flag = 0;
        abort_flag[1] = p.w.status[kHookWord] == PLORA_HOOK_WITHHOLD_RELEASE;   // test hook: warp 0 never hands a stage back
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the unit list comes from the prep kernel
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int n_units = *p.w.n_units;
    const int n_items = n_units * p.n_kv_heads;

    if (warp == kConsumerWarps) {
        // ------------------------------- producer warp (one lane) -------------------------------
        if (lane != 0) return;
        uint32_t it = 0;
        bool stopped = false;   // a wait ran out somewhere in this CTA: nothing more is issued
        for (int item = blockIdx.x; item < n_items && !stopped; item += gridDim.x) {
            const int unit = item / p.n_kv_heads, head = item - unit * p.n_kv_heads;
            const int req = p.w.unit_req[unit], chunk = p.w.unit_chunk[unit];
            int len = p.kv_len[req];
            len = len > p.max_kv_len ? p.max_kv_len : len;
            const int tok0 = chunk * kChunkTokens;
            const int n_in_chunk = min(kChunkTokens, len - tok0);
            const int n_tiles = (n_in_chunk + kTileTokens - 1) / kTileTokens;
            const uint16_t* qsrc = p.q + ((size_t)req * p.n_kv_heads + head) * G * kHeadDim;
            for (int t = 0; t < n_tiles; ++t, ++it) {
                const uint32_t slot = it % kStages, dst = slots + slot * kSlotBytes, bar = full + slot * 8;
                if (!mbar_wait(empty + slot * 8, ((it / kStages) & 1) ^ 1, abort_flag, p.w.status)) {
                    stopped = true;
                    break;
                }
                const int flags = (t == 0 ? kFlagFirst : 0) | (t == n_tiles - 1 ? kFlagLast : 0);
                sts128(dst + kHdrOffset, (uint32_t)flags, (uint32_t)unit, (uint32_t)head,
                       (uint32_t)min(kTileTokens, n_in_chunk - t * kTileTokens));
                mbar_arrive_expect_tx(bar, 2 * kKBytes + G * kHeadDim * 2);
                const int tok = tok0 + t * kTileTokens;
                tma_box4(dst, &tm_k, 0, tok, head, req, bar);
                tma_box4(dst + kKBytes / 2, &tm_k, 64, tok, head, req, bar);
                tma_box4(dst + kKBytes, &tm_v, 0, tok, head, req, bar);
                tma_box4(dst + kKBytes + kKBytes / 2, &tm_v, 64, tok, head, req, bar);
                bulk_g2s(dst + kQOffset, qsrc, G * kHeadDim * 2, bar);
            }
        }
        const uint32_t slot = it % kStages;   // tell the consumers that nothing follows
        if (!stopped && mbar_wait(empty + slot * 8, ((it / kStages) & 1) ^ 1, abort_flag, p.w.status)) {
            sts128(slots + slot * kSlotBytes + kHdrOffset, (uint32_t)kFlagEnd, 0u, 0u, 0u);
            mbar_arrive(full + slot * 8);
            ++it;   // the closing stage counts as armed: its slot's barrier has moved on one phase
        }
        // Before the thread leaves, the copies of the stages it armed last (stages it - 1, it - 2, ...) must
        // have landed: the CTA's shared memory goes to another CTA when its last warp is gone.  In an orderly
        // run these waits return at once or overlap the consumers' last tiles.
        const long long limit = wait_limit(p.w.status);
        for (uint32_t k = 1; k <= (uint32_t)kStages && k <= it; ++k) {
            const uint32_t j = it - k;
            if (!mbar_drain(full + (j % kStages) * 8, (j / kStages) & 1, limit)) atomicCAS(p.w.status, 0, PLORA_ERR_TIMEOUT);
        }
        return;
    }

    // ------------------------------- consumer warps -------------------------------
    // scores: lane (tk, qr) = (lane & 7, lane >> 3) takes token 8 * warp + tk and dims [32 qr, 32 qr + 32);
    // values: lane owns dims 4 * lane .. 4 * lane + 3 of the output
    const int tk = lane & 7, qr = lane >> 3, trow = warp * 8 + tk;
    const uint32_t k_off = (uint32_t)(qr >> 1) * (kKBytes / 2) + trow * 128;   // sub-tile and row of the lane's K piece
    const uint32_t v_sub = (uint32_t)(lane >> 4) * (kKBytes / 2);
    const int v_chunk = (lane >> 1) & 7, v_byte = (lane & 1) * 8;
    float m_run[G], l_run[G], o_run[G][4];
    // grouped queries (G > 1), tensor-core path: lane (g, c) = (lane / 4, lane % 4) holds, for query head g, the
    // anchor and the sum of its warp's tokens, the output dims 8 n + 2 c, 8 n + 2 c + 1 (n = 0..15), and the
    // query fragments of the eight 16-dim steps
    const int mg = lane >> 2, mc = lane & 3;
    float mm = -INFINITY, ml = 0.f, mo[16][2];
    uint32_t qf[8][2];
    uint32_t meetings = 0;
    bool alive = true;
    // test hook: warp 0 never hands a stage back, so the copy thread's wait for a free stage runs out
    // (the hook's flag sits in shared memory next to the abort flag and is looked up at every release: a value kept in
    // a register for the whole kernel pushed the grouped-query variants, which are at their register limit, into spills)
    volatile int* hook_flag = abort_flag + 1;
    // A lane whose wait for a stage fails leaves the loop and, with it, the kernel, without another
    // warp-level operation (shuffles and warp barriers are defined over the lanes that have not exited);
    // at the meetings, which are rare, the warp votes so that its lanes go on or stop together.
    auto consumer_meet = [&]() {
        __syncwarp();
        if (lane == 0) mbar_arrive(meet);
        alive = __all_sync(0xffffffffu, alive && mbar_wait(meet, meetings & 1, abort_flag, p.w.status));
        ++meetings;
    };
    for (uint32_t it = 0; alive; ++it) {
        const uint32_t slot = it % kStages;
        if (!mbar_wait(full + slot * 8, (it / kStages) & 1, abort_flag, p.w.status)) break;
        const uint32_t st = slots + slot * kSlotBytes;
        const uint4 hw = lds128(st + kHdrOffset);
        StageHdr h;
        h.flags = (int)hw.x; h.unit = (int)hw.y; h.head = (int)hw.z; h.n_tok = (int)hw.w;
        if (h.flags & kFlagEnd) break;
        if (h.flags & kFlagFirst) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
                m_run[g] = -INFINITY;
                l_run[g] = 0.f;
                o_run[g][0] = o_run[g][1] = o_run[g][2] = o_run[g][3] = 0.f;
            }
        }
        if constexpr (G == 1) {
            // K piece of this lane: 32 dims = 4 chunks of 16 bytes, chunk c of row r stored at c ^ (r & 7)
            uint4 kraw[4];
    #pragma unroll
            for (int i = 0; i < 4; ++i) kraw[i] = lds128(st + k_off + ((((qr & 1) * 4 + i) ^ (trow & 7)) << 4));
            // V pieces of the warp's 8 tokens for this lane's 4 dims
            uint2 vraw[8];
    #pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int r = warp * 8 + j;
                vraw[j] = lds64(st + kKBytes + v_sub + r * 128 + ((v_chunk ^ (r & 7)) << 4) + v_byte);
                if (r >= h.n_tok) vraw[j] = make_uint2(0u, 0u);   // beyond the cache's end: whatever lies there must not reach the sum
            }
            const bool valid = trow < h.n_tok;
    #pragma unroll
            for (int g = 0; g < G; ++g) {
                // q piece: dims [32 qr, +32) of query head g, bf16 in the stage
                // packed multiply-adds (two fp32 FMAs per instruction on sm_100): the even and the odd dims
                // of a 32-bit word advance together, two chains of 16 instead of one of 32
                float2 s2 = make_float2(0.f, 0.f);
    #pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint4 qw = lds128(st + kQOffset + g * (kHeadDim * 2) + qr * 64 + i * 16);
                    s2 = __ffma2_rn(make_float2(bf_lo(qw.x), bf_hi(qw.x)), make_float2(bf_lo(kraw[i].x), bf_hi(kraw[i].x)), s2);
                    s2 = __ffma2_rn(make_float2(bf_lo(qw.y), bf_hi(qw.y)), make_float2(bf_lo(kraw[i].y), bf_hi(kraw[i].y)), s2);
                    s2 = __ffma2_rn(make_float2(bf_lo(qw.z), bf_hi(qw.z)), make_float2(bf_lo(kraw[i].z), bf_hi(kraw[i].z)), s2);
                    s2 = __ffma2_rn(make_float2(bf_lo(qw.w), bf_hi(qw.w)), make_float2(bf_lo(kraw[i].w), bf_hi(kraw[i].w)), s2);
                }
                float s = s2.x + s2.y;
                s += __shfl_xor_sync(0xffffffffu, s, 8);
                s += __shfl_xor_sync(0xffffffffu, s, 16);
                s = valid ? s * p.scale_log2e : -INFINITY;      // every lane of a token now holds its score
                float mx = s;
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                const float m_new = fmaxf(m_run[g], mx);
                // a warp whose tokens are all beyond the tile's end keeps its state (m_new may still be -inf)
                const float alpha = m_new == -INFINITY ? 1.f : exp2f(m_run[g] - m_new);
                const float pt = valid ? exp2f(s - m_new) : 0.f;
                float psum = pt;
                psum += __shfl_xor_sync(0xffffffffu, psum, 1);
                psum += __shfl_xor_sync(0xffffffffu, psum, 2);
                psum += __shfl_xor_sync(0xffffffffu, psum, 4);
                l_run[g] = l_run[g] * alpha + psum;
                float2 o01 = make_float2(o_run[g][0] * alpha, o_run[g][1] * alpha), o23 = make_float2(o_run[g][2] * alpha, o_run[g][3] * alpha);
    #pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float pj = __shfl_sync(0xffffffffu, pt, j);     // lane j (quarter 0) holds token j's weight
                    const float2 pp = make_float2(pj, pj);
                    o01 = __ffma2_rn(pp, make_float2(bf_lo(vraw[j].x), bf_hi(vraw[j].x)), o01);
                    o23 = __ffma2_rn(pp, make_float2(bf_lo(vraw[j].y), bf_hi(vraw[j].y)), o23);
                }
                o_run[g][0] = o01.x; o_run[g][1] = o01.y; o_run[g][2] = o23.x; o_run[g][3] = o23.y;
                m_run[g] = m_new;
            }
        } else {
            // ---- grouped queries: S = Q K^T and O += P V on the tensor cores (mma.sync), this warp's 8 tokens ----
            // The G query heads are the first rows of the 16-row operand (the others are zero registers).
            // Scores: 16-dim steps over K, B fragments by ldmatrix from the swizzled rows of the warp's
            // tokens.  Values: the probabilities, as bf16 hi + lo halves (two MMAs, fp32-grade accuracy),
            // against 8-dim blocks of V by ldmatrix.trans.  The instruction count no longer grows with G.
            if (h.flags & kFlagFirst) {
                mm = -INFINITY;
                ml = 0.f;
#pragma unroll
                for (int n = 0; n < 16; ++n) mo[n][0] = mo[n][1] = 0.f;
                const uint32_t qa = st + kQOffset + mg * (kHeadDim * 2) + mc * 4;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    qf[ks][0] = mg < G ? lds32(qa + ks * 32) : 0u;
                    qf[ks][1] = mg < G ? lds32(qa + ks * 32 + 16) : 0u;
                }
            }
            const int row0 = warp * 8;
            if (row0 + 8 > h.n_tok) {
                // beyond the cache's end: whatever lies there must not reach the sum (0 * NaN); this warp alone reads these rows
                for (int i = lane; i < 8 * 16; i += 32) {
                    const int r = row0 + (i >> 4), c = i & 15;
                    if (r >= h.n_tok) sts128(st + kKBytes + (c >> 3) * (kKBytes / 2) + r * 128 + ((c & 7) << 4), 0u, 0u, 0u, 0u);
                }
                __syncwarp();
            }
            // the lane's row of the 8 x 8 blocks it addresses: token row0 + (lane & 7), 16-byte chunk 4 i + (lane >> 3)
            const int lrow = row0 + (lane & 7), lch = lane >> 3;
            float sc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int ch = 4 * i + lch;
                uint32_t b[4];
                ldmatrix_x4(st + (ch >> 3) * (kKBytes / 2) + lrow * 128 + (((ch & 7) ^ (lrow & 7)) << 4), b);
                mma_16816(sc, qf[2 * i][0], qf[2 * i][1], b[0], b[1]);
                mma_16816(sc, qf[2 * i + 1][0], qf[2 * i + 1][1], b[2], b[3]);
            }
            const int t0 = row0 + 2 * mc;
            const float s0 = t0 < h.n_tok ? sc[0] * p.scale_log2e : -INFINITY;
            const float s1 = t0 + 1 < h.n_tok ? sc[1] * p.scale_log2e : -INFINITY;
            float mx = fmaxf(s0, s1);
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float m_new = fmaxf(mm, mx);
            const float alpha = m_new == -INFINITY ? 1.f : exp2f(mm - m_new);
            const float p0 = t0 < h.n_tok ? exp2f(s0 - m_new) : 0.f;
            const float p1 = t0 + 1 < h.n_tok ? exp2f(s1 - m_new) : 0.f;
            float psum = p0 + p1;
            psum += __shfl_xor_sync(0xffffffffu, psum, 1);
            psum += __shfl_xor_sync(0xffffffffu, psum, 2);
            ml = ml * alpha + psum;
            mm = m_new;
            const uint32_t h0 = bf16_rn_bits(p0), h1 = bf16_rn_bits(p1);
            const uint32_t p_hi = h0 | (h1 << 16);
            const uint32_t p_lo = bf16_rn_bits(p0 - __uint_as_float(h0 << 16)) | (bf16_rn_bits(p1 - __uint_as_float(h1 << 16)) << 16);
            // the hi halves ride in rows 0..7 of the operand and the lo halves in rows 8..15 (there are at most
            // eight query heads): one MMA per block gives both products, in rows g and g + 8 of the result
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int ch = 4 * i + lch;
                uint32_t b[4];
                ldmatrix_x4_trans(st + kKBytes + (ch >> 3) * (kKBytes / 2) + lrow * 128 + (((ch & 7) ^ (lrow & 7)) << 4), b);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int n = 4 * i + j;
                    float d0 = mo[n][0] * alpha, d1 = mo[n][1] * alpha, d2 = 0.f, d3 = 0.f;
                    mma_1688(d0, d1, d2, d3, p_hi, p_lo, b[j]);
                    mo[n][0] = d0 + d2;
                    mo[n][1] = d1 + d3;
                }
            }
        }
        if constexpr (G > 1) {
            if (h.flags & kFlagLast) {
                // Anchor merge of the eight warps' shares, all query heads at once.  The item's last tile is
                // consumed, so its stage (34 KB of K, V and q) serves as the meeting place: every warp
                // puts its G triples there, then warp g combines query head g.  Two meetings per item.
                consumer_meet();   // nobody reads the tile any more
                float* scr = reinterpret_cast<float*>(base + slot * kSlotBytes);
                static_assert(kConsumerWarps * kMaxQPerKv * kMergeStride * 4 <= kHdrOffset, "the meeting place fits in a stage");
                if (mg < G) {
                    float* mine = scr + (warp * G + mg) * kMergeStride;
#pragma unroll
                    for (int n = 0; n < 16; ++n) *reinterpret_cast<float2*>(mine + 8 * n + 2 * mc) = make_float2(mo[n][0], mo[n][1]);
                    if (mc == 0) {
                        mine[kHeadDim] = mm;
                        mine[kHeadDim + 1] = ml;
                    }
                }
                consumer_meet();
                if (warp < G && alive) {
                    const int g = warp;
                    float M = -INFINITY;
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, scr[(w * G + g) * kMergeStride + kHeadDim]);
                    float L = 0.f;
                    float4 O = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) {
                        const float* src = scr + (w * G + g) * kMergeStride;
                        const float mw = src[kHeadDim];
                        const float f = mw == -INFINITY ? 0.f : exp2f(mw - M);
                        L = fmaf(f, src[kHeadDim + 1], L);
                        const float4 ow = *reinterpret_cast<const float4*>(src + 4 * lane);
                        O.x = fmaf(f, ow.x, O.x); O.y = fmaf(f, ow.y, O.y); O.z = fmaf(f, ow.z, O.z); O.w = fmaf(f, ow.w, O.w);
                    }
                    float* dst = p.w.partials + ((size_t)h.unit * (p.n_kv_heads * G) + h.head * G + g) * kPartFloats;
                    *reinterpret_cast<float4*>(dst + 4 * lane) = O;
                    if (lane == 0) {
                        dst[kHeadDim] = M;
                        dst[kHeadDim + 1] = L;
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the stage goes back to the copy engine
            }
            __syncwarp();
            if (lane == 0 && !(warp == 0 && *hook_flag)) mbar_arrive(empty + slot * 8);
        } else {
            __syncwarp();
            if (lane == 0 && !(warp == 0 && *hook_flag)) mbar_arrive(empty + slot * 8);
            if (h.flags & kFlagLast) {
                // anchor merge of the eight warps' shares of this item
                float* mine = merge + warp * kMergeStride;
                *reinterpret_cast<float4*>(mine + 4 * lane) = make_float4(o_run[0][0], o_run[0][1], o_run[0][2], o_run[0][3]);
                if (lane == 0) {
                    mine[kHeadDim] = m_run[0];
                    mine[kHeadDim + 1] = l_run[0];
                }
                consumer_meet();
                if (warp == 0) {
                    float M = -INFINITY;
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, merge[w * kMergeStride + kHeadDim]);
                    float L = 0.f;
                    float4 O = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int w = 0; w < kConsumerWarps; ++w) {
                        const float mw = merge[w * kMergeStride + kHeadDim];
                        const float f = mw == -INFINITY ? 0.f : exp2f(mw - M);
                        L = fmaf(f, merge[w * kMergeStride + kHeadDim + 1], L);
                        const float4 ow = *reinterpret_cast<const float4*>(merge + w * kMergeStride + 4 * lane);
                        O.x = fmaf(f, ow.x, O.x); O.y = fmaf(f, ow.y, O.y); O.z = fmaf(f, ow.z, O.z); O.w = fmaf(f, ow.w, O.w);
                    }
                    float* dst = p.w.partials + ((size_t)h.unit * p.n_kv_heads + h.head) * kPartFloats;
                    *reinterpret_cast<float4*>(dst + 4 * lane) = O;
                    if (lane == 0) {
                        dst[kHeadDim] = M;
                        dst[kHeadDim + 1] = L;
                    }
                }
                consumer_meet();
            }
        }
    }
}

// ---- merge: rescale the chunks' partial outputs by their anchors ----------------------------------------
__global__ void __launch_bounds__(128) merge_kernel(const Params p) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int n_q_heads = p.n_kv_heads * p.q_per_kv;
    const int pair = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (pair >= p.n_req * n_q_heads) return;
    const int req = pair / n_q_heads, hq = pair - req * n_q_heads;
    const int u0 = p.w.unit_start[req], u1 = p.w.unit_start[req + 1];
    float M = -INFINITY;
    for (int u = u0; u < u1; ++u) M = fmaxf(M, p.w.partials[((size_t)u * n_q_heads + hq) * kPartFloats + kHeadDim]);
    float L = 0.f;
    float4 O = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int u = u0; u < u1; ++u) {
        const float* src = p.w.partials + ((size_t)u * n_q_heads + hq) * kPartFloats;
        const float mu = src[kHeadDim];
        const float f = mu == -INFINITY ? 0.f : exp2f(mu - M);
        L = fmaf(f, src[kHeadDim + 1], L);
        const float4 ou = *reinterpret_cast<const float4*>(src + 4 * lane);
        O.x = fmaf(f, ou.x, O.x); O.y = fmaf(f, ou.y, O.y); O.z = fmaf(f, ou.z, O.z); O.w = fmaf(f, ou.w, O.w);
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;    // an empty cache leaves a zero row
    float* dst = p.out + ((size_t)req * n_q_heads + hq) * kHeadDim;
    *reinterpret_cast<float4*>(dst + 4 * lane) = make_float4(O.x * inv, O.y * inv, O.z * inv, O.w * inv);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess) f = nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

static size_t up256(size_t v) { return (v + 255) & ~(size_t)255; }
static size_t max_units(int n_req, int max_kv_len) { return (size_t)n_req * ((max_kv_len + kChunkTokens - 1) / kChunkTokens); }

static Work carve(void* ws, int n_req, int max_kv_len, int n_q_heads) {
    uint8_t* b = static_cast<uint8_t*>(ws);
    const size_t U = max_units(n_req, max_kv_len);
    Work w;
    w.status = reinterpret_cast<int32_t*>(b);
    w.n_units = w.status + 1;
    size_t o = 256;
    w.unit_req = reinterpret_cast<int32_t*>(b + o); o += up256(U * 4);
    w.unit_chunk = reinterpret_cast<int32_t*>(b + o); o += up256(U * 4);
    w.unit_start = reinterpret_cast<int32_t*>(b + o); o += up256(((size_t)n_req + 1) * 4);
    w.partials = reinterpret_cast<float*>(b + o);
    (void)n_q_heads;
    return w;
}

}  // namespace attn
}  // namespace plora

using namespace plora::attn;

extern "C" PLORA_API size_t plora_attn_workspace_bytes(int32_t n_req, int32_t max_kv_len, int32_t n_kv_heads, int32_t q_per_kv) {
    if (n_req < 1 || max_kv_len < 1 || n_kv_heads < 1 || q_per_kv < 1) return 0;
    const size_t U = max_units(n_req, max_kv_len);
    return 256 + 2 * up256(U * 4) + up256(((size_t)n_req + 1) * 4) +
           up256(U * (size_t)n_kv_heads * q_per_kv * kPartFloats * sizeof(float));
}

extern "C" PLORA_API plora_status plora_attn_decode(const void* q, const void* k_cache, const void* v_cache,
                                                    const int32_t* kv_len, int32_t n_req, int32_t max_kv_len,
                                                    int32_t n_kv_heads, int32_t q_per_kv, int32_t head_dim, float scale,
                                                    float* out, void* workspace, size_t workspace_bytes, void* stream) {
    if (!q || !k_cache || !v_cache || !kv_len || !out || !workspace || n_req < 1 || max_kv_len < 1 || n_kv_heads < 1)
        return PLORA_ERR_INVALID_ARG;
    if (head_dim != kHeadDim || (q_per_kv != 1 && q_per_kv != 2 && q_per_kv != 4 && q_per_kv != 8)) return PLORA_ERR_UNSUPPORTED;
    if (((uintptr_t)q & 15) || ((uintptr_t)k_cache & 15) || ((uintptr_t)v_cache & 15) || ((uintptr_t)out & 15) ||
        ((uintptr_t)workspace & 255))
        return PLORA_ERR_INVALID_ARG;
    if (workspace_bytes < plora_attn_workspace_bytes(n_req, max_kv_len, n_kv_heads, q_per_kv)) return PLORA_ERR_WORKSPACE;
    if (!encode_tiled()) return PLORA_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Params p;
    p.w = carve(workspace, n_req, max_kv_len, n_kv_heads * q_per_kv);
    p.q = static_cast<const uint16_t*>(q);
    p.kv_len = kv_len;
    p.out = out;
    p.n_req = n_req;
    p.max_kv_len = max_kv_len;
    p.n_kv_heads = n_kv_heads;
    p.q_per_kv = q_per_kv;
    p.scale_log2e = scale * 1.4426950408889634f;
    // K and V as 4-D tensors [request][KV head][token][dim] of bf16; a box is 64 dims x 64 tokens of one
    // head, 128-byte swizzled (tokens beyond max_kv_len read as zeros)
    CUtensorMap tm[2];
    const cuuint64_t dims[4] = {(cuuint64_t)kHeadDim, (cuuint64_t)max_kv_len, (cuuint64_t)n_kv_heads, (cuuint64_t)n_req};
    const cuuint64_t strides[3] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)max_kv_len * kHeadDim * 2,
                                   (cuuint64_t)n_kv_heads * max_kv_len * kHeadDim * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)kTileTokens, 1, 1};
    const cuuint32_t es[4] = {1, 1, 1, 1};
    const void* bases[2] = {k_cache, v_cache};
    for (int i = 0; i < 2; ++i)
        if (encode_tiled()(&tm[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(bases[i]), dims, strides, box, es,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return PLORA_ERR_INVALID_ARG;

    int dev = 0, sm_count = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return PLORA_ERR_CUDA;
    prep_kernel<<<1, 1024, 0, st>>>(p);
    if (cudaGetLastError() != cudaSuccess) return PLORA_ERR_CUDA;

    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    void (*kern)(const CUtensorMap, const CUtensorMap, const Params) =
        q_per_kv == 1 ? partial_kernel<1> : q_per_kv == 2 ? partial_kernel<2> : q_per_kv == 4 ? partial_kernel<4> : partial_kernel<8>;
    static bool configured[4] = {false, false, false, false};
    const int ki = q_per_kv == 1 ? 0 : q_per_kv == 2 ? 1 : q_per_kv == 4 ? 2 : 3;
    if (!configured[ki]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) return PLORA_ERR_CUDA;
        configured[ki] = true;
    }
    const long long items = (long long)max_units(n_req, max_kv_len) * n_kv_heads;
    int grid = 2 * sm_count;
    if (grid > items) grid = (int)items;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = st;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, tm[0], tm[1], p) != cudaSuccess) return PLORA_ERR_CUDA;

    cudaLaunchConfig_t mc{};
    mc.gridDim = dim3((n_req * n_kv_heads * q_per_kv + 3) / 4);
    mc.blockDim = dim3(128);
    mc.stream = st;
    mc.attrs = attr;
    mc.numAttrs = 1;
    if (cudaLaunchKernelEx(&mc, merge_kernel, p) != cudaSuccess) return PLORA_ERR_CUDA;
    return PLORA_OK;
}

extern "C" PLORA_API plora_status plora_attn_set_debug(void* workspace, int64_t cycles, int32_t hook, void* stream) {
    if (!workspace || cycles < 0 || (hook != PLORA_HOOK_NONE && hook != PLORA_HOOK_WITHHOLD_RELEASE)) return PLORA_ERR_INVALID_ARG;
    if (hook != PLORA_HOOK_NONE && (cycles < 1 || cycles > PLORA_HOOK_MAX_CYCLES)) return PLORA_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t* w = static_cast<int32_t*>(workspace);
    const long long lim = cycles;
    if (cudaMemcpyAsync(w + kHookWord, &hook, 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(w + kLimitWord, &lim, 8, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return PLORA_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? PLORA_OK : PLORA_ERR_CUDA;
}

extern "C" PLORA_API plora_status plora_attn_status(void* workspace, void* stream, int32_t* host_out) {
    if (!workspace || !host_out) return PLORA_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(host_out, workspace, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return PLORA_ERR_CUDA;
    if (cudaMemsetAsync(workspace, 0, 4, st) != cudaSuccess) return PLORA_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? PLORA_OK : PLORA_ERR_CUDA;
}
