/*
 * plora.h — C ABI of the B200 (sm_100a) batched heterogeneous-adapter LoRA delta.
 *
 * For a batch of tokens, each tagged with an adapter id a_t, the library computes
 *
 *        y_t  +=  s_a * ( (x_t * A_a) * B_a ),        a = a_t
 *
 * over a pool of adapters held in this GPU's HBM.  A_a is [d_in, r_a], B_a is
 * [r_a, d_out] (paper Section II-A: y = x (W + A B); Section III-A: Y = X A B).
 * This is the paper's placement P1 / strategy E1 (Section V-A): both matrices are
 * resident in GPU memory and the GPU computes the delta without touching any
 * other device.  The shrink m = x A and expand y = m B halves (Section V-A,
 * strategy E4) are also exported on their own.
 *
 * General conventions
 *   - "dev" pointers are CUDA device pointers on the context's device; "host"
 *     pointers are ordinary host memory.  The library never takes ownership of a
 *     caller's buffer.
 *   - bf16 tensors are raw 16-bit patterns; x is [n_tok, d_in] row-major
 *     contiguous, y is fp32 [n_tok, d_out] row-major contiguous.  d_in and d_out
 *     must be multiples of 8.
 *   - adapter ids are int32 in [-1, n_adapters); -1 means "no adapter": the
 *     token's row of y is left as it is.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Unless stated otherwise a call only enqueues work on `stream` and returns
 *     without synchronising.
 *   - Every function returns a plora_status (0 = ok, negative = error) and never
 *     throws or aborts.  Errors that the host can see are returned before
 *     anything is launched.  Conditions only the device can see (an id outside
 *     [-1, n_adapters), a bounded wait that ran out) set a sticky device status
 *     word, read with plora_device_status; the kernels stay inside their buffers
 *     in that case (an out-of-range id is treated as -1).
 *   - One context serves one stream at a time; calls on one context are not
 *     thread-safe.
 */
#ifndef PLORA_H_
#define PLORA_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define PLORA_API __attribute__((visibility("default")))
#else
#define PLORA_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct plora_ctx plora_ctx; /* opaque, owned by the library */
typedef int32_t plora_status;

enum {
    PLORA_OK = 0,
    PLORA_ERR_INVALID_ARG = -1,    /* null pointer, negative size, size above the context's limits */
    PLORA_ERR_NOT_REGISTERED = -2, /* no pool registered for (layer, proj) */
    PLORA_ERR_BAD_ADAPTER_ID = -3, /* device status: an id outside [-1, n_adapters) was seen */
    PLORA_ERR_WORKSPACE = -4,      /* slab or workspace too small */
    PLORA_ERR_CUDA = -5,           /* a CUDA runtime call failed */
    PLORA_ERR_TIMEOUT = -6,        /* device status: a bounded device-side wait ran out */
    PLORA_ERR_UNSUPPORTED = -7,    /* shape outside what the kernels handle (rank > 128, d not multiple of 8, ...) */
    PLORA_ERR_DEBUG_CHECK = -8     /* device status, debug build only (compiled with -DPLORA_DEBUG): a kernel was about to
                                      read or write outside a buffer; the access was skipped */
};

/* Which kernels plora_lora_delta uses. */
enum {
    PLORA_PATH_AUTO = 0,    /* fused BGMV for short segments; in batches of 1024+ tokens the tensor-core
                               segmented GEMM takes the long ones: a CTA per tile of 64 rows when they make
                               at least 128 tiles together, a cluster of eight CTAs per tile when fewer */
    PLORA_PATH_UNFUSED = 1, /* BGMV shrink kernel then BGMV expand kernel, m in HBM workspace */
    PLORA_PATH_FUSED = 2,   /* fused BGMV for every segment */
    PLORA_PATH_SGMV = 3,    /* tensor-core segmented GEMM for every segment, a CTA per tile */
    PLORA_PATH_SGMV_SPLIT = 4 /* tensor-core segmented GEMM for every segment, a cluster of eight CTAs per tile */
};

/*
 * Create a context on CUDA device `device`.  Allocates the bucketing buffers
 * and kernel workspace for batches of up to `max_tokens` tokens over pools of up
 * to `max_adapters` adapters.  Synchronous.  *out is set only on success.
 */
PLORA_API plora_status plora_create(plora_ctx **out, int device, int32_t max_tokens, int32_t max_adapters);

/* Free everything the context owns (not the caller's slabs).  Synchronises the device. */
PLORA_API plora_status plora_destroy(plora_ctx *ctx);

/*
 * Adapter-pool registry (the paper keeps each adapter as a matrix pair (A, B)
 * attached to every injected weight of every layer, Sections II-A and VII-A; here
 * one pool = all adapters of one (layer, projection)).
 *
 * plora_pool_desc describes one pool in the paper's logical layout.  All arrays
 * are HOST arrays of length n_adapters; A[a] / B[a] point to bf16 matrices
 * [d_in, ranks[a]] and [ranks[a], d_out], row-major contiguous, in host memory
 * (ab_on_device = 0) or device memory (ab_on_device = 1).  Ranks must lie in
 * [1, 128].  scales[a] is s_a (for instance alpha / r_a).
 */
typedef struct {
    int32_t layer, proj;
    int32_t d_in, d_out;
    int32_t n_adapters;
    int32_t ab_on_device;
    const int32_t *ranks;
    const float *scales;
    const void *const *A;
    const void *const *B;
} plora_pool_desc;

/*
 * Bytes of device memory the library's private slab layout needs for this pool
 * (only layer..n_adapters and ranks are read).  Returns 0 if the description is
 * invalid or unsupported.  The caller allocates that much device memory,
 * 256-byte aligned, and keeps it alive while the pool is registered.
 */
PLORA_API size_t plora_pool_slab_bytes(const plora_pool_desc *desc);

/*
 * Repack the pool into `slab_dev` (library-private tiled layout, ranks padded
 * with zeros) and record its offset table under (layer, proj), replacing any
 * earlier registration of that pair.  The source matrices are not needed after
 * the call returns: it synchronises `stream` (registration is a set-up step).
 * From then on the slab is read-only for the library and must not be written by
 * the caller while the pool is registered: the delta kernels fetch adapter tiles
 * before they have joined the stream's order behind the preceding kernel.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE (slab_bytes too small or more
 * adapters than the context allows), CUDA.
 */
PLORA_API plora_status plora_register_pool(plora_ctx *ctx, const plora_pool_desc *desc, void *slab_dev, size_t slab_bytes,
                                 void *stream);

/* Padded maximum rank of a registered pool: the leading dimension `ldm` that
 * plora_shrink / plora_expand need at least.  Negative status on error. */
PLORA_API int32_t plora_pool_max_rank(plora_ctx *ctx, int32_t layer, int32_t proj);

/*
 * Token bucketing (once per step; every layer and projection of the step reuses
 * it).  The per-adapter request count B_i of the paper's cost model (Section
 * VI-B) is the length of adapter i's segment.
 *
 * adapter_ids_dev: int32 [n_tok] on the device.  Produces, in context-owned
 * device memory:
 *   perm         int32 [n_tok]      token indices ordered by (id, token index), id -1 last
 *   seg_adapter  int32 [cap]        ascending distinct ids >= 0 present; tail = -1
 *   seg_start    int32 [cap + 1]    start of each segment in perm; entry n_seg and tail = n_active
 *   n_seg, n_active  int32 scalars  segments, tokens with id >= 0
 * with cap = min(n_tok, n_adapters).  The result is unique (stable order) and
 * deterministic.  Errors: INVALID_ARG (null, n_tok < 0 or > max_tokens,
 * n_adapters < 1 or > max_adapters).
 *
 * Reuse rule.  A bucket made by plora_bucket is the caller's statement that the ids
 * buffer keeps its contents: every later delta call that passes the same
 * (adapter_ids_dev, n_tok) and a pool of the same n_adapters uses it as it is, until
 * the next plora_bucket.  Call plora_bucket again after writing new ids into the
 * buffer, also when the pointer is unchanged.  A delta call that finds no such bucket
 * buckets for itself, and that bucket serves this one call only (all projections of a
 * grouped call share it): the library cannot see whether the buffer was rewritten, or
 * its address given to another tensor, before the next call.
 *
 * The bucket, and for pools of mixed ranks the ordering of its work units by rank
 * that the first delta call on such a pool adds to it, are device state of the
 * context, produced in stream order.  The library tracks on the host which ids
 * and which pool ranks that state belongs to and rebuilds it when a call needs
 * another; a captured CUDA graph replays only the launches that were needed at
 * capture time, so a graph should contain its own plora_bucket call (then it is
 * self-contained), or nothing that changes the bucket or uses a pool with other
 * ranks may run on the context between its replays.
 */
PLORA_API plora_status plora_bucket(plora_ctx *ctx, const int32_t *adapter_ids_dev, int32_t n_tok, int32_t n_adapters,
                          void *stream);

/* Device pointers to the current bucket's arrays (valid until the next plora_bucket
 * or plora_destroy; written by work enqueued on the bucket's stream). */
PLORA_API plora_status plora_bucket_view(plora_ctx *ctx, const int32_t **perm, const int32_t **seg_adapter,
                               const int32_t **seg_start, const int32_t **n_seg, const int32_t **n_active);

/*
 * The LoRA delta of one projection (Section V-A, strategy E1):
 *     y[t, :] += s_a * ((x[t, :] * A_a) * B_a),  a = adapter_ids[t]
 * x_dev bf16 [n_tok, d_in], y_dev fp32 [n_tok, d_out] (holds the base projection
 * output on entry), both on the device; d_in/d_out are the registered pool's.
 * Uses the context's current bucket when plora_bucket was last called with this
 * same (adapter_ids_dev, n_tok) and the pool's n_adapters; otherwise buckets
 * first, for this call only (see the reuse rule at plora_bucket).  Every adapter
 * present in the batch is read from HBM once per call, whatever its number of tokens
 * (Section VI-B).  Each element of y receives exactly one addition, so results are
 * bit-reproducible run to run.
 * Tensor memory.  Segments that take the tensor-core path (PLORA_PATH_AUTO on batches
 * of 1024+ tokens, PLORA_PATH_SGMV and PLORA_PATH_SGMV_SPLIT always) run in a kernel whose CTAs each allocate 256
 * of an SM's 512 tensor-memory columns, two CTAs per SM (one per SM for pools with
 * ranks above 64).  The allocation instruction has no time limit: it blocks while
 * another kernel resident on the same SM (a base-model GEMM on a second stream, say)
 * holds the columns it needs, and goes on when they are freed.  Do not run this call
 * concurrently with a kernel that keeps more than half of the tensor memory for its
 * whole lifetime and itself waits for this call.
 * Errors: INVALID_ARG, NOT_REGISTERED, CUDA.
 */
PLORA_API plora_status plora_lora_delta(plora_ctx *ctx, const void *x_dev, const int32_t *adapter_ids_dev, int32_t n_tok,
                              int32_t layer, int32_t proj, float *y_dev, void *stream);

/*
 * The LoRA delta of several projections that do not depend on one another, in one call (the
 * paper attaches adapters to the query, key and value generation, the output projection and
 * the FFN weights of every layer, Section II-A: q, k and v of a layer read the same activations
 * and can run together, and so can up and gate).  Equivalent to n calls of plora_lora_delta;
 * projections whose pools have the same shape (d_in, d_out, adapter count, largest rank) share
 * one kernel launch, which matters at decode sizes where a launch is only a few microseconds
 * of work.  x_dev[g], layers[g], projs[g], y_dev[g] describe projection g; the arrays are HOST
 * arrays of length n, 1 <= n <= 4; the x_dev[g] may or may not be the same buffer; the y_dev[g]
 * must be distinct.  Same bucket rule and errors as plora_lora_delta.
 */
PLORA_API plora_status plora_lora_delta_group(plora_ctx *ctx, int32_t n, const void *const *x_dev,
                                              const int32_t *adapter_ids_dev, int32_t n_tok, const int32_t *layers,
                                              const int32_t *projs, float *const *y_dev, void *stream);

/*
 * The two halves on their own (Section V-A, strategy E4: m = x A, then y = m B).
 * m_dev is fp32 [n_tok, ldm] on the device, ldm >= plora_pool_max_rank.
 * plora_shrink writes m[t, k] = sum_i x[t, i] A_a[i, k] (unscaled) for k < r_a and 0
 * for the other columns and for tokens with id -1.  plora_expand computes
 * y[t, :] += s_a * (m[t, :r_a] * B_a).  Same bucket rule and errors as above.
 */
PLORA_API plora_status plora_shrink(plora_ctx *ctx, const void *x_dev, const int32_t *adapter_ids_dev, int32_t n_tok,
                          int32_t layer, int32_t proj, float *m_dev, int32_t ldm, void *stream);
PLORA_API plora_status plora_expand(plora_ctx *ctx, const float *m_dev, int32_t ldm, const int32_t *adapter_ids_dev,
                          int32_t n_tok, int32_t layer, int32_t proj, float *y_dev, void *stream);

/* The same split with a 2-byte m, as the paper's strategy E4 ships it between the two halves
 * (Section VI-B: its transfer term counts S = 2 bytes per value of m).
 * plora_shrink_m16: m_bf16[t, 0..ldm) = bf16(x_t A[a_t]), rounded to nearest even from the fp32 sum;
 * zeros beyond the adapter's rank and for tokens without an adapter.  plora_expand_m16:
 * y_t += s * m_bf16[t] * B[a_t], values beyond the adapter's rank ignored.  m_bf16: device, bf16
 * [n_tok, ldm] row-major, 16-byte aligned, ldm >= the pool's largest padded rank and a multiple of 8.
 * One rounding of m to bf16 costs about 2e-3 of max|delta| (inside the 5e-3 contract, far above the
 * fp32 path's 2e-7).  Same errors and stream semantics as plora_shrink / plora_expand. */
PLORA_API plora_status plora_shrink_m16(plora_ctx *ctx, const void *x_bf16_dev, const int32_t *adapter_ids_dev,
                                        int32_t n_tok, int32_t layer, int32_t proj, void *m_bf16_dev, int32_t ldm,
                                        void *stream);
PLORA_API plora_status plora_expand_m16(plora_ctx *ctx, const void *m_bf16_dev, int32_t ldm,
                                        const int32_t *adapter_ids_dev, int32_t n_tok, int32_t layer, int32_t proj,
                                        float *y_dev, void *stream);

/*
 * Same operation as plora_lora_delta with HOST buffers: copies x, ids and y to
 * context-owned device staging buffers, buckets, runs the delta and copies y
 * back, then waits until y_host holds the result.  Pinned host memory makes
 * the copies asynchronous to each other but is not required.
 */
PLORA_API plora_status plora_lora_delta_host(plora_ctx *ctx, const void *x_host, const int32_t *adapter_ids_host,
                                   int32_t n_tok, int32_t layer, int32_t proj, float *y_host, void *stream);

/*
 * The pipelined form of the above, for a step that makes many such calls (one per layer and
 * projection, Section II-A).  It queues the work and returns; y_host[g] holds its result only
 * after plora_host_sync.  n projections (1..4) that share one input are served together:
 * x_host is copied once, y_host[g] += delta of pool (layers[g], projs[g]); all n pools must have
 * the same d_in.  The copies to the device run on a stream of the context's own, the kernels on
 * `stream`, the copies back on a second stream of the context's own, over a ring of four staging
 * sets, so one call's copy back, the next call's kernels and the following call's copy in overlap
 * (both directions of the host link in use at once).  x_host, adapter_ids_host and y_host[g]
 * must stay untouched until plora_host_sync returns, and should be pinned: from pageable memory
 * the copies are correct but each blocks the calling thread.  The same ids may be passed to
 * every call of a step; they are bucketed again per call.
 * Errors as plora_lora_delta_group; PLORA_ERR_INVALID_ARG also if the pools' d_in differ.
 * The first call at a new largest shape allocates staging memory and synchronises.
 *
 * plora_host_sync: blocks the calling thread until every queued call's result is in host memory.
 */
PLORA_API plora_status plora_lora_delta_host_async(plora_ctx *ctx, int32_t n, const void *x_host,
                                                   const int32_t *adapter_ids_host, int32_t n_tok, const int32_t *layers,
                                                   const int32_t *projs, float *const *y_host, void *stream);
PLORA_API plora_status plora_host_sync(plora_ctx *ctx);

/*
 * The LoRA delta for callers that must not allocate device memory.  (The paper has no
 * counterpart for this entry point; it exists for the way the library is embedded.)
 *
 * Some hosts of this library cannot call cudaMalloc at the point where they need the
 * delta: a serving loop that may not stall (cudaMalloc and cudaFree synchronise the whole
 * device), a process whose device memory was handed out in full at start-up, or code
 * running under an allocator it does not control.  This call computes what
 * plora_lora_delta computes (the same result within the tolerance of the fp32 paths: the
 * order of the additions differs), by the shrink kernel followed by the expand kernel, and keeps
 * the intermediate m = x A in a fixed array that is part of the library image instead of
 * in allocated workspace.  It calls no cudaMalloc, no cudaFree and no allocating library
 * routine; it only enqueues kernels on `stream` (bucketing first if the context's current
 * bucket does not match, as plora_lora_delta does).
 *
 * The array holds PLORA_NOALLOC_SCRATCH_FLOATS floats (1 MiB) and every GPU that loads the
 * library carries it until the process exits.  The call needs n_tok * R floats of it, R
 * being the pool's padded maximum rank (plora_pool_max_rank): for instance 16384 tokens at
 * rank 16 or 2048 tokens at rank 128.  A larger request is refused with
 * PLORA_ERR_WORKSPACE before anything is launched.
 *
 * The first call on a device looks up the array's device address (once per device) before
 * it launches; that lookup may make the CUDA runtime load the library's device code onto the
 * device, which allocates and synchronises inside the driver, so only the calls after the first
 * are free of allocation.  Make the first call during set-up, outside any stream capture, and not
 * at the same time as another thread's first call on that device (the address is cached without
 * a lock; later calls only read it).  All calls, on all
 * contexts of a device, share the one array, and it keeps what the previous call left in
 * it: the shrink kernel rewrites every row the expand kernel will read (rows of tokens
 * without an adapter are written as zeros), so nothing has to be cleared between calls,
 * but two calls whose kernels overlap on the GPU (different streams, no ordering between
 * them) race on it and give wrong results.  Keep them on one stream or order them with
 * events.
 *
 * Arguments, bucket rule and other errors are those of plora_lora_delta.
 */
#define PLORA_NOALLOC_SCRATCH_FLOATS (1 << 18)
PLORA_API plora_status plora_lora_delta_noalloc(plora_ctx *ctx, const void *x_dev, const int32_t *adapter_ids_dev,
                                                int32_t n_tok, int32_t layer, int32_t proj, float *y_dev, void *stream);

/* Choose the kernels plora_lora_delta uses (PLORA_PATH_*); takes effect at the next
 * plora_bucket.  `sgmv_min_rows` (> 0) is the segment length from which AUTO sends a
 * segment to the tensor-core path; pass 0 to keep the default. */
PLORA_API plora_status plora_set_path(plora_ctx *ctx, int32_t path, int32_t sgmv_min_rows);

/* The 16-bit type of x, A and B: bf16 (the default) or IEEE half, the paper's own FP16 (its cost model
 * counts S = 2 bytes per value either way).  Pools are stored as 16-bit patterns, so the setting only
 * tells the kernels how to read them: it applies to every later call on this context and must match
 * what the caller registered and passes.  Accumulation and y stay fp32; the tensor-core path then
 * carries m as half hi + lo.  plora_shrink_m16 / plora_expand_m16 keep a bf16 m. */
#define PLORA_INPUT_BF16 0
#define PLORA_INPUT_FP16 1
PLORA_API plora_status plora_set_input_type(plora_ctx *ctx, int32_t type);

/*
 * Hint about the inputs of the following calls (no counterpart in the paper; default 0).  The fused decode
 * kernels are launched so that they may start while the previous kernel of the stream is still running
 * (programmatic dependent launch).  By default they read x only after that kernel has completed, because
 * it may be the kernel that produces x.  With resident = 1 the caller states that the x of every
 * following call was complete in memory before the previous kernel of the stream began: true when deltas
 * are issued back to back on inputs produced earlier (q/k/v of a layer, a benchmark on resident inputs),
 * false when the kernel right before a call writes its x and signals its dependents early.  The kernels
 * then stream and multiply x while the previous kernel drains; they still write nothing (workspace, y)
 * and read no y before it has completed, and the results are bit-identical to those with resident = 0.
 * Wrong use is a data race on x, nothing else.  The tensor-core path and the unfused halves ignore the hint.
 * Host-side setting of the context, no device work; PLORA_ERR_INVALID_ARG for a null context or a value
 * other than 0 or 1.
 */
PLORA_API plora_status plora_set_inputs_resident(plora_ctx *ctx, int32_t resident);

/*
 * Diagnostics of the bounded device-side waits (no counterpart in the paper).  Every wait inside the
 * kernels (on a shared-memory barrier, or on partial sums from another CTA) gives up after a number of
 * SM clock cycles, records PLORA_ERR_TIMEOUT in the status word, and the kernel winds down: no role
 * issues further copies, the copies already issued are waited for, tensor memory is freed, y may hold
 * partial results for that call.  The context stays usable.
 * plora_set_wait_limit: cycles > 0 sets the limit for this context's later launches; 0 restores the
 * default (4e9, about two seconds).
 * plora_set_test_hook: for tests only.  PLORA_HOOK_WITHHOLD_RELEASE makes one consumer of every CTA
 * never hand its stages back to the copy warp, so that the copy warp's wait for a free stage runs out
 * (at that point every copy it issued has landed).  Accepted only while a wait limit of at most
 * PLORA_HOOK_MAX_CYCLES is set; PLORA_HOOK_NONE switches it off.
 */
#define PLORA_HOOK_NONE 0
#define PLORA_HOOK_WITHHOLD_RELEASE 1
#define PLORA_HOOK_MAX_CYCLES (1 << 24)
PLORA_API plora_status plora_set_wait_limit(plora_ctx *ctx, int64_t cycles);
PLORA_API plora_status plora_set_test_hook(plora_ctx *ctx, int32_t hook);

/*
 * Read-bandwidth probe (no counterpart in the paper; a measuring aid for the roofline).  Reads
 * `bytes` bytes (a multiple of 16, 16-byte aligned) of device memory at buf_dev once, with 16-byte
 * loads from every SM, and folds them into a checksum in sink_dev (device, at least 4 bytes per
 * launched block: 64 KiB always suffices), so the loads cannot be optimised away.  The caller times
 * it with events on `stream`; bytes / time is what a kernel that only reads can get from HBM on this
 * part, which is the fair ceiling for the decode path (its traffic is almost all adapter reads),
 * whereas a copy's figure counts reads and writes.  Runs on the current device.
 */
PLORA_API plora_status plora_stream_read(const void *buf_dev, size_t bytes, void *sink_dev, size_t sink_bytes,
                                         void *stream);

/* Synchronise `stream`, copy the sticky device status word to *host_out (0 or a
 * PLORA_ERR_* value) and clear it. */
PLORA_API plora_status plora_device_status(plora_ctx *ctx, void *stream, int32_t *host_out);

/* Kernels launched by this context since creation (host-side counter). */
PLORA_API int64_t plora_launch_count(plora_ctx *ctx);

PLORA_API const char *plora_status_string(plora_status s);

/* ---- Cost model of the LoRA computation (paper Section VI-B: the table of per-strategy cost terms
 * and the equation T_LoRA = max{T_Base, T_LoRA_dev} + T_LoRA_GPU).  Host arithmetic only: nothing
 * is launched, no context is needed.  The benchmark's roofline is strategy E1's memory term of this
 * model (every adapter present is read once per step, S bytes per value) plus the activations.
 *
 * Hardware: throughputs in flop/s, bandwidths in byte/s, latency in seconds. */
typedef struct {
    double c_gpu, w_gpu;    /* GPU compute throughput and HBM bandwidth */
    double c_dev, w_dram;   /* per-device near-data compute throughput and DRAM bandwidth */
    double n_dev;           /* number of devices */
    double l_link, w_link;  /* one-way link latency and link bandwidth */
} plora_cost_hw;

/* Per strategy j = 0..3 (the paper's E1..E4): GPU time, device compute time, device-to-GPU transfer
 * time; then the sums over the strategies and the total. */
typedef struct {
    double t_gpu[4], t_dev_cpt[4], t_dev_trs[4];
    double t_lora_gpu, t_lora_dev, t_lora;
} plora_cost_terms;

/* ranks: host [n_adapters], R_i >= 1.  batch: host [n_adapters][4] row-major, batch[i][j] = requests of
 * adapter i served under strategy E(j+1), >= 0.  d: model dimension D.  value_bytes: S (2 under FP16).
 * t_base: profiled base-model GPU time.  A strategy nobody uses contributes zero to every term; a
 * memory argument sums only over the adapters that serve a request under that strategy.
 * Returns PLORA_ERR_INVALID_ARG for null pointers, non-positive hardware parameters, d, value_bytes or
 * ranks, or negative batch entries. */
PLORA_API plora_status plora_cost_model(const plora_cost_hw *hw, int32_t n_adapters, const int32_t *ranks,
                                        const double *batch, double d, double value_bytes, double t_base,
                                        plora_cost_terms *out);

/* ---- Decode attention (paper Section V-B): for every request, one query token against the request's
 * KV cache, O = softmax(scale * q K^T) V per head.  The cache is streamed once (the path is bound by
 * HBM bandwidth on the KV bytes); chunks of 256 tokens of one (request, KV head) are the partitions of
 * the paper's integral execution strategy: each runs all three steps with a partial softmax that keeps
 * its anchor (maximum), a second kernel rescales the partial outputs into the exact result.
 *
 * q        device bf16 [n_req][n_kv_heads * q_per_kv][head_dim]; query head h reads KV head h / q_per_kv
 * k_cache  device bf16 [n_req][n_kv_heads][max_kv_len][head_dim] (v_cache alike); 16-byte aligned
 * kv_len   device int32 [n_req]: tokens of the request's cache that are valid (clamped to [0, max_kv_len]);
 *          0 leaves a zero row of out.  What lies beyond kv_len is never used.
 * out      device fp32 [n_req][n_kv_heads * q_per_kv][head_dim], overwritten
 * workspace  device, 256-byte aligned, at least plora_attn_workspace_bytes(...) bytes; its first 256
 *          bytes must be zero before the first call (they hold the sticky status word); contents are
 *          scratch between calls.  One workspace serves one stream at a time.
 * head_dim must be 128 and q_per_kv one of 1, 2, 4, 8 (else PLORA_ERR_UNSUPPORTED).  Work is only
 * enqueued on `stream`.  A bounded device wait that runs out sets PLORA_ERR_TIMEOUT in the status word
 * (plora_attn_status synchronises the stream, returns the word and clears it). */
PLORA_API size_t plora_attn_workspace_bytes(int32_t n_req, int32_t max_kv_len, int32_t n_kv_heads, int32_t q_per_kv);
PLORA_API plora_status plora_attn_decode(const void *q_bf16_dev, const void *k_cache_dev, const void *v_cache_dev,
                                         const int32_t *kv_len_dev, int32_t n_req, int32_t max_kv_len,
                                         int32_t n_kv_heads, int32_t q_per_kv, int32_t head_dim, float scale,
                                         float *out_dev, void *workspace_dev, size_t workspace_bytes, void *stream);
PLORA_API plora_status plora_attn_status(void *workspace_dev, void *stream, int32_t *host_out);
/* The wait limit and test hook of plora_set_wait_limit / plora_set_test_hook for the attention kernels,
 * which have no context: the settings live in the workspace's header (zero = defaults) and hold for later
 * calls with this workspace.  cycles 0 restores the default limit; a hook other than PLORA_HOOK_NONE needs
 * 0 < cycles <= PLORA_HOOK_MAX_CYCLES.  Synchronises `stream`. */
PLORA_API plora_status plora_attn_set_debug(void *workspace_dev, int64_t cycles, int32_t hook, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* PLORA_H_ */
