/*
 * libape -- APE (Adaptive Parallel Encoding, arxiv 2502.05431) attention for NVIDIA B200 (sm_100a).
 *
 * C ABI: plain pointers and sizes only.  Unless said otherwise a pointer is a DEVICE pointer that the
 * caller owns; arrays of descriptors (requests, spans) are HOST arrays that are read during the call and
 * may be freed as soon as it returns.  Every function returns APE_OK (0) or a negative ape_status code;
 * nothing throws, aborts, traps or prints.  All tensors are bf16 with the head dimension contiguous;
 * strides are in ELEMENTS.
 *
 * Data model (paper, section "Parallel Encoding": a query is augmented by a subset of independently
 * pre-cached contexts; section "Prepending Shared Prefix": one shared prefix in front of all of them):
 *   - one KV pool  K, V : [n_tokens, H_kv, d]  holds every cached token of every request;
 *   - the shared prefix, each cached context C_i and the query's own K/V are SPANS (start, len) of pool
 *     tokens.  Contexts are addressed through the span table only, never re-packed, so inserting,
 *     removing or re-ordering contexts is an edit of that table;
 *   - query rows Q and outputs O : [rows, H_q, d]; consecutive query heads share a KV head
 *     (g = h / (H_q / H_kv)).
 *
 * Two operations, each split into a plan (host work: validation, tile lists, upload; may block) and
 * a launch (asynchronous on the caller's stream, no allocation, no host synchronisation):
 *
 *   ape_attend           Eq. 5 of the paper (section "Formulation"): softmax attention of the query rows over
 *                        [prefix | all contexts | causal query segment] in which context logits are
 *                        divided by the temperature T and the summed context weight Z_C enters as Z_C^S.
 *   ape_encode_contexts  the pre-caching attention (section "Parallel Encoding", first step): every
 *                        context row attends to the whole prefix and causally to its own context only.
 */
#ifndef APE_H_
#define APE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ape_handle_s *ape_handle_t;
typedef struct ape_plan_s *ape_plan_t;

enum ape_status {
    APE_OK = 0,
    APE_ERR_INVALID_ARG = -1, /* null pointer, negative count, span outside the pool, len < q_len ...      */
    APE_ERR_SHAPE = -2,       /* H_q % H_kv != 0, H_q/H_kv not a power of two <= 16, head_dim not 64 or 128 */
    APE_ERR_ALIGN = -3,       /* pointer not 16-byte aligned or stride not a multiple of 8 elements        */
    APE_ERR_RANGE = -4,       /* T or S not finite and > 0, kv_extra outside the reserved capacity         */
    APE_ERR_LAYOUT = -5,      /* a tensor cannot be described to the copy engine (extent over 2^31 ...)     */
    APE_ERR_WORKSPACE = -6,   /* workspace missing, misaligned (256 B) or too small                        */
    APE_ERR_CUDA = -7,        /* a CUDA runtime or driver call failed                                      */
    APE_ERR_TIMEOUT = -8,     /* a kernel gave up on a bounded wait (reported by ape_get_status)           */
    APE_ERR_NOMEM = -9,       /* host or device allocation failed while planning                           */
    APE_ERR_MODE = -10        /* plan used with the wrong entry point                                      */
};

typedef enum { APE_PREFILL = 0, APE_DECODE = 1 } ape_mode_t;

typedef struct {
    int32_t n_q_heads;   /* H_q                                                  */
    int32_t n_kv_heads;  /* H_kv, divides H_q; H_q/H_kv a power of two <= 16     */
    int32_t head_dim;    /* d: 64 or 128                                         */
    float softmax_scale; /* logit scale c; 0 selects 1/sqrt(d) (Eq. 1)           */
} ape_shape_t;

typedef struct { int64_t start, len; } ape_span_t;        /* tokens of the KV pool, len >= 0 */

typedef struct {          /* K and V share geometry: element (t, g, e) at base[t*token_stride + g*head_stride + e] */
    const void *k, *v;
    int64_t n_tokens, token_stride, head_stride;
} ape_kv_pool_t;

typedef struct {          /* Q or O rows: element (r, h, e) at data[r*token_stride + h*head_stride + e] */
    void *data;
    int64_t n_rows, token_stride, head_stride;
} ape_rows_t;

typedef struct {          /* one request (HOST struct; ctx is a HOST array) */
    int64_t q_start, q_len;        /* its rows of Q and O; q_len >= 1 (decode: q_len == 1)                     */
    ape_span_t prefix;             /* shared prefix P, len may be 0                                            */
    const ape_span_t *ctx;         /* the N cached contexts C_1..C_N in any order; entries may be empty        */
    int32_t n_ctx;                 /* N >= 0                                                                   */
    ape_span_t query_kv;           /* the query segment's own K/V, len l_k >= q_len; row i sees keys            */
                                   /* j <= i + (l_k - q_len) (causal, aligned to the end)                      */
    int64_t query_kv_capacity;     /* >= query_kv.len: pool tokens reserved from query_kv.start for appends    */
} ape_request_t;

/* Library instance bound to one device.  Allocates a 4-byte device status word.  `device` is a CUDA ordinal.
 * Every entry point makes its handle's device current while it runs and puts the caller's current device back before
 * it returns. */
int ape_create(ape_handle_t *handle, int device);
int ape_destroy(ape_handle_t handle);

/*
 * Plans made after this call use at most n_sm thread blocks (one per SM) instead of the whole GPU, e.g. to leave SMs to
 * a collective or another stream that runs beside the attention; 0 restores the device's SM count.  The split of the
 * key/value stream over thread blocks (the split-KV of the appendix "Hierarchical Formula for Softmax Attention")
 * follows the budget, the result does not depend on it beyond rounding.  1 <= n_sm <= SMs of the device, else
 * APE_ERR_INVALID_ARG.  Plans that already exist keep their split.
 */
int ape_set_sm_budget(ape_handle_t handle, int32_t n_sm);

/*
 * Plan an attend over n_req independent requests that share one pool and one Q / O tensor.
 * mode APE_PREFILL: tensor-core kernel for q_len rows per request.  mode APE_DECODE: q_len must be 1;
 * split-KV streaming kernel.  `lse` (nullable, device, fp32 [q rows, H_q]) receives the natural log of
 * Eq. 5's denominator.  Builds tile lists and work assignments, uploads them (cudaMalloc + blocking copy).
 * The plan keeps the device pointers given here; their contents may change between launches.
 */
int ape_attend_plan(ape_handle_t handle, const ape_shape_t *shape, const ape_kv_pool_t *pool,
                    const ape_rows_t *q, const ape_rows_t *out, float *lse,
                    const ape_request_t *requests, int32_t n_req, ape_mode_t mode, ape_plan_t *plan);

/*
 * Same as ape_attend_plan, for the per-context form of the appendix "Hierarchical Formula for APE" (Eq. 11-12): every
 * context C_i keeps its own softmax and enters the final merge with S * LogSumExp_i, i.e. the context mass is
 * sum_i Z_i^S instead of Eq. 5's (sum_i Z_i)^S.  The two forms agree when S = 1 or when there is one context; this
 * form depends on the context boundaries (contexts are never fused), and is the building block of the
 * tree-structured merge the paper names as a future direction.  Launch with ape_attend as usual.
 * APE_PREFILL plans run in two passes (ape_attend then launches four kernels): per query row the log-sum-exp of every
 * context, then the same attention as ape_attend_plan with (S - 1) * LogSumExp_i added to the logits of context i, which
 * gives its tokens exactly the weights of Eq. 11-12; the plan's workspace also holds 16 bytes per (context, query row,
 * query head).  APE_DECODE plans keep one partial per context and cut their work items at every context boundary.
 */
int ape_attend_plan_per_context(ape_handle_t handle, const ape_shape_t *shape, const ape_kv_pool_t *pool,
                                const ape_rows_t *q, const ape_rows_t *out, float *lse,
                                const ape_request_t *requests, int32_t n_req, ape_mode_t mode, ape_plan_t *plan);

/*
 * Same as ape_attend_plan, for contexts that form trees (appendix "Future Directions": each context a tree-like
 * hierarchy, evaluated along each branch with intermediate results merged on the way; built on the appendix
 * "Hierarchical Formula for APE", Eq. 11-12).  requests[r].ctx[i] is node i of request r: its own tokens (the span may be
 * empty: a node that only groups its children); parent[r][i] is its parent node, -1 for a top-level node, and
 * parent[r][i] < i (children are listed after their parent).  At most 16 levels.
 * Evaluation, per query row: inside a node its members -- its own tokens (logits divided by T) and its finished child
 * nodes -- merge by the plain hierarchical softmax identity into the node's output V_n and log-sum-exp A_n; a node with
 * scaled[r][i] != 0 enters its parent's merge with S * A_n (the A^{h'} = S * LogSumExp of Eq. 11), the others with A_n;
 * the top-level nodes and the non-context segment meet in the final softmax.  `scaled` (or scaled[r]) may be NULL: then
 * exactly the top-level nodes are scaled, i.e. every top-level tree is one context of Eq. 11-12.  Two ends of this
 * family are printed formulas: one node per context gives Eq. 11-12 (ape_attend_plan_per_context), one tree over all
 * contexts gives Eq. 5 (ape_attend_plan).  The paper prints no formula for deeper hierarchies; where S applies along a
 * branch is this library's reading, made explicit by `scaled`.
 * Launch with ape_attend.  APE_PREFILL plans run in two passes like the per-context form (the bias of a node's tokens is
 * the sum of (S - 1) * A_a over the scaled nodes a on its path to the top, itself included; 16 bytes of workspace per
 * (node, query row, query head)); APE_DECODE plans cut their work items at node boundaries and merge the partials with a
 * stack of accumulators.  APE_ERR_INVALID_ARG for a malformed tree.
 */
int ape_attend_plan_tree(ape_handle_t handle, const ape_shape_t *shape, const ape_kv_pool_t *pool,
                         const ape_rows_t *q, const ape_rows_t *out, float *lse,
                         const ape_request_t *requests, int32_t n_req,
                         const int32_t *const *parent, const uint8_t *const *scaled, ape_mode_t mode, ape_plan_t *plan);

/*
 * Decode for a batch of requests that attend to the SAME cached contexts (the serving case the paper's cache argument
 * describes: many queries over one set of pre-encoded documents or shots; section "Parallel Encoding", pre-caching).
 * Every request has q_len 1, its row of Q directly follows the previous request's (q_start = requests[0].q_start + r),
 * and the context tokens of all requests are the same set (any split into contexts, any order); prefixes and query
 * segments are per request.  The context K/V is then read ONCE for the whole batch: the context pass runs on the tensor
 * cores with the batch's query rows as one block of rows, the rest (prefix + the request's own growing query segment)
 * runs per request, and one merge applies Eq. 5 per request.  Launch with ape_attend (T, S, kv_extra as for APE_DECODE).
 * APE_ERR_INVALID_ARG if the requests do not share their contexts or their rows are not consecutive.
 */
int ape_attend_plan_shared(ape_handle_t handle, const ape_shape_t *shape, const ape_kv_pool_t *pool,
                           const ape_rows_t *q, const ape_rows_t *out, float *lse,
                           const ape_request_t *requests, int32_t n_req, ape_plan_t *plan);

/*
 * Plan the block-diagonal encoding of n_ctx contexts against one shared prefix.  `q` and `out` are aligned
 * with the pool: row t belongs to pool token t (only rows inside the context spans are read / written).
 * `lse` (nullable, fp32 [pool rows, H_q]) receives each row's log-sum-exp.
 */
int ape_encode_plan(ape_handle_t handle, const ape_shape_t *shape, const ape_kv_pool_t *pool,
                    const ape_rows_t *q, const ape_rows_t *out, float *lse,
                    const ape_span_t *prefix, const ape_span_t *ctx, int32_t n_ctx, ape_plan_t *plan);

/* Bytes of device scratch a launch of this plan needs (a multiple of 256; may be 0). */
int ape_plan_workspace_bytes(ape_plan_t plan, size_t *bytes);
int ape_plan_destroy(ape_plan_t plan);

/*
 * Launch APE attention (Eq. 5; the two-accumulator + log-sum-exp merge of the appendix "Efficient
 * Implementation").  T: attention temperature, S: scaling factor (the exponent of the context mass in
 * Eq. 5; a caller who tuned with the paper's S*T parametrisation passes that product).  Both finite, > 0.
 * kv_extra: tokens appended to every request's query segment since planning (decode step t passes t;
 * 0 <= kv_extra <= capacity - len; prefill plans require 0).  `workspace`: device, 256-byte aligned,
 * at least ape_plan_workspace_bytes; contents undefined afterwards.  `stream`: a cudaStream_t (0 = default).
 * Asynchronous; launches that share a workspace must be stream-ordered.
 */
int ape_attend(ape_plan_t plan, float T, float S, int64_t kv_extra,
               void *workspace, size_t workspace_bytes, void *stream);

/*
 * The whole of Eq. 5 in one call, for callers who do not keep a plan: the arguments are the paper's statement of the
 * problem (section "Formulation": the query rows, the shared prefix, the contexts, the query's own keys, T and S) in
 * the layout of ape_attend_plan.  Plans, allocates the plan's scratch, launches on `stream`, waits for the stream,
 * frees everything again.  Synchronous, and it pays the planning and two device allocations on every call: loops
 * (a decode loop above all) should plan once and call ape_attend.  APE_DECODE here means kv_extra = 0.
 */
int ape_attend_once(ape_handle_t handle, const ape_shape_t *shape, const ape_kv_pool_t *pool,
                    const ape_rows_t *q, const ape_rows_t *out, float *lse,
                    const ape_request_t *requests, int32_t n_req, ape_mode_t mode, float T, float S, void *stream);

/* Launch the context pre-encoding attention of an encode plan.  No T, no S (they apply to queries only).  An encode
 * plan writes its outputs directly and needs no scratch (ape_plan_workspace_bytes gives 0): `workspace` and
 * `workspace_bytes` are accepted so that all launches look alike, and are ignored (NULL / 0 are fine). */
int ape_encode_contexts(ape_plan_t plan, void *workspace, size_t workspace_bytes, void *stream);

/*
 * End-to-end variant for callers whose tensors live in HOST memory: copies h_q (the Q tensor) and the
 * K / V pools host-to-device into the plan's device buffers, launches ape_attend, copies O back to h_out,
 * all on `stream`, then synchronises the stream.  Host buffers have the same geometry as the device
 * tensors (dense: token_stride = heads * d, head_stride = d) and should be pinned.
 * *h2d_bytes / *d2h_bytes (nullable) receive the bytes moved.
 */
int ape_attend_host(ape_plan_t plan, float T, float S, int64_t kv_extra, void *workspace, size_t workspace_bytes,
                    const void *h_q, const void *h_k_pool, const void *h_v_pool, void *h_out,
                    size_t *h2d_bytes, size_t *d2h_bytes, void *stream);

/*
 * One decode step for callers whose per-step tensors live in HOST memory (the cache itself stays on the device, that is
 * what makes it a cache).  For a decode plan or a shared-context plan: copies the new token's query rows h_q
 * [n_req, H_q, d] to the requests' rows of Q; if h_k_new / h_v_new are given (both or neither; [n_req, H_kv, d], dense),
 * appends them to the requests' query segments at the position step `kv_extra` adds (the "append" that precedes a
 * decode step: the row of the newest token at planning time + kv_extra); launches ape_attend; copies the requests' rows
 * of O to h_out [n_req, H_q, d]; synchronises `stream`.  Request r's rows are the r-th of every host array.  Host buffers
 * should be pinned.  No allocation.  *h2d_bytes / *d2h_bytes (nullable) receive the bytes moved.
 */
int ape_decode_step_host(ape_plan_t plan, float T, float S, int64_t kv_extra, void *workspace, size_t workspace_bytes,
                         const void *h_q, const void *h_k_new, const void *h_v_new, void *h_out,
                         size_t *h2d_bytes, size_t *d2h_bytes, void *stream);

/*
 * Allocation-free decode step.  (The paper has no counterpart to this entry point; it exists for the callers
 * described here.)  Some hosts of this library must not allocate device memory at call time: an inference server
 * that has handed the whole GPU to its own memory pool (a cudaMalloc there fails or fragments the pool), a
 * latency-critical decode loop that cannot afford the device-wide synchronisation an allocation may imply, or a
 * plug-in that runs under a policy forbidding the allocator.  ape_create and the plan calls above allocate (status
 * word, plan metadata) and take a caller-provided workspace; this call needs none of them.  It computes exactly
 * what an APE_DECODE plan followed by ape_attend computes (one query row per request, Eq. 5), with the same kernels,
 * but keeps the plan metadata, the split-KV partials and the status word in a fixed 8 MiB device array that is
 * part of the library image.  Every GPU that loads the library holds those 8 MiB until the process exits.
 *
 *   - Arguments as in ape_attend_plan (mode APE_DECODE) and ape_attend; `device` is the CUDA ordinal the tensors
 *     live on; `lse` is nullable.  The caller still owns and passes every input and output tensor.
 *   - Limits: the tile lists and work items of the batch must fit 4 MiB and the partials the other 4 MiB
 *     (roughly: up to ~250,000 64-token tiles over all requests, i.e. about 16M cached tokens, and
 *     (SMs + 2 * n_req * H_kv) * (H_q / H_kv) * d * 4 bytes of partials).  A larger batch is rejected with
 *     APE_ERR_WORKSPACE before anything is launched; nothing is ever allocated instead.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress) and the device's
 *     properties.  With lazy module loading this lookup is also the moment the runtime materialises the array, so the
 *     driver's free-memory figure drops by 8 MiB once.  Later calls only do host work, one stream-ordered copy into the
 *     array and two kernel launches on `stream`.
 *   - `stream` must not be capturing: the metadata is rebuilt from the host arrays on every call and uploaded from a
 *     buffer that dies with the call, so the work cannot be recorded for replay.  A capturing stream is refused with
 *     APE_ERR_MODE before anything is enqueued.
 *   - Calls no cudaMalloc, cudaFree, or any other allocating routine.  Host descriptors are read during the call.
 *   - All calls on a device share the one array, and it keeps the previous call's contents: each call rewrites
 *     the metadata it uses.  Two calls whose GPU work may overlap (different streams, or different threads) race on
 *     the array: order them on one stream or with events.
 *   - Host-side blocking: the metadata (16 bytes per 64-token tile, about 0.5 MB for sixteen 128K-token requests) is
 *     uploaded from pageable host memory, so the call returns only after the work enqueued earlier on `stream` has
 *     drained and the bytes are staged.  The kernels it launches then run asynchronously, like those of ape_attend.  A
 *     decode loop that needs the host to run ahead of the GPU plans once with ape_attend_plan instead.
 *   - Status word: a kernel that gives up on a bounded wait sets the array's status word, and the word STAYS set, also
 *     across later calls, until a call reads it.  With a non-NULL `device_status` (HOST pointer) the call synchronises
 *     `stream` after its launches, stores the word there (0 or APE_ERR_TIMEOUT) and clears it.  With NULL nothing is
 *     read or cleared; a timeout raised by such a call is reported by the next call that passes `device_status`.
 */
int ape_decode_noalloc(const ape_shape_t *shape, const ape_kv_pool_t *pool, const ape_rows_t *q,
                       const ape_rows_t *out, float *lse, const ape_request_t *requests, int32_t n_req,
                       float T, float S, int64_t kv_extra, int device, void *stream, int32_t *device_status);

/*
 * Context-sharded attend (section "Parallel Encoding": hundreds of contexts, or more context than one GPU holds): each
 * shard -- another GPU, or another part of one GPU's pool -- holds a subset of the contexts and plans an ordinary attend
 * over that subset; ape_attend_partial runs the shard and, instead of the merged output, hands out the two segments of
 * Eq. 5 separately per query row and head: the context segment's own softmax output and the natural-log LSE of its logits
 * (temperature applied), and the same for the non-context segment (prefix + query, identical on every shard).
 * The caller gathers o_ctx / lse_ctx of all shards (one all-gather; 4 * (d + 1) bytes per row and head per shard) and
 * calls ape_merge_shards, which combines the shards' context segments by the hierarchical softmax identity (appendix
 * "Hierarchical Formula for Softmax Attention"), applies the scaling factor S to the combined context LSE and merges with
 * the non-context segment (Eq. 5).  The result equals ape_attend over all contexts.  All four arrays are DEVICE, fp32,
 * caller-owned: o_* [q rows, H_q, d], lse_* [q rows, H_q], indexed like Q; a segment without keys has lse = -inf.
 * Not available for per-context and tree plans (APE_ERR_MODE).
 */
typedef struct { float *o_ctx, *lse_ctx, *o_oth, *lse_oth; } ape_partials_t;

int ape_attend_partial(ape_plan_t plan, float T, int64_t kv_extra, void *workspace, size_t workspace_bytes,
                       const ape_partials_t *partials, void *stream);

/* o_ctx_all [n_shards, n_rows, H_q, d], lse_ctx_all [n_shards, n_rows, H_q] (shard-major, as an all-gather leaves them);
 * o_oth / lse_oth of any one shard; out bf16 rows (16-byte aligned like every tensor), lse nullable. */
int ape_merge_shards(ape_handle_t handle, const ape_shape_t *shape, int64_t n_rows, int32_t n_shards,
                     const float *o_ctx_all, const float *lse_ctx_all, const float *o_oth, const float *lse_oth,
                     float S, const ape_rows_t *out, float *lse, void *stream);

/*
 * Rotary position embedding with position re-use, fused with the write into the cache (the step right before
 * ape_encode_contexts: it makes the K, V and Q that the pre-caching attention and, later, ape_attend read).
 *
 * Section "Position Embedding" of the paper names the rotary embedding (Su et al.); the section "Parallel Encoding"
 * item "Re-using Positions for Long Context" places every context in the same range of positions.  Together with the
 * shared prefix of section "Prepending Shared Prefix" the positions of a request are: prefix 0 .. l_P-1, EVERY context
 * l_P .. l_P+l_i-1, query l_P + max_i l_i onward.  The pairing is the half-split one of the paper's base models
 * (component i with i + d/2, angle pos * theta^(-2i/d)).
 *
 * A run copies `len` rows, source row src_start+j to destination row dst_start+j, rotated for position pos0+j.
 */
typedef struct { int64_t src_start, dst_start, len, pos0; } ape_rope_run_t;

/*
 * The runs of one request under position re-use (HOST helper, no GPU work): source rows are packed in the order
 * prefix, context 1..N, query K/V, starting at row `src_start`; destinations are the request's pool spans.
 * `runs` is a HOST array of `capacity` entries; *n_runs receives the count (N + 2, empty spans included with len 0).
 * APE_ERR_INVALID_ARG if capacity is too small or a span is malformed.
 */
int ape_rope_runs_for_request(const ape_request_t *request, int64_t src_start, ape_rope_run_t *runs,
                              int32_t capacity, int32_t *n_runs);

/*
 * Plan for a set of runs (HOST array, read during the call): cuts them into work items and uploads those
 * (cudaMalloc + blocking copy).  head_dim 64 or 128; theta > 1 is the base of the embedding (500000 for Llama-3).
 * Every row index must fit 31 bits.  Destroy with ape_plan_destroy.
 */
int ape_rope_plan(ape_handle_t handle, int32_t head_dim, double theta, const ape_rope_run_t *runs, int32_t n_runs,
                  ape_plan_t *plan);

/*
 * Apply the plan to one tensor: src and dst are bf16 [rows, n_heads, head_dim] with strides in elements (16-byte
 * aligned, strides multiples of 8); rotate = 1 for K and Q, 0 for V (plain copy through the same runs).  src and dst
 * must not overlap.  Asynchronous on `stream`; allocates nothing.  Rows outside the runs are not touched.
 * APE_ERR_INVALID_ARG if a run reaches past src->n_rows or dst->n_rows.
 */
int ape_rope_write(ape_plan_t plan, const ape_rows_t *src, const ape_rows_t *dst, int32_t n_heads, int32_t rotate,
                   void *stream);

/* Kernels launched by the last ape_attend / ape_encode_contexts call on this plan. */
int ape_plan_last_launches(ape_plan_t plan, int32_t *n_launches);

/*
 * Self-test of the error path every kernel of the library shares: launches one warp that waits, with the library's
 * bounded wait, on a barrier nothing ever completes.  After the bound (about a second) the wait gives up, the kernel
 * returns normally and ape_get_status reports APE_ERR_TIMEOUT; the context stays usable.  Nothing faults, traps or
 * hangs.  Asynchronous on `stream`.
 */
int ape_selftest_timeout(ape_handle_t handle, void *stream);
/* The same probe aimed at the status word of ape_decode_noalloc's fixed array on `device` (no handle exists there). */
int ape_selftest_timeout_noalloc(int device, void *stream);

/* Synchronises the WHOLE device (cudaDeviceSynchronize: every stream, also those this library never saw) and returns the
 * device status word (0, or APE_ERR_TIMEOUT) in *device_status; clears it. */
int ape_get_status(ape_handle_t handle, int32_t *device_status);
/* The same for a caller that must not stall its other streams: reads the word in stream order on `stream` and waits for
 * that stream only, so it reports what the launches enqueued on `stream` before this call have raised.  A word that was
 * set is cleared by a stream-ordered write on `stream`.  APE_ERR_MODE if `stream` is being captured. */
int ape_get_status_stream(ape_handle_t handle, void *stream, int32_t *device_status);
const char *ape_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* APE_H_ */
