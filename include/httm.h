/*
 * httm.h - C ABI of the B200 (sm_100a) library for one VGGT-style global-attention
 * layer with head-wise temporal token merging (HTTM).
 *
 * The path behind these calls is Algorithm 1 of the HTTM paper between its projections:
 *   temporal reorder (Sec. 3.3) -> per-head, per-block cosine matching of Q and of K
 *   (Eq. 1) -> [optional: outlier filtering of the queries, Sec. 3.4 / Algorithm 2, see
 *   httm_set_outlier_fraction] -> mean merge of Q, K, V (V follows K, Sec. 3.2) -> softmax
 *   attention on the merged sets (Eq. 3-4) -> head-wise unmerge (Eq. 5-7) + inverse reorder.
 * The projections themselves are offered as httm_linear.
 *
 * Conventions common to all calls
 *   - S frames; every frame has n_camera + n_register special tokens followed by a
 *     grid_h x grid_w patch grid (row-major).  P = specials + grid_h*grid_w tokens per
 *     frame, N = S*P tokens, token index i = frame*P + index_in_frame.
 *   - Q, K, V are bf16 DEVICE tensors addressed as ptr[head*stride_head +
 *     token*stride_token + channel], strides in ELEMENTS, channels contiguous.
 *     ptr must be 16-byte aligned and both strides multiples of 8 elements.
 *   - The output is bf16, addressed the same way; the paper's concatenated layout
 *     [N][heads*head_dim] (Eq. 7) is stride_head = head_dim, stride_token =
 *     heads*head_dim.  It must not overlap an input.
 *   - Calls enqueue work on the given CUDA stream (a cudaStream_t passed as void*;
 *     NULL = the legacy default stream) and return without waiting for it.  The caller
 *     owns the tensors and keeps them alive until the stream has passed the call.
 *   - The context owns all scratch memory (sized at httm_create; nothing is allocated
 *     in the attention calls) and is not thread-safe; separate contexts are independent.
 *   - Every function returns HTTM_OK (0) or a negative httm_status.  Arguments are
 *     checked on the host before anything is launched.  Nothing aborts or throws.
 */
#ifndef HTTM_H_
#define HTTM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    HTTM_OK = 0,
    HTTM_ERR_INVALID_ARG = -1, /* null pointer, value out of range, overlapping output */
    HTTM_ERR_UNSUPPORTED = -2, /* head_dim != 64, block of more than 4096 tokens, ... */
    HTTM_ERR_ALIGNMENT = -3,   /* pointer not 16-byte aligned / stride not multiple of 8 */
    HTTM_ERR_NOMEM = -4,       /* device or host allocation failed                     */
    HTTM_ERR_CUDA = -5,        /* a CUDA runtime / driver call failed (see last_error)  */
    HTTM_ERR_TIMEOUT = -6      /* a bounded device-side wait gave up (status word set)  */
} httm_status;

typedef struct httm_ctx httm_ctx; /* opaque; created and destroyed by the library */

typedef struct {
    int32_t frames;               /* S >= 1                                            */
    int32_t n_camera, n_register; /* special tokens per frame (VGGT: 1 and 4); >= 0    */
    int32_t grid_h, grid_w;       /* patch grid, >= 1                                  */
    int32_t heads, head_dim;      /* head_dim must be 64                               */
    int32_t blk_frames, blk_h, blk_w; /* merging block: frames x patch window, >= 1;
                                     blocks are clipped at the grid / sequence end     */
    double ratio_q, ratio_kv;     /* fraction of tokens merged away, in [0, 1)         */
    int32_t device;               /* CUDA device ordinal                               */
    int32_t anchor_first_frame;   /* 0, or 1: first-frame anchoring (the paper's appendix on error mitigation): in every
                                     merging block that contains frame 0 the dst tokens are exactly the block's tokens of
                                     frame 0 and every other token of the block is a src token, so the reference frame is
                                     never merged away and similar tokens of later frames merge INTO it; there the budget
                                     is r = min(floor(ratio*n + 1e-9), n - n0) with n0 the block's tokens of frame 0.
                                     Any block shape of up to 256 tokens is accepted (blocks of one frame then merge
                                     nothing in the first frame group); blocks of more than 256 tokens may hold at most
                                     1024 tokens of frame 0 (UNSUPPORTED otherwise), and httm_global_attention_static
                                     has no anchoring.  (The field takes the struct's former padding.)  */
} httm_config;

typedef struct {
    void* ptr;            /* device pointer to bf16 data (inputs are only read)        */
    int64_t stride_head;  /* elements between heads                                    */
    int64_t stride_token; /* elements between tokens                                   */
} httm_tensor;

/* httm_query selectors */
enum {
    HTTM_Q_TOKENS = 0,          /* N                                                   */
    HTTM_Q_MERGED_Q = 1,        /* M_q: merged query length (same for every head)      */
    HTTM_Q_MERGED_K = 2,        /* M_k: merged key/value length                        */
    HTTM_Q_BLOCKS = 3,          /* merging blocks per head                             */
    HTTM_Q_WORKSPACE_BYTES = 4, /* device bytes owned by the context                   */
    HTTM_Q_MAX_BLOCK_TOKENS = 5,
    HTTM_Q_DEVICE_STATUS = 6,   /* syncs the device; 0 or the first device-side error   */
    HTTM_Q_MERGED_Q_ROWS = 7,   /* rows per head of HTTM_X_Q_MERGED / HTTM_X_O_MERGED: M_q, or N while query
                                   outlier filtering is on (the merged length then differs per head)    */
    HTTM_Q_OUTLIERS = 8         /* syncs the device; query tokens (of the merging blocks, all heads) that the
                                   last call's filtering took out of their groups                      */
};

/* httm_export selectors: intermediates of the LAST httm_global_attention call.
 * Index arrays are int32, tensors bf16 bit patterns (uint16). */
enum {
    HTTM_X_PI = 0,         /* [N]       reordered position -> original token index      */
    HTTM_X_PI_INV = 1,     /* [N]       original token index -> reordered position      */
    HTTM_X_BLOCK_START = 2,/* [blocks+1] reordered position of each block's first token */
    HTTM_X_ASSIGN_Q = 3,   /* [H][N]    reordered position each token is merged into     */
    HTTM_X_ASSIGN_K = 4,
    HTTM_X_RANK_Q = 5,     /* [H][N]    merged row of each reordered token               */
    HTTM_X_Q_REORDERED = 6,/* [H][N][D]                                                  */
    HTTM_X_K_REORDERED = 7,
    HTTM_X_V_REORDERED = 8,
    HTTM_X_Q_MERGED = 9,   /* [H][M_q][D]                                                */
    HTTM_X_K_MERGED = 10,  /* [H][M_k][D]                                                */
    HTTM_X_V_MERGED = 11,
    HTTM_X_O_MERGED = 12,  /* [H][M_q][D] attention output before unmerge               */
    /* query outlier filtering (Sec. 3.4); with it on, items 9 and 12 are [H][N][D] and head h's first
     * HTTM_X_MERGED_Q_HEAD[h] rows are valid */
    HTTM_X_DEVIATION = 13,     /* [H][N] float: distance of each reordered query token to its group's mean */
    HTTM_X_THRESHOLD = 14,     /* [1]    float: tau, the (K+1)-th largest deviation (+inf: K = 0)           */
    HTTM_X_MERGED_Q_HEAD = 15, /* [H]    int32: merged query length of every head                         */
    HTTM_X_ASSIGN_Q_INITIAL = 16 /* [H][N] int32: the query map before the outliers left (3 holds the map after) */
};

/* httm_launch_stage selectors.  0-4: the five separate kernels of the path (match and merge read the
 * reordered copies written by the reorder kernel).  5, 6: the match and merge kernels reading their blocks
 * straight from q, k, v (the temporal reorder folded into their tiled loads; UNSUPPORTED only for scenes of
 * more than 32767 frames, patch rows or patch columns, or more than 32 special tokens per frame).
 * httm_global_attention runs 5, 6, 3, 4 (0, 1, 2, 3, 4 for such scenes); both orders give the same maps. */
enum {
    HTTM_STAGE_REORDER = 0,
    HTTM_STAGE_MATCH = 1,
    HTTM_STAGE_MERGE = 2,
    HTTM_STAGE_ATTENTION = 3,
    HTTM_STAGE_UNMERGE = 4,
    HTTM_STAGE_MATCH_DIRECT = 5,
    HTTM_STAGE_MERGE_DIRECT = 6,
    HTTM_STAGE_OUTLIER_FILTER = 7,/* between 5 and 6, only after httm_set_outlier_fraction(> 0): five small kernels
                                     (six between 9 and 2 for blocks of more than 256 tokens) */
    /* merging blocks of 257 .. 4096 tokens (the paper's runs of 128 tokens over 30 frames, Sec. 4.1): stages 1, 5, 6 are
     * UNSUPPORTED; the order is 0, 8, 9, 2, 3, 4.  8: cosine of every token with every dst token of its block on the
     * tensor cores + best dst per token; 9: the r best src of every block merge (map written) */
    HTTM_STAGE_BIG_SCORES = 8,
    HTTM_STAGE_BIG_SELECT = 9,
    HTTM_STAGE_ATTENTION_UNMERGE = 10 /* stages 3 and 4 as one kernel: the attention epilogue writes every merged query row to its
                                         member tokens in `out` (contexts with blocks of at most 32 tokens, outlier filtering off;
                                         UNSUPPORTED otherwise); needs the member lists the last merge stage (2 or 6) left */
};

/*
 * Create a context for one problem geometry (Algorithm 1's inputs: block shape
 * B_s x B_t and the merge budgets).  Host work only plus device allocation and a few
 * small uploads: builds the reorder index pi (Sec. 3.3), the block table and the
 * per-block merge budget r = min(floor(ratio*n + 1e-9), n-1) with
 * n_dst = min(ceil(n/4), n-r) evenly spaced destination tokens (Sec. 3.2).
 * On success *out owns the context; free it with httm_destroy.
 * Errors: INVALID_ARG, UNSUPPORTED, NOMEM, CUDA.  On error *out is NULL.
 */
int httm_create(const httm_config* cfg, httm_ctx** out);

/*
 * HTTM global attention (Algorithm 1 between the QKV and output projections).
 * q, k, v: device tensors of the context's geometry; out: device output, all N
 * tokens, every head.  Kernels enqueued on `stream`:
 *   [reorder (Sec. 3.3)] -> match Q, K (Eq. 1, top-r of Sec. 3.2) -> merge Q, K, V
 *   (mean of constituents) -> attention on merged sets (Eq. 3-4) -> unmerge +
 *   inverse reorder + head concat (Eq. 5-7).
 * Match and merge load each block's patch window straight from q, k, v and no reordered
 * copy is written (HTTM_X_*_REORDERED hold what the last HTTM_STAGE_REORDER wrote); scenes of
 * more than 32767 frames / patch rows / patch columns, or with more than 32 special tokens per
 * frame, run the reorder kernel first.  With blocks of at most 32 tokens (and outlier filtering
 * off) the unmerge runs in the attention kernel's epilogue: every merged query row is written
 * straight to its member tokens in `out`, three kernels in all; the merged attention output
 * (HTTM_X_O_MERGED) is then computed only when it is exported.  Larger blocks: four kernels.
 * With ratio_q = ratio_kv = 0 the result equals httm_dense_attention up to rounding.
 * Errors: INVALID_ARG, ALIGNMENT, CUDA (launch failure); device-side wait time-outs
 * are reported by the next httm_query(HTTM_Q_DEVICE_STATUS) / httm_export.
 */
int httm_global_attention(httm_ctx* ctx, httm_tensor q, httm_tensor k, httm_tensor v, httm_tensor out,
                          void* cuda_stream);

/*
 * Adaptive outlier filtering for the query tokens (Sec. 3.4, Algorithm 2); off (fraction 0) after httm_create.
 * With 0 < fraction <= 1 every later httm_global_attention / httm_attention_host call inserts, between match and
 * merge: the deviation of every query token from the mean of the group it was merged into (0 for a token on its
 * own), the threshold tau = the (K+1)-th largest deviation over ALL heads with K = floor(fraction * heads * N + 1e-9),
 * and the map update: tokens with deviation > tau leave their groups and stay unmerged; a group that loses its
 * destination token continues under its remaining member with the lowest reordered position.  Only queries are
 * filtered; K and V are untouched.  The merged query length then differs from head to head (HTTM_X_MERGED_Q_HEAD).
 * The first call with fraction > 0 allocates the extra workspace (device allocation: call it outside timed regions).
 * Blocks of at most 32 tokens that are loaded straight from q, k, v take five small warp-per-block kernels; every
 * other geometry (larger blocks, or scenes that go over the reordered copies) takes six kernels that work on the sorted
 * groups of a block and merges from the reordered copies.
 * Errors: INVALID_ARG (fraction outside [0, 1]), NOMEM, CUDA.
 */
int httm_set_outlier_fraction(httm_ctx* ctx, double fraction);

/*
 * Head-sharded layers (Sec. 3.2: every head matches, merges, attends and unmerges on its own).  A context created
 * with heads = H / G serves the heads one GPU owns: hand it head-strided views of Q, K, V and of the output (its
 * column slice of [tokens][H x 64]); no kernel reads another shard's data and nothing is exchanged inside the layer.
 * The one quantity that spans the heads is the outlier budget of Sec. 3.4 (item 3: the gamma-quantile is taken
 * "across all heads"): with outlier filtering on, tell the context how many heads the whole layer has and give it a
 * function that sums a vector of int32 counters over all shards.  The threshold selection then builds each of its
 * three radix histograms (2048, 2048, 1024 counters) locally, calls
 *     exchange(user, device_counts, n_counts, cuda_stream)
 * and chooses the bin from the summed histogram, so that every shard arrives at the same threshold: exactly the
 * one a single context with all the heads finds.  exchange must enqueue, on cuda_stream, an in-place sum of the
 * n_counts int32 values at device_counts (device memory owned by the context) over all shards, e.g. an NCCL
 * all-reduce, and return 0; every shard calls it three times per httm_global_attention, in the same order.
 * total_heads = 0 and exchange = NULL switch sharding off.  Without outlier filtering the setting has no effect.
 * Errors: INVALID_ARG (fewer heads than the context has; more without an exchange function), UNSUPPORTED (total
 * heads x tokens >= 2^31); a non-zero return of exchange makes the attention call fail with HTTM_ERR_CUDA.
 */
typedef int (*httm_exchange_fn)(void* user, void* device_counts, int32_t n_counts, void* cuda_stream);
int httm_set_head_shard(httm_ctx* ctx, int32_t total_heads, httm_exchange_fn exchange, void* user);

/*
 * The projections around the path (Algorithm 1: Q, K, V = x W_qkv before it, out = Attn W_o after it) for callers
 * that want no library matmul next to the path:  y[n_rows][out_features] = x[n_rows][in_features] . w^T  with the
 * weight given as w[out_features][in_features] (the layout a linear layer stores), all bf16 on the context's device,
 * fp32 accumulation, one rounding to bf16; ldx / ldw / ldy are the row strides in elements.  No bias.  One kernel on
 * `stream` (tcgen05 GEMM).  x and w are only read; y must not overlap them.
 * Errors: INVALID_ARG, ALIGNMENT (pointers 16-byte aligned, strides multiples of 8), UNSUPPORTED (in_features must be
 * a multiple of 64, out_features a multiple of 8), CUDA; a device-side wait time-out is reported like the others.
 */
int httm_linear(httm_ctx* ctx, const void* x, int64_t ldx, const void* w, int64_t ldw, void* y, int64_t ldy,
                int64_t n_rows, int32_t in_features, int32_t out_features, void* cuda_stream);

/*
 * Exact multi-head softmax attention over all N tokens (the unmerged baseline the
 * paper's speed-ups are measured against, Sec. 4.1), same attention kernel, output
 * written directly in `out`'s layout.  Same argument rules and errors as above.
 */
int httm_dense_attention(httm_ctx* ctx, httm_tensor q, httm_tensor k, httm_tensor v, httm_tensor out,
                         void* cuda_stream);

/*
 * The same two operations for callers whose tensors live in HOST memory (pinned memory
 * makes the copies asynchronous).  q, k, v: bf16 [heads][N][head_dim] contiguous;
 * out: bf16 [N][heads*head_dim] contiguous.  Each call copies the inputs to
 * context-owned device buffers, runs the path on `stream` and copies the result back;
 * the caller synchronises `stream` before reading `out`.  The copies run on two streams
 * of the context's own over two sets of buffers (all created at the first such call),
 * so that consecutive calls overlap: one call's host-to-device copy runs during the
 * previous call's kernels and device-to-host copy.  Consequences: the input buffers
 * must hold their data when the call is made (their copy does not wait for earlier
 * work on `stream`) and must stay unchanged, like `out` unread, until `stream` has
 * been synchronised.  dense != 0 selects httm_dense_attention.
 * Errors: INVALID_ARG, NOMEM, CUDA.
 */
int httm_attention_host(httm_ctx* ctx, const void* q_host, const void* k_host, const void* v_host,
                        void* out_host, int dense, void* cuda_stream);

/*
 * Enqueue one of the five stages of httm_global_attention on its own, reading and
 * writing the context's intermediates of the previous stages (for per-kernel timing
 * and profiling; calling stages 0..4 in order equals httm_global_attention).
 * q, k, v are read by HTTM_STAGE_REORDER only, out is written by HTTM_STAGE_UNMERGE only;
 * the other stages ignore them.
 */
int httm_launch_stage(httm_ctx* ctx, int stage, httm_tensor q, httm_tensor k, httm_tensor v,
                      httm_tensor out, void* cuda_stream);

/* Sizes and status, see HTTM_Q_*.  Errors: INVALID_ARG, CUDA, TIMEOUT (device status). */
int httm_query(httm_ctx* ctx, int what, int64_t* value);

/*
 * Copy an intermediate of the last call (HTTM_X_*) to host memory.  Waits for `stream`
 * first.  `bytes` must be exactly the size of the item (int32 or bf16 elements).
 * Errors: INVALID_ARG (wrong size / selector), CUDA, TIMEOUT (device status word set).
 */
int httm_export(httm_ctx* ctx, int what, void* host_dst, size_t bytes, void* cuda_stream);

/* Message of the last error on this context (or of the last failed httm_create when ctx
 * is NULL).  The string is owned by the library and valid until the next call. */
const char* httm_last_error(const httm_ctx* ctx);

/* Number of kernels launched by the library on this context since it was created. */
int64_t httm_launch_count(const httm_ctx* ctx);

/*
 * (No counterpart in the paper: a packaging variant of httm_global_attention.)
 * The same HTTM global attention for callers that cannot allocate device memory at the time
 * of the call and therefore cannot use httm_create, which calls cudaMalloc: for example code
 * that runs after a serving process has handed the whole device to its own memory pool, or a
 * latency-critical loop in which cudaMalloc's device-wide synchronisation is not acceptable.
 * This call allocates nothing on the device (no cudaMalloc / cudaFree, no library allocator):
 * every intermediate of the path lives in one array of HTTM_STATIC_SCRATCH_BYTES that is built
 * into the library's device image, so every GPU that loads the library holds that much memory
 * until the process exits.
 *   - cfg describes the problem exactly as for httm_create (cfg->device selects the GPU);
 *     q, k, v, out follow the rules at the top of this file and stay owned by the caller.
 *   - Problems whose intermediates do not fit the array (roughly heads * N * 128 bytes * 5;
 *     the tiny 1044-token, 16-head configuration needs about 11 MiB) are rejected with
 *     HTTM_ERR_UNSUPPORTED before anything is launched; use a context for those.
 *   - The first call on a device looks up the array's device address and sets kernel
 *     attributes; make that first call before any stream capture begins.
 *   - The array also holds the plan tables of one configuration per device (reorder index and
 *     block table).  A call whose configuration differs from the one resident on that device
 *     (the first call included) uploads them: three host-to-device copies from pageable memory
 *     on `cuda_stream`, which the runtime stages on the host before it returns.  Calls that
 *     repeat the resident configuration enqueue kernels only, and return without waiting for
 *     earlier work on the stream.
 *   - All calls share the one array and it keeps the previous call's contents (the call
 *     resets what must start clean).  Two calls that overlap on the GPU, e.g. on different
 *     streams, race on it: serialise them.  Calls are serialised on the host by a lock.
 *   - Intermediates cannot be exported and the device status word is not reported.
 * Errors: INVALID_ARG, ALIGNMENT, UNSUPPORTED, CUDA; message via httm_last_error(NULL).
 */
#define HTTM_STATIC_SCRATCH_BYTES (16u << 20)
int httm_global_attention_static(const httm_config* cfg, httm_tensor q, httm_tensor k, httm_tensor v,
                                 httm_tensor out, void* cuda_stream);

/*
 * Times of the kernels INSIDE a call of httm_global_attention (the paper's Table 3 splits a layer the same way: attention,
 * matching, aggregation).  httm_set_call_timing(ctx, 1) makes every later httm_global_attention on this context record
 * a CUDA event on the caller's stream before its first kernel and after each part of the call (a part is one kernel;
 * the five small kernels of the outlier filter count as one part); the events are created by this call, none per
 * httm_global_attention.  httm_call_times waits for the last call's final event and returns, for its parts in launch
 * order, the time between consecutive events in milliseconds (ms[i]) and a name (names[i], static strings such as
 * "match_direct", "merge_direct", "attention_unmerge"; names may be NULL); *count = number of parts of the last call,
 * of which at most `capacity` are written.  Host pointers.  The times are those of the kernels as they run in the
 * call, one behind the other (caches as the previous kernel left them), which the one-kernel launches of
 * httm_launch_stage are not.  Off by default; enable = 0 switches it off again.
 * Errors: INVALID_ARG (null arguments, timing off), CUDA.
 */
int httm_set_call_timing(httm_ctx* ctx, int32_t enable);
int httm_call_times(httm_ctx* ctx, float* ms, const char** names, int32_t capacity, int32_t* count);

/*
 * Aids for testing the error paths (host-side injection; nothing here faults or hangs the device).
 *   httm_fail_nth_allocation(n): the n-th device allocation the library makes from now on (in this process) fails as if
 *     the device were out of memory: the call that needed it returns HTTM_ERR_NOMEM and releases what it had taken.
 *     n = 0 switches it off.
 *   httm_expire_a_wait(ctx, stream): enqueues a one-tile kernel whose producer issues two of the three loads its
 *     barrier expects, so that the kernel's bounded wait runs out (about two seconds): it records the time-out in the
 *     context's status word, releases its tensor memory and returns.  The next httm_query(HTTM_Q_DEVICE_STATUS) /
 *     httm_export then reports HTTM_ERR_TIMEOUT; the context stays usable (the status word keeps the first error).
 * Errors: INVALID_ARG, UNSUPPORTED (a context with fewer than 384 token-heads), CUDA.
 */
int httm_fail_nth_allocation(int32_t n);
int httm_expire_a_wait(httm_ctx* ctx, void* cuda_stream);

/*
 * Diagnostic: one 128-row tile through the tensor-core building blocks of the attention kernel
 * (Eq. 3-4 on a single tile): s_out[128][128] = Q K^T and o_out[128][64] = bf16(s_out) V in fp32,
 * with q, k, v contiguous bf16 [128][64] DEVICE arrays (16-byte aligned), s_out / o_out / status_dev
 * device arrays owned by the caller.  *status_dev is set non-zero if a bounded wait gave up.
 * Errors: INVALID_ARG, CUDA.
 */
int httm_selftest_tensor_core(const void* q, const void* k, const void* v, float* s_out, float* o_out,
                              int* status_dev, void* cuda_stream);

/* Free the context and everything it owns.  The caller first synchronises every stream
 * the context was used on.  NULL is accepted. */
int httm_destroy(httm_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* HTTM_H_ */
