// Internal declarations shared by the translation units of libhttm (not part of the ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace httm {

constexpr int kHeadDim = 64;          // channels per head the kernels are written for
constexpr int kRowBytes = kHeadDim * 2;  // one token of one head, bf16
constexpr int kMaxBlockTokens = 256;  // largest merging block the warp-per-block match / merge kernels stage
constexpr int kMaxBigBlockTokens = 4096;   // largest merging block of the large-block path (Sec. 4.1: 128 tokens x 30 frames = 3840)
constexpr int kMaxBigDst = 1024;           // its dst tokens (a quarter of the block) stay in shared memory
constexpr int kBigSliceRows = 4096;        // rows of a block one work item of the score kernel handles (the whole block)

// Device status word values (first error wins).
enum : int {
    kDevOk = 0,
    kDevTimeoutMatchLoad = 1,   // match kernel: bulk copy of a block did not complete in time
    kDevTimeoutAttention = 2,   // attention kernel: a pipeline barrier did not complete in time
    kDevBadIndex = 3,           // an index read from a map was out of range (skipped)
    kDevTimeoutBigMatch = 4,    // large-block score kernel: a pipeline barrier did not complete in time
    kDevTimeoutLinear = 5       // projection GEMM: a pipeline barrier did not complete in time
};

// One merging block (Sec. 3.3): tokens [start, start + n) of the reordered sequence.
// r_* = number of src tokens merged away, nd_* = number of dst tokens,
// moff_* = merged row of the block's first kept token (closed form: the per-block kept
// count n - r is the same for every head).
struct BlockInfo {
    int32_t start, n;
    int32_t r_q, nd_q, moff_q;
    int32_t r_k, nd_k, moff_k;
    // dst positions: j is a dst token iff j < n_rule and floor((j + 1) n_dst / n_rule) > floor(j n_dst / n_rule).
    // n_rule = n: n_dst evenly spaced tokens (Sec. 3.2 reading); n_rule = n_dst: the first n_dst tokens of the block,
    // i.e. its tokens of frame 0 (first-frame anchoring).
    int32_t n_rule;
};

// Where a merging block sits in the original layout (used when the kernels read the blocks straight from
// Q/K/V with tiled TMA loads instead of from the reordered copies): first frame, first patch row and
// column, and the clipped extents.
struct BlockGeom {
    int16_t s0, y0, x0, frames, rows, cols;   // rows x cols patches over `frames` frames; 12 bytes
};
// Geometry of the original token layout: token (frame s, in-frame index p) is row s * tokens_per_frame + p;
// patch (y, x) has p = n_special + y * grid_w + x.
struct SourceLayout {
    int32_t frames, grid_h, grid_w, n_special, tokens_per_frame;
    int32_t blk_frames, blk_h, blk_w;
};

struct TensorView {          // bf16, element strides
    const __nv_bfloat16* ptr;
    int64_t stride_head, stride_token;
};

struct ReorderArgs {
    TensorView src[3];
    __nv_bfloat16* dst[3];   // [H][N][64] contiguous
    const int32_t* pi;       // [N]
    int32_t n_tokens, heads;
    float* inv_norm[2];      // optional, [H][N] each: 1 / max(|x|, 1e-12) of the reordered Q and K tokens (large-block path)
};

// Large-block path (blocks of 257 .. 4096 tokens; Sec. 4.1's 128 x 30 regime): matching as a dense contraction.
struct BigItem {
    int32_t block, row0;     // rows [row0, row0 + kBigSliceRows) of this block
};
struct BigMatchArgs {
    const __nv_bfloat16* xr[2];   // reordered Q, K [H][N][64]
    const float* inv_norm[2];     // [H][N]
    uint32_t* best_key[2];        // [H][N] order-preserving key of every token's best cosine to a dst token
    int32_t* best_pos[2];         // [H][N] token number, inside the block, of that dst
    int32_t* assign[2];           // [H][N] out (select kernel)
    const BlockInfo* blocks;
    const BigItem* items;         // the slices of all blocks (the same list for every tensor and head)
    int32_t n_items, n_blocks, n_tokens, heads;
    int32_t* status;
};

struct MatchArgs {
    // direct mode (geom != nullptr): blocks are read from the original tensors src[0..1]; else from xr
    const BlockGeom* geom;
    TensorView src[2];
    SourceLayout layout;
    const __nv_bfloat16* xr[2];   // reordered Q, K  [H][N][64]
    int32_t* assign[2];           // A_q, A_k        [H][N]
    const BlockInfo* blocks;
    int32_t n_blocks, n_tokens, heads;
    int32_t* status;
};

struct MergeArgs {
    // direct mode (geom != nullptr): blocks and special tokens are read from the original tensors src[0..2]
    const BlockGeom* geom;
    TensorView src[3];
    SourceLayout layout;
    const __nv_bfloat16* xr[3];   // reordered Q, K, V
    const int32_t* assign[2];     // A_q, A_k (V uses A_k)
    __nv_bfloat16* merged[3];     // Q_m [H][M_q][64], K_m, V_m [H][M_k][64]
    int32_t* rank_q;              // [H][N] merged row of every reordered token (written for Q)
    const int32_t* moff_q_var;    // optional [H][blocks]: per-head merged offsets of Q (outlier filtering); then m_q is the row stride of merged[0]
    // optional (blocks of at most 32 tokens): the members of every merged query row, for the unmerge in the attention epilogue:
    // group_start[h][m] .. group_start[h][m + 1] index group_member[h][], which holds ORIGINAL token numbers (pi: [N])
    int32_t* group_start;         // [H][M_q + 1]; entry M_q (= N) is written once when the workspace is set up
    int32_t* group_member;        // [H][N]
    const int32_t* pi;
    const BlockInfo* blocks;
    int32_t n_blocks, n_tokens, heads, n_special_total, m_q, m_k;
    int32_t* status;
};

// Query outlier filtering (Sec. 3.4): deviations, global threshold, map rewrite, per-head merged offsets.
// layout of OutlierArgs::sel (int32 words)
constexpr int kSelOutliers = 0;    // tokens the filter took out of their groups
constexpr int kSelDone = 1;        // [3] CTAs that have finished level 0, 1, 2
constexpr int kSelPrefix = 4;      // [2] bits of tau fixed after level 0, 1
constexpr int kSelRank = 6;        // [2] rank (counted from the largest) still to be skipped inside that prefix
constexpr int kSelOffsetsDone = 9; // heads whose block offsets are complete
constexpr int kSelFinished = 8;    // tau is final (budget 0 or everything): the refinement kernels return at once
constexpr int kSelHist = 16;       // [3][2048] histograms of bits 31-21, 20-10, 9-0
constexpr int kSelWords = kSelHist + 3 * 2048;

struct OutlierArgs {
    const BlockGeom* geom;
    const BlockInfo* blocks;
    TensorView src_q;             // original Q
    SourceLayout layout;
    const int32_t* assign_q;      // [H][N] map of the initial merging
    int32_t* assign_q_out;        // [H][N] map after the outliers left (special tokens: identity, written once at creation)
    float* eps;                   // [H][N] deviations (special tokens: 0, written once at creation)
    float* tau;                   // [1] threshold
    int32_t* kept_cnt;            // [H][blocks] kept tokens per block after filtering
    int32_t* moff_var;            // [H][blocks] merged row of each block's first kept token
    int32_t* mq_head;             // [H] merged query length
    int32_t* tile_prefix;         // [H + 1] index of each head's first 128-row query tile
    int32_t* sel;                 // [kSelWords] selection state, zeroed before every call: outlier counter, per-level
                                  // CTA counters, prefixes, remaining ranks, then the three radix histograms
    int64_t budget;               // K: number of tokens, over all heads, that may be outliers
    int32_t n_blocks, n_tokens, heads, n_special_total;
    int32_t* status;
    // Head-sharded layers (this context holds some of the heads, the budget is one for ALL heads, Sec. 3.4 item 3):
    // total_count = deviations of all shards (total heads x tokens); defer_select: the kernels only build their
    // histograms, the bin is chosen by a kernel of its own once the histograms of all shards have been summed
    int64_t total_count;
    int32_t defer_select;
};

struct UnmergeArgs {
    const __nv_bfloat16* o_m;     // [H][M_q][64]
    const int32_t* rank_q;        // [H][N]
    const int32_t* pi_inv;        // [N]
    __nv_bfloat16* out;
    int64_t out_stride_head, out_stride_token;
    int32_t n_tokens, heads, m_q;
    int32_t* status;
};

struct AttentionArgs {
    TensorView q, k, v;
    __nv_bfloat16* out;
    int64_t out_stride_head, out_stride_token;
    int32_t m_q, m_k, heads;
    float scale_log2;             // log2(e) / sqrt(head_dim)
    int32_t* status;
    // optional (outlier filtering): per-head query lengths [H] and first-tile indices [H + 1] in device memory;
    // then m_q is the row stride of q / out and an upper bound of every head's length
    const int32_t* mq_head;
    const int32_t* tile_prefix;
    // optional (unmerge folded into the epilogue, Eq. 5-7): every merged query row is written to each of its member tokens
    // at out + head * out_stride_head + token * out_stride_token instead of to its own row; see MergeArgs
    const int32_t* group_start;
    const int32_t* group_member;
    int32_t n_tokens;
};

struct LinearArgs {   // y[n_rows][out] = x[n_rows][in] . w[out][in]^T, leading dimensions in elements
    const __nv_bfloat16 *x, *w;
    __nv_bfloat16* y;
    int64_t ldx, ldw, ldy, n_rows;
    int32_t in_features, out_features;
    int32_t* status;
};

// Launchers (each enqueues exactly one kernel on `stream`; returns the CUDA error).
cudaError_t launch_reorder(const ReorderArgs& a, cudaStream_t stream);
cudaError_t launch_match(const MatchArgs& a, int max_block_tokens, int sm_count, cudaStream_t stream);
// first-frame anchoring: the blocks of the first frame group (the first n_anchor blocks) whose dst tokens exceed main_capacity,
// from the original tensors through the reorder index pi
cudaError_t launch_match_anchor(const MatchArgs& a, const TensorView& src_q, const TensorView& src_k, const int32_t* pi, int n_anchor,
                                int main_capacity, int max_block_tokens, cudaStream_t stream);
cudaError_t launch_merge(const MergeArgs& a, int max_block_tokens, int sm_count, cudaStream_t stream);
cudaError_t launch_unmerge(const UnmergeArgs& a, cudaStream_t stream);
cudaError_t launch_deviation(const OutlierArgs& a, int sm_count, cudaStream_t stream);
cudaError_t launch_threshold(const OutlierArgs& a, int sm_count, cudaStream_t stream);
cudaError_t launch_filter(const OutlierArgs& a, cudaStream_t stream);   // map rewrite + per-head offsets (two kernels)
cudaError_t launch_offsets(const OutlierArgs& a, cudaStream_t stream);  // per-head offsets alone
cudaError_t launch_threshold0(const OutlierArgs& a, int sm_count, cudaStream_t stream);   // threshold with the level-0 histogram taken from the deviations (three kernels)
cudaError_t launch_refine_level(const OutlierArgs& a, int level, int sm_count, cudaStream_t stream);   // histogram of one level alone (0, 1, 2)
cudaError_t launch_select_level(const OutlierArgs& a, int level, cudaStream_t stream);                 // choose the bin of one level from its (summed) histogram
cudaError_t launch_big_deviation(const OutlierArgs& a, int max_block_tokens, cudaStream_t stream);   // large blocks: deviations
cudaError_t launch_big_filter(const OutlierArgs& a, int max_block_tokens, cudaStream_t stream);      // large blocks: map rewrite + kept counts
cudaError_t launch_big_scores(const BigMatchArgs& a, int sm_count, cudaStream_t stream);   // tcgen05 contraction + row argmax
cudaError_t launch_big_select(const BigMatchArgs& a, cudaStream_t stream);                  // top-r per (tensor, head, block)
cudaError_t launch_big_merge(const MergeArgs& a, int max_block_tokens, cudaStream_t stream);                      // sort by merged row + gather means
cudaError_t configure_big_blocks();
cudaError_t launch_linear(const LinearArgs& a, int sm_count, cudaStream_t stream);   // tcgen05 GEMM for the projections
cudaError_t configure_linear();
cudaError_t launch_attention(const AttentionArgs& a, int sm_count, cudaStream_t stream);   // tcgen05 / TMEM kernel
cudaError_t configure_attention();
cudaError_t configure_kernels();   // one-time function attributes (dynamic shared memory sizes)
cudaError_t launch_wait_expiry(const void* tiles, float* scratch, int32_t* status, cudaStream_t stream);   // time-out path test, see httm_umma_selftest.cu

}  // namespace httm
