// C ABI of libhttm: context (plan + workspace), argument checks, stage launches, exports.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "../../include/httm.h"
#include "httm_internal.h"
#include "httm_plan.h"

using namespace httm;

namespace {
thread_local std::string g_create_error;
int g_fail_allocation = 0;   // httm_fail_nth_allocation: counts down to the device allocation that is made to fail

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};
}  // namespace

struct httm_ctx {
    httm_config cfg{};
    int32_t n_special = 0, tokens_per_frame = 0, n_tokens = 0, n_blocks = 0, max_block = 0;
    int32_t m_q = 0, m_k = 0;
    int sm_count = 148;
    std::vector<int32_t> pi, pi_inv, blk_start;
    std::vector<BlockInfo> blocks;
    std::vector<BlockGeom> geom;
    BlockGeom* d_geom = nullptr;
    // device workspace
    int32_t *d_pi = nullptr, *d_pi_inv = nullptr, *d_assign_q = nullptr, *d_assign_k = nullptr, *d_rank_q = nullptr;
    int32_t* d_status = nullptr;
    BlockInfo* d_blocks = nullptr;
    __nv_bfloat16 *d_qr = nullptr, *d_kr = nullptr, *d_vr = nullptr;
    __nv_bfloat16 *d_qm = nullptr, *d_km = nullptr, *d_vm = nullptr, *d_om = nullptr;
    // Members of every merged query row (blocks of at most 32 tokens): the attention epilogue writes each row straight to
    // its tokens (unmerge + inverse reorder, Eq. 5-7, without the O_m round trip).  om_stale: the last call took that
    // path, so O_m does not hold its attention output (httm_export recomputes it on request).
    int32_t *d_group_start = nullptr, *d_group_member = nullptr;
    bool om_stale = false;
    // first-frame anchoring: blocks of the first frame group (the first n_anchor blocks) with more dst tokens than the
    // match kernel holds (match_capacity) are matched by a kernel of their own, launched behind it
    int32_t n_anchor = 0, match_capacity = 0;
    // head-sharded layer (httm_set_head_shard): heads of the whole layer, and the caller's sum over the shards
    int32_t total_heads = 0;
    httm_exchange_fn exchange = nullptr;
    void* exchange_user = nullptr;
    // query outlier filtering (Sec. 3.4): off while fraction == 0; its workspace is allocated when it is first switched on.
    // The merged query length then differs per head: Q_m and O_m get N rows per head.
    double outlier_fraction = 0.0;
    int32_t *d_assign_qf = nullptr, *d_kept_cnt = nullptr, *d_moff_var = nullptr, *d_mq_head = nullptr, *d_tile_prefix = nullptr;
    int32_t* d_sel = nullptr;   // state of the threshold selection, first word = outlier counter
    float *d_eps = nullptr, *d_tau = nullptr;
    __nv_bfloat16 *d_qm_var = nullptr, *d_om_var = nullptr;
    // large merging blocks (257 .. 4096 tokens, Sec. 4.1): matching as a tensor-core contraction, see httm_big_blocks.cu
    std::vector<BigItem> big_items;
    BigItem* d_big_items = nullptr;
    float *d_inv_norm_q = nullptr, *d_inv_norm_k = nullptr;
    uint32_t *d_best_key_q = nullptr, *d_best_key_k = nullptr;
    int32_t *d_best_pos_q = nullptr, *d_best_pos_k = nullptr;
    bool big() const { return max_block > kMaxBlockTokens; }
    bool filtering() const { return outlier_fraction > 0.0; }
    int32_t q_rows() const { return filtering() ? n_tokens : m_q; }   // rows per head of Q_m and O_m
    // staging for the host-buffer entry point (allocated on first use)
    // Two sets of device buffers, two copy streams and events, so that one call's host-to-device copy overlaps the
    // previous call's kernels and device-to-host copy (PCIe is full duplex; the copies are 6x the kernel time).
    struct HostSet {
        __nv_bfloat16 *q = nullptr, *k = nullptr, *v = nullptr, *out = nullptr;
        cudaEvent_t loaded = nullptr, consumed = nullptr, computed = nullptr, returned = nullptr;
        bool used = false;
    } hs[2];
    cudaStream_t s_h2d = nullptr, s_d2h = nullptr;
    int64_t host_calls = 0;
    int64_t workspace_bytes = 0;
    int64_t launches = 0;
    // optional: events between the kernels of httm_global_attention (httm_set_call_timing)
    static constexpr int kMaxCallParts = 12;
    bool call_timing = false;
    cudaEvent_t call_ev[kMaxCallParts + 1] = {};
    const char* call_part[kMaxCallParts] = {};
    int call_parts = 0;
    std::string error;

    int fail(int code, const char* fmt, ...) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        error = buf;
        return code;
    }
    template <typename T>
    int alloc(T** p, size_t count) {
        const size_t bytes = (count ? count : 1) * sizeof(T);
        cudaError_t e = g_fail_allocation > 0 && --g_fail_allocation == 0 ? cudaErrorMemoryAllocation
                                                                          : cudaMalloc(reinterpret_cast<void**>(p), bytes);
        if (e != cudaSuccess) {
            *p = nullptr;
            cudaGetLastError();
            return fail(e == cudaErrorMemoryAllocation ? HTTM_ERR_NOMEM : HTTM_ERR_CUDA, "cudaMalloc(%zu bytes): %s", bytes,
                        cudaGetErrorString(e));
        }
        workspace_bytes += (int64_t)bytes;
        return HTTM_OK;
    }
    void release() {
        void* ptrs[] = {d_geom, d_pi, d_pi_inv, d_assign_q, d_assign_k, d_rank_q, d_status, d_blocks, d_qr, d_kr,
                        d_vr, d_qm,     d_km,       d_vm,       d_om,     hs[0].q,  hs[0].k,  hs[0].v, hs[0].out, hs[1].q, hs[1].k, hs[1].v, hs[1].out,
                        d_assign_qf, d_kept_cnt, d_moff_var, d_mq_head, d_tile_prefix, d_sel, d_eps, d_tau, d_qm_var, d_om_var,
                        d_big_items, d_inv_norm_q, d_inv_norm_k, d_best_key_q, d_best_key_k, d_best_pos_q, d_best_pos_k,
                        d_group_start, d_group_member};
        for (void* p : ptrs)
            if (p) cudaFree(p);
        for (HostSet& h : hs)
            for (cudaEvent_t e : {h.loaded, h.consumed, h.computed, h.returned})
                if (e) cudaEventDestroy(e);
        for (cudaEvent_t& e : call_ev) {
            if (e) cudaEventDestroy(e);
            e = nullptr;
        }
        if (s_h2d) cudaStreamDestroy(s_h2d);
        if (s_d2h) cudaStreamDestroy(s_d2h);
    }
};

namespace {

int check_cuda(httm_ctx* c, cudaError_t e, const char* what) {
    if (e == cudaSuccess) return HTTM_OK;
    cudaGetLastError();
    return c->fail(HTTM_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

bool overlaps(const void* a, int64_t a_bytes, const void* b, int64_t b_bytes) {
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + (uintptr_t)b_bytes && b0 < a0 + (uintptr_t)a_bytes;
}

int64_t span_bytes(const httm_ctx* c, const httm_tensor& t) {
    return ((int64_t)(c->cfg.heads - 1) * t.stride_head + (int64_t)(c->n_tokens - 1) * t.stride_token + kHeadDim) * 2;
}

int check_tensor(httm_ctx* c, const httm_tensor& t, const char* name) {
    const int rc = check_tensor_layout(t, c->cfg.heads, name, &c->error);
    return rc;
}

int check_io(httm_ctx* c, const httm_tensor& q, const httm_tensor& k, const httm_tensor& v, const httm_tensor& out) {
    int rc;
    if ((rc = check_tensor(c, q, "q")) || (rc = check_tensor(c, k, "k")) || (rc = check_tensor(c, v, "v")) ||
        (rc = check_tensor(c, out, "out")))
        return rc;
    const httm_tensor* in[3] = {&q, &k, &v};
    for (const httm_tensor* t : in)
        if (overlaps(out.ptr, span_bytes(c, out), t->ptr, span_bytes(c, *t)))
            return c->fail(HTTM_ERR_INVALID_ARG, "out overlaps an input tensor");
    return HTTM_OK;
}

TensorView view(const httm_tensor& t) {
    return TensorView{reinterpret_cast<const __nv_bfloat16*>(t.ptr), t.stride_head, t.stride_token};
}
TensorView view(const __nv_bfloat16* p, int64_t rows) { return TensorView{p, rows * kHeadDim, kHeadDim}; }

float scale_log2() { return 1.4426950408889634f / std::sqrt((float)kHeadDim); }

int stage_reorder(httm_ctx* c, const httm_tensor& q, const httm_tensor& k, const httm_tensor& v, cudaStream_t s) {
    ReorderArgs a{};
    a.src[0] = view(q);
    a.src[1] = view(k);
    a.src[2] = view(v);
    a.dst[0] = c->d_qr;
    a.dst[1] = c->d_kr;
    a.dst[2] = c->d_vr;
    a.pi = c->d_pi;
    a.n_tokens = c->n_tokens;
    a.heads = c->cfg.heads;
    a.inv_norm[0] = c->d_inv_norm_q;   // (null unless the context has large blocks)
    a.inv_norm[1] = c->d_inv_norm_k;
    c->launches++;
    return check_cuda(c, launch_reorder(a, s), "reorder launch");
}

SourceLayout source_layout(const httm_ctx* c) {
    SourceLayout L{};
    L.frames = c->cfg.frames;
    L.grid_h = c->cfg.grid_h;
    L.grid_w = c->cfg.grid_w;
    L.n_special = c->n_special;
    L.tokens_per_frame = c->tokens_per_frame;
    L.blk_frames = c->cfg.blk_frames;
    L.blk_h = c->cfg.blk_h;
    L.blk_w = c->cfg.blk_w;
    return L;
}

// The match and merge kernels read every block straight from Q/K/V (tiled TMA loads of the block's patch window):
// the reordered copies are not needed on the hot path (the 16-bit block coordinates bound the scene size).
// A frame's special tokens are staged by one load of n_special rows into the 32-row stage of the merge kernel: more of
// them per frame take the path over the reordered copies (special tokens in chunks of 32).
bool direct_mode(const httm_ctx* c) {
    return c->cfg.frames <= 32767 && c->cfg.grid_h <= 32767 && c->cfg.grid_w <= 32767 && c->n_special <= 32;
}

// Outlier filtering runs on the warp-per-block kernels where blocks have at most 32 tokens and are loaded straight from
// Q/K/V; everywhere else (larger blocks, or scenes that take the reordered copies) on the sorted-group kernels of the
// large-block path, which handle any block size from the reordered copy.
bool sorted_filter(const httm_ctx* c) { return c->filtering() && !(c->max_block <= 32 && direct_mode(c)); }

// The unmerge runs in the attention epilogue where the merge kernel leaves the member lists of the merged query rows:
// blocks of at most 32 tokens, every head with the same merged length (no outlier filtering).
bool fused_unmerge(const httm_ctx* c) { return c->d_group_start != nullptr && !c->filtering(); }

BigMatchArgs big_match_args(httm_ctx* c) {
    BigMatchArgs a{};
    a.xr[0] = c->d_qr;
    a.xr[1] = c->d_kr;
    a.inv_norm[0] = c->d_inv_norm_q;
    a.inv_norm[1] = c->d_inv_norm_k;
    a.best_key[0] = c->d_best_key_q;
    a.best_key[1] = c->d_best_key_k;
    a.best_pos[0] = c->d_best_pos_q;
    a.best_pos[1] = c->d_best_pos_k;
    a.assign[0] = c->d_assign_q;
    a.assign[1] = c->d_assign_k;
    a.blocks = c->d_blocks;
    a.items = c->d_big_items;
    a.n_items = (int32_t)c->big_items.size();
    a.n_blocks = c->n_blocks;
    a.n_tokens = c->n_tokens;
    a.heads = c->cfg.heads;
    a.status = c->d_status;
    return a;
}
int stage_big_scores(httm_ctx* c, cudaStream_t s) {
    c->launches++;
    return check_cuda(c, launch_big_scores(big_match_args(c), c->sm_count, s), "large-block score launch");
}
int stage_big_select(httm_ctx* c, cudaStream_t s) {
    c->launches++;
    return check_cuda(c, launch_big_select(big_match_args(c), s), "large-block select launch");
}

// src: the original Q, K, V (direct mode) or nullptr (blocks come from the reordered copies)
int stage_match(httm_ctx* c, cudaStream_t s, const httm_tensor* src = nullptr) {
    if (c->big()) return c->fail(HTTM_ERR_UNSUPPORTED, "blocks of more than 256 tokens are matched by the large-block stages");
    MatchArgs a{};
    if (src) {
        a.geom = c->d_geom;
        a.src[0] = view(src[0]);
        a.src[1] = view(src[1]);
        a.layout = source_layout(c);
    }
    a.xr[0] = c->d_qr;
    a.xr[1] = c->d_kr;
    a.assign[0] = c->d_assign_q;
    a.assign[1] = c->d_assign_k;
    a.blocks = c->d_blocks;
    a.n_blocks = c->n_blocks;
    a.n_tokens = c->n_tokens;
    a.heads = c->cfg.heads;
    a.status = c->d_status;
    c->launches++;
    int rc = check_cuda(c, launch_match(a, c->max_block, c->sm_count, s), "match launch");
    if (rc || c->n_anchor == 0) return rc;
    c->launches++;
    if (src)
        return check_cuda(c, launch_match_anchor(a, view(src[0]), view(src[1]), c->d_pi, c->n_anchor, c->match_capacity, c->max_block, s), "anchor match launch");
    return check_cuda(c, launch_match_anchor(a, view(c->d_qr, c->n_tokens), view(c->d_kr, c->n_tokens), nullptr, c->n_anchor, c->match_capacity, c->max_block, s),
                      "anchor match launch");
}

int stage_merge(httm_ctx* c, cudaStream_t s, const httm_tensor* src = nullptr) {
    if ((c->big() || sorted_filter(c)) && src)
        return c->fail(HTTM_ERR_UNSUPPORTED, "this context merges from the reordered copies (blocks of more than 256 tokens, or outlier filtering with blocks of more than 32)");
    MergeArgs a{};
    if (src) {
        a.geom = c->d_geom;
        a.src[0] = view(src[0]);
        a.src[1] = view(src[1]);
        a.src[2] = view(src[2]);
        a.layout = source_layout(c);
    }
    a.xr[0] = c->d_qr;
    a.xr[1] = c->d_kr;
    a.xr[2] = c->d_vr;
    a.assign[0] = c->filtering() ? c->d_assign_qf : c->d_assign_q;
    a.assign[1] = c->d_assign_k;
    a.merged[0] = c->filtering() ? c->d_qm_var : c->d_qm;
    a.moff_q_var = c->filtering() ? c->d_moff_var : nullptr;
    a.merged[1] = c->d_km;
    a.merged[2] = c->d_vm;
    a.rank_q = c->d_rank_q;
    if (fused_unmerge(c)) {
        a.group_start = c->d_group_start;
        a.group_member = c->d_group_member;
        a.pi = c->d_pi;
    }
    a.blocks = c->d_blocks;
    a.n_blocks = c->n_blocks;
    a.n_tokens = c->n_tokens;
    a.heads = c->cfg.heads;
    a.n_special_total = c->cfg.frames * c->n_special;
    a.m_q = c->q_rows();
    a.m_k = c->m_k;
    a.status = c->d_status;
    c->launches++;
    if (c->big() || sorted_filter(c)) return check_cuda(c, launch_big_merge(a, c->max_block, s), "sorted-group merge launch");
    return check_cuda(c, launch_merge(a, c->max_block, c->sm_count, s), "merge launch");
}

// final_out: null = the merged output O_m is written (unmerged by the next stage); else the epilogue writes every merged row
// to its member tokens in the caller's output tensor (needs fused_unmerge)
int stage_attention(httm_ctx* c, cudaStream_t s, const httm_tensor* final_out = nullptr) {
    AttentionArgs a{};
    a.q = view(c->filtering() ? c->d_qm_var : c->d_qm, c->q_rows());
    a.k = view(c->d_km, c->m_k);
    a.v = view(c->d_vm, c->m_k);
    if (final_out) {
        if (!fused_unmerge(c)) return c->fail(HTTM_ERR_UNSUPPORTED, "unmerge in the attention epilogue needs blocks of at most 32 tokens and no outlier filtering");
        a.out = reinterpret_cast<__nv_bfloat16*>(final_out->ptr);
        a.out_stride_head = final_out->stride_head;
        a.out_stride_token = final_out->stride_token;
        a.group_start = c->d_group_start;
        a.group_member = c->d_group_member;
        a.n_tokens = c->n_tokens;
    } else {
        a.out = c->filtering() ? c->d_om_var : c->d_om;
        a.out_stride_head = (int64_t)c->q_rows() * kHeadDim;
        a.out_stride_token = kHeadDim;
    }
    c->om_stale = final_out != nullptr;
    a.m_q = c->q_rows();
    if (c->filtering()) {
        a.mq_head = c->d_mq_head;
        a.tile_prefix = c->d_tile_prefix;
    }
    a.m_k = c->m_k;
    a.heads = c->cfg.heads;
    a.scale_log2 = scale_log2();
    a.status = c->d_status;
    c->launches++;
    return check_cuda(c, launch_attention(a, c->sm_count, s), "attention launch");
}

int stage_unmerge(httm_ctx* c, const httm_tensor& out, cudaStream_t s) {
    if (c->om_stale) return c->fail(HTTM_ERR_INVALID_ARG, "the merged output is not there: the last attention launch unmerged in its epilogue (run HTTM_STAGE_ATTENTION first)");
    UnmergeArgs a{};
    a.o_m = c->filtering() ? c->d_om_var : c->d_om;
    a.rank_q = c->d_rank_q;
    a.pi_inv = c->d_pi_inv;
    a.out = reinterpret_cast<__nv_bfloat16*>(out.ptr);
    a.out_stride_head = out.stride_head;
    a.out_stride_token = out.stride_token;
    a.n_tokens = c->n_tokens;
    a.heads = c->cfg.heads;
    a.m_q = c->q_rows();
    a.status = c->d_status;
    c->launches++;
    return check_cuda(c, launch_unmerge(a, s), "unmerge launch");
}

// Sec. 3.4 / Algorithm 2 between match and merge: deviations, global threshold, map update, per-head offsets
int stage_outlier(httm_ctx* c, const httm_tensor& q, cudaStream_t s) {
    OutlierArgs a{};
    a.geom = c->d_geom;
    a.blocks = c->d_blocks;
    a.src_q = view(q);
    a.layout = source_layout(c);
    a.assign_q = c->d_assign_q;
    a.assign_q_out = c->d_assign_qf;
    a.eps = c->d_eps;
    a.tau = c->d_tau;
    a.kept_cnt = c->d_kept_cnt;
    a.moff_var = c->d_moff_var;
    a.mq_head = c->d_mq_head;
    a.tile_prefix = c->d_tile_prefix;
    a.sel = c->d_sel;
    const int64_t all_heads = c->total_heads > 0 ? c->total_heads : c->cfg.heads;
    a.budget = (int64_t)std::floor(c->outlier_fraction * (double)all_heads * (double)c->n_tokens + 1e-9);
    a.total_count = all_heads * (int64_t)c->n_tokens;
    a.defer_select = c->exchange != nullptr;
    a.n_blocks = c->n_blocks;
    a.n_tokens = c->n_tokens;
    a.heads = c->cfg.heads;
    a.n_special_total = c->cfg.frames * c->n_special;
    a.status = c->d_status;
    int rc;
    if ((rc = check_cuda(c, cudaMemsetAsync(c->d_sel, 0, kSelWords * sizeof(int32_t), s), "selection state reset"))) return rc;
    if (c->exchange) {
        // Head-sharded layer: the threshold is one for all heads, so every level's histogram is summed over the shards
        // (the caller's exchange, in stream order) before its bin is chosen.  Nine kernels (ten over the reordered copies).
        const bool sorted = sorted_filter(c);
        if (sorted) {
            a.src_q = view(c->d_qr, c->n_tokens);
            if ((rc = check_cuda(c, launch_big_deviation(a, c->max_block, s), "large-block deviation launch"))) return rc;
            if ((rc = check_cuda(c, launch_refine_level(a, 0, c->sm_count, s), "threshold launch"))) return rc;
            c->launches += 2;
        } else {
            if ((rc = check_cuda(c, launch_deviation(a, c->sm_count, s), "deviation launch"))) return rc;
            c->launches += 1;
        }
        for (int level = 0; level < 3; ++level) {
            if (level > 0) {
                if ((rc = check_cuda(c, launch_refine_level(a, level, c->sm_count, s), "threshold launch"))) return rc;
                c->launches += 1;
            }
            if (c->exchange(c->exchange_user, c->d_sel + kSelHist + level * 2048, level == 2 ? 1024 : 2048, s) != 0)
                return c->fail(HTTM_ERR_CUDA, "the histogram exchange of level %d failed", level);
            if ((rc = check_cuda(c, launch_select_level(a, level, s), "threshold selection launch"))) return rc;
            c->launches += 1;
        }
        c->launches += 2;
        if (sorted) {
            if ((rc = check_cuda(c, launch_big_filter(a, c->max_block, s), "large-block filter launch"))) return rc;
            return check_cuda(c, launch_offsets(a, s), "offsets launch");
        }
        return check_cuda(c, launch_filter(a, s), "filter launch");
    }
    if (sorted_filter(c)) {   // the blocks are runs of rows of the reordered copy; six kernels
        a.src_q = view(c->d_qr, c->n_tokens);
        if ((rc = check_cuda(c, launch_big_deviation(a, c->max_block, s), "large-block deviation launch"))) return rc;
        if ((rc = check_cuda(c, launch_threshold0(a, c->sm_count, s), "threshold launch"))) return rc;
        if ((rc = check_cuda(c, launch_big_filter(a, c->max_block, s), "large-block filter launch"))) return rc;
        c->launches += 6;
        return check_cuda(c, launch_offsets(a, s), "offsets launch");
    }
    if ((rc = check_cuda(c, launch_deviation(a, c->sm_count, s), "deviation launch"))) return rc;
    if ((rc = check_cuda(c, launch_threshold(a, c->sm_count, s), "threshold launch"))) return rc;
    c->launches += 5;
    return check_cuda(c, launch_filter(a, s), "filter launch");
}

int dense_impl(httm_ctx* c, const httm_tensor& q, const httm_tensor& k, const httm_tensor& v, const httm_tensor& out,
               cudaStream_t s) {
    AttentionArgs a{};
    a.q = view(q);
    a.k = view(k);
    a.v = view(v);
    a.out = reinterpret_cast<__nv_bfloat16*>(out.ptr);
    a.out_stride_head = out.stride_head;
    a.out_stride_token = out.stride_token;
    a.m_q = c->n_tokens;
    a.m_k = c->n_tokens;
    a.heads = c->cfg.heads;
    a.scale_log2 = scale_log2();
    a.status = c->d_status;
    c->launches++;
    return check_cuda(c, launch_attention(a, c->sm_count, s), "dense attention launch");
}

int global_impl(httm_ctx* c, const httm_tensor& q, const httm_tensor& k, const httm_tensor& v, const httm_tensor& out,
                cudaStream_t s) {
    // With call timing on, an event follows every part of the call (a part is one kernel, or the five small kernels of
    // the outlier filter); part(rc, name) passes the stage's return code through.
    c->call_parts = 0;
    if (c->call_timing) cudaEventRecord(c->call_ev[0], s);
    auto part = [&](int rc, const char* name) {
        if (rc == HTTM_OK && c->call_timing && c->call_parts < httm_ctx::kMaxCallParts) {
            c->call_part[c->call_parts++] = name;
            cudaEventRecord(c->call_ev[c->call_parts], s);
        }
        return rc;
    };
    int rc;
    if (c->big()) {   // six kernels: reorder (+ norms), scores, select, merge, attention, unmerge
        if ((rc = part(stage_reorder(c, q, k, v, s), "reorder"))) return rc;
        if ((rc = part(stage_big_scores(c, s), "big_scores"))) return rc;
        if ((rc = part(stage_big_select(c, s), "big_select"))) return rc;
        if (c->filtering() && (rc = part(stage_outlier(c, q, s), "outlier_filter"))) return rc;
        if ((rc = part(stage_merge(c, s), "merge"))) return rc;
        if ((rc = part(stage_attention(c, s), "attention"))) return rc;
        return part(stage_unmerge(c, out, s), "unmerge");
    }
    if (sorted_filter(c)) {   // outlier filtering with blocks of 33 .. 256 tokens: everything from the reordered copies
        if ((rc = part(stage_reorder(c, q, k, v, s), "reorder"))) return rc;
        if ((rc = part(stage_match(c, s), "match"))) return rc;
        if ((rc = part(stage_outlier(c, q, s), "outlier_filter"))) return rc;
        if ((rc = part(stage_merge(c, s), "merge"))) return rc;
        if ((rc = part(stage_attention(c, s), "attention"))) return rc;
        return part(stage_unmerge(c, out, s), "unmerge");
    }
    if (direct_mode(c)) {   // the temporal reorder is folded into the block loads of match and merge
        const httm_tensor src[3] = {q, k, v};
        if ((rc = part(stage_match(c, s, src), "match_direct"))) return rc;
        if (c->filtering() && (rc = part(stage_outlier(c, q, s), "outlier_filter"))) return rc;
        if ((rc = part(stage_merge(c, s, src), "merge_direct"))) return rc;
    } else {
        if ((rc = part(stage_reorder(c, q, k, v, s), "reorder"))) return rc;
        if ((rc = part(stage_match(c, s), "match"))) return rc;
        if ((rc = part(stage_merge(c, s), "merge"))) return rc;
    }
    // ... and the unmerge into the attention epilogue: three kernels
    if (fused_unmerge(c)) return part(stage_attention(c, s, &out), "attention_unmerge");
    if ((rc = part(stage_attention(c, s), "attention"))) return rc;
    return part(stage_unmerge(c, out, s), "unmerge");
}

int device_status(httm_ctx* c, int32_t* value) {
    cudaError_t e = cudaMemcpy(value, c->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost);   // syncs
    return check_cuda(c, e, "read device status");
}

}  // namespace

namespace httm {
// lets other translation units of the library report through httm_last_error(NULL)
void set_global_error(const std::string& msg) { g_create_error = msg; }
}  // namespace httm

extern "C" {

int httm_create(const httm_config* cfg, httm_ctx** out) {
    if (out) *out = nullptr;
    if (!cfg || !out) {
        g_create_error = "httm_create: null argument";
        return HTTM_ERR_INVALID_ARG;
    }
    auto bad = [&](int code, const char* msg) {
        g_create_error = std::string("httm_create: ") + msg;
        return code;
    };
    {
        std::string why;
        const int rc = check_config(*cfg, &why);
        if (rc != HTTM_OK) return bad(rc, why.c_str());
    }
    const int64_t bf = std::min<int64_t>(cfg->blk_frames, cfg->frames), bh = std::min<int64_t>(cfg->blk_h, cfg->grid_h),
                  bw = std::min<int64_t>(cfg->blk_w, cfg->grid_w);
    if (bf * bh * bw > kMaxBigBlockTokens) return bad(HTTM_ERR_UNSUPPORTED, "a merging block may hold at most 4096 tokens");
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || cfg->device < 0 || cfg->device >= n_dev) {
        cudaGetLastError();
        return bad(HTTM_ERR_INVALID_ARG, "device ordinal out of range (or no CUDA device)");
    }

    httm_ctx* c = new (std::nothrow) httm_ctx();
    if (!c) return bad(HTTM_ERR_NOMEM, "host allocation failed");
    c->cfg = *cfg;
    int anchored_nd_max = 0;
    {   // reorder index, block table and merge budgets (Sec. 3.2 / 3.3)
        HostPlan plan;
        build_host_plan(*cfg, &plan);
        c->n_special = plan.n_special;
        c->tokens_per_frame = plan.tokens_per_frame;
        c->n_tokens = plan.n_tokens;
        c->n_blocks = plan.n_blocks;
        c->max_block = plan.max_block;
        c->m_q = plan.m_q;
        c->m_k = plan.m_k;
        anchored_nd_max = plan.anchored_dst_max;
        c->pi = std::move(plan.pi);
        c->pi_inv = std::move(plan.pi_inv);
        c->blk_start = std::move(plan.blk_start);
        c->blocks = std::move(plan.blocks);
        c->geom = std::move(plan.geom);
        for (int32_t b = 0; b < c->n_blocks; ++b)
            for (int row0 = 0; row0 < c->blocks[b].n; row0 += kBigSliceRows) c->big_items.push_back(BigItem{b, row0});
    }
    {   // the match kernels hold a quarter of their largest block as dst tokens (the large-block path 1024); anchored blocks of
        // up to 256 tokens with more (two or three frames per block) go to a kernel of their own
        const int cap = c->max_block > kMaxBlockTokens ? kMaxBigDst : (c->max_block <= 32 ? 8 : (c->max_block <= 64 ? 16 : (c->max_block <= 128 ? 32 : 64)));
        c->match_capacity = cap;
        if (anchored_nd_max > cap) {
            if (c->max_block > kMaxBlockTokens) {
                delete c;
                return bad(HTTM_ERR_UNSUPPORTED, "first-frame anchoring: blocks of more than 256 tokens may hold at most 1024 tokens of frame 0");
            }
            const int64_t groups = (cfg->frames + cfg->blk_frames - 1) / cfg->blk_frames;
            c->n_anchor = (int32_t)(c->n_blocks / groups);   // the blocks of the first frame group come first
        }
    }
    DeviceGuard guard(cfg->device);
    int rc = HTTM_OK;
    auto done = [&](int code) -> int {
        if (code != HTTM_OK) {
            g_create_error = "httm_create: " + c->error;
            c->release();
            delete c;
            return code;
        }
        *out = c;
        return HTTM_OK;
    };
    if (!guard.ok) return done(c->fail(HTTM_ERR_CUDA, "cudaSetDevice failed"));
    cudaDeviceProp prop{};
    if ((rc = check_cuda(c, cudaGetDeviceProperties(&prop, cfg->device), "cudaGetDeviceProperties"))) return done(rc);
    if (prop.major != 10) return done(c->fail(HTTM_ERR_UNSUPPORTED, "device is sm_%d%d; this library is built for sm_100a only",
                                               prop.major, prop.minor));
    c->sm_count = prop.multiProcessorCount;
    if ((rc = check_cuda(c, configure_kernels(), "cudaFuncSetAttribute"))) return done(rc);
    if ((rc = check_cuda(c, configure_big_blocks(), "cudaFuncSetAttribute"))) return done(rc);
    if ((rc = check_cuda(c, configure_linear(), "cudaFuncSetAttribute"))) return done(rc);

    const size_t H = cfg->heads, N = c->n_tokens;
    if ((rc = c->alloc(&c->d_pi, N)) || (rc = c->alloc(&c->d_pi_inv, N)) || (rc = c->alloc(&c->d_blocks, c->blocks.size())) || (rc = c->alloc(&c->d_geom, c->geom.size())) ||
        (rc = c->alloc(&c->d_status, 4)) || (rc = c->alloc(&c->d_assign_q, H * N)) || (rc = c->alloc(&c->d_assign_k, H * N)) ||
        (rc = c->alloc(&c->d_rank_q, H * N)) || (rc = c->alloc(&c->d_qr, H * N * kHeadDim)) ||
        (rc = c->alloc(&c->d_kr, H * N * kHeadDim)) || (rc = c->alloc(&c->d_vr, H * N * kHeadDim)) ||
        (rc = c->alloc(&c->d_qm, H * c->m_q * kHeadDim)) || (rc = c->alloc(&c->d_km, H * c->m_k * kHeadDim)) ||
        (rc = c->alloc(&c->d_vm, H * c->m_k * kHeadDim)) || (rc = c->alloc(&c->d_om, H * c->m_q * kHeadDim)))
        return done(rc);

    if (c->max_block <= 32) {   // member lists of the merged query rows; entry M_q of every head is the constant N
        if ((rc = c->alloc(&c->d_group_start, H * (size_t)(c->m_q + 1))) || (rc = c->alloc(&c->d_group_member, H * N))) return done(rc);
        std::vector<int32_t> gs(H * (size_t)(c->m_q + 1), 0);
        for (size_t hd = 0; hd < H; ++hd) gs[hd * (size_t)(c->m_q + 1) + c->m_q] = c->n_tokens;
        if ((rc = check_cuda(c, cudaMemcpy(c->d_group_start, gs.data(), gs.size() * 4, cudaMemcpyHostToDevice), "group table upload"))) return done(rc);
    }
    if (c->big()) {
        if ((rc = c->alloc(&c->d_big_items, c->big_items.size())) || (rc = c->alloc(&c->d_inv_norm_q, H * N)) ||
            (rc = c->alloc(&c->d_inv_norm_k, H * N)) || (rc = c->alloc(&c->d_best_key_q, H * N)) || (rc = c->alloc(&c->d_best_key_k, H * N)) ||
            (rc = c->alloc(&c->d_best_pos_q, H * N)) || (rc = c->alloc(&c->d_best_pos_k, H * N)))
            return done(rc);
        if ((rc = check_cuda(c, cudaMemcpy(c->d_big_items, c->big_items.data(), c->big_items.size() * sizeof(BigItem), cudaMemcpyHostToDevice),
                             "item table upload")))
            return done(rc);
    }
    // uploads; special tokens are never merged: their map entries are constants, written once
    std::vector<int32_t> ident(H * N);
    for (size_t hd = 0; hd < H; ++hd)
        for (size_t p = 0; p < N; ++p) ident[hd * N + p] = (int32_t)p;
    cudaError_t e = cudaSuccess;
    auto up = [&](void* dst, const void* src, size_t bytes) {
        if (e == cudaSuccess && bytes) e = cudaMemcpy(dst, src, bytes, cudaMemcpyHostToDevice);
    };
    up(c->d_pi, c->pi.data(), N * 4);
    up(c->d_pi_inv, c->pi_inv.data(), N * 4);
    up(c->d_blocks, c->blocks.data(), c->blocks.size() * sizeof(BlockInfo));
    up(c->d_geom, c->geom.data(), c->geom.size() * sizeof(BlockGeom));
    up(c->d_assign_q, ident.data(), H * N * 4);
    up(c->d_assign_k, ident.data(), H * N * 4);
    up(c->d_rank_q, ident.data(), H * N * 4);
    if (e == cudaSuccess) e = cudaMemset(c->d_status, 0, 16);
    if ((rc = check_cuda(c, e, "workspace upload"))) return done(rc);
    return done(HTTM_OK);
}

int httm_global_attention(httm_ctx* c, httm_tensor q, httm_tensor k, httm_tensor v, httm_tensor out, void* cuda_stream) {
    if (!c) return HTTM_ERR_INVALID_ARG;
    int rc = check_io(c, q, k, v, out);
    if (rc) return rc;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return c->fail(HTTM_ERR_CUDA, "cudaSetDevice failed");
    return global_impl(c, q, k, v, out, static_cast<cudaStream_t>(cuda_stream));
}

int httm_set_outlier_fraction(httm_ctx* c, double fraction) {
    if (!c) return HTTM_ERR_INVALID_ARG;
    if (!(fraction >= 0.0 && fraction <= 1.0)) return c->fail(HTTM_ERR_INVALID_ARG, "outlier fraction must lie in [0, 1]");
    if (fraction == 0.0) {
        c->outlier_fraction = 0.0;
        return HTTM_OK;
    }
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return c->fail(HTTM_ERR_CUDA, "cudaSetDevice failed");
    if (!c->d_eps) {
        const size_t H = c->cfg.heads, N = c->n_tokens, B = c->n_blocks;
        int rc;
        const int64_t before = c->workspace_bytes;
        if ((rc = c->alloc(&c->d_assign_qf, H * N)) || (rc = c->alloc(&c->d_kept_cnt, H * B)) || (rc = c->alloc(&c->d_moff_var, H * B)) ||
            (rc = c->alloc(&c->d_mq_head, H)) || (rc = c->alloc(&c->d_tile_prefix, H + 1)) || (rc = c->alloc(&c->d_sel, kSelWords)) ||
            (rc = c->alloc(&c->d_tau, 1)) || (rc = c->alloc(&c->d_qm_var, H * N * kHeadDim)) || (rc = c->alloc(&c->d_om_var, H * N * kHeadDim)) ||
            (rc = c->alloc(&c->d_eps, H * N))) {
            // give back what this attempt took: a later call starts from nothing again
            void** taken[] = {(void**)&c->d_assign_qf, (void**)&c->d_kept_cnt, (void**)&c->d_moff_var, (void**)&c->d_mq_head, (void**)&c->d_tile_prefix,
                              (void**)&c->d_sel, (void**)&c->d_tau, (void**)&c->d_qm_var, (void**)&c->d_om_var, (void**)&c->d_eps};
            for (void** p : taken) {
                if (*p) cudaFree(*p);
                *p = nullptr;
            }
            c->workspace_bytes = before;
            return rc;
        }
        // special tokens: never merged (identity map entries, deviation 0), written here once; rows of Q_m past a head's
        // merged length are read by the last query tile of the head (their results are discarded): give them a value
        std::vector<int32_t> ident(H * N);
        for (size_t hd = 0; hd < H; ++hd)
            for (size_t p = 0; p < N; ++p) ident[hd * N + p] = (int32_t)p;
        cudaError_t e = cudaMemcpy(c->d_assign_qf, ident.data(), H * N * 4, cudaMemcpyHostToDevice);
        if (e == cudaSuccess) e = cudaMemset(c->d_eps, 0, H * N * 4);
        if (e == cudaSuccess) e = cudaMemset(c->d_qm_var, 0, H * N * kRowBytes);
        if (e == cudaSuccess) e = cudaMemset(c->d_sel, 0, kSelWords * sizeof(int32_t));
        if ((rc = check_cuda(c, e, "outlier workspace setup"))) return rc;
    }
    c->outlier_fraction = fraction;
    return HTTM_OK;
}

int httm_set_call_timing(httm_ctx* c, int32_t enable) {
    if (!c) return HTTM_ERR_INVALID_ARG;
    if (enable != 0 && enable != 1) return c->fail(HTTM_ERR_INVALID_ARG, "enable must be 0 or 1");
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return c->fail(HTTM_ERR_CUDA, "cudaSetDevice failed");
    if (enable && !c->call_ev[0]) {
        for (cudaEvent_t& e : c->call_ev) {
            const int rc = check_cuda(c, cudaEventCreate(&e), "cudaEventCreate");
            if (rc) return rc;
        }
    }
    c->call_timing = enable != 0;
    c->call_parts = 0;
    return HTTM_OK;
}

int httm_call_times(httm_ctx* c, float* ms, const char** names, int32_t capacity, int32_t* count) {
    if (!c) return HTTM_ERR_INVALID_ARG;
    if (!ms || !count || capacity < 0) return c->fail(HTTM_ERR_INVALID_ARG, "httm_call_times: null argument");
    if (!c->call_timing) return c->fail(HTTM_ERR_INVALID_ARG, "call timing is off (httm_set_call_timing)");
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return c->fail(HTTM_ERR_CUDA, "cudaSetDevice failed");
    *count = c->call_parts;
    if (c->call_parts == 0) return HTTM_OK;
    int rc = check_cuda(c, cudaEventSynchronize(c->call_ev[c->call_parts]), "cudaEventSynchronize");
    for (int i = 0; rc == HTTM_OK && i < c->call_parts && i < capacity; ++i) {
        rc = check_cuda(c, cudaEventElapsedTime(&ms[i], c->call_ev[i], c->call_ev[i + 1]), "cudaEventElapsedTime");
        if (names) names[i] = c->call_part[i];
    }
    return rc;
}

int httm_fail_nth_allocation(int32_t n) {
    g_fail_allocation = n > 0 ? n : 0;
    return HTTM_OK;
}

int httm_expire_a_wait(httm_ctx* c, void* cuda_stream) {
    if (!c) return HTTM_ERR_INVALID_ARG;
    if ((int64_t)c->cfg.heads * c->n_tokens < 3 * 128) return c->fail(HTTM_ERR_UNSUPPORTED, "the context's workspace is smaller than three 128-token tiles");
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return c->fail(HTTM_ERR_CUDA, "cudaSetDevice failed");
    c->launches++;
    return check_cuda(c, launch_wait_expiry(c->d_qr, reinterpret_cast<float*>(c->d_kr), c->d_status, static_cast<cudaStream_t>(cuda_stream)),
                      "wait-expiry launch");
}

int httm_set_head_shard(httm_ctx* c, int32_t total_heads, httm_exchange_fn exchange, void* user) {
    if (!c) return HTTM_ERR_INVALID_ARG;
    if (total_heads == 0 && !exchange) {   // back to a layer of its own
        c->total_heads = 0;
        c->exchange = nullptr;
        c->exchange_user = nullptr;
        return HTTM_OK;
    }
    if (total_heads < c->cfg.heads) return c->fail(HTTM_ERR_INVALID_ARG, "head shard: the layer cannot have fewer heads than this context");
    if ((int64_t)total_heads * c->n_tokens > (1ll << 31) - 1) return c->fail(HTTM_ERR_UNSUPPORTED, "head shard: total heads x tokens must stay below 2^31");
    if (total_heads > c->cfg.heads && !exchange) return c->fail(HTTM_ERR_INVALID_ARG, "head shard: an exchange function is needed when other shards hold heads");
    c->total_heads = total_heads;
    c->exchange = exchange;
    c->exchange_user = user;
    return HTTM_OK;
}

int httm_linear(httm_ctx* c, const void* x, int64_t ldx, const void* w, int64_t ldw, void* y, int64_t ldy, int64_t n_rows,
                int32_t in_features, int32_t out_features, void* cuda_stream) {
    if (!c) return HTTM_ERR_INVALID_ARG;
    if (n_rows < 0 || in_features < 1 || out_features < 1 || n_rows > (1ll << 31) - 256)
        return c->fail(HTTM_ERR_INVALID_ARG, "linear: sizes out of range");
    if (n_rows == 0) return HTTM_OK;   // nothing to do (an empty matrix may come with a null pointer)
    if (!x || !w || !y) return c->fail(HTTM_ERR_INVALID_ARG, "linear: null pointer");
    if (in_features % 64 != 0 || out_features % 8 != 0)
        return c->fail(HTTM_ERR_UNSUPPORTED, "linear: in_features must be a multiple of 64 and out_features a multiple of 8");
    if ((((uintptr_t)x | (uintptr_t)w | (uintptr_t)y) & 15u) != 0 || ldx % 8 != 0 || ldw % 8 != 0 || ldy % 8 != 0)
        return c->fail(HTTM_ERR_ALIGNMENT, "linear: pointers must be 16-byte aligned and leading dimensions multiples of 8");
    if (ldx < in_features || ldw < in_features || ldy < out_features)
        return c->fail(HTTM_ERR_INVALID_ARG, "linear: a leading dimension is smaller than its row");
    if (overlaps(y, ((n_rows - 1) * ldy + out_features) * 2, x, ((n_rows - 1) * ldx + in_features) * 2) ||
        overlaps(y, ((n_rows - 1) * ldy + out_features) * 2, w, ((int64_t)(out_features - 1) * ldw + in_features) * 2))
        return c->fail(HTTM_ERR_INVALID_ARG, "linear: y overlaps an input");
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return c->fail(HTTM_ERR_CUDA, "cudaSetDevice failed");
    LinearArgs a{};
    a.x = static_cast<const __nv_bfloat16*>(x);
    a.w = static_cast<const __nv_bfloat16*>(w);
    a.y = static_cast<__nv_bfloat16*>(y);
    a.ldx = ldx;
    a.ldw = ldw;
    a.ldy = ldy;
    a.n_rows = n_rows;
    a.in_features = in_features;
    a.out_features = out_features;
    a.status = c->d_status;
    c->launches++;
    return check_cuda(c, launch_linear(a, c->sm_count, static_cast<cudaStream_t>(cuda_stream)), "linear launch");
}

int httm_dense_attention(httm_ctx* c, httm_tensor q, httm_tensor k, httm_tensor v, httm_tensor out, void* cuda_stream) {
    if (!c) return HTTM_ERR_INVALID_ARG;
    int rc = check_io(c, q, k, v, out);
    if (rc) return rc;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return c->fail(HTTM_ERR_CUDA, "cudaSetDevice failed");
    return dense_impl(c, q, k, v, out, static_cast<cudaStream_t>(cuda_stream));
}

int httm_attention_host(httm_ctx* c, const void* q_host, const void* k_host, const void* v_host, void* out_host, int dense,
                        void* cuda_stream) {
    if (!c) return HTTM_ERR_INVALID_ARG;
    if (!q_host || !k_host || !v_host || !out_host) return c->fail(HTTM_ERR_INVALID_ARG, "null host pointer");
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return c->fail(HTTM_ERR_CUDA, "cudaSetDevice failed");
    const size_t elems = (size_t)c->cfg.heads * c->n_tokens * kHeadDim;
    int rc;
    if (!c->s_h2d) {   // first call: buffers, streams, events
        for (httm_ctx::HostSet& h : c->hs)
            if ((rc = c->alloc(&h.q, elems)) || (rc = c->alloc(&h.k, elems)) || (rc = c->alloc(&h.v, elems)) || (rc = c->alloc(&h.out, elems)))
                return rc;
        cudaError_t e = cudaStreamCreateWithFlags(&c->s_h2d, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->s_d2h, cudaStreamNonBlocking);
        for (httm_ctx::HostSet& h : c->hs)
            for (cudaEvent_t* ev : {&h.loaded, &h.consumed, &h.computed, &h.returned})
                if (e == cudaSuccess) e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming);
        if ((rc = check_cuda(c, e, "copy streams and events"))) return rc;
    }
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    httm_ctx::HostSet& h = c->hs[c->host_calls & 1];
    ++c->host_calls;
    // host -> device on the copy stream, once the call that used this set two calls ago has read its inputs.  The
    // copy does NOT wait for earlier work on `stream`: the host buffers must hold their data when the call is made.
    cudaError_t e = cudaSuccess;
    if (h.used) e = cudaStreamWaitEvent(c->s_h2d, h.consumed, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h.q, q_host, elems * 2, cudaMemcpyHostToDevice, c->s_h2d);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h.k, k_host, elems * 2, cudaMemcpyHostToDevice, c->s_h2d);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h.v, v_host, elems * 2, cudaMemcpyHostToDevice, c->s_h2d);
    if (e == cudaSuccess) e = cudaEventRecord(h.loaded, c->s_h2d);
    // kernels on the caller's stream, after the inputs have landed and after this set's previous result has left
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s, h.loaded, 0);
    if (e == cudaSuccess && h.used) e = cudaStreamWaitEvent(s, h.returned, 0);
    if ((rc = check_cuda(c, e, "host to device copy"))) return rc;
    const int64_t N = c->n_tokens, H = c->cfg.heads;
    httm_tensor q{h.q, N * kHeadDim, kHeadDim}, k{h.k, N * kHeadDim, kHeadDim}, v{h.v, N * kHeadDim, kHeadDim};
    httm_tensor o{h.out, kHeadDim, H * kHeadDim};
    rc = dense ? dense_impl(c, q, k, v, o, s) : global_impl(c, q, k, v, o, s);
    if (rc) return rc;
    // (the workspace between the kernels is shared by consecutive calls: they run in order on the caller's stream)
    e = cudaEventRecord(h.computed, s);
    if (e == cudaSuccess) e = cudaEventRecord(h.consumed, s);
    // device -> host on the second copy stream; the caller's stream waits for it, so that synchronising `stream`
    // (or anything enqueued on it later) sees the result
    if (e == cudaSuccess) e = cudaStreamWaitEvent(c->s_d2h, h.computed, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out_host, h.out, elems * 2, cudaMemcpyDeviceToHost, c->s_d2h);
    if (e == cudaSuccess) e = cudaEventRecord(h.returned, c->s_d2h);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s, h.returned, 0);
    h.used = true;
    return check_cuda(c, e, "device to host copy");
}

int httm_launch_stage(httm_ctx* c, int stage, httm_tensor q, httm_tensor k, httm_tensor v, httm_tensor out, void* cuda_stream) {
    if (!c) return HTTM_ERR_INVALID_ARG;
    DeviceGuard guard(c->cfg.device);
    if (!guard.ok) return c->fail(HTTM_ERR_CUDA, "cudaSetDevice failed");
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    int rc;
    switch (stage) {
        case HTTM_STAGE_REORDER:
            if ((rc = check_tensor(c, q, "q")) || (rc = check_tensor(c, k, "k")) || (rc = check_tensor(c, v, "v"))) return rc;
            return stage_reorder(c, q, k, v, s);
        case HTTM_STAGE_MATCH:
            return stage_match(c, s);
        case HTTM_STAGE_MERGE:
            return stage_merge(c, s);
        case HTTM_STAGE_ATTENTION:
            return stage_attention(c, s);
        case HTTM_STAGE_UNMERGE:
            if ((rc = check_tensor(c, out, "out"))) return rc;
            return stage_unmerge(c, out, s);
        case HTTM_STAGE_ATTENTION_UNMERGE:
            if ((rc = check_tensor(c, out, "out"))) return rc;
            return stage_attention(c, s, &out);
        case HTTM_STAGE_BIG_SCORES:
        case HTTM_STAGE_BIG_SELECT:
            if (!c->big()) return c->fail(HTTM_ERR_UNSUPPORTED, "the large-block stages need merging blocks of more than 256 tokens");
            return stage == HTTM_STAGE_BIG_SCORES ? stage_big_scores(c, s) : stage_big_select(c, s);
        case HTTM_STAGE_OUTLIER_FILTER:
            if (!c->filtering()) return c->fail(HTTM_ERR_INVALID_ARG, "outlier filtering is off: call httm_set_outlier_fraction first");
            if ((rc = check_tensor(c, q, "q"))) return rc;
            return stage_outlier(c, q, s);
        case HTTM_STAGE_MATCH_DIRECT:
        case HTTM_STAGE_MERGE_DIRECT: {
            if (!direct_mode(c)) return c->fail(HTTM_ERR_UNSUPPORTED, "direct stages need a scene of at most 32767 frames / patch rows / patch columns and at most 32 special tokens per frame");
            if ((rc = check_tensor(c, q, "q")) || (rc = check_tensor(c, k, "k")) || (rc = check_tensor(c, v, "v"))) return rc;
            const httm_tensor src[3] = {q, k, v};
            return stage == HTTM_STAGE_MATCH_DIRECT ? stage_match(c, s, src) : stage_merge(c, s, src);
        }
        default:
            return c->fail(HTTM_ERR_INVALID_ARG, "unknown stage %d", stage);
    }
}

int httm_query(httm_ctx* c, int what, int64_t* value) {
    if (!c) return HTTM_ERR_INVALID_ARG;
    if (!value) return c->fail(HTTM_ERR_INVALID_ARG, "null value pointer");
    switch (what) {
        case HTTM_Q_TOKENS: *value = c->n_tokens; return HTTM_OK;
        case HTTM_Q_MERGED_Q: *value = c->m_q; return HTTM_OK;
        case HTTM_Q_MERGED_K: *value = c->m_k; return HTTM_OK;
        case HTTM_Q_BLOCKS: *value = c->n_blocks; return HTTM_OK;
        case HTTM_Q_WORKSPACE_BYTES: *value = c->workspace_bytes; return HTTM_OK;
        case HTTM_Q_MAX_BLOCK_TOKENS: *value = c->max_block; return HTTM_OK;
        case HTTM_Q_MERGED_Q_ROWS: *value = c->q_rows(); return HTTM_OK;
        case HTTM_Q_OUTLIERS: {
            *value = 0;
            if (!c->filtering()) return HTTM_OK;
            DeviceGuard guard(c->cfg.device);
            int32_t cnt = 0;
            int rc = check_cuda(c, cudaMemcpy(&cnt, c->d_sel + kSelOutliers, sizeof cnt, cudaMemcpyDeviceToHost), "read outlier count");
            *value = cnt;
            return rc;
        }
        case HTTM_Q_DEVICE_STATUS: {
            DeviceGuard guard(c->cfg.device);
            int32_t st = 0;
            int rc = device_status(c, &st);
            if (rc) return rc;
            *value = st;
            if (st != kDevOk)
                return c->fail(st == kDevBadIndex ? HTTM_ERR_CUDA : HTTM_ERR_TIMEOUT, "device status word = %d", st);
            return HTTM_OK;
        }
        default: return c->fail(HTTM_ERR_INVALID_ARG, "unknown query %d", what);
    }
}

int httm_export(httm_ctx* c, int what, void* host_dst, size_t bytes, void* cuda_stream) {
    if (!c) return HTTM_ERR_INVALID_ARG;
    if (!host_dst) return c->fail(HTTM_ERR_INVALID_ARG, "null destination");
    const size_t H = c->cfg.heads, N = c->n_tokens;
    const void* src = nullptr;
    size_t need = 0;
    bool host_src = false;
    switch (what) {
        case HTTM_X_PI: src = c->pi.data(); need = N * 4; host_src = true; break;
        case HTTM_X_PI_INV: src = c->pi_inv.data(); need = N * 4; host_src = true; break;
        case HTTM_X_BLOCK_START: src = c->blk_start.data(); need = c->blk_start.size() * 4; host_src = true; break;
        case HTTM_X_ASSIGN_Q: src = c->filtering() ? c->d_assign_qf : c->d_assign_q; need = H * N * 4; break;
        case HTTM_X_ASSIGN_Q_INITIAL: src = c->d_assign_q; need = H * N * 4; break;
        case HTTM_X_DEVIATION: src = c->d_eps; need = H * N * 4; break;
        case HTTM_X_THRESHOLD: src = c->d_tau; need = 4; break;
        case HTTM_X_MERGED_Q_HEAD: src = c->d_mq_head; need = H * 4; break;
        case HTTM_X_ASSIGN_K: src = c->d_assign_k; need = H * N * 4; break;
        case HTTM_X_RANK_Q: src = c->d_rank_q; need = H * N * 4; break;
        case HTTM_X_Q_REORDERED: src = c->d_qr; need = H * N * kRowBytes; break;
        case HTTM_X_K_REORDERED: src = c->d_kr; need = H * N * kRowBytes; break;
        case HTTM_X_V_REORDERED: src = c->d_vr; need = H * N * kRowBytes; break;
        case HTTM_X_Q_MERGED: src = c->filtering() ? c->d_qm_var : c->d_qm; need = H * (size_t)c->q_rows() * kRowBytes; break;
        case HTTM_X_K_MERGED: src = c->d_km; need = H * (size_t)c->m_k * kRowBytes; break;
        case HTTM_X_V_MERGED: src = c->d_vm; need = H * (size_t)c->m_k * kRowBytes; break;
        case HTTM_X_O_MERGED: src = c->filtering() ? c->d_om_var : c->d_om; need = H * (size_t)c->q_rows() * kRowBytes; break;
        default: return c->fail(HTTM_ERR_INVALID_ARG, "unknown export %d", what);
    }
    if (!src) return c->fail(HTTM_ERR_INVALID_ARG, "export %d needs outlier filtering switched on", what);
    if (bytes != need) return c->fail(HTTM_ERR_INVALID_ARG, "export %d needs %zu bytes, got %zu", what, need, bytes);
    if (what == HTTM_X_O_MERGED && c->om_stale) {
        // the last call unmerged in the attention epilogue and left O_m alone: compute it now from the merged Q, K, V of that call
        DeviceGuard guard(c->cfg.device);
        const int rc = stage_attention(c, static_cast<cudaStream_t>(cuda_stream));
        if (rc) return rc;
    }
    if (host_src) {
        memcpy(host_dst, src, need);
        return HTTM_OK;
    }
    DeviceGuard guard(c->cfg.device);
    int rc;
    if ((rc = check_cuda(c, cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)), "stream synchronize"))) return rc;
    if ((rc = check_cuda(c, cudaMemcpy(host_dst, src, need, cudaMemcpyDeviceToHost), "export copy"))) return rc;
    int32_t st = 0;
    if ((rc = device_status(c, &st))) return rc;
    if (st != kDevOk) return c->fail(st == kDevBadIndex ? HTTM_ERR_CUDA : HTTM_ERR_TIMEOUT, "device status word = %d", st);
    return HTTM_OK;
}

const char* httm_last_error(const httm_ctx* c) { return c ? c->error.c_str() : g_create_error.c_str(); }

int64_t httm_launch_count(const httm_ctx* c) { return c ? c->launches : 0; }

int httm_destroy(httm_ctx* c) {
    if (!c) return HTTM_OK;
    {
        DeviceGuard guard(c->cfg.device);
        c->release();
    }
    delete c;
    return HTTM_OK;
}

}  // extern "C"
