// Host-side plan of a scene: the temporal-reorder permutation and the block table (Sec. 3.3), the merge budgets
// (Sec. 3.2) and the layout checks of the caller's tensors.  One copy, used by every entry point of the library.
#pragma once

#include <algorithm>
#include <cmath>
#include <string>
#include <vector>

#include "../../include/httm.h"
#include "httm_internal.h"

namespace httm {

// Merge budget of a block of n tokens (Sec. 3.2, r = N - M): r src tokens are merged away,
// n_dst evenly spaced tokens act as destinations.
inline void block_budget(int n, double ratio, int32_t* r, int32_t* nd) {
    int64_t rr = (int64_t)std::floor(ratio * (double)n + 1e-9);
    rr = std::max<int64_t>(0, std::min<int64_t>(rr, n - 1));
    const int64_t d = std::min<int64_t>((n + 3) / 4, n - rr);
    *r = (int32_t)rr;
    *nd = (int32_t)d;
}

struct HostPlan {
    int32_t n_special = 0, tokens_per_frame = 0, n_tokens = 0, n_blocks = 0, max_block = 0;
    int32_t m_q = 0, m_k = 0;          // merged lengths (closed form: the same for every head)
    int32_t anchored_dst_max = 0;      // largest dst count of a block under first-frame anchoring
    std::vector<int32_t> pi, pi_inv;   // reordered position -> original index and back
    std::vector<int32_t> blk_start;    // n_blocks + 1 entries
    std::vector<BlockInfo> blocks;
    std::vector<BlockGeom> geom;
};

// Reorder index pi (Sec. 3.3): special tokens first (frame-major), then the blocks in (frame group, window row,
// window column) order, inside a block frame / y / x; windows and frame groups are clipped at the edges.
// With cfg.anchor_first_frame the blocks of the first frame group take their tokens of frame 0 as dst tokens.
// The caller has validated cfg (positive sizes, N < 2^31).
inline void build_host_plan(const httm_config& cfg, HostPlan* p) {
    const int S = cfg.frames, h = cfg.grid_h, w = cfg.grid_w;
    p->n_special = cfg.n_camera + cfg.n_register;
    p->tokens_per_frame = p->n_special + h * w;
    p->n_tokens = S * p->tokens_per_frame;
    const int nsp = p->n_special, P = p->tokens_per_frame;
    p->pi.assign(p->n_tokens, 0);
    p->pi_inv.assign(p->n_tokens, 0);
    p->blk_start.clear();
    p->blocks.clear();
    p->geom.clear();
    p->max_block = 0;
    p->anchored_dst_max = 0;
    int32_t pos = 0;
    for (int s = 0; s < S; ++s)
        for (int j = 0; j < nsp; ++j) p->pi[pos++] = s * P + j;
    int32_t moff_q = pos, moff_k = pos;
    for (int g0 = 0; g0 < S; g0 += cfg.blk_frames) {
        const int f = std::min(cfg.blk_frames, S - g0);
        for (int y0 = 0; y0 < h; y0 += cfg.blk_h) {
            const int hh = std::min(cfg.blk_h, h - y0);
            for (int x0 = 0; x0 < w; x0 += cfg.blk_w) {
                const int ww = std::min(cfg.blk_w, w - x0);
                BlockInfo bi{};
                bi.start = pos;
                bi.n = f * hh * ww;
                bi.n_rule = bi.n;
                block_budget(bi.n, cfg.ratio_q, &bi.r_q, &bi.nd_q);
                block_budget(bi.n, cfg.ratio_kv, &bi.r_k, &bi.nd_k);
                if (cfg.anchor_first_frame && g0 == 0) {   // the block's tokens of frame 0 are its dst tokens, all others src
                    const int n0 = hh * ww;
                    bi.n_rule = n0;
                    bi.nd_q = bi.nd_k = n0;
                    bi.r_q = (int32_t)std::min<int64_t>((int64_t)std::floor(cfg.ratio_q * (double)bi.n + 1e-9), bi.n - n0);
                    bi.r_k = (int32_t)std::min<int64_t>((int64_t)std::floor(cfg.ratio_kv * (double)bi.n + 1e-9), bi.n - n0);
                    p->anchored_dst_max = std::max(p->anchored_dst_max, n0);
                }
                bi.moff_q = moff_q;
                bi.moff_k = moff_k;
                moff_q += bi.n - bi.r_q;
                moff_k += bi.n - bi.r_k;
                p->max_block = std::max(p->max_block, bi.n);
                p->blk_start.push_back(pos);
                p->blocks.push_back(bi);
                p->geom.push_back(BlockGeom{(int16_t)g0, (int16_t)y0, (int16_t)x0, (int16_t)f, (int16_t)hh, (int16_t)ww});
                for (int tl = 0; tl < f; ++tl)
                    for (int yl = 0; yl < hh; ++yl)
                        for (int xl = 0; xl < ww; ++xl) p->pi[pos++] = (g0 + tl) * P + nsp + (y0 + yl) * w + (x0 + xl);
            }
        }
    }
    p->blk_start.push_back(pos);
    p->n_blocks = (int32_t)p->blocks.size();
    p->m_q = moff_q;
    p->m_k = moff_k;
    for (int32_t i = 0; i < p->n_tokens; ++i) p->pi_inv[p->pi[i]] = i;
}

// Layout rules of a caller's tensor (bf16, [heads][tokens][64] through two element strides).  Returns HTTM_OK or
// the error code, with the reason in *why.
inline int check_tensor_layout(const httm_tensor& t, int heads, const char* name, std::string* why) {
    auto bad = [&](int code, const char* msg) {
        *why = std::string(name) + ": " + msg;
        return code;
    };
    if (!t.ptr) return bad(HTTM_ERR_INVALID_ARG, "null pointer");
    if (((uintptr_t)t.ptr & 15u) != 0) return bad(HTTM_ERR_ALIGNMENT, "pointer is not 16-byte aligned");
    if (t.stride_head % 8 != 0 || t.stride_token % 8 != 0) return bad(HTTM_ERR_ALIGNMENT, "strides must be multiples of 8 elements");
    if (t.stride_token < kHeadDim || t.stride_head < 0) return bad(HTTM_ERR_INVALID_ARG, "stride_token must be >= head_dim and stride_head >= 0");
    if (heads > 1 && t.stride_head < kHeadDim) return bad(HTTM_ERR_INVALID_ARG, "stride_head must be >= head_dim");
    return HTTM_OK;
}

// The checks of a configuration that do not depend on the device.  Returns HTTM_OK or the error code.
inline int check_config(const httm_config& cfg, std::string* why) {
    auto bad = [&](int code, const char* msg) {
        *why = msg;
        return code;
    };
    if (cfg.frames < 1 || cfg.n_camera < 0 || cfg.n_register < 0 || cfg.grid_h < 1 || cfg.grid_w < 1 || cfg.heads < 1 ||
        cfg.blk_frames < 1 || cfg.blk_h < 1 || cfg.blk_w < 1)
        return bad(HTTM_ERR_INVALID_ARG, "sizes must be positive (special-token counts non-negative)");
    if (!(cfg.ratio_q >= 0.0 && cfg.ratio_q < 1.0) || !(cfg.ratio_kv >= 0.0 && cfg.ratio_kv < 1.0))
        return bad(HTTM_ERR_INVALID_ARG, "merge ratios must lie in [0, 1)");
    if (cfg.anchor_first_frame != 0 && cfg.anchor_first_frame != 1) return bad(HTTM_ERR_INVALID_ARG, "anchor_first_frame must be 0 or 1");
    if (cfg.head_dim != kHeadDim) return bad(HTTM_ERR_UNSUPPORTED, "head_dim must be 64");
    if (cfg.heads > 65535) return bad(HTTM_ERR_UNSUPPORTED, "at most 65535 heads");
    const int64_t per_frame = (int64_t)cfg.n_camera + cfg.n_register + (int64_t)cfg.grid_h * cfg.grid_w;
    const int64_t n_tokens = per_frame * cfg.frames;
    if (n_tokens > (1ll << 24) || n_tokens * cfg.heads > (1ll << 31) - 1)
        return bad(HTTM_ERR_UNSUPPORTED, "too many tokens (N <= 2^24 and N*heads < 2^31)");
    return HTTM_OK;
}

}  // namespace httm
