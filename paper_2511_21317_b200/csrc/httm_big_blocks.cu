// Matching and merging for LARGE merging blocks (257 .. 4096 tokens): the paper's own regime of runs of
// n_s = 128 tokens over n_t = 30 frames, 3840 tokens per block (Sec. 3.3, Sec. 4.1).  A block no longer fits one
// warp's stage, and its similarity step (Eq. 1) is a real dense contraction: n tokens x n_dst dst tokens x 64.
//
//   big_scores_kernel   cosine of every token of a block with every dst token of the block on the 5th-generation
//                       tensor cores (tcgen05.mma, accumulators in tensor memory; the dst tokens enter scaled by
//                       their inverse norms, split exactly into three bf16 planes), fused with the row-wise
//                       arg-max: per token the best dst and the best cosine
//   big_select_kernel   the r src tokens with the best cosines merge (Sec. 3.2): exact radix select per block,
//                       ties by position; writes the assignment map
//   big_merge_kernel    mean of every group (Sec. 3.2): tokens sorted by (merged row, position), one warp
//                       gathers the members of a row in that order; writes merged Q / K / V and rank_q
// All three read the reordered copies (a block is a contiguous run of rows there).
#include "httm_internal.h"
#include "tc_sm100.cuh"

namespace httm {

namespace {

// ------------------------------------------------------------------------------------------------ shared helpers
__device__ __forceinline__ uint32_t score_key(float s) {   // unsigned keys order like the floats
    const uint32_t b = __float_as_uint(s);
    return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}
// token number (inside its block) of dst d of n_dst dst tokens: the positions j < n_rule with
// floor((j + 1) n_dst / n_rule) > floor(j n_dst / n_rule), i.e. j = ceil((d + 1) n_rule / n_dst) - 1.  n_rule is the
// block length (evenly spaced dst tokens) or n_dst (the first n_dst tokens: first-frame anchoring), see BlockInfo.
__device__ __forceinline__ int dst_position(int d, int n_rule, int nd) { return ((d + 1) * n_rule + nd - 1) / nd - 1; }
__device__ __forceinline__ bool is_dst_position(int j, int n_rule, int nd) {
    return j < n_rule && ((j + 1) * nd) / n_rule > (j * nd) / n_rule;
}

// ------------------------------------------------------------------------------------------------ scores
// cos(i, d) |x_i| = sum_k x_ik (w_d x_dk) with w_d = 1 / max(|x_d|, 1e-12).  The dst rows are multiplied by their
// inverse norms when they are gathered, and the fp32 products are split EXACTLY into three bf16 planes (8 + 8 + 8
// significant bits), so that three accumulating MMAs per K step give the scaled scores straight in tensor memory: the
// arg-max warps neither load weights nor multiply (the tensor cores are idle most of the time in this kernel, the
// arg-max warps are what bounds it).  The dst tokens of a block are taken 256 at a time (three planes of 32 KB); the
// token tiles of the slice are streamed once per such chunk, and every token's best so far waits in shared memory.
constexpr int TILE = 128;                        // rows of an operand tile
constexpr int TILE_BYTES = TILE * kRowBytes;     // 16 KB
constexpr int kChunkDst = 256;                   // dst tokens per chunk = columns of a score buffer
constexpr int kPlaneBytes = kChunkDst * kRowBytes;       // 32 KB
constexpr int kSrcTilesPerItem = kBigSliceRows / TILE;   // 32: a work item is a whole block
constexpr int SC_THREADS = 320;                  // warp 0: TMA producer, warp 1: MMA issuer, warps 2-9: arg-max (two column halves x four lane quadrants)
constexpr int SC_TMEM_COLS = 512;                // two score buffers of 256 columns
constexpr int SC_STAGES = 4;                     // ring of token tiles: a tile's load takes longer than its MMAs and its arg-max

struct ScoreBars {
    uint64_t a_full[SC_STAGES], a_empty[SC_STAGES];   // ring of token tiles
    uint64_t s_full[2], s_empty[2];   // score buffers
    uint64_t x_full[2], x_done[2];    // exchange of the two column halves' results, by token-tile parity
    uint32_t tmem_base;
    int abort_flag;
};
constexpr int SC_OFF_A = 3 * kPlaneBytes;                        // token tiles behind the three planes
constexpr int SC_OFF_BEST = SC_OFF_A + SC_STAGES * TILE_BYTES;   // float [2 halves][tokens of the item]: best score so far
constexpr int SC_OFF_ARG = SC_OFF_BEST + 2 * kBigSliceRows * 4;  // uint16 [2][tokens]: its dst (n_dst <= 1024)
constexpr int SC_OFF_XCH = SC_OFF_ARG + 2 * kBigSliceRows * 2;   // [2][128] (best, arg) of column half 1
constexpr int SC_OFF_BARS = SC_OFF_XCH + 2 * TILE * 8;
constexpr int SC_SMEM = SC_OFF_BARS + 256 + 1024 /*alignment slack*/;

__device__ __forceinline__ uint32_t bf16_bits_rn(float f) {
    const __nv_bfloat16 h = __float2bfloat16_rn(f);
    return (uint32_t)*reinterpret_cast<const unsigned short*>(&h);
}

__global__ void __launch_bounds__(SC_THREADS, 1)
big_scores_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, const BigMatchArgs a) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t s_b = tc::smem_addr(smem), s_a = s_b + SC_OFF_A;
    float* best_s = reinterpret_cast<float*>(smem + SC_OFF_BEST);
    uint16_t* arg_s = reinterpret_cast<uint16_t*>(smem + SC_OFF_ARG);
    float2* xch = reinterpret_cast<float2*>(smem + SC_OFF_XCH);
    ScoreBars* bars = reinterpret_cast<ScoreBars*>(smem + SC_OFF_BARS);
    volatile int* abort_flag = &bars->abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        bars->abort_flag = 0;
        for (int i = 0; i < SC_STAGES; ++i) {
            tc::mbar_init(tc::smem_addr(&bars->a_full[i]), 1);
            tc::mbar_init(tc::smem_addr(&bars->a_empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            tc::mbar_init(tc::smem_addr(&bars->s_full[i]), 1);
            tc::mbar_init(tc::smem_addr(&bars->s_empty[i]), 256);
            tc::mbar_init(tc::smem_addr(&bars->x_full[i]), 128);
            tc::mbar_init(tc::smem_addr(&bars->x_done[i]), 128);
        }
        tc::fence_barrier_init();
        tc::prefetch_tensormap(&map_q);
        tc::prefetch_tensormap(&map_k);
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_addr(&bars->tmem_base), SC_TMEM_COLS);
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem = bars->tmem_base;

    // completions so far of every barrier (each role counts its own): they give the phase parities across chunks and items
    uint32_t n_tiles_done = 0;   // token tiles so far: tile k uses ring stage k % SC_STAGES and score buffer k & 1
    uint32_t n_x[2] = {0, 0};    // exchanges per parity slot
    const int64_t total = 2ll * a.heads * a.n_items;
    constexpr uint32_t idesc = tc::idesc_bf16(128, kChunkDst, false, false);
    constexpr uint64_t kTileStep = TILE_BYTES >> 4, kPlaneStep = kPlaneBytes >> 4;   // descriptor address fields count 16-byte units

    for (int64_t item = blockIdx.x;; item += gridDim.x) {
        __syncthreads();
        if (item >= total || bars->abort_flag) break;   // (the flag is only set between two barriers: same answer in every thread)
        const int t = (int)(item / ((int64_t)a.heads * a.n_items));
        const int64_t rem = item - (int64_t)t * a.heads * a.n_items;
        const int h = (int)(rem / a.n_items);
        const BigItem it = a.items[rem - (int64_t)h * a.n_items];
        const BlockInfo bi = a.blocks[it.block];
        const int n = bi.n, r = t == 0 ? bi.r_q : bi.r_k, nd = t == 0 ? bi.nd_q : bi.nd_k;
        if (r == 0) continue;   // nothing merges in this block (uniform)
        const int n_chunks = (nd + kChunkDst - 1) / kChunkDst;
        const int n_st = min(kSrcTilesPerItem, (n - it.row0 + TILE - 1) / TILE);  // token tiles of this slice
        const int64_t head_row0 = (int64_t)h * a.n_tokens + bi.start;             // row of the block's first token in [H][N]

        for (int chunk = 0; chunk < n_chunks; ++chunk) {
            const int d_lo = chunk * kChunkDst, d_cnt = min(kChunkDst, nd - d_lo);   // this chunk's dst tokens
            if (chunk > 0) {
                __syncthreads();   // every role is done with the previous chunk's planes
                if (bars->abort_flag) break;   // (uniform, as above)
            }
            // ---- dst tokens of the chunk, scaled and split, -> three resident planes (128-byte swizzle, as a tiled bulk
            //      copy would leave them)
            {
                const __nv_bfloat16* x = a.xr[t] + head_row0 * kHeadDim;
                const float* inv = a.inv_norm[t] + head_row0;
                const int c16 = tid & 7;
                constexpr int kRowsPerPass = SC_THREADS / 8, kPasses = (kChunkDst + kRowsPerPass - 1) / kRowsPerPass;
                uint4 v[kPasses];   // all of this thread's loads are issued before the first is used
                float w[kPasses];
#pragma unroll
                for (int u = 0; u < kPasses; ++u) {
                    const int dl = (tid >> 3) + u * kRowsPerPass;
                    v[u] = make_uint4(0u, 0u, 0u, 0u);
                    w[u] = 0.f;
                    if (dl < d_cnt) {
                        const int pos = dst_position(d_lo + dl, bi.n_rule, nd);
                        v[u] = __ldg(reinterpret_cast<const uint4*>(x + (int64_t)pos * kHeadDim) + c16);
                        w[u] = __ldg(inv + pos);
                    }
                }
#pragma unroll
                for (int u = 0; u < kPasses; ++u) {
                    const int dl = (tid >> 3) + u * kRowsPerPass;
                    if (dl >= kChunkDst) continue;
                    // rows past the last dst token come out as zeros (x = 0, w = 0); their columns are masked below
                    const uint32_t in[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                    uint32_t o0[4], o1[4], o2[4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint32_t b0[2], b1[2], b2[2];
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const float xv = __uint_as_float(e == 0 ? in[q] << 16 : in[q] & 0xffff0000u);
                            const float p = xv * w[u];                                // one rounding to fp32 (24 bits)
                            b0[e] = bf16_bits_rn(p);
                            const float r1 = p - __uint_as_float(b0[e] << 16);        // exact
                            b1[e] = bf16_bits_rn(r1);
                            const float r2 = r1 - __uint_as_float(b1[e] << 16);       // exact, at most 8 significant bits
                            b2[e] = bf16_bits_rn(r2);
                        }
                        o0[q] = b0[0] | (b0[1] << 16);
                        o1[q] = b1[0] | (b1[1] << 16);
                        o2[q] = b2[0] | (b2[1] << 16);
                    }
                    unsigned char* dst = smem + dl * kRowBytes + ((c16 ^ (dl & 7)) << 4);
                    *reinterpret_cast<uint4*>(dst) = make_uint4(o0[0], o0[1], o0[2], o0[3]);
                    *reinterpret_cast<uint4*>(dst + kPlaneBytes) = make_uint4(o1[0], o1[1], o1[2], o1[3]);
                    *reinterpret_cast<uint4*>(dst + 2 * kPlaneBytes) = make_uint4(o2[0], o2[1], o2[2], o2[3]);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor cores read the planes through the async proxy
            }
            __syncthreads();

            if (warp == 0) {
                // -------------------------------------------------------------- producer: the token tiles of the slice, once per chunk
                if (tc::elect_one()) {
                    for (int i = 0; i < n_st; ++i) {
                        const uint32_t k = n_tiles_done + i, st = k % SC_STAGES, ph = (k / SC_STAGES) & 1u;
                        if (!tc::mbar_wait(tc::smem_addr(&bars->a_empty[st]), ph ^ 1u, abort_flag)) break;
                        const uint32_t bar = tc::smem_addr(&bars->a_full[st]);
                        tc::mbar_expect_tx(bar, TILE_BYTES);
                        // rows past the block's end belong to the next block (finite, results dropped) or are zero filled past N
                        tc::tma_load_3d(s_a + st * TILE_BYTES, t == 0 ? &map_q : &map_k, bar, 0, bi.start + it.row0 + i * TILE, h);
                    }
                }
                __syncwarp();
            } else if (warp == 1) {
                // -------------------------------------------------------------- issuer: S = X_tile . (hi + mid + lo)^T
                if (tc::elect_one()) {
                    const uint64_t da0 = tc::smem_desc_sw128(s_a), db0 = tc::smem_desc_sw128(s_b);
                    bool ok = true;
                    for (int i = 0; ok && i < n_st; ++i) {
                        const uint32_t k = n_tiles_done + i, st = k % SC_STAGES, b = k & 1u;
                        ok = tc::mbar_wait(tc::smem_addr(&bars->a_full[st]), (k / SC_STAGES) & 1u, abort_flag) &&
                             tc::mbar_wait(tc::smem_addr(&bars->s_empty[b]), ((k >> 1) & 1u) ^ 1u, abort_flag);
                        if (!ok) break;
                        tc::fence_after_sync();
                        const uint64_t da = da0 + (uint64_t)st * kTileStep;
#pragma unroll
                        for (int pl = 0; pl < 3; ++pl)
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks)   // K = 16 steps over the 64 channels: 32 bytes = 2 descriptor units
                                tc::mma_ss(tmem + b * kChunkDst, da + 2 * ks, db0 + (uint64_t)pl * kPlaneStep + 2 * ks, idesc, (pl | ks) ? 1u : 0u);
                        tc::mma_commit(tc::smem_addr(&bars->a_empty[st]));   // the tile may be refilled when these MMAs are done
                        tc::mma_commit(tc::smem_addr(&bars->s_full[b]));
                    }
                }
                __syncwarp();
            } else {
                // -------------------------------------------------------------- arg-max over the chunk's dst tokens, one thread per
                // token and column half; the scores arrive scaled
                const int half = (warp - 2) >> 2;
                const int row = (warp & 3) * 32 + lane;            // row of the token tile = lane of tensor memory
                const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
                const bool last_chunk = chunk == n_chunks - 1;
                bool ok = true;
                for (int i = 0; ok && i < n_st; ++i) {
                    const uint32_t k = n_tiles_done + i, b = k & 1u;
                    const int mine = half * kBigSliceRows + i * TILE + row;
                    float best = -INFINITY;
                    int arg = 0;
                    if (chunk > 0) {
                        best = best_s[mine];
                        arg = arg_s[mine];
                    }
                    ok = tc::mbar_wait(tc::smem_addr(&bars->s_full[b]), (k >> 1) & 1u, abort_flag);
                    if (!ok) break;
                    tc::fence_after_sync();
#pragma unroll
                    for (int part = 0; part < 2; ++part) {
                        uint32_t raw[64];
                        const uint32_t taddr = tmem + b * kChunkDst + half * TILE + part * 64 + lane_addr;
                        tc::tmem_ld32(taddr, raw);
                        tc::tmem_ld32(taddr + 32, raw + 32);
                        tc::tmem_wait_ld();
                        if (part == 1) {   // both parts are in registers: the buffer can take the next scores
                            tc::fence_before_sync();
                            tc::mbar_arrive(tc::smem_addr(&bars->s_empty[b]));
                        }
                        const int c0 = half * TILE + part * 64;   // first column of these 64 inside the chunk
                        if (c0 < d_cnt) {                         // (uniform in the warp)
                            if (c0 + 64 > d_cnt) {                // the block's last dst tokens: mask the columns behind them
#pragma unroll
                                for (int c = 0; c < 64; ++c)
                                    if (c0 + c >= d_cnt) raw[c] = 0xff800000u;   // -inf
                            }
                            // maxima of the four groups of 16 columns (independent chains), then of the part
                            float g0 = -INFINITY, g1 = -INFINITY, g2 = -INFINITY, g3 = -INFINITY;
#pragma unroll
                            for (int c = 0; c < 16; c += 2) {
                                g0 = tc::fmax3(g0, __uint_as_float(raw[c]), __uint_as_float(raw[c + 1]));
                                g1 = tc::fmax3(g1, __uint_as_float(raw[16 + c]), __uint_as_float(raw[17 + c]));
                                g2 = tc::fmax3(g2, __uint_as_float(raw[32 + c]), __uint_as_float(raw[33 + c]));
                                g3 = tc::fmax3(g3, __uint_as_float(raw[48 + c]), __uint_as_float(raw[49 + c]));
                            }
                            const float m = fmaxf(tc::fmax3(g0, g1, g2), g3);
                            if (m > best) {   // find the first column holding the maximum (ties: lowest dst): first group, then
                                best = m;     // the first of its 16 columns (the search runs whenever any row of the warp improves)
                                const bool in0 = g0 == m, in1 = g1 == m, in2 = g2 == m;
                                const int group = in0 ? 0 : (in1 ? 1 : (in2 ? 2 : 3));
                                int first = 15;
#pragma unroll
                                for (int c = 14; c >= 0; --c) {
                                    const uint32_t v = in0 ? raw[c] : (in1 ? raw[16 + c] : (in2 ? raw[32 + c] : raw[48 + c]));
                                    if (__uint_as_float(v) == m) first = c;
                                }
                                arg = d_lo + c0 + 16 * group + first;
                            }
                        }
                    }
                    if (!last_chunk) {
                        best_s[mine] = best;
                        arg_s[mine] = (uint16_t)arg;
                        continue;
                    }
                    // the two column halves of a token meet: half 1 hands (best, arg) over, half 0 decides (ties: lowest dst)
                    const int slot = i & 1;
                    if (half == 1) {
                        ok = tc::mbar_wait(tc::smem_addr(&bars->x_done[slot]), (n_x[slot] & 1u) ^ 1u, abort_flag);
                        if (!ok) break;
                        xch[slot * TILE + row] = make_float2(best, __int_as_float(arg));
                        tc::mbar_arrive(tc::smem_addr(&bars->x_full[slot]));
                    } else {
                        ok = tc::mbar_wait(tc::smem_addr(&bars->x_full[slot]), n_x[slot] & 1u, abort_flag);
                        if (!ok) break;
                        const float2 o = xch[slot * TILE + row];
                        tc::mbar_arrive(tc::smem_addr(&bars->x_done[slot]));
                        const int oarg = __float_as_int(o.y);
                        if (o.x > best || (o.x == best && oarg < arg)) {
                            best = o.x;
                            arg = oarg;
                        }
                        const int p = it.row0 + i * TILE + row;   // token number inside the block
                        if (p < n) {
                            const float w = __ldg(a.inv_norm[t] + head_row0 + p);
                            a.best_key[t][head_row0 + p] = score_key(best * w);
                            a.best_pos[t][head_row0 + p] = dst_position(arg, bi.n_rule, nd);
                        }
                    }
                    ++n_x[slot];
                }
            }
            n_tiles_done += n_st;   // (every thread keeps the count, whatever its role)
        }
    }
    tc::fence_before_sync();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem, SC_TMEM_COLS);
    if (tid == 0 && bars->abort_flag) atomicCAS(a.status, kDevOk, kDevTimeoutBigMatch);
}

// ------------------------------------------------------------------------------------------------ selection
// One CTA per (tensor, head, block); thread i owns tokens 4 i .. 4 i + 3 of the block, so that counts taken in
// thread order are counts in position order.
constexpr int SEL_THREADS = 1024;

// one warp: walking down from the largest of 256 bins, the bin in which the running count reaches `want`
// (1 <= want <= total); *bin_out = that bin, *want_out = want minus the count of all higher bins
__device__ __forceinline__ void pick_bin(const int* h, int want, int* bin_out, int* want_out) {
    const int lane = threadIdx.x & 31, lo = lane * 8;
    int c = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) c += h[lo + i];
    int incl = c;   // this lane's bins and all higher ones
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_down_sync(0xffffffffu, incl, off);
        if (lane + off < 32) incl += o;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, incl >= want);
    if (hit == 0) {   // cannot happen for want <= total; keep the result defined
        if (lane == 0) {
            *bin_out = 0;
            *want_out = 1;
        }
        return;
    }
    if (lane == 31 - __clz(hit)) {
        int above = incl - c, b = lo + 7;
        for (; b > lo; --b) {
            if (above + h[b] >= want) break;
            above += h[b];
        }
        *bin_out = b;
        *want_out = want - above;
    }
}

__global__ void __launch_bounds__(SEL_THREADS, 1) big_select_kernel(const BigMatchArgs a) {
    __shared__ int hist[256];
    __shared__ int warp_sum[32];
    __shared__ int s_bin, s_want;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int per_tensor = a.heads * a.n_blocks;
    const int t = blockIdx.x / per_tensor, h = (blockIdx.x % per_tensor) / a.n_blocks, b = blockIdx.x % a.n_blocks;
    const BlockInfo bi = a.blocks[b];
    const int n = bi.n, r = t == 0 ? bi.r_q : bi.r_k, nd = t == 0 ? bi.nd_q : bi.nd_k;
    const int64_t base = (int64_t)h * a.n_tokens + bi.start;
    int32_t* A = a.assign[t] + base;
    if (r == 0) {   // nothing merges: identity
        for (int j = tid; j < n; j += SEL_THREADS) A[j] = bi.start + j;
        return;
    }
    uint32_t key[4];
    bool src[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int j = 4 * tid + e;
        src[e] = j < n && !is_dst_position(j, bi.n_rule, nd);
        key[e] = src[e] ? a.best_key[t][base + j] : 0u;
    }
    const int n_src = n - nd;
    bool merged[4] = {src[0], src[1], src[2], src[3]};
    if (r < n_src) {
        // T = the r-th largest key: radix select, 8 bits a pass
        uint32_t prefix = 0, mask = 0;
        int want = r;
        for (int shift = 24; shift >= 0; shift -= 8) {
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool in = src[e] && (key[e] & mask) == prefix;
                const int bin = in ? (int)((key[e] >> shift) & 255u) : -1;
                const unsigned peers = __match_any_sync(0xffffffffu, bin);   // one atomic per distinct bin of the warp
                if (in && lane == __ffs(peers) - 1) atomicAdd(&hist[bin], __popc(peers));
            }
            __syncthreads();
            if (warp == 0) pick_bin(hist, want, &s_bin, &s_want);
            __syncthreads();
            prefix |= (uint32_t)s_bin << shift;
            mask |= 255u << shift;
            want = s_want;
            __syncthreads();   // s_bin, s_want and hist are rewritten in the next pass
        }
        // keys above T merge; of the keys equal to T the first `want` in position order (Sec. 3.2 ties: lowest position)
        int eq = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) eq += (src[e] && key[e] == prefix) ? 1 : 0;
        int incl = eq;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += o;
        }
        if (lane == 31) warp_sum[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int w = warp_sum[lane];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, w, off);
                if (lane >= off) w += o;
            }
            warp_sum[lane] = w;
        }
        __syncthreads();
        int before = (warp > 0 ? warp_sum[warp - 1] : 0) + incl - eq;   // equal keys at lower positions
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (src[e] && key[e] == prefix) {
                merged[e] = before < want;
                ++before;
            } else {
                merged[e] = src[e] && key[e] > prefix;
            }
        }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int j = 4 * tid + e;
        if (j < n) {
            int target = j;
            if (merged[e]) {
                target = a.best_pos[t][base + j];
                if (target < 0 || target >= n) {   // cannot happen after the score kernel; never write a bad index
                    atomicCAS(a.status, kDevOk, kDevBadIndex);
                    target = j;
                }
            }
            A[j] = bi.start + target;
        }
    }
}

// ------------------------------------------------------------------------------------------------ merging
// One CTA per (map in {Q, K}, head, block) - the K map also merges V - plus CTAs that copy the special tokens.
// The sorted-group kernels are templated on T, the threads of a CTA; a CTA holds one block of up to 4 T tokens (thread i
// owns tokens 4 i .. 4 i + 3).  T is chosen from the largest block of the context: 1024 for blocks of 4096 tokens, 64 for
// blocks of up to 256, so that small blocks get many small CTAs per SM.
__host__ __device__ constexpr int mg_smem_bytes(int T) { return 4 * T * 4 /*keys*/ + 4 * T * 2 /*row of kept token*/ + (4 * T + 4) * 4 /*segments*/ + 256; }
__host__ __device__ constexpr int of_smem_bytes(int T) { return mg_smem_bytes(T) + 4 * T * 2 /*position of every row's kept token*/ + 4 * T /*outlier flags*/ + 4 * T * 2 /*new representative of every row*/; }

__device__ __forceinline__ void unpack8f(const uint4& raw, float* f) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        f[2 * i] = __uint_as_float(w[i] << 16);
        f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// The groups of one block from its map A (every thread of the T-thread CTA calls this): merged row of every kept token =
// its rank among the kept tokens in position order (row_of; -1 for merged tokens); all tokens sorted by (merged row,
// position) in keys[] = (row << 12) | position, so that the members of a row are one ascending run; seg[row] = first
// sorted index of the row, seg[n_kept] = n.  rep_of_row (optional) gets the position of every row's kept token; rank_out
// (optional) the merged row of every token plus moff.  Returns the number of kept tokens, at most `limit` (tokens whose
// row would lie beyond it, or whose target is not a kept token, are recorded as a corrupt map and left out).
template <int T>
__device__ int build_groups(const int32_t* A, int block_start, int n, int limit, uint32_t* keys, int16_t* row_of, int* seg, int* warp_sum,
                            int16_t* rep_of_row, int32_t* status, int32_t* rank_out, int moff) {
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    int rep[4];
    int kept = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int j = 4 * tid + e;
        rep[e] = -1;
        if (j < n) {
            rep[e] = A[j] - block_start;
            if (rep[e] < 0 || rep[e] >= n) {   // corrupt map: record, treat as kept
                atomicCAS(status, kDevOk, kDevBadIndex);
                rep[e] = j;
            }
            kept += rep[e] == j ? 1 : 0;
        }
    }
    int incl = kept;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += o;
    }
    __syncthreads();   // (the scratch arrays may still be in use by a previous call's readers)
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = lane < T / 32 ? warp_sum[lane] : 0;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, w, off);
            if (lane >= off) w += o;
        }
        if (lane < T / 32) warp_sum[lane] = w;
    }
    __syncthreads();
    const int n_kept = min(warp_sum[T / 32 - 1], limit);
    int next_row = (warp > 0 ? warp_sum[warp - 1] : 0) + incl - kept;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int j = 4 * tid + e;
        if (j < n) {
            const bool is_kept = rep[e] == j;
            row_of[j] = is_kept ? (int16_t)next_row : (int16_t)-1;
            if (is_kept) {
                if (rep_of_row && next_row < n_kept) rep_of_row[next_row] = (int16_t)j;
                ++next_row;
            }
        }
    }
    __syncthreads();
    int P = 32;
    while (P < n) P <<= 1;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int j = 4 * tid + e;
        uint32_t key = 0xffffffffu;
        if (j < n) {
            int row = row_of[rep[e]];
            if (row < 0 || row >= n_kept) {   // target is not a kept token, or more kept tokens than a valid map has
                atomicCAS(status, kDevOk, kDevBadIndex);
                row = 0xfffff;                // sorts behind every valid row, is never gathered
            } else if (rank_out) {
                rank_out[j] = moff + row;
            }
            key = ((uint32_t)row << 12) | (uint32_t)j;
        }
        if (j < P) keys[j] = key;
    }
    __syncthreads();
    for (int k = 2; k <= P; k <<= 1) {   // bitonic sort: the keys are distinct, so the order is unique
        for (int jj = k >> 1; jj > 0; jj >>= 1) {
            for (int c = tid; c < (P >> 1); c += T) {   // comparator c of this stage: elements i and i + jj (bit jj of i clear)
                const int i = ((c & ~(jj - 1)) << 1) | (c & (jj - 1));
                const uint32_t x = keys[i], y = keys[i + jj];
                if ((x > y) == ((i & k) == 0)) {
                    keys[i] = y;
                    keys[i + jj] = x;
                }
            }
            __syncthreads();
        }
    }
    for (int i = tid; i <= n; i += T) {
        const int row = i < n ? (int)(keys[i] >> 12) : n_kept;
        const int prev = i > 0 ? (int)(keys[i - 1] >> 12) : -1;
        if (row != prev && prev < n_kept)   // every row from prev + 1 to row starts here (rows without members cannot occur in a valid map)
            for (int q = prev + 1; q <= min(row, n_kept); ++q) seg[q] = i;
    }
    __syncthreads();
    return n_kept;
}

template <int T>
__global__ void __launch_bounds__(T, 1) big_merge_kernel(const MergeArgs a, int sp_chunks) {
    extern __shared__ __align__(16) unsigned char mg_smem[];
    uint32_t* keys = reinterpret_cast<uint32_t*>(mg_smem);                                     // [P] (merged row << 12) | position
    int16_t* row_of = reinterpret_cast<int16_t*>(mg_smem + (4 * T) * 4);            // [n] merged row of a kept token, -1
    int* seg = reinterpret_cast<int*>(mg_smem + (4 * T) * 6);                       // [n_kept + 1] first sorted index of every merged row
    int* warp_sum = seg + (4 * T) + 4;                                              // [32]
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_block_ctas = 2 * a.heads * a.n_blocks;
    const int ch = lane & 7, sub = lane >> 3;   // 16-byte chunk of a row; which of four rows in flight

    if ((int)blockIdx.x >= n_block_ctas) {
        // special tokens: never merged, first in the merged order; T / 8 rows of one head per CTA, all three tensors
        const int idx = blockIdx.x - n_block_ctas, h = idx / sp_chunks, row = (idx % sp_chunks) * (T / 8) + (tid >> 3);
        if (row < a.n_special_total) {
            for (int t = 0; t < 3; ++t) {
                const int m_len = t == 0 ? a.m_q : a.m_k;
                const uint4 v = __ldg(reinterpret_cast<const uint4*>(a.xr[t] + ((int64_t)h * a.n_tokens + row) * kHeadDim) + (tid & 7));
                reinterpret_cast<uint4*>(a.merged[t] + ((int64_t)h * m_len + row) * kHeadDim)[tid & 7] = v;
            }
        }
        return;
    }
    const int per_map = a.heads * a.n_blocks;
    const int m = blockIdx.x / per_map, h = (blockIdx.x % per_map) / a.n_blocks, b = blockIdx.x % a.n_blocks;
    const BlockInfo bi = a.blocks[b];
    const int n = bi.n, r = m == 0 ? bi.r_q : bi.r_k, m_len = m == 0 ? a.m_q : a.m_k;
    const bool variable = m == 0 && a.moff_q_var != nullptr;   // after outlier filtering the kept count of a block varies by head
    const int moff = m == 0 ? (variable ? __ldg(a.moff_q_var + (int64_t)h * a.n_blocks + b) : bi.moff_q) : bi.moff_k;
    const int limit = variable ? n : n - r;                    // most kept tokens a valid map can have
    const int64_t base = (int64_t)h * a.n_tokens + bi.start;
    const int32_t* A = a.assign[m] + base;

    const int n_kept = build_groups<T>(A, bi.start, n, limit, keys, row_of, seg, warp_sum, nullptr, a.status, m == 0 ? a.rank_q + base : nullptr, moff);
    // eight lanes per merged row (a lane owns one 16-byte chunk of the row), four rows per warp at a time, four
    // members of a row in flight: the gather is bound by load latency, so it needs many loads in the air.  Member
    // i of a row goes to accumulator i mod 4; the four are added in a fixed order: the result does not depend on
    // scheduling.
    for (int t = (m == 0 ? 0 : 1); t <= (m == 0 ? 0 : 2); ++t) {
        const __nv_bfloat16* x = a.xr[t] + base * kHeadDim;
        __nv_bfloat16* out = a.merged[t] + ((int64_t)h * m_len + moff) * kHeadDim;
        for (int row = warp * 4 + sub; row < n_kept; row += (T / 32) * 4) {
            const int i0 = seg[row], i1 = seg[row + 1];
            float acc[4][8];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[u][e] = 0.f;
            for (int i = i0; i < i1; i += 4) {
                uint4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    v[u] = make_uint4(0u, 0u, 0u, 0u);
                    if (i + u < i1) v[u] = __ldg(reinterpret_cast<const uint4*>(x + (int64_t)(keys[i + u] & 4095u) * kHeadDim) + ch);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float f[8];
                    unpack8f(v[u], f);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[u][e] += f[e];
                }
            }
            if (i1 > i0) {
                const float inv = 1.0f / (float)(i1 - i0);
                float r8[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) r8[e] = ((acc[0][e] + acc[1][e]) + (acc[2][e] + acc[3][e])) * inv;
                uint4 o;
                o.x = pack2(r8[0], r8[1]);
                o.y = pack2(r8[2], r8[3]);
                o.z = pack2(r8[4], r8[5]);
                o.w = pack2(r8[6], r8[7]);
                reinterpret_cast<uint4*>(out + (int64_t)row * kHeadDim)[ch] = o;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------ outlier filtering
// Query outlier filtering (Sec. 3.4, Algorithm 2) for large blocks: the same steps as for small blocks - deviation of
// every query token from the mean of its group, one threshold over all heads (the refinement kernels of the small-block
// path, which work on the array of deviations), outliers leave their groups - on the sorted group structure of the merge
// kernel.  One CTA per (head, block).

// eps[h][p] = || q_p - mean of the group p was merged into ||_2 in fp32; 0 for a token on its own
template <int T>
__global__ void __launch_bounds__(T, 1) big_deviation_kernel(const OutlierArgs a) {
    extern __shared__ __align__(16) unsigned char mg_smem[];
    uint32_t* keys = reinterpret_cast<uint32_t*>(mg_smem);
    int16_t* row_of = reinterpret_cast<int16_t*>(mg_smem + (4 * T) * 4);
    int* seg = reinterpret_cast<int*>(mg_smem + (4 * T) * 6);
    int* warp_sum = seg + (4 * T) + 4;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int ch = lane & 7, sub = lane >> 3;
    const int h = blockIdx.x / a.n_blocks, b = blockIdx.x % a.n_blocks;
    const BlockInfo bi = a.blocks[b];
    const int n = bi.n;
    const int64_t base = (int64_t)h * a.n_tokens + bi.start;
    float* eps = a.eps + base;
    if (bi.r_q == 0) {   // nothing merged in this block (uniform)
        for (int j = tid; j < n; j += T) eps[j] = 0.f;
        return;
    }
    const int n_kept = build_groups<T>(a.assign_q + base, bi.start, n, n, keys, row_of, seg, warp_sum, nullptr, a.status, nullptr, 0);
    const __nv_bfloat16* x = a.src_q.ptr + (int64_t)h * a.src_q.stride_head + (int64_t)bi.start * a.src_q.stride_token;
    const int64_t st = a.src_q.stride_token;
    // eight lanes per group (a lane owns 8 of the 64 channels), four groups per warp at a time
    for (int row = warp * 4 + sub; row < ((n_kept + 3) & ~3); row += (T / 32) * 4) {   // (whole sub-groups stay together for the shuffles)
        const bool live = row < n_kept;
        const int i0 = live ? seg[row] : 0, i1 = live ? seg[row + 1] : 0;
        const int cnt = i1 - i0;
        float mean[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) mean[e] = 0.f;
        if (cnt >= 2) {
            float acc[4][8];
#pragma unroll
            for (int u = 0; u < 4; ++u)
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[u][e] = 0.f;
            for (int i = i0; i < i1; i += 4) {
                uint4 v[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    v[u] = make_uint4(0u, 0u, 0u, 0u);
                    if (i + u < i1) v[u] = __ldg(reinterpret_cast<const uint4*>(x + (int64_t)(keys[i + u] & 4095u) * st) + ch);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float f[8];
                    unpack8f(v[u], f);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[u][e] += f[e];
                }
            }
            const float inv = 1.0f / (float)cnt;
#pragma unroll
            for (int e = 0; e < 8; ++e) mean[e] = ((acc[0][e] + acc[1][e]) + (acc[2][e] + acc[3][e])) * inv;   // kept in fp32
        }
        // (the eight lanes of a group walk its members together: the trip count is the same in all of them); four members
        // at a time, so that four loads are in flight
        const unsigned group_mask = 0xffu << (8 * sub);
        for (int i = i0; i < i1; i += 4) {
            uint4 v[4];
            int pos[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                pos[u] = i + u < i1 ? (int)(keys[i + u] & 4095u) : -1;
                v[u] = make_uint4(0u, 0u, 0u, 0u);
                if (cnt >= 2 && pos[u] >= 0) v[u] = __ldg(reinterpret_cast<const uint4*>(x + (int64_t)pos[u] * st) + ch);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float f[8];
                unpack8f(v[u], f);
                float d2 = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float d = f[e] - mean[e];
                    d2 = fmaf(d, d, d2);
                }
                d2 += __shfl_xor_sync(group_mask, d2, 1);
                d2 += __shfl_xor_sync(group_mask, d2, 2);
                d2 += __shfl_xor_sync(group_mask, d2, 4);
                if (ch == 0 && pos[u] >= 0) eps[pos[u]] = cnt >= 2 ? sqrtf(d2) : 0.f;
            }
        }
    }
}

// Outliers (eps > tau) leave their groups: an outlier maps to itself; the other tokens of a group stay together, under
// their old representative if it is not an outlier, else under the remaining member with the lowest position.
template <int T>
__global__ void __launch_bounds__(T, 1) big_filter_kernel(const OutlierArgs a) {
    extern __shared__ __align__(16) unsigned char mg_smem[];
    uint32_t* keys = reinterpret_cast<uint32_t*>(mg_smem);
    int16_t* row_of = reinterpret_cast<int16_t*>(mg_smem + (4 * T) * 4);
    int* seg = reinterpret_cast<int*>(mg_smem + (4 * T) * 6);
    int* warp_sum = seg + (4 * T) + 4;
    int16_t* rep_of_row = reinterpret_cast<int16_t*>(mg_smem + mg_smem_bytes(T));
    unsigned char* outl = mg_smem + mg_smem_bytes(T) + (4 * T) * 2;
    int16_t* new_rep = reinterpret_cast<int16_t*>(mg_smem + mg_smem_bytes(T) + (4 * T) * 3);
    __shared__ int s_kept, s_out;
    const int tid = threadIdx.x;
    const int h = blockIdx.x / a.n_blocks, b = blockIdx.x % a.n_blocks;
    const BlockInfo bi = a.blocks[b];
    const int n = bi.n;
    const int64_t base = (int64_t)h * a.n_tokens + bi.start;
    const int32_t* A = a.assign_q + base;
    int32_t* A_out = a.assign_q_out + base;
    if (bi.r_q == 0) {   // nothing merged, every deviation is 0: nothing to filter unless everything is an outlier, which changes nothing here
        for (int j = tid; j < n; j += T) A_out[j] = bi.start + j;
        if (tid == 0) a.kept_cnt[(int64_t)h * a.n_blocks + b] = n;
        return;
    }
    if (tid == 0) {
        s_kept = 0;
        s_out = 0;
    }
    const float tau = *a.tau;
    const int n_kept = build_groups<T>(A, bi.start, n, n, keys, row_of, seg, warp_sum, rep_of_row, a.status, nullptr, 0);
    int n_out = 0;
    for (int j = tid; j < n; j += T) {
        const bool o = a.eps[base + j] > tau;
        outl[j] = o ? 1 : 0;
        n_out += o ? 1 : 0;
    }
    __syncthreads();
    for (int row = tid; row < n_kept; row += T) {   // a thread per group: groups are short, the rare long one costs its thread a scan
        const int rp = rep_of_row[row];
        int nr = rp;
        if (outl[rp]) {
            nr = -1;
            for (int i = seg[row]; i < seg[row + 1]; ++i) {
                const int pos = (int)(keys[i] & 4095u);
                if (!outl[pos]) {
                    nr = pos;
                    break;
                }
            }
        }
        new_rep[row] = (int16_t)nr;
    }
    __syncthreads();
    int kept = 0;
    for (int j = tid; j < n; j += T) {
        int target = j;
        if (!outl[j]) {
            int rp = A[j] - bi.start;
            if (rp < 0 || rp >= n) rp = j;                  // (recorded by build_groups)
            const int row = row_of[rp];
            if (row >= 0 && row < n_kept) target = new_rep[row];   // never -1 here: j itself is a remaining member
            if (target < 0) target = j;
        }
        A_out[j] = bi.start + target;
        kept += target == j ? 1 : 0;
    }
    atomicAdd(&s_kept, kept);
    atomicAdd(&s_out, n_out);
    __syncthreads();
    if (tid == 0) {
        a.kept_cnt[(int64_t)h * a.n_blocks + b] = s_kept;
        if (s_out) atomicAdd(a.sel + kSelOutliers, s_out);
    }
}

}  // namespace

// threads per CTA for blocks of up to max_block tokens
template <typename F>
cudaError_t with_cta_size(int max_block, F&& f) {
    if (max_block <= 256) return f(std::integral_constant<int, 64>{});
    if (max_block <= 512) return f(std::integral_constant<int, 128>{});
    if (max_block <= 1024) return f(std::integral_constant<int, 256>{});
    if (max_block <= 2048) return f(std::integral_constant<int, 512>{});
    return f(std::integral_constant<int, 1024>{});
}

cudaError_t launch_big_deviation(const OutlierArgs& a, int max_block, cudaStream_t stream) {
    return with_cta_size(max_block, [&](auto t) {
        constexpr int T = decltype(t)::value;
        big_deviation_kernel<T><<<a.heads * a.n_blocks, T, mg_smem_bytes(T), stream>>>(a);
        return cudaGetLastError();
    });
}

cudaError_t launch_big_filter(const OutlierArgs& a, int max_block, cudaStream_t stream) {
    return with_cta_size(max_block, [&](auto t) {
        constexpr int T = decltype(t)::value;
        big_filter_kernel<T><<<a.heads * a.n_blocks, T, of_smem_bytes(T), stream>>>(a);
        return cudaGetLastError();
    });
}

template <int T>
cudaError_t configure_sorted_group_kernels() {
    cudaError_t e = cudaFuncSetAttribute(big_merge_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, mg_smem_bytes(T));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(big_deviation_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, mg_smem_bytes(T));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(big_filter_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, of_smem_bytes(T));
}

cudaError_t configure_big_blocks() {
    cudaError_t e = cudaFuncSetAttribute(big_scores_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SC_SMEM);
    if (e == cudaSuccess) e = configure_sorted_group_kernels<64>();
    if (e == cudaSuccess) e = configure_sorted_group_kernels<128>();
    if (e == cudaSuccess) e = configure_sorted_group_kernels<256>();
    if (e == cudaSuccess) e = configure_sorted_group_kernels<512>();
    if (e == cudaSuccess) e = configure_sorted_group_kernels<1024>();
    return e;
}

cudaError_t launch_big_scores(const BigMatchArgs& a, int sm_count, cudaStream_t stream) {
    CUtensorMap mq, mk;
    if (!encode_rows_tensor_map(&mq, a.xr[0], a.n_tokens, a.heads, kHeadDim, (int64_t)a.n_tokens * kHeadDim, TILE) ||
        !encode_rows_tensor_map(&mk, a.xr[1], a.n_tokens, a.heads, kHeadDim, (int64_t)a.n_tokens * kHeadDim, TILE))
        return cudaErrorInvalidValue;
    const int64_t total = 2ll * a.heads * a.n_items;
    int ctas = sm_count < 1 ? 1 : sm_count;
    if (ctas > total) ctas = (int)total;
    if (ctas < 1) ctas = 1;
    big_scores_kernel<<<ctas, SC_THREADS, SC_SMEM, stream>>>(mq, mk, a);
    return cudaGetLastError();
}

cudaError_t launch_big_select(const BigMatchArgs& a, cudaStream_t stream) {
    big_select_kernel<<<2 * a.heads * a.n_blocks, SEL_THREADS, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_big_merge(const MergeArgs& a, int max_block, cudaStream_t stream) {
    return with_cta_size(max_block, [&](auto t) {
        constexpr int T = decltype(t)::value;
        const int sp_chunks = (a.n_special_total + T / 8 - 1) / (T / 8);
        big_merge_kernel<T><<<2 * a.heads * a.n_blocks + a.heads * sp_chunks, T, mg_smem_bytes(T), stream>>>(a, sp_chunks);
        return cudaGetLastError();
    });
}

}  // namespace httm
