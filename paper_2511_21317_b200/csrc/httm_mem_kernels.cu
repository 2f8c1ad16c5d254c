// HBM-bound kernels of the HTTM path: temporal reorder (gather), per-(head, block)
// cosine matching, mean merge, and unmerge + inverse reorder.  sm_100a only.
#include "httm_internal.h"
#include "tc_sm100.cuh"   // mbarrier / TMA wrappers (device), tensor-map encoders (host)

namespace httm {

// ------------------------------------------------------------------------------------
// small device helpers (mbarrier and address wrappers: tc_sm100.cuh)
// ------------------------------------------------------------------------------------
using tc::mbar_expect_tx;
using tc::mbar_init;
using tc::mbar_try_wait;
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return tc::smem_addr(p); }
// Bounded wait of the warp-per-block kernels: gives up after about two seconds, records `code` in the
// status word and returns false.  Never spins forever.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t mbar, uint32_t parity, int32_t* status, int code) {
    if (mbar_try_wait(mbar, parity)) return true;
    const uint64_t t0 = tc::timer_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(mbar, parity)) return true;
        if (tc::timer_ns() - t0 > 2000000000ull) {
            atomicCAS(status, kDevOk, code);
            return false;
        }
    }
}
__device__ __forceinline__ void unpack8(const uint4& raw, float* f) {
    f[0] = __uint_as_float(raw.x << 16);
    f[1] = __uint_as_float(raw.x & 0xffff0000u);
    f[2] = __uint_as_float(raw.y << 16);
    f[3] = __uint_as_float(raw.y & 0xffff0000u);
    f[4] = __uint_as_float(raw.z << 16);
    f[5] = __uint_as_float(raw.z & 0xffff0000u);
    f[6] = __uint_as_float(raw.w << 16);
    f[7] = __uint_as_float(raw.w & 0xffff0000u);
}

// ------------------------------------------------------------------------------------
// a1. Temporal reorder (Sec. 3.3; Algorithm 1 "Reorder"): xr[h][p'] = x[h][pi[p']]
//     One 16-byte chunk per thread, 8 threads per token row, 4 rows in flight per thread.
// ------------------------------------------------------------------------------------
constexpr int kReorderThreads = 256;
constexpr int kReorderUnroll = 4;
constexpr int kReorderTokensPerCta = (kReorderThreads / 8) * kReorderUnroll;

template <bool NORMS>   // NORMS: also write 1 / max(|x|, 1e-12) of every Q and K token (the large-block matcher needs them)
__global__ void __launch_bounds__(kReorderThreads) reorder_kernel(const __grid_constant__ ReorderArgs a) {
    const int t = blockIdx.z, h = blockIdx.y;
    const int chunk = threadIdx.x & 7, slot = threadIdx.x >> 3;
    const int base = blockIdx.x * kReorderTokensPerCta;
    const __nv_bfloat16* src = a.src[t].ptr + (int64_t)h * a.src[t].stride_head + chunk * 8;
    const int64_t st = a.src[t].stride_token;
    __nv_bfloat16* dst = a.dst[t] + (int64_t)h * a.n_tokens * kHeadDim + chunk * 8;
    uint4 v[kReorderUnroll];
#pragma unroll
    for (int u = 0; u < kReorderUnroll; ++u) {
        const int p = base + u * (kReorderThreads / 8) + slot;
        v[u] = make_uint4(0u, 0u, 0u, 0u);
        if (p < a.n_tokens) v[u] = __ldg(reinterpret_cast<const uint4*>(src + (int64_t)__ldg(a.pi + p) * st));
    }
#pragma unroll
    for (int u = 0; u < kReorderUnroll; ++u) {
        const int p = base + u * (kReorderThreads / 8) + slot;
        if (p < a.n_tokens) *reinterpret_cast<uint4*>(dst + (int64_t)p * kHeadDim) = v[u];
        if (NORMS && t < 2) {   // the eight threads of a row are neighbouring lanes
            float x[8];
            unpack8(v[u], x);
            float s = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) s = fmaf(x[e], x[e], s);
            s += __shfl_xor_sync(0xffffffffu, s, 1);
            s += __shfl_xor_sync(0xffffffffu, s, 2);
            s += __shfl_xor_sync(0xffffffffu, s, 4);
            if (chunk == 0 && p < a.n_tokens) a.inv_norm[t][(int64_t)h * a.n_tokens + p] = fminf(rsqrtf(s), 1e12f);
        }
    }
}

cudaError_t launch_reorder(const ReorderArgs& a, cudaStream_t stream) {
    dim3 grid((a.n_tokens + kReorderTokensPerCta - 1) / kReorderTokensPerCta, a.heads, 3);
    if (a.inv_norm[0])
        reorder_kernel<true><<<grid, kReorderThreads, 0, stream>>>(a);
    else
        reorder_kernel<false><<<grid, kReorderThreads, 0, stream>>>(a);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------
// Task cursor: (tensor t, head h, unit u) of a linear task index that advances by a fixed
// stride, kept up to date with carries instead of 64-bit divisions in the loop.
// ------------------------------------------------------------------------------------
struct TaskCursor {
    int t, h, u;
    int st, sh, su;        // the stride, decomposed the same way
    int heads, units;
    __device__ void init(int64_t first, int64_t stride, int heads_, int units_) {
        heads = heads_;
        units = units_;
        const int64_t per_tensor = (int64_t)heads * units;
        t = (int)(first / per_tensor);
        int64_t rem = first - t * per_tensor;
        h = (int)(rem / units);
        u = (int)(rem - (int64_t)h * units);
        st = (int)(stride / per_tensor);
        rem = stride - st * per_tensor;
        sh = (int)(rem / units);
        su = (int)(rem - (int64_t)sh * units);
    }
    __device__ __forceinline__ void advance() {
        u += su;
        if (u >= units) {
            u -= units;
            ++h;
        }
        h += sh;
        if (h >= heads) {
            h -= heads;
            ++t;
        }
        t += st;
    }
};

// ------------------------------------------------------------------------------------
// a2. Block-wise bipartite matching (Eq. 1; Sec. 3.2 top-r rule), one warp per
//     (tensor in {Q, K}, head, block).  The block (n x 64 bf16, contiguous after the
//     reorder) is staged in shared memory by a tiled TMA load with the 128-byte swizzle,
//     double buffered per warp.  The dot products of every token with every dst token are
//     a small dense contraction (n x n_dst x 64): they run on the tensor cores as
//     m16n8k16 bf16 MMAs with fp32 accumulation, operands fetched with ldmatrix straight
//     from the swizzled stage (conflict free); the dst rows are gathered by giving
//     ldmatrix their row addresses.  Products of bf16 values are exact in fp32, and the
//     accumulation error measured on this hardware is below that of an fp32 FMA chain.
//     Squared norms are the diagonal of the same kind of MMA (a tile of rows against
//     itself).  Similarity = dot * inv_norm(src) * inv_norm(dst).
//     argmax ties -> lowest dst; top-r ties -> lowest src.  The r merged src are found by
//     min(r, n_src - r) rounds of a warp-wide max (or min) extraction.
//     Token j of a block is owned, for the selection, by lane (j & 7) * 4 + ((j >> 3) & 1),
//     slot j >> 4: the lane where the MMA accumulator layout leaves row j's results.
// ------------------------------------------------------------------------------------
// warps per CTA (one CTA per SM): as many as the shared memory takes at two stages per warp; a warp works alone on its
// blocks, so the number of warps per scheduler is what hides its instruction latencies
__host__ __device__ constexpr int match_warps_per_cta(int nmax) { return nmax <= 32 ? 8 : (nmax <= 64 ? 16 : (nmax <= 128 ? 12 : 6)); }
// stages per warp: blocks of more than 64 tokens keep a warp busy for many microseconds, far longer than a load takes; one
// stage there buys twice the warps for the same shared memory
__host__ __device__ constexpr int match_stages(int nmax) { return nmax <= 32 ? 2 : 1; }
__host__ __device__ constexpr int match_aux_bytes(int nmax) { return nmax * 4 + 16; }   // inverse norms + 2 mbarriers
__host__ __device__ constexpr int match_smem_bytes(int nmax) {
    return match_warps_per_cta(nmax) * (match_stages(nmax) * nmax * kRowBytes + match_aux_bytes(nmax)) + 1024 /*alignment slack*/;
}

// tiled TMA load {64 channels, rows, heads} -> this CTA's shared memory; the channel coordinate is 0
__device__ __forceinline__ void tma_rows_load(uint32_t dst_smem, const CUtensorMap* map, uint32_t mbar, int row, int head) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(
                     dst_smem),
                 "l"(reinterpret_cast<uint64_t>(map)), "r"(mbar), "r"(0), "r"(row), "r"(head)
                 : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t* r, uint32_t saddr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(saddr)
                 : "memory");
}
// c (16x8 fp32) += a (16x16 bf16, row) * b (16x8 bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// tiled TMA load of one merging block straight from an original tensor: {64 channels, x, y, frame, head}
__device__ __forceinline__ void tma_block_load(uint32_t dst_smem, const CUtensorMap* map, uint32_t mbar, int x0, int y0, int s0, int head) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], [%2];" ::"r"(dst_smem),
        "l"(reinterpret_cast<uint64_t>(map)), "r"(mbar), "r"(0), "r"(x0), "r"(y0), "r"(s0), "r"(head)
        : "memory");
}
// Direct mode: a block arrives as the box [box_frames][box_h][box_w] of 128-byte rows (zero rows where the block
// is clipped by the grid edge or the last frame); its tokens are numbered in the same (frame, row, column)
// order without the holes.  For a block that is not clipped both numberings coincide.
struct BoxMap {
    int box_h, box_w;          // rows and columns of the box
    int rows, cols;            // of this block
    uint32_t m_plane, m_cols;  // multipliers for floor(j / (rows * cols)) and floor(j / cols), j < 256
    bool clipped;
    __device__ void set(int box_frames, int bh, int bw, int frames, int r, int c) {
        box_h = bh;
        box_w = bw;
        rows = r;
        cols = c;
        clipped = frames != box_frames || r != bh || c != bw;
        if (clipped) {
            m_plane = 65536u / (uint32_t)(r * c) + 1u;
            m_cols = 65536u / (uint32_t)c + 1u;
        }
    }
    // token number -> box row
    __device__ __forceinline__ int row_of_token(int j) const {
        if (!clipped) return j;
        const int t = (int)(((uint32_t)j * m_plane) >> 16), rem = j - t * rows * cols;
        const int y = (int)(((uint32_t)rem * m_cols) >> 16), x = rem - y * cols;
        return (t * box_h + y) * box_w + x;
    }
};
// monotone map float -> uint32 (larger float <-> larger key); every real score maps to a key >= 1
__device__ __forceinline__ uint32_t score_key(float s) {
    const uint32_t b = __float_as_uint(s);
    return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}

template <int PASSES, bool DIRECT>
__global__ void __launch_bounds__(match_warps_per_cta(32 * PASSES) * 32, PASSES == 1 ? 2 : 1)   // 3 CTAs/SM would need 80 registers: spills cost more than the third CTA gains
match_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, const MatchArgs a) {
    constexpr int NMAX = 32 * PASSES;
    constexpr int WARPS = match_warps_per_cta(NMAX);
    constexpr int MT = NMAX / 16;        // 16-token row tiles
    constexpr int NT = NMAX / 32;        // 8-dst column tiles (n_dst <= NMAX / 4)
    constexpr bool KEEP_A = PASSES == 1; // row-tile fragments stay in registers between the two passes
    constexpr int STAGES = match_stages(NMAX);
    constexpr uint32_t STAGE_BYTES = NMAX * kRowBytes;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;   // accumulator layout: rows g, g + 8; columns 2 tq, 2 tq + 1
    unsigned char* aux = smem + (size_t)WARPS * STAGES * STAGE_BYTES + (size_t)warp * match_aux_bytes(NMAX);
    float* invn = reinterpret_cast<float*>(aux);                                   // [NMAX]
    const uint32_t mbar0 = smem_u32(aux + NMAX * 4);                               // 2 mbarriers (one used with a single stage)
    const uint32_t stage0 = smem_u32(smem + (size_t)warp * STAGES * STAGE_BYTES);  // [STAGES][NMAX][128], 1024-aligned

    if (lane == 0) {
        mbar_init(mbar0, 1);
        mbar_init(mbar0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    const int64_t n_tasks = 2ll * a.heads * a.n_blocks;
    const int64_t stride = (int64_t)gridDim.x * WARPS;
    const int64_t first = (int64_t)blockIdx.x * WARPS + warp;
    TaskCursor cur, nxt;   // the task being processed; the task whose load is issued next
    cur.init(first, stride, a.heads, a.n_blocks);
    nxt = cur;

    // direct mode: box extents (clipped to the scene once) and the box coordinates of the rows this lane owns
    const int box_f = DIRECT ? min(a.layout.blk_frames, a.layout.frames) : 1, box_h = DIRECT ? min(a.layout.blk_h, a.layout.grid_h) : 1,
              box_w = DIRECT ? min(a.layout.blk_w, a.layout.grid_w) : 1;
    const int box_rows = box_f * box_h * box_w;
    const uint32_t box_bytes = (uint32_t)box_rows * kRowBytes;
    int own_t[MT], own_y[MT], own_x[MT];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        const int rho = mt * 16 + (tq & 1) * 8 + g;
        own_t[mt] = DIRECT ? rho / (box_h * box_w) : 0;
        own_y[mt] = DIRECT ? (rho / box_w) % box_h : 0;
        own_x[mt] = DIRECT ? rho % box_w : 0;
    }
    BoxMap bm;
    bm.clipped = false;
    auto issue = [&](const TaskCursor& c, int buf) {   // lane 0 only; the whole box is transferred (rows past the head's end are zero filled)
        const uint32_t mb = mbar0 + 8 * buf;
        if (DIRECT) {
            const BlockGeom bg = a.geom[c.u];
            mbar_expect_tx(mb, box_bytes);
            tma_block_load(stage0 + buf * STAGE_BYTES, c.t == 0 ? &map_q : &map_k, mb, bg.x0, bg.y0, bg.s0, c.h);
        } else {
            const int start = __ldg(&a.blocks[c.u].start);
            mbar_expect_tx(mb, STAGE_BYTES);
            tma_rows_load(stage0 + buf * STAGE_BYTES, c.t == 0 ? &map_q : &map_k, mb, start, c.h);
        }
    };
    if (first < n_tasks && lane == 0) issue(nxt, 0);
    nxt.advance();
    if (STAGES == 2) {
        if (first + stride < n_tasks && lane == 0) issue(nxt, 1);
        nxt.advance();
    }

    int cached_n = -1, cached_nd = -1;
    uint32_t magic_n = 0, magic_nd = 0;

    int it = 0;
    bool failed = false;
    for (int64_t task = first; task < n_tasks; task += stride, ++it, cur.advance(), nxt.advance()) {
        const int buf = STAGES == 2 ? (it & 1) : 0;
        const uint32_t parity = STAGES == 2 ? ((it >> 1) & 1) : (it & 1);
        const bool more = task + STAGES * stride < n_tasks;
        const BlockInfo bi = a.blocks[cur.u];
        const int n = bi.n, r = cur.t == 0 ? bi.r_q : bi.r_k, nd = cur.t == 0 ? bi.nd_q : bi.nd_k;
        int32_t* A = a.assign[cur.t] + (int64_t)cur.h * a.n_tokens + bi.start;
        if (!mbar_wait_bounded(mbar0 + 8 * buf, parity, a.status, kDevTimeoutMatchLoad)) {
            failed = true;
            break;
        }
        if (r == 0) {
#pragma unroll
            for (int p = 0; p < PASSES; ++p) {
                const int j = lane + 32 * p;
                if (j < n) A[j] = bi.start + j;
            }
            __syncwarp();
            if (more && lane == 0) issue(nxt, buf);
            continue;
        }
        if (nd > NT * 8) {   // first-frame anchoring with more dst tokens than a quarter of the largest block: match_anchor_kernel
            __syncwarp();
            if (more && lane == 0) issue(nxt, buf);
            continue;
        }
        // floor(x / n) and floor(x / n_dst) by multiplication: exact for the operand ranges below (n <= 256, n_dst <= 64)
        const int n_rule = bi.n_rule;   // n (evenly spaced dst tokens) or n_dst (the first n_dst tokens: first-frame anchoring)
        if (n_rule != cached_n || nd != cached_nd) {
            cached_n = n_rule;
            cached_nd = nd;
            magic_n = (1u << 23) / (uint32_t)n_rule + 1u;
            magic_nd = (1u << 23) / (uint32_t)nd + 1u;
        }
        BlockGeom bg{};
        if (DIRECT) {
            bg = a.geom[cur.u];
            bm.set(box_f, box_h, box_w, bg.frames, bg.rows, bg.cols);
        }
        const int n_rows = DIRECT ? box_rows : n;   // rows of the stage that may hold tokens
        auto div_n = [&](int x) { return (int)(((uint32_t)x * magic_n) >> 23); };          // floor(x / n_rule), x < (n_rule + 1) * n_dst
        auto pos_of = [&](int d) { return (int)(((uint32_t)((d + 1) * n_rule + nd - 1) * magic_nd) >> 23) - 1; };   // position of dst d
        const uint32_t blk = stage0 + buf * STAGE_BYTES;
        // ldmatrix address of 16-byte chunk `chunk` of row `row` (chunk c of row j sits at c ^ (j & 7))
        auto chunk_addr = [&](int row, int chunk) { return blk + row * kRowBytes + ((chunk ^ (row & 7)) << 4); };

        // ---- pass 1: squared norms of every token = diagonal of (row tile) x (row tile)^T
        uint32_t af[KEEP_A ? MT : 1][4][4];   // [tile][k step][a0..a3]
        auto load_a = [&](int mt, uint32_t (*dstf)[4]) {
            // matrices of one ldmatrix.x4: rows 0-7 / 8-15 of the tile (lane bit 3), k chunk 2 ks / 2 ks + 1 (lane bit 4)
            const int row = mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) ldmatrix_x4(dstf[ks], chunk_addr(row, 2 * ks + (lane >> 4)));
        };
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            if (mt * 16 < n_rows) {   // warp-uniform
                uint32_t(*fr)[4] = af[KEEP_A ? mt : 0];
                load_a(mt, fr);
                float lo[4] = {0.f, 0.f, 0.f, 0.f}, hi[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    mma_bf16_16816(lo, fr[ks], fr[ks][0], fr[ks][2]);   // against rows 0-7 of the tile
                    mma_bf16_16816(hi, fr[ks], fr[ks][1], fr[ks][3]);   // against rows 8-15
                }
                if (tq == (g >> 1)) {   // this lane holds the diagonal entries of rows g and g + 8
                    const float s_lo = (g & 1) ? lo[1] : lo[0], s_hi = (g & 1) ? hi[3] : hi[2];
                    // 1 / max(|x|, 1e-12): rsqrt.approx is within 2 ulp, far inside the 1e-5 margin rule
                    invn[mt * 16 + g] = fminf(rsqrtf(s_lo), 1e12f);
                    invn[mt * 16 + 8 + g] = fminf(rsqrtf(s_hi), 1e12f);
                }
            }
        }
        // ---- dst fragments: column tile nt holds dst 8 nt .. 8 nt + 7, gathered by row address
        uint32_t bf[NT][4][2];   // [tile][k step][b0, b1]
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            if (nt * 8 < nd) {
                const int d = min(nt * 8 + (lane & 7), nd - 1);
                const int row = DIRECT ? bm.row_of_token(pos_of(d)) : pos_of(d);
#pragma unroll
                for (int kp = 0; kp < 2; ++kp) {   // one ldmatrix.x4 = k steps 2 kp and 2 kp + 1
                    uint32_t rr[4];
                    ldmatrix_x4(rr, chunk_addr(row, 4 * kp + (lane >> 3)));
                    bf[nt][2 * kp][0] = rr[0];
                    bf[nt][2 * kp][1] = rr[1];
                    bf[nt][2 * kp + 1][0] = rr[2];
                    bf[nt][2 * kp + 1][1] = rr[3];
                }
            }
        }
        __syncwarp();   // inverse norms visible; with one pass, every fragment is now in registers
        if (KEEP_A) {
            if (more && lane == 0) issue(nxt, buf);
        }

        // ---- pass 2: similarities, best dst of every token (kept by the owner lane of the token)
        float wd[NT][2];   // inverse norms of this lane's dst columns
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int d = nt * 8 + 2 * tq + e;
                wd[nt][e] = d < nd ? invn[DIRECT ? bm.row_of_token(pos_of(d)) : pos_of(d)] : 0.f;
            }
        uint32_t key[MT];
        int best[MT], tok[MT];   // tok: number of the owned token in the block, -1 if the row holds none
        bool is_src[MT];
        const int own_half = tq & 1;   // owner of rows g (tq == 0) or g + 8 (tq == 1); lanes with tq >= 2 own nothing
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            key[mt] = 0;
            best[mt] = 0;
            tok[mt] = -1;
            is_src[mt] = false;
            if (mt * 16 < n_rows) {
                uint32_t(*fr)[4] = af[KEEP_A ? mt : 0];
                if (!KEEP_A) load_a(mt, fr);
                float top[2] = {-INFINITY, -INFINITY};   // rows g, g + 8
                int arg[2] = {0, 0};
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    if (nt * 8 < nd) {
                        float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) mma_bf16_16816(c, fr[ks], bf[nt][ks][0], bf[nt][ks][1]);
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int d = nt * 8 + 2 * tq + e;
                            if (d < nd) {
                                const float w = wd[nt][e];
                                const float s0 = c[e] * w, s1 = c[2 + e] * w;
                                if (s0 > top[0]) {
                                    top[0] = s0;
                                    arg[0] = d;
                                }
                                if (s1 > top[1]) {
                                    top[1] = s1;
                                    arg[1] = d;
                                }
                            }
                        }
                    }
                }
                // combine the four lanes of a row (ties: lowest dst)
#pragma unroll
                for (int hrow = 0; hrow < 2; ++hrow) {
#pragma unroll
                    for (int off = 1; off <= 2; off <<= 1) {
                        const float ov = __shfl_xor_sync(0xffffffffu, top[hrow], off);
                        const int oa = __shfl_xor_sync(0xffffffffu, arg[hrow], off);
                        if (ov > top[hrow] || (ov == top[hrow] && oa < arg[hrow])) {
                            top[hrow] = ov;
                            arg[hrow] = oa;
                        }
                    }
                }
                const int rho = mt * 16 + own_half * 8 + g;   // row of the stage; j: number of the token in the block
                const bool valid = DIRECT ? (own_t[mt] < bg.frames && own_y[mt] < bg.rows && own_x[mt] < bg.cols) : rho < n;
                const int j = DIRECT ? (own_t[mt] * bg.rows + own_y[mt]) * bg.cols + own_x[mt] : rho;
                tok[mt] = valid ? j : -1;
                if (tq < 2 && valid) {
                    const int jr = min(j, n_rule);   // (positions from n_rule on are src tokens; the clamp keeps the operand in range)
                    const int dj = div_n(jr * nd);
                    if (!(j < n_rule && div_n((jr + 1) * nd) > dj)) {   // not a dst position: a src token
                        is_src[mt] = true;
                        key[mt] = score_key((own_half ? top[1] : top[0]) * invn[rho]);
                        best[mt] = pos_of(own_half ? arg[1] : arg[0]);
                    }
                }
            }
        }

        // ---- the r src with the best scores merge (ties: lowest position first)
        const int n_src = n - nd, n_out = n_src - r;
        bool merged[MT];
        if (r <= n_out) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) merged[mt] = false;
            for (int round = 0; round < r; ++round) {
                uint32_t loc = 0;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) loc = max(loc, (is_src[mt] && !merged[mt]) ? key[mt] : 0u);
                const uint32_t m = __reduce_max_sync(0xffffffffu, loc);
                int cand = 0x7fffffff;   // lowest own position holding the maximum
#pragma unroll
                for (int mt = MT - 1; mt >= 0; --mt)
                    if (is_src[mt] && !merged[mt] && key[mt] == m) cand = mt * 16 + own_half * 8 + g;
                const int win = __reduce_min_sync(0xffffffffu, cand);
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
                    if (is_src[mt] && win == mt * 16 + own_half * 8 + g) merged[mt] = true;
            }
        } else {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) merged[mt] = is_src[mt];
            for (int round = 0; round < n_out; ++round) {
                uint32_t loc = 0xffffffffu;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) loc = min(loc, merged[mt] ? key[mt] : 0xffffffffu);
                const uint32_t m = __reduce_min_sync(0xffffffffu, loc);
                int cand = -1;           // highest own position holding the minimum
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
                    if (merged[mt] && key[mt] == m) cand = mt * 16 + own_half * 8 + g;
                const int win = __reduce_max_sync(0xffffffffu, cand);
#pragma unroll
                for (int mt = 0; mt < MT; ++mt)
                    if (merged[mt] && win == mt * 16 + own_half * 8 + g) merged[mt] = false;
            }
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            if (tq < 2 && tok[mt] >= 0) A[tok[mt]] = bi.start + (merged[mt] ? best[mt] : tok[mt]);
        }
        __syncwarp();   // every lane is done with the inverse norms (and, with several passes, the stage buffer)
        if (!KEEP_A) {
            if (more && lane == 0) issue(nxt, buf);
        }
    }
    if (failed) {
        // give copies that may still be in flight a bounded chance to land before the CTA's
        // shared memory is released
        mbar_wait_bounded(mbar0, STAGES == 2 ? ((it >> 1) & 1) : (it & 1), a.status, kDevTimeoutMatchLoad);
        if (STAGES == 2) mbar_wait_bounded(mbar0 + 8, (it >> 1) & 1, a.status, kDevTimeoutMatchLoad);
    }
}

// 5-D map of the patch tokens of an original tensor with one merging block as the box
static bool encode_block_map(CUtensorMap* map, const TensorView& t, const SourceLayout& L, int heads) {
    const int bw = L.blk_w < L.grid_w ? L.blk_w : L.grid_w, bh = L.blk_h < L.grid_h ? L.blk_h : L.grid_h,
              bf = L.blk_frames < L.frames ? L.blk_frames : L.frames;
    return encode_patch_tensor_map(map, t.ptr + (int64_t)L.n_special * t.stride_token, L.grid_w, L.grid_h, L.frames, heads, t.stride_token,
                                   L.tokens_per_frame, t.stride_head, bw, bh, bf);
}

template <int PASSES>
static cudaError_t launch_match_t(const MatchArgs& a, int sm_count, cudaStream_t stream) {
    constexpr int NMAX = 32 * PASSES;
    constexpr int WARPS = match_warps_per_cta(NMAX);
    const size_t smem = match_smem_bytes(NMAX);
    const bool direct = a.geom != nullptr;
    CUtensorMap mq, mk;
    const int64_t N = a.n_tokens;
    if (direct) {
        if (!encode_block_map(&mq, a.src[0], a.layout, a.heads) || !encode_block_map(&mk, a.src[1], a.layout, a.heads)) return cudaErrorInvalidValue;
    } else if (!encode_rows_tensor_map(&mq, a.xr[0], N, a.heads, kHeadDim, N * kHeadDim, NMAX) ||
               !encode_rows_tensor_map(&mk, a.xr[1], N, a.heads, kHeadDim, N * kHeadDim, NMAX)) {
        return cudaErrorInvalidValue;
    }
    const int64_t n_tasks = 2ll * a.heads * a.n_blocks;
    int ctas_per_sm = (int)((224 * 1024) / (smem + 1024));
    ctas_per_sm = ctas_per_sm < 1 ? 1 : (ctas_per_sm > 16 / WARPS ? (16 / WARPS < 1 ? 1 : 16 / WARPS) : ctas_per_sm);
    int64_t grid = (n_tasks + WARPS - 1) / WARPS;
    const int64_t cap = (int64_t)sm_count * ctas_per_sm;
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    if (direct)
        match_kernel<PASSES, true><<<(unsigned)grid, WARPS * 32, smem, stream>>>(mq, mk, a);
    else
        match_kernel<PASSES, false><<<(unsigned)grid, WARPS * 32, smem, stream>>>(mq, mk, a);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------
// a2 under first-frame anchoring (the paper's appendix on error mitigation: all tokens of frame 0 are dst tokens), for the
//     blocks of the first frame group whose dst tokens exceed what match_kernel holds (a quarter of the largest block:
//     blocks of two or three frames).  Same rule, plain formulation: one CTA per (tensor, head, block), the block's rows
//     gathered through the reorder index into shared memory, inverse norms, for every src token the dot products with
//     the dst tokens (the block's first n_dst tokens) by fp32 FMAs on exact bf16 products, best dst (ties: lowest),
//     then the r best src by rank counting (ties: lowest position).  These blocks are 1 / (frame groups) of the scene.
// ------------------------------------------------------------------------------------
constexpr int kAnchorThreads = 128;
constexpr int kAnchorPitch = kRowBytes + 16;   // row pitch in shared memory: 16-byte accesses of neighbouring rows on distinct banks
__host__ __device__ constexpr int anchor_smem_bytes(int nmax) { return nmax * (kAnchorPitch + 12); }   // rows, inverse norms, scores, best dst

__global__ void __launch_bounds__(kAnchorThreads) match_anchor_kernel(const MatchArgs a, const TensorView src_q, const TensorView src_k,
                                                                       const int32_t* __restrict__ pi, int n_anchor, int main_capacity, int nmax) {
    extern __shared__ __align__(16) unsigned char sm_anchor[];
    const int task = blockIdx.x;
    const int b = task % n_anchor, h = (task / n_anchor) % a.heads, t = task / (n_anchor * a.heads);
    const BlockInfo bi = a.blocks[b];
    const int n = bi.n, nd = t == 0 ? bi.nd_q : bi.nd_k, r = t == 0 ? bi.r_q : bi.r_k;
    if (bi.n_rule == n || nd <= main_capacity || r == 0 || n > nmax) return;   // match_kernel has written this block's map
    unsigned char* rows = sm_anchor;
    float* inv = reinterpret_cast<float*>(sm_anchor + (size_t)nmax * kAnchorPitch);
    float* score = inv + nmax;
    int* best = reinterpret_cast<int*>(score + nmax);
    const TensorView& sv = t == 0 ? src_q : src_k;
    const __nv_bfloat16* base = sv.ptr + (int64_t)h * sv.stride_head;
    for (int q = threadIdx.x; q < n * 8; q += kAnchorThreads) {
        const int row = q >> 3, c = q & 7;
        const int64_t orig = pi ? __ldg(pi + bi.start + row) : bi.start + row;   // (no index: the tensors are the reordered copies)
        *reinterpret_cast<uint4*>(rows + row * kAnchorPitch + c * 16) = __ldg(reinterpret_cast<const uint4*>(base + orig * sv.stride_token + c * 8));
    }
    __syncthreads();
    for (int j = threadIdx.x; j < n; j += kAnchorThreads) {
        float ss = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            float x[8];
            unpack8(*reinterpret_cast<const uint4*>(rows + j * kAnchorPitch + c * 16), x);
#pragma unroll
            for (int e = 0; e < 8; ++e) ss = fmaf(x[e], x[e], ss);
        }
        inv[j] = fminf(rsqrtf(ss), 1e12f);   // 1 / max(|x|, 1e-12)
    }
    __syncthreads();
    for (int j = nd + threadIdx.x; j < n; j += kAnchorThreads) {   // src tokens: everything behind the block's tokens of frame 0
        float xs[64];
#pragma unroll
        for (int c = 0; c < 8; ++c) unpack8(*reinterpret_cast<const uint4*>(rows + j * kAnchorPitch + c * 16), xs + 8 * c);
        float top = -INFINITY;
        int arg = 0;
        for (int d = 0; d < nd; ++d) {
            float dot = 0.f;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                float xd[8];
                unpack8(*reinterpret_cast<const uint4*>(rows + d * kAnchorPitch + c * 16), xd);   // (the same row for every thread: a broadcast)
#pragma unroll
                for (int e = 0; e < 8; ++e) dot = fmaf(xs[8 * c + e], xd[e], dot);
            }
            const float sim = dot * inv[d];
            if (sim > top) {
                top = sim;
                arg = d;
            }
        }
        score[j] = top * inv[j];
        best[j] = arg;
    }
    __syncthreads();
    int32_t* A = a.assign[t] + (int64_t)h * a.n_tokens + bi.start;
    for (int j = threadIdx.x; j < n; j += kAnchorThreads) {
        if (j < nd) {
            A[j] = bi.start + j;
            continue;
        }
        const uint32_t key = score_key(score[j]);
        int rank = 0;   // src tokens that come before this one: better score, or the same score at a lower position
        for (int i = nd; i < n; ++i) {
            const uint32_t ki = score_key(score[i]);
            rank += (ki > key || (ki == key && i < j)) ? 1 : 0;
        }
        A[j] = bi.start + (rank < r ? best[j] : j);
    }
}

cudaError_t launch_match_anchor(const MatchArgs& a, const TensorView& src_q, const TensorView& src_k, const int32_t* pi, int n_anchor,
                                int main_capacity, int max_block_tokens, cudaStream_t stream) {
    if (n_anchor <= 0) return cudaSuccess;
    const int nmax = max_block_tokens < kMaxBlockTokens ? max_block_tokens : kMaxBlockTokens;
    match_anchor_kernel<<<2 * a.heads * n_anchor, kAnchorThreads, anchor_smem_bytes(nmax), stream>>>(a, src_q, src_k, pi, n_anchor, main_capacity, nmax);
    return cudaGetLastError();
}

cudaError_t launch_match(const MatchArgs& a, int max_block_tokens, int sm_count, cudaStream_t stream) {
    if (max_block_tokens <= 32) return launch_match_t<1>(a, sm_count, stream);
    if (max_block_tokens <= 64) return launch_match_t<2>(a, sm_count, stream);
    if (max_block_tokens <= 128) return launch_match_t<4>(a, sm_count, stream);
    return launch_match_t<8>(a, sm_count, stream);
}

// ------------------------------------------------------------------------------------
// a3 (blocks of at most 32 tokens).  The group sums of a block are one small dense
//     contraction: merged_sum[kept row][channel] = sum_token W[row][token] x[token][channel]
//     with the 0/1 assignment matrix W.  It runs on the tensor cores (m16n8k16, bf16 inputs,
//     fp32 accumulation: W is exact in bf16, the products are exact, and the measured
//     accumulation error is below that of an fp32 add chain).  W is built in registers from
//     the map; x comes from the swizzled TMA stage through ldmatrix.trans (conflict free).
//     The mean is the sum times the reciprocal of the group size, rounded once to bf16.
//     One warp per (tensor, head, block); kept tokens are compacted in reordered order.
// ------------------------------------------------------------------------------------
constexpr int kMergeTcWarps = 8;
constexpr int kMergeTcAux = 32 * 4 + 16 + 32 * 4;   // reciprocal group sizes per kept row + 2 mbarriers + group sizes / starts
constexpr int kMergeTcSmem = kMergeTcWarps * (2 * 32 * kRowBytes + kMergeTcAux) + 1024 /*alignment slack*/;

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t* r, uint32_t saddr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(saddr)
                 : "memory");
}

// DIRECT: the blocks come straight from the original tensors (5-D block maps), the special tokens frame by
// frame (4-D frame maps sq, sk, sv); otherwise from the reordered copies, specials in chunks of 32.
template <bool DIRECT>
__global__ void __launch_bounds__(kMergeTcWarps * 32, 2)
merge_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_sq,
                const __grid_constant__ CUtensorMap map_sk, const __grid_constant__ CUtensorMap map_sv, const MergeArgs a) {
    constexpr uint32_t STAGE_BYTES = 32 * kRowBytes;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;   // accumulator layout: rows g, g + 8; columns 2 tq, 2 tq + 1
    unsigned char* stage = smem + (size_t)warp * 2 * STAGE_BYTES;                       // [2][32][128], 1024-aligned, swizzled
    unsigned char* aux = smem + (size_t)kMergeTcWarps * 2 * STAGE_BYTES + (size_t)warp * kMergeTcAux;
    float* rcnt = reinterpret_cast<float*>(aux);                                        // [32] 1 / group size of kept row
    const uint32_t mbar0 = smem_u32(aux + 32 * 4), stage0 = smem_u32(stage);
    int* gsz = reinterpret_cast<int*>(aux + 32 * 4 + 16);                               // [32] size, then first member, of kept row

    if (lane == 0) {
        mbar_init(mbar0, 1);
        mbar_init(mbar0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    // task -> (tensor t, head h, unit u); units 0 .. n_blocks-1 are merging blocks, the rest are
    // chunks of 32 special tokens (never merged: rows 0 .. n_special_total-1 are copied)
    const int sp_chunks = DIRECT ? (a.layout.n_special > 0 ? a.layout.frames : 0) : (a.n_special_total + 31) / 32;
    const int per_head = a.n_blocks + sp_chunks;
    const int box_f = DIRECT ? min(a.layout.blk_frames, a.layout.frames) : 1, box_h = DIRECT ? min(a.layout.blk_h, a.layout.grid_h) : 1,
              box_w = DIRECT ? min(a.layout.blk_w, a.layout.grid_w) : 1;
    const int box_rows = box_f * box_h * box_w;
    const int own_t = DIRECT ? lane / (box_h * box_w) : 0, own_y = DIRECT ? (lane / box_w) % box_h : 0, own_x = DIRECT ? lane % box_w : 0;
    if (DIRECT) {   // stage rows that no block load writes enter the MMAs with weight 0: they must hold finite values
        for (int q = box_rows * 8 + lane; q < 32 * 8; q += 32) {   // (a load of special tokens may overwrite some of them later)
            *reinterpret_cast<uint4*>(stage + q * 16) = make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(stage + STAGE_BYTES + q * 16) = make_uint4(0u, 0u, 0u, 0u);
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
    }
    BoxMap bm;
    bm.clipped = false;
    const int64_t n_tasks = 3ll * a.heads * per_head;
    const int64_t stride = (int64_t)gridDim.x * kMergeTcWarps;
    const int64_t first = (int64_t)blockIdx.x * kMergeTcWarps + warp;
    TaskCursor cur, nxt;   // the task being processed; the task whose load is issued next
    cur.init(first, stride, a.heads, per_head);
    nxt = cur;

    auto unit_start = [&](const TaskCursor& c) { return c.u >= a.n_blocks ? (c.u - a.n_blocks) * 32 : __ldg(&a.blocks[c.u].start); };
    auto issue = [&](const TaskCursor& c, int buf) {   // lane 0 only; the whole 32-row box is transferred (rows past the head's end are zero filled)
        const uint32_t mb = mbar0 + 8 * buf;
        if (!DIRECT) {
            mbar_expect_tx(mb, STAGE_BYTES);
            tma_rows_load(stage0 + buf * STAGE_BYTES, c.t == 0 ? &map_q : (c.t == 1 ? &map_k : &map_v), mb, unit_start(c), c.h);
        } else if (c.u >= a.n_blocks) {   // the special tokens of frame u - n_blocks
            mbar_expect_tx(mb, (uint32_t)a.layout.n_special * kRowBytes);
            const CUtensorMap* m = c.t == 0 ? &map_sq : (c.t == 1 ? &map_sk : &map_sv);
            asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(
                             stage0 + buf * STAGE_BYTES),
                         "l"(reinterpret_cast<uint64_t>(m)), "r"(mb), "r"(0), "r"(0), "r"(c.u - a.n_blocks), "r"(c.h)
                         : "memory");
        } else {
            const BlockGeom bg = a.geom[c.u];
            mbar_expect_tx(mb, (uint32_t)box_rows * kRowBytes);
            tma_block_load(stage0 + buf * STAGE_BYTES, c.t == 0 ? &map_q : (c.t == 1 ? &map_k : &map_v), mb, bg.x0, bg.y0, bg.s0, c.h);
        }
    };
    if (first < n_tasks && lane == 0) issue(nxt, 0);
    nxt.advance();
    if (first + stride < n_tasks && lane == 0) issue(nxt, 1);
    nxt.advance();

    // Everything a task needs besides the staged rows: its place in the tables, and this lane's map entry.
    // Both are fetched one task ahead (table entry at the start of the previous task, map entry behind its
    // MMAs), so that their global-memory latency is not paid between waiting for a stage and using it.
    struct Meta {
        int t, h, start, n, r, moff;
        bool special;
        BlockGeom bg;
    };
    auto load_meta = [&](const TaskCursor& c) {
        Meta m{};
        m.t = c.t;
        m.h = c.h;
        m.special = c.u >= a.n_blocks;
        if (m.special) {
            m.start = DIRECT ? (c.u - a.n_blocks) * a.layout.n_special : (c.u - a.n_blocks) * 32;
            m.n = DIRECT ? a.layout.n_special : min(32, a.n_special_total - m.start);
            m.r = 0;
            m.moff = m.start;
        } else {
            if (DIRECT) m.bg = a.geom[c.u];
            const BlockInfo bi = a.blocks[c.u];
            m.start = bi.start;
            m.n = bi.n;
            m.r = c.t == 0 ? bi.r_q : bi.r_k;
            m.moff = c.t == 0 ? (a.moff_q_var ? __ldg(a.moff_q_var + (int64_t)c.h * a.n_blocks + c.u) : bi.moff_q) : bi.moff_k;
        }
        return m;
    };
    // lane = row of the stage; number of the token it holds in the block (-1: none)
    auto token_of_lane = [&](const Meta& m) {
        return !DIRECT || m.special ? (lane < m.n ? lane : -1)
                                    : ((own_t < m.bg.frames && own_y < m.bg.rows && own_x < m.bg.cols) ? (own_t * m.bg.rows + own_y) * m.bg.cols + own_x : -1);
    };
    auto load_target = [&](const Meta& m) {   // token this lane's token is merged into (number in the block), -1 if the lane holds none
        const int tok = token_of_lane(m);
        return m.r > 0 && tok >= 0 ? __ldg(a.assign[m.t == 0 ? 0 : 1] + (int64_t)m.h * a.n_tokens + m.start + tok) - m.start : -1;
    };
    Meta meta_next{};
    int target_next = -1;
    if (first < n_tasks) {
        meta_next = load_meta(cur);
        target_next = load_target(meta_next);
    }
    TaskCursor ahead = cur;   // the task after the current one
    ahead.advance();

    int it = 0;
    bool failed = false;
    for (int64_t task = first; task < n_tasks; task += stride, ++it, cur.advance(), nxt.advance(), ahead.advance()) {
        const int buf = it & 1;
        const uint32_t parity = (it >> 1) & 1;
        const bool more = task + 2 * stride < n_tasks, has_next = task + stride < n_tasks;
        const Meta meta = meta_next;
        int rep = target_next;
        if (has_next) meta_next = load_meta(ahead);   // in flight while this task is processed
        const int t = meta.t, h = meta.h, start = meta.start, n = meta.n, r = meta.r, moff = meta.moff;
        const bool special = meta.special;
        const BlockGeom bg = meta.bg;
        if (DIRECT && !special) bm.set(box_f, box_h, box_w, bg.frames, bg.rows, bg.cols);
        if (special) bm.clipped = false;
        const int m_len = t == 0 ? a.m_q : a.m_k;
        uint32_t* out = reinterpret_cast<uint32_t*>(a.merged[t] + ((int64_t)h * m_len + moff) * kHeadDim);   // 32 words per row
        const uint32_t blk = stage0 + buf * STAGE_BYTES;
        const int tok = token_of_lane(meta);
        // rep = ROW of the stage holding the token this lane's token is merged into
        if (r > 0 && tok >= 0) {
            if (rep < 0 || rep >= n) {   // corrupt map: record, treat as kept
                atomicCAS(a.status, kDevOk, kDevBadIndex);
                rep = tok;
            }
            if (DIRECT) rep = bm.row_of_token(rep);
        } else {
            rep = -1;
        }
        if (!mbar_wait_bounded(mbar0 + 8 * buf, parity, a.status, kDevTimeoutMatchLoad)) {
            failed = true;
            break;
        }
        if (r == 0) {   // nothing merges here: copy the rows, 16 bytes per lane (chunk c of row j sits at c ^ (j & 7))
            const unsigned char* sb = stage + buf * STAGE_BYTES;
            uint4* o4 = reinterpret_cast<uint4*>(out);
            for (int q = lane; q < n * 8; q += 32) {
                const int row = DIRECT ? bm.row_of_token(q >> 3) : q >> 3, ch = q & 7;
                o4[q] = *reinterpret_cast<const uint4*>(sb + row * kRowBytes + ((ch ^ (row & 7)) << 4));
            }
            if (t == 0 && !special && lane < n) a.rank_q[(int64_t)h * a.n_tokens + start + lane] = moff + lane;
            if (t == 0 && a.group_start && lane < n) {   // every token is a group of its own
                a.group_start[(int64_t)h * (a.m_q + 1) + moff + lane] = start + lane;
                a.group_member[(int64_t)h * a.n_tokens + start + lane] = __ldg(a.pi + start + lane);
            }
            if (has_next) target_next = load_target(meta_next);
        } else {
            // merged row of every token: rank of its representative among the kept tokens
            const unsigned kept = __ballot_sync(0xffffffffu, rep == lane);   // rep == -1 for lanes >= n
            const int n_kept = __popc(kept);
            const int row_of = rep >= 0 ? __popc(kept & ((1u << rep) - 1u)) : -1;
            if (t == 0 && tok >= 0) a.rank_q[(int64_t)h * a.n_tokens + start + tok] = moff + row_of;
            const unsigned group = __match_any_sync(0xffffffffu, row_of);
            if (rep == lane) rcnt[row_of] = 1.0f / (float)__popc(group);
            if (t == 0 && a.group_start) {
                // member lists of the merged rows: the block's tokens group by group, kept rows in rank order
                // (first member of row k = tokens of the rows before it: a warp scan over the group sizes)
                if (rep == lane) gsz[row_of] = __popc(group);
                __syncwarp();
                const int sz = lane < n_kept ? gsz[lane] : 0;
                int incl = sz;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const int v = __shfl_up_sync(0xffffffffu, incl, off);
                    if (lane >= off) incl += v;
                }
                __syncwarp();   // every size has been read
                if (lane < n_kept) {
                    gsz[lane] = incl - sz;
                    a.group_start[(int64_t)h * (a.m_q + 1) + moff + lane] = start + incl - sz;
                }
                __syncwarp();
                if (tok >= 0) {   // the token's number in the original order: from the block's place in the scene, or through the reorder index
                    const int orig = DIRECT ? (bg.s0 + own_t) * a.layout.tokens_per_frame + a.layout.n_special + (bg.y0 + own_y) * a.layout.grid_w + bg.x0 + own_x
                                            : __ldg(a.pi + start + tok);
                    a.group_member[(int64_t)h * a.n_tokens + start + gsz[row_of] + __popc(group & ((1u << lane) - 1u))] = orig;
                }
            }
            // x fragments: for k step ks (16 tokens) and channel tile pair np, one ldmatrix.x4.trans gives
            // b0, b1 of channel tile 2 np and b0, b1 of channel tile 2 np + 1
            uint32_t bf[2][4][4];
            const int n_ks = (DIRECT ? box_rows : n) > 16 ? 2 : 1;   // rows of the stage that may hold tokens
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                if (ks < n_ks) {
                    const int tok = 16 * ks + (lane & 7) + ((lane >> 3) & 1) * 8;
                    const uint32_t rowaddr = blk + tok * kRowBytes;
#pragma unroll
                    for (int np = 0; np < 4; ++np) ldmatrix_x4_trans(bf[ks][np], rowaddr + (((2 * np + (lane >> 4)) ^ (tok & 7)) << 4));
                }
            }
            // W fragments need the rows of tokens 16 ks + {2 tq, 2 tq + 1, 2 tq + 8, 2 tq + 9}
            int rw[2][4];
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                rw[ks][0] = __shfl_sync(0xffffffffu, row_of, 16 * ks + 2 * tq);
                rw[ks][1] = __shfl_sync(0xffffffffu, row_of, 16 * ks + 2 * tq + 1);
                rw[ks][2] = __shfl_sync(0xffffffffu, row_of, 16 * ks + 2 * tq + 8);
                rw[ks][3] = __shfl_sync(0xffffffffu, row_of, 16 * ks + 2 * tq + 9);
            }
            __syncwarp();   // reciprocal group sizes visible; every lane has its fragments: the stage can be refilled
            if (more && lane == 0) issue(nxt, buf);
            const int n_mt = n_kept > 16 ? 2 : 1;
#pragma unroll 1
            for (int mt = 0; mt < n_mt; ++mt) {
                const int r0 = 16 * mt + g, r1 = r0 + 8;   // this lane's two accumulator rows
                float c[8][4];
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
#pragma unroll
                for (int ks = 0; ks < 2; ++ks) {
                    if (ks < n_ks) {
                        uint32_t af[4];   // bf16 1.0 = 0x3f80
                        af[0] = (rw[ks][0] == r0 ? 0x3f80u : 0u) | (rw[ks][1] == r0 ? 0x3f800000u : 0u);
                        af[1] = (rw[ks][0] == r1 ? 0x3f80u : 0u) | (rw[ks][1] == r1 ? 0x3f800000u : 0u);
                        af[2] = (rw[ks][2] == r0 ? 0x3f80u : 0u) | (rw[ks][3] == r0 ? 0x3f800000u : 0u);
                        af[3] = (rw[ks][2] == r1 ? 0x3f80u : 0u) | (rw[ks][3] == r1 ? 0x3f800000u : 0u);
#pragma unroll
                        for (int nt = 0; nt < 8; ++nt)
                            mma_bf16_16816(c[nt], af, bf[ks][nt >> 1][2 * (nt & 1)], bf[ks][nt >> 1][2 * (nt & 1) + 1]);
                    }
                }
                if (mt == 0 && has_next) target_next = load_target(meta_next);   // behind this task's MMAs
                const int cap = t == 0 && a.moff_q_var ? n : n - r;   // (a corrupt map cannot overrun; after outlier filtering more than n - r may be kept)
                const bool w0 = r0 < n_kept && r0 < cap, w1 = r1 < n_kept && r1 < cap;
                const float i0 = w0 ? rcnt[r0] : 0.f, i1 = w1 ? rcnt[r1] : 0.f;
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) {
                    if (w0) {
                        const __nv_bfloat162 o = __floats2bfloat162_rn(c[nt][0] * i0, c[nt][1] * i0);
                        out[r0 * 32 + nt * 4 + tq] = *reinterpret_cast<const uint32_t*>(&o);
                    }
                    if (w1) {
                        const __nv_bfloat162 o = __floats2bfloat162_rn(c[nt][2] * i1, c[nt][3] * i1);
                        out[r1 * 32 + nt * 4 + tq] = *reinterpret_cast<const uint32_t*>(&o);
                    }
                }
            }
            __syncwarp();   // every lane is done with the reciprocals before the next task rewrites them
            continue;
        }
        __syncwarp();   // every lane is done reading this stage buffer
        if (more && lane == 0) issue(nxt, buf);
    }
    if (failed) {
        mbar_wait_bounded(mbar0, (it >> 1) & 1, a.status, kDevTimeoutMatchLoad);
        mbar_wait_bounded(mbar0 + 8, (it >> 1) & 1, a.status, kDevTimeoutMatchLoad);
    }
}

static cudaError_t launch_merge_tc(const MergeArgs& a, int sm_count, cudaStream_t stream) {
    CUtensorMap m[3], sp[3];
    const int64_t N = a.n_tokens;
    const bool direct = a.geom != nullptr;
    const int sp_units = direct ? (a.layout.n_special > 0 ? a.layout.frames : 0) : (a.n_special_total + 31) / 32;
    for (int t = 0; t < 3; ++t) {
        if (direct) {
            if (!encode_block_map(&m[t], a.src[t], a.layout, a.heads)) return cudaErrorInvalidValue;
            if (a.layout.n_special > 0 &&
                !encode_frame_tensor_map(&sp[t], a.src[t].ptr, a.layout.tokens_per_frame, a.layout.frames, a.heads, a.src[t].stride_token,
                                         a.src[t].stride_head, a.layout.n_special))
                return cudaErrorInvalidValue;
            if (a.layout.n_special <= 0) sp[t] = m[t];   // never used
        } else {
            if (!encode_rows_tensor_map(&m[t], a.xr[t], N, a.heads, kHeadDim, N * kHeadDim, 32)) return cudaErrorInvalidValue;
            sp[t] = m[t];   // not used
        }
    }
    const int64_t n_tasks = 3ll * a.heads * (a.n_blocks + sp_units);
    int64_t grid = (n_tasks + kMergeTcWarps - 1) / kMergeTcWarps;
    const int64_t cap = (int64_t)sm_count * 2;
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    if (direct)
        merge_tc_kernel<true><<<(unsigned)grid, kMergeTcWarps * 32, kMergeTcSmem, stream>>>(m[0], m[1], m[2], sp[0], sp[1], sp[2], a);
    else
        merge_tc_kernel<false><<<(unsigned)grid, kMergeTcWarps * 32, kMergeTcSmem, stream>>>(m[0], m[1], m[2], sp[0], sp[1], sp[2], a);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------
// a3 (blocks of 33 to 256 tokens).  The same contraction as above, merged_sum = W x, for blocks that
//     take several 32-token passes: lane l holds the map entries of tokens l, l + 32, ...; the kept rows
//     are walked in tiles of 16, the tokens in steps of 16, and the x fragments are fetched per
//     (row tile, token step) with ldmatrix.trans from the swizzled TMA stage (blocks come from the
//     reordered copies).  Group sizes are counted with shared-memory atomics.
// ------------------------------------------------------------------------------------
__host__ __device__ constexpr int merge_multi_warps(int nmax) { return nmax <= 64 ? 16 : (nmax <= 128 ? 12 : 6); }   // as for the match kernel
__host__ __device__ constexpr int merge_multi_stages(int nmax) { return nmax <= 32 ? 2 : 1; }                          // (see match_stages)
__host__ __device__ constexpr int merge_multi_aux(int nmax) { return nmax * 8 + 16; }   // counts, reciprocals, 2 mbarriers
__host__ __device__ constexpr int merge_multi_smem(int nmax) {
    return merge_multi_warps(nmax) * (merge_multi_stages(nmax) * nmax * kRowBytes + merge_multi_aux(nmax)) + 1024 /*alignment slack*/;
}

template <int PASSES, bool DIRECT>
__global__ void __launch_bounds__(merge_multi_warps(32 * PASSES) * 32, 1)
merge_multi_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                   const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_sq,
                   const __grid_constant__ CUtensorMap map_sk, const __grid_constant__ CUtensorMap map_sv, const MergeArgs a) {
    constexpr int NMAX = 32 * PASSES;
    constexpr int WARPS = merge_multi_warps(NMAX);
    constexpr int STAGES = merge_multi_stages(NMAX);
    constexpr int KS = NMAX / 16;   // token steps
    constexpr uint32_t STAGE_BYTES = NMAX * kRowBytes;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;   // accumulator layout: rows g, g + 8; columns 2 tq, 2 tq + 1
    unsigned char* stage = smem + (size_t)warp * STAGES * STAGE_BYTES;                  // [STAGES][NMAX][128], 1024-aligned, swizzled
    unsigned char* aux = smem + (size_t)WARPS * STAGES * STAGE_BYTES + (size_t)warp * merge_multi_aux(NMAX);
    int* cnt = reinterpret_cast<int*>(aux);                                             // [NMAX] group size of kept row
    float* rcnt = reinterpret_cast<float*>(aux + NMAX * 4);                             // [NMAX] its reciprocal
    const uint32_t mbar0 = smem_u32(aux + NMAX * 8), stage0 = smem_u32(stage);

    if (lane == 0) {
        mbar_init(mbar0, 1);
        mbar_init(mbar0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    // task -> (tensor t, head h, unit u); units 0 .. n_blocks-1 are merging blocks, the rest are
    // chunks of 32 special tokens (never merged: rows 0 .. n_special_total-1 are copied)
    const int sp_chunks = DIRECT ? (a.layout.n_special > 0 ? a.layout.frames : 0) : (a.n_special_total + 31) / 32;
    const int per_head = a.n_blocks + sp_chunks;
    // direct mode: box extents and the box coordinates of the stage rows lane + 32 p
    const int box_f = DIRECT ? min(a.layout.blk_frames, a.layout.frames) : 1, box_h = DIRECT ? min(a.layout.blk_h, a.layout.grid_h) : 1,
              box_w = DIRECT ? min(a.layout.blk_w, a.layout.grid_w) : 1;
    const int box_rows = box_f * box_h * box_w;
    int own_t[PASSES], own_y[PASSES], own_x[PASSES];
#pragma unroll
    for (int p = 0; p < PASSES; ++p) {
        const int rho = lane + 32 * p;
        own_t[p] = DIRECT ? rho / (box_h * box_w) : 0;
        own_y[p] = DIRECT ? (rho / box_w) % box_h : 0;
        own_x[p] = DIRECT ? rho % box_w : 0;
    }
    if (DIRECT) {   // stage rows that no block load writes enter the MMAs with weight 0: they must hold finite values
        for (int q = box_rows * 8 + lane; q < NMAX * 8; q += 32) {   // (a load of special tokens may overwrite some of them later)
            *reinterpret_cast<uint4*>(stage + q * 16) = make_uint4(0u, 0u, 0u, 0u);
            if (STAGES == 2) *reinterpret_cast<uint4*>(stage + STAGE_BYTES + q * 16) = make_uint4(0u, 0u, 0u, 0u);   // (one stage: there is no second buffer)
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
    }
    BoxMap bm;
    bm.clipped = false;
    const int64_t n_tasks = 3ll * a.heads * per_head;
    const int64_t stride = (int64_t)gridDim.x * WARPS;
    const int64_t first = (int64_t)blockIdx.x * WARPS + warp;
    TaskCursor cur, nxt;   // the task being processed; the task whose load is issued next
    cur.init(first, stride, a.heads, per_head);
    nxt = cur;

    auto issue = [&](const TaskCursor& c, int buf) {   // lane 0 only; the whole NMAX-row box is transferred (rows past the head's end are zero filled)
        const uint32_t mb = mbar0 + 8 * buf;
        if (!DIRECT) {
            const int start = c.u >= a.n_blocks ? (c.u - a.n_blocks) * 32 : __ldg(&a.blocks[c.u].start);
            mbar_expect_tx(mb, STAGE_BYTES);
            tma_rows_load(stage0 + buf * STAGE_BYTES, c.t == 0 ? &map_q : (c.t == 1 ? &map_k : &map_v), mb, start, c.h);
        } else if (c.u >= a.n_blocks) {   // the special tokens of frame u - n_blocks
            mbar_expect_tx(mb, (uint32_t)a.layout.n_special * kRowBytes);
            const CUtensorMap* m = c.t == 0 ? &map_sq : (c.t == 1 ? &map_sk : &map_sv);
            asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];" ::"r"(
                             stage0 + buf * STAGE_BYTES),
                         "l"(reinterpret_cast<uint64_t>(m)), "r"(mb), "r"(0), "r"(0), "r"(c.u - a.n_blocks), "r"(c.h)
                         : "memory");
        } else {
            const BlockGeom bg = a.geom[c.u];
            mbar_expect_tx(mb, (uint32_t)box_rows * kRowBytes);
            tma_block_load(stage0 + buf * STAGE_BYTES, c.t == 0 ? &map_q : (c.t == 1 ? &map_k : &map_v), mb, bg.x0, bg.y0, bg.s0, c.h);
        }
    };
    if (first < n_tasks && lane == 0) issue(nxt, 0);
    nxt.advance();
    if (STAGES == 2) {
        if (first + stride < n_tasks && lane == 0) issue(nxt, 1);
        nxt.advance();
    }

    int it = 0;
    bool failed = false;
    for (int64_t task = first; task < n_tasks; task += stride, ++it, cur.advance(), nxt.advance()) {
        const int buf = STAGES == 2 ? (it & 1) : 0;
        const uint32_t parity = STAGES == 2 ? ((it >> 1) & 1) : (it & 1);
        const bool more = task + STAGES * stride < n_tasks;
        const int t = cur.t, h = cur.h;
        const bool special = cur.u >= a.n_blocks;
        int start, n, r, moff;
        BlockGeom bg{};
        bm.clipped = false;
        if (special) {
            start = DIRECT ? (cur.u - a.n_blocks) * a.layout.n_special : (cur.u - a.n_blocks) * 32;
            n = DIRECT ? a.layout.n_special : min(32, a.n_special_total - start);
            r = 0;
            moff = start;
        } else {
            if (DIRECT) {
                bg = a.geom[cur.u];
                bm.set(box_f, box_h, box_w, bg.frames, bg.rows, bg.cols);
            }
            const BlockInfo bi = a.blocks[cur.u];
            start = bi.start;
            n = bi.n;
            r = t == 0 ? bi.r_q : bi.r_k;
            moff = t == 0 ? bi.moff_q : bi.moff_k;
        }
        const int m_len = t == 0 ? a.m_q : a.m_k;
        uint32_t* out = reinterpret_cast<uint32_t*>(a.merged[t] + ((int64_t)h * m_len + moff) * kHeadDim);   // 32 words per row
        const uint32_t blk = stage0 + buf * STAGE_BYTES;

        // the map entries do not depend on the staged rows: fetch them before waiting
        // stage row lane + 32 p holds token tok[p] of the block (-1: none), merged into the token in stage ROW rep[p]
        int rep[PASSES], tok[PASSES];
#pragma unroll
        for (int p = 0; p < PASSES; ++p) {
            const int rho = lane + 32 * p;
            tok[p] = !DIRECT || special ? (rho < n ? rho : -1)
                                        : ((own_t[p] < bg.frames && own_y[p] < bg.rows && own_x[p] < bg.cols) ? (own_t[p] * bg.rows + own_y[p]) * bg.cols + own_x[p] : -1);
            rep[p] = -1;
            if (r > 0 && tok[p] >= 0) {
                rep[p] = __ldg(a.assign[t == 0 ? 0 : 1] + (int64_t)h * a.n_tokens + start + tok[p]) - start;
                if (rep[p] < 0 || rep[p] >= n) {   // corrupt map: record, treat as kept
                    atomicCAS(a.status, kDevOk, kDevBadIndex);
                    rep[p] = tok[p];
                }
                if (DIRECT) rep[p] = bm.row_of_token(rep[p]);
            }
        }
        if (!mbar_wait_bounded(mbar0 + 8 * buf, parity, a.status, kDevTimeoutMatchLoad)) {
            failed = true;
            break;
        }
        if (r == 0) {   // nothing merges here: copy the rows, 16 bytes per lane (chunk c of row j sits at c ^ (j & 7))
            const unsigned char* sb = stage + buf * STAGE_BYTES;
            uint4* o4 = reinterpret_cast<uint4*>(out);
            for (int q = lane; q < n * 8; q += 32) {
                const int row = DIRECT ? bm.row_of_token(q >> 3) : q >> 3, ch = q & 7;
                o4[q] = *reinterpret_cast<const uint4*>(sb + row * kRowBytes + ((ch ^ (row & 7)) << 4));
            }
            if (t == 0 && !special)
                for (int j = lane; j < n; j += 32) a.rank_q[(int64_t)h * a.n_tokens + start + j] = moff + j;
        } else {
            // merged row of every token: rank of its representative among the kept tokens
            unsigned kept[PASSES];
            int kept_before[PASSES], n_kept = 0;
#pragma unroll
            for (int p = 0; p < PASSES; ++p) {
                kept[p] = __ballot_sync(0xffffffffu, rep[p] == lane + 32 * p);   // rep == -1 for positions >= n
                kept_before[p] = n_kept;
                n_kept += __popc(kept[p]);
                cnt[lane + 32 * p] = 0;
            }
            __syncwarp();
            int row_of[PASSES];
#pragma unroll
            for (int p = 0; p < PASSES; ++p) {
                row_of[p] = -1;
                if (rep[p] >= 0) {
#pragma unroll
                    for (int pp = 0; pp < PASSES; ++pp)
                        if ((rep[p] >> 5) == pp) row_of[p] = kept_before[pp] + __popc(kept[pp] & ((1u << (rep[p] & 31)) - 1u));
                    atomicAdd(&cnt[row_of[p]], 1);
                    if (t == 0) a.rank_q[(int64_t)h * a.n_tokens + start + tok[p]] = moff + row_of[p];
                }
            }
            __syncwarp();
#pragma unroll
            for (int p = 0; p < PASSES; ++p)
                if (lane + 32 * p < n_kept) rcnt[lane + 32 * p] = 1.0f / (float)cnt[lane + 32 * p];
            __syncwarp();
            const int n_ks = ((DIRECT ? box_rows : n) + 15) >> 4, n_mt = (n_kept + 15) >> 4;   // stage rows that may hold tokens
            const int n_out = min(n_kept, n - r);   // (a corrupt map cannot overrun)
#pragma unroll 1
            for (int mt = 0; mt < n_mt; ++mt) {
                const int r0 = 16 * mt + g, r1 = r0 + 8;   // this lane's two accumulator rows
                float c[8][4];
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    if (ks < n_ks) {   // warp-uniform
                        // W fragment: rows of tokens 16 ks + {2 tq, 2 tq + 1, 2 tq + 8, 2 tq + 9} (held by pass ks / 2, lane 16 (ks & 1) + ..)
                        const int src = 16 * (ks & 1) + 2 * tq;
                        const int w0 = __shfl_sync(0xffffffffu, row_of[ks >> 1], src), w1 = __shfl_sync(0xffffffffu, row_of[ks >> 1], src + 1);
                        const int w2 = __shfl_sync(0xffffffffu, row_of[ks >> 1], src + 8), w3 = __shfl_sync(0xffffffffu, row_of[ks >> 1], src + 9);
                        uint32_t af[4];   // bf16 1.0 = 0x3f80
                        af[0] = (w0 == r0 ? 0x3f80u : 0u) | (w1 == r0 ? 0x3f800000u : 0u);
                        af[1] = (w0 == r1 ? 0x3f80u : 0u) | (w1 == r1 ? 0x3f800000u : 0u);
                        af[2] = (w2 == r0 ? 0x3f80u : 0u) | (w3 == r0 ? 0x3f800000u : 0u);
                        af[3] = (w2 == r1 ? 0x3f80u : 0u) | (w3 == r1 ? 0x3f800000u : 0u);
                        if (__any_sync(0xffffffffu, (af[0] | af[1] | af[2] | af[3]) != 0u)) {   // no token of this step belongs to this row tile: skip
                            const int tok = 16 * ks + (lane & 7) + ((lane >> 3) & 1) * 8;
                            const uint32_t rowaddr = blk + tok * kRowBytes;
#pragma unroll
                            for (int np = 0; np < 4; ++np) {
                                uint32_t bf[4];
                                ldmatrix_x4_trans(bf, rowaddr + (((2 * np + (lane >> 4)) ^ (tok & 7)) << 4));
                                mma_bf16_16816(c[2 * np], af, bf[0], bf[1]);
                                mma_bf16_16816(c[2 * np + 1], af, bf[2], bf[3]);
                            }
                        }
                    }
                }
                const bool s0 = r0 < n_out, s1 = r1 < n_out;
                const float i0 = s0 ? rcnt[r0] : 0.f, i1 = s1 ? rcnt[r1] : 0.f;
#pragma unroll
                for (int nt = 0; nt < 8; ++nt) {
                    if (s0) {
                        const __nv_bfloat162 o = __floats2bfloat162_rn(c[nt][0] * i0, c[nt][1] * i0);
                        out[r0 * 32 + nt * 4 + tq] = *reinterpret_cast<const uint32_t*>(&o);
                    }
                    if (s1) {
                        const __nv_bfloat162 o = __floats2bfloat162_rn(c[nt][2] * i1, c[nt][3] * i1);
                        out[r1 * 32 + nt * 4 + tq] = *reinterpret_cast<const uint32_t*>(&o);
                    }
                }
            }
        }
        __syncwarp();   // every lane is done reading this stage buffer and the per-row tables
        if (more && lane == 0) issue(nxt, buf);
    }
    if (failed) {
        mbar_wait_bounded(mbar0, STAGES == 2 ? ((it >> 1) & 1) : (it & 1), a.status, kDevTimeoutMatchLoad);
        if (STAGES == 2) mbar_wait_bounded(mbar0 + 8, (it >> 1) & 1, a.status, kDevTimeoutMatchLoad);
    }
}

template <int PASSES>
static cudaError_t launch_merge_multi(const MergeArgs& a, int sm_count, cudaStream_t stream) {
    constexpr int NMAX = 32 * PASSES;
    constexpr int WARPS = merge_multi_warps(NMAX);
    constexpr int STAGES = merge_multi_stages(NMAX);
    CUtensorMap m[3], sp[3];
    const int64_t N = a.n_tokens;
    const bool direct = a.geom != nullptr;
    for (int t = 0; t < 3; ++t) {
        if (direct) {
            if (!encode_block_map(&m[t], a.src[t], a.layout, a.heads)) return cudaErrorInvalidValue;
            if (a.layout.n_special > 0 &&
                !encode_frame_tensor_map(&sp[t], a.src[t].ptr, a.layout.tokens_per_frame, a.layout.frames, a.heads, a.src[t].stride_token,
                                         a.src[t].stride_head, a.layout.n_special))
                return cudaErrorInvalidValue;
            if (a.layout.n_special <= 0) sp[t] = m[t];   // never used
        } else {
            if (!encode_rows_tensor_map(&m[t], a.xr[t], N, a.heads, kHeadDim, N * kHeadDim, NMAX)) return cudaErrorInvalidValue;
            sp[t] = m[t];   // not used
        }
    }
    const int sp_units = direct ? (a.layout.n_special > 0 ? a.layout.frames : 0) : (a.n_special_total + 31) / 32;
    const int64_t n_tasks = 3ll * a.heads * (a.n_blocks + sp_units);
    int64_t grid = (n_tasks + WARPS - 1) / WARPS;
    if (grid > sm_count) grid = sm_count;
    if (grid < 1) grid = 1;
    if (direct)
        merge_multi_kernel<PASSES, true><<<(unsigned)grid, WARPS * 32, merge_multi_smem(NMAX), stream>>>(m[0], m[1], m[2], sp[0], sp[1], sp[2], a);
    else
        merge_multi_kernel<PASSES, false><<<(unsigned)grid, WARPS * 32, merge_multi_smem(NMAX), stream>>>(m[0], m[1], m[2], sp[0], sp[1], sp[2], a);
    return cudaGetLastError();
}

cudaError_t launch_merge(const MergeArgs& a, int max_block_tokens, int sm_count, cudaStream_t stream) {
    if (max_block_tokens <= 32) return launch_merge_tc(a, sm_count, stream);
    if (max_block_tokens <= 64) return launch_merge_multi<2>(a, sm_count, stream);
    if (max_block_tokens <= 128) return launch_merge_multi<4>(a, sm_count, stream);
    return launch_merge_multi<8>(a, sm_count, stream);
}

// ------------------------------------------------------------------------------------
// Adaptive outlier filtering for the query tokens (Sec. 3.4, Algorithm 2), blocks of at most 32 tokens.
//   deviation_kernel   eps[h][p] = || q_p - mean of the group p was merged into ||_2 (0 for a group of one)
//   threshold_kernel   tau = the (K+1)-th largest eps over all heads (K = the global budget): radix select
//   filter_kernel      outliers (eps > tau) leave their groups; the map is rewritten, the kept tokens of
//                      every (head, block) are counted
//   offsets_kernel     per head: merged row of every block's first kept token (prefix sum over the blocks),
//                      merged length, and the head's first 128-row query tile (for the attention kernel)
// ------------------------------------------------------------------------------------
__device__ void finish_level(const OutlierArgs& a, int level, int* hist);   // (threshold selection, below)
constexpr int kDevWarps = 6;     // 6 x 16.2 KB of shared memory: two CTAs per SM
constexpr int kDevStages = 3;    // block loads in flight per warp (the kernel is bound by bytes in flight)
constexpr int kCentStride = 65;  // floats per mean: odd, so that reads of different means spread over the banks
constexpr int kDevAux = 16 * kCentStride * 4 + 16 * 4 + 32;   // means of the groups of two or more (at most 16 in 32 tokens), reciprocal sizes, mbarriers
constexpr int kDevSmem = kDevWarps * (kDevStages * 32 * kRowBytes + kDevAux) + 2048 * 4 /*histogram*/ + 1024 /*alignment slack*/;

__global__ void __launch_bounds__(kDevWarps * 32, 2)
deviation_kernel(const __grid_constant__ CUtensorMap map_q, const OutlierArgs a) {
    constexpr uint32_t STAGE_BYTES = 32 * kRowBytes;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, tq = lane & 3;   // MMA accumulator layout: rows g, g + 8; columns 2 tq, 2 tq + 1
    unsigned char* stage = smem + (size_t)warp * kDevStages * STAGE_BYTES;
    unsigned char* aux = smem + (size_t)kDevWarps * kDevStages * STAGE_BYTES + (size_t)warp * kDevAux;
    float* cent = reinterpret_cast<float*>(aux);                   // [16][65] group means
    float* rcnt = cent + 16 * kCentStride;                         // [16] 1 / group size
    int* hist = reinterpret_cast<int*>(smem + (size_t)kDevWarps * (kDevStages * STAGE_BYTES + kDevAux));   // [2048] bits 31-21 of this CTA's deviations
    for (int i = threadIdx.x; i < 2048; i += kDevWarps * 32) hist[i] = 0;
    __syncthreads();
    const uint32_t mbar0 = smem_u32(aux + 16 * kCentStride * 4 + 16 * 4), stage0 = smem_u32(stage);
    if (lane == 0) {
        for (int st = 0; st < kDevStages; ++st) mbar_init(mbar0 + 8 * st, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();
    const SourceLayout& L = a.layout;
    const int box_f = min(L.blk_frames, L.frames), box_h = min(L.blk_h, L.grid_h), box_w = min(L.blk_w, L.grid_w);
    const int box_rows = box_f * box_h * box_w;
    const int own_t = lane / (box_h * box_w), own_y = (lane / box_w) % box_h, own_x = lane % box_w;
    for (int q = box_rows * 8 + lane; q < 32 * 8; q += 32)   // rows no load ever writes enter the MMAs with weight 0: keep them finite
        for (int st = 0; st < kDevStages; ++st) *reinterpret_cast<uint4*>(stage + st * STAGE_BYTES + q * 16) = make_uint4(0u, 0u, 0u, 0u);
    __syncwarp();
    BoxMap bm;
    bm.clipped = false;

    const int64_t n_tasks = (int64_t)a.heads * a.n_blocks;   // (head, block), queries only
    const int64_t stride = (int64_t)gridDim.x * kDevWarps;
    const int64_t first = (int64_t)blockIdx.x * kDevWarps + warp;
    TaskCursor cur, nxt;
    cur.init(first, stride, a.heads, a.n_blocks);   // one "tensor": t stays 0 while the task index is in range
    nxt = cur;
    auto issue = [&](const TaskCursor& c, int buf) {   // lane 0 only
        const BlockGeom bg = a.geom[c.u];
        const uint32_t mb = mbar0 + 8 * buf;
        mbar_expect_tx(mb, (uint32_t)box_rows * kRowBytes);
        tma_block_load(stage0 + buf * STAGE_BYTES, &map_q, mb, bg.x0, bg.y0, bg.s0, c.h);
    };
#pragma unroll
    for (int st = 0; st < kDevStages; ++st) {
        if (first + st * stride < n_tasks && lane == 0) issue(nxt, st);
        nxt.advance();
    }

    int buf = 0;
    uint32_t parity = 0;
    bool failed = false;
    for (int64_t task = first; task < n_tasks; task += stride, cur.advance(), nxt.advance()) {
        const bool more = task + kDevStages * stride < n_tasks;
        const int h = cur.h;
        const BlockInfo bi = a.blocks[cur.u];
        const BlockGeom bg = a.geom[cur.u];
        bm.set(box_f, box_h, box_w, bg.frames, bg.rows, bg.cols);
        const int n = bi.n, r = bi.r_q;
        const int tok = (own_t < bg.frames && own_y < bg.rows && own_x < bg.cols) ? (own_t * bg.rows + own_y) * bg.cols + own_x : -1;
        float* eps = a.eps + (int64_t)h * a.n_tokens + bi.start;
        int rep = -1;   // stage ROW of the token this lane's token was merged into
        if (r > 0 && tok >= 0) {
            rep = __ldg(a.assign_q + (int64_t)h * a.n_tokens + bi.start + tok) - bi.start;
            if (rep < 0 || rep >= n) {
                atomicCAS(a.status, kDevOk, kDevBadIndex);
                rep = tok;
            }
            rep = bm.row_of_token(rep);
        }
        if (!mbar_wait_bounded(mbar0 + 8 * buf, parity, a.status, kDevTimeoutMatchLoad)) {
            failed = true;
            break;
        }
        if (r == 0) {   // nothing merged in this block: every deviation is 0
            if (tok >= 0) eps[tok] = 0.f;
        } else {
            const uint32_t blk = stage0 + buf * STAGE_BYTES;
            // groups of two or more tokens get a mean; row of the mean = rank of the group's representative among them
            const unsigned group = __match_any_sync(0xffffffffu, rep);   // (lanes without a token share rep = -1: ignored below)
            const int group_size = rep >= 0 ? __popc(group) : 0;
            const unsigned multi = __ballot_sync(0xffffffffu, rep == lane && group_size >= 2);
            const int row_of = group_size >= 2 ? __popc(multi & ((1u << rep) - 1u)) : -1;
            if (rep == lane && group_size >= 2) rcnt[row_of] = 1.0f / (float)group_size;
            // group sums = W x on the tensor cores, as in merge_tc_kernel: W [16 means][32 tokens] of zeros and ones
            uint32_t bf[2][4][4];
            const int n_ks = box_rows > 16 ? 2 : 1;
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                if (ks < n_ks) {
                    const int row = 16 * ks + (lane & 7) + ((lane >> 3) & 1) * 8;
                    const uint32_t rowaddr = blk + row * kRowBytes;
#pragma unroll
                    for (int np = 0; np < 4; ++np) ldmatrix_x4_trans(bf[ks][np], rowaddr + (((2 * np + (lane >> 4)) ^ (row & 7)) << 4));
                }
            }
            float c[8][4];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
            const int r0 = g, r1 = g + 8;
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {
                if (ks < n_ks) {
                    const int w0 = __shfl_sync(0xffffffffu, row_of, 16 * ks + 2 * tq), w1 = __shfl_sync(0xffffffffu, row_of, 16 * ks + 2 * tq + 1);
                    const int w2 = __shfl_sync(0xffffffffu, row_of, 16 * ks + 2 * tq + 8), w3 = __shfl_sync(0xffffffffu, row_of, 16 * ks + 2 * tq + 9);
                    uint32_t af[4];
                    af[0] = (w0 == r0 ? 0x3f80u : 0u) | (w1 == r0 ? 0x3f800000u : 0u);
                    af[1] = (w0 == r1 ? 0x3f80u : 0u) | (w1 == r1 ? 0x3f800000u : 0u);
                    af[2] = (w2 == r0 ? 0x3f80u : 0u) | (w3 == r0 ? 0x3f800000u : 0u);
                    af[3] = (w2 == r1 ? 0x3f80u : 0u) | (w3 == r1 ? 0x3f800000u : 0u);
#pragma unroll
                    for (int nt = 0; nt < 8; ++nt) mma_bf16_16816(c[nt], af, bf[ks][nt >> 1][2 * (nt & 1)], bf[ks][nt >> 1][2 * (nt & 1) + 1]);
                }
            }
            __syncwarp();   // reciprocal group sizes visible
            const int n_cent = __popc(multi);
            const float i0 = r0 < n_cent ? rcnt[r0] : 0.f, i1 = r1 < n_cent ? rcnt[r1] : 0.f;
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {   // the means stay in fp32 (no rounding to bf16 before the distance)
                if (r0 < n_cent) {
                    cent[r0 * kCentStride + nt * 8 + 2 * tq] = c[nt][0] * i0;
                    cent[r0 * kCentStride + nt * 8 + 2 * tq + 1] = c[nt][1] * i0;
                }
                if (r1 < n_cent) {
                    cent[r1 * kCentStride + nt * 8 + 2 * tq] = c[nt][2] * i1;
                    cent[r1 * kCentStride + nt * 8 + 2 * tq + 1] = c[nt][3] * i1;
                }
            }
            __syncwarp();   // means visible
            float dev = 0.f;
            if (tok >= 0) {
                float d2 = 0.f;
                if (row_of >= 0) {   // distance of this lane's token (stage row `lane`) to its group's mean
                    const unsigned char* row = stage + buf * STAGE_BYTES + lane * kRowBytes;
                    const float* cr = cent + row_of * kCentStride;
#pragma unroll
                    for (int ch = 0; ch < 8; ++ch) {
                        float x[8];
                        unpack8(*reinterpret_cast<const uint4*>(row + ((ch ^ (lane & 7)) << 4)), x);
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const float d = x[e] - cr[ch * 8 + e];
                            d2 = fmaf(d, d, d2);
                        }
                    }
                }
                dev = sqrtf(d2);
                eps[tok] = dev;
            }
            // level 0 of the threshold selection: histogram of the top 11 bits (zeros are not counted), one atomic per distinct bin
            const int bin = (int)(__float_as_uint(dev) >> 21);
            const unsigned peers = __match_any_sync(0xffffffffu, bin);
            if (bin > 0 && lane == __ffs(peers) - 1) atomicAdd(&hist[bin], __popc(peers));
        }
        __syncwarp();   // every lane is done with the stage and the tables
        if (more && lane == 0) issue(nxt, buf);
        if (++buf == kDevStages) {
            buf = 0;
            parity ^= 1u;
        }
    }
    if (failed) {   // give copies that may still be in flight a bounded chance to land before the shared memory is released
        for (int st = 0; st < kDevStages; ++st) {
            mbar_wait_bounded(mbar0 + 8 * st, parity, a.status, kDevTimeoutMatchLoad);
            mbar_wait_bounded(mbar0 + 8 * st, parity ^ 1u, a.status, kDevTimeoutMatchLoad);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 2048; i += kDevWarps * 32) {
        const int c = hist[i];
        if (c) atomicAdd(a.sel + kSelHist + i, c);
    }
    finish_level(a, 0, hist);
}

// ---- tau = the (K+1)-th largest deviation over all heads (K = the budget): radix select on the bit patterns of the
// non-negative floats (they order like the values), 11 + 11 + 10 bits.  Level 0's histogram is built by the
// deviation kernel while it writes the deviations; two refinement kernels rescan them (2 MB, resident in L2) for the
// elements inside the prefix chosen so far.  In each kernel the CTA that finishes last walks the histogram down from
// the largest bin until the remaining rank falls inside one, and leaves prefix and rank for the next level.
// Zeros are never counted at level 0: the walk ends in bin 0 whatever it holds.

// One warp: bin and remaining rank for histogram h[nb] (shared memory), as the sequential walk
//   above = 0; for (bin = nb - 1; bin > 0 && above + h[bin] <= rank; --bin) above += h[bin];  rank -= above
__device__ __forceinline__ void select_bin(const int* h, int nb, int rank, int* bin_out, int* rank_out) {
    const int lane = threadIdx.x & 31, per = nb >> 5, lo = lane * per;
    int c = 0;
    for (int i = 0; i < per; ++i) c += h[lo + i];
    if (lane == 0) c -= h[0];   // bin 0 ends the walk: it is never added
    int incl = c;               // this lane's bins and all higher ones
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int o = __shfl_down_sync(0xffffffffu, incl, off);
        if (lane + off < 32) incl += o;
    }
    const unsigned hit = __ballot_sync(0xffffffffu, incl > rank);
    if (hit == 0) {             // fewer than rank + 1 elements above bin 0
        if (lane == 0) {
            *bin_out = 0;
            *rank_out = rank - incl;
        }
        return;
    }
    if (lane == 31 - __clz(hit)) {   // the walk stops inside this lane's bins
        int above = incl - c, b = lo + per - 1;
        for (; b > lo; --b) {
            if (above + h[b] > rank) break;
            above += h[b];
        }
        *bin_out = b;
        *rank_out = rank - above;
    }
}

// The bin of one level from its complete histogram (one CTA; hist: 2048 ints of shared memory).
__device__ void select_level(const OutlierArgs& a, int level, int* hist) {
    __shared__ int s_bin, s_rank;
    const int64_t count = a.total_count;
    if (level == 0 && (a.budget <= 0 || a.budget >= count)) {   // nothing is an outlier (tau = +inf) / everything is (tau = -1)
        if (threadIdx.x == 0) {
            *a.tau = a.budget <= 0 ? INFINITY : -1.0f;
            a.sel[kSelFinished] = 1;
        }
        return;
    }
    if (level > 0 && __ldcg(a.sel + kSelFinished)) return;
    const int nb = level == 2 ? 1024 : 2048, shift = level == 0 ? 21 : (level == 1 ? 10 : 0);
    for (int i = threadIdx.x; i < nb; i += blockDim.x) hist[i] = __ldcg(a.sel + kSelHist + level * 2048 + i);
    __syncthreads();
    if (threadIdx.x < 32) {
        const int rank = level == 0 ? (int)a.budget : __ldcg(a.sel + kSelRank + level - 1);
        select_bin(hist, nb, rank, &s_bin, &s_rank);
        __syncwarp();
        if (threadIdx.x == 0) {
            const uint32_t prefix = (level == 0 ? 0u : (uint32_t)__ldcg(a.sel + kSelPrefix + level - 1)) | ((uint32_t)s_bin << shift);
            if (level < 2) {
                a.sel[kSelPrefix + level] = (int)prefix;
                a.sel[kSelRank + level] = s_rank;
            } else {
                *a.tau = __uint_as_float(prefix);
            }
        }
    }
}

// End of a level, called by every thread of every CTA after the CTA's histogram has been added to the global one:
// the CTA that arrives last selects the bin - unless the selection is deferred (head-sharded layers: the histograms
// of the other shards are still to be added; select_level_kernel runs behind the exchange).
__device__ void finish_level(const OutlierArgs& a, int level, int* hist) {
    __shared__ int s_last;
    if (a.defer_select) return;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        s_last = atomicAdd(a.sel + kSelDone + level, 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    select_level(a, level, hist);
}
__global__ void __launch_bounds__(256) select_level_kernel(const OutlierArgs a, int level) {
    __shared__ int hist[2048];
    select_level(a, level, hist);
}

constexpr int kRefineThreads = 256;
// LEVEL 1: histogram of bits 20-10 of the deviations whose bits 31-21 equal the level-0 choice; LEVEL 2: of bits 9-0
// of those whose bits 31-10 equal the choice so far.  LEVEL 0 (only where the deviation kernel does not build it on the
// fly: the large-block path): histogram of bits 31-21 of all deviations.
template <int LEVEL>
__global__ void __launch_bounds__(kRefineThreads) refine_kernel(const OutlierArgs a) {
    __shared__ int hist[2048];
    if (__ldcg(a.sel + kSelFinished)) return;   // (same answer in every thread of every CTA)
    constexpr int NB = LEVEL == 2 ? 1024 : 2048, SHIFT = LEVEL == 0 ? 21 : (LEVEL == 1 ? 10 : 0);
    constexpr uint32_t MASK = LEVEL == 0 ? 0u : (LEVEL == 1 ? 0xffe00000u : 0xfffffc00u);
    for (int i = threadIdx.x; i < NB; i += kRefineThreads) hist[i] = 0;
    __syncthreads();
    const uint32_t prefix = LEVEL == 0 ? 0u : (uint32_t)__ldcg(a.sel + kSelPrefix + (LEVEL > 0 ? LEVEL - 1 : 0));
    const int64_t count = (int64_t)a.heads * a.n_tokens, quads = count >> 2;
    const uint4* bits4 = reinterpret_cast<const uint4*>(a.eps);   // (the array comes from cudaMalloc: 16-byte aligned)
    auto tally = [&](uint32_t b) {
        if ((b & MASK) == prefix) atomicAdd(&hist[(b >> SHIFT) & (NB - 1)], 1);
    };
    for (int64_t i = (int64_t)blockIdx.x * kRefineThreads + threadIdx.x; i < quads; i += (int64_t)gridDim.x * kRefineThreads) {
        const uint4 b = __ldg(bits4 + i);
        tally(b.x);
        tally(b.y);
        tally(b.z);
        tally(b.w);
    }
    if (blockIdx.x == 0 && threadIdx.x < (int)(count & 3)) tally(__float_as_uint(a.eps[(quads << 2) + threadIdx.x]));
    __syncthreads();
    for (int i = threadIdx.x; i < NB; i += kRefineThreads) {
        const int c = hist[i];
        if (c) atomicAdd(a.sel + kSelHist + LEVEL * 2048 + i, c);
    }
    finish_level(a, LEVEL, hist);
}

// Outliers leave their groups (Sec. 3.4 item 4): one warp per (head, block), lane = token of the block.
// An outlier maps to itself; the other tokens of a group stay together, under their old representative if
// that is not an outlier, else under the remaining member with the lowest position.
__global__ void __launch_bounds__(256) filter_kernel(const OutlierArgs a) {
    const int lane = threadIdx.x & 31;
    const int64_t task = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (task >= (int64_t)a.heads * a.n_blocks) return;
    const int h = (int)(task / a.n_blocks), b = (int)(task - (int64_t)h * a.n_blocks);
    const BlockInfo bi = a.blocks[b];
    const int n = bi.n;
    const float tau = *a.tau;
    const int32_t* A = a.assign_q + (int64_t)h * a.n_tokens + bi.start;
    int32_t* A_out = a.assign_q_out + (int64_t)h * a.n_tokens + bi.start;
    int rep = -1 - lane;   // lanes without a token match nobody
    bool outl = false;
    if (lane < n) {
        rep = A[lane] - bi.start;
        if (rep < 0 || rep >= n) {
            atomicCAS(a.status, kDevOk, kDevBadIndex);
            rep = lane;
        }
        outl = a.eps[(int64_t)h * a.n_tokens + bi.start + lane] > tau;
    }
    const unsigned out_mask = __ballot_sync(0xffffffffu, outl);
    const unsigned group = __match_any_sync(0xffffffffu, rep);
    int now = lane;
    if (lane < n && !outl) now = ((out_mask >> rep) & 1u) ? __ffs(group & ~out_mask) - 1 : rep;
    const unsigned kept = __ballot_sync(0xffffffffu, lane < n && now == lane);
    if (lane < n) A_out[lane] = bi.start + now;
    if (lane == 0) {
        a.kept_cnt[(int64_t)h * a.n_blocks + b] = __popc(kept);
        if (out_mask) atomicAdd(a.sel + kSelOutliers, __popc(out_mask));
    }
}

// Per head (one CTA each): merged row of every block's first kept token = specials + exclusive prefix sum of the kept
// counts, and the merged length.  The CTA that finishes last builds, over the heads, the index of each head's first
// 128-row query tile (for the attention kernel).
constexpr int kOffsetsThreads = 1024;
__global__ void __launch_bounds__(kOffsetsThreads, 1) offsets_kernel(const OutlierArgs a) {
    __shared__ int warp_sum[32];
    __shared__ int s_last;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, h = blockIdx.x;
    const int32_t* cnt = a.kept_cnt + (int64_t)h * a.n_blocks;
    int32_t* moff = a.moff_var + (int64_t)h * a.n_blocks;
    int running = a.n_special_total;
    for (int b0 = 0; b0 < a.n_blocks; b0 += kOffsetsThreads) {
        const int b = b0 + threadIdx.x;
        const int c = b < a.n_blocks ? cnt[b] : 0;
        int incl = c;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int o = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += o;
        }
        if (lane == 31) warp_sum[warp] = incl;
        __syncthreads();
        if (warp == 0) {   // inclusive scan of the 32 warp totals
            int w = warp_sum[lane];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int o = __shfl_up_sync(0xffffffffu, w, off);
                if (lane >= off) w += o;
            }
            warp_sum[lane] = w;
        }
        __syncthreads();
        if (b < a.n_blocks) moff[b] = running + (warp > 0 ? warp_sum[warp - 1] : 0) + incl - c;
        running += warp_sum[31];
        __syncthreads();   // the totals are read before the next chunk overwrites them
    }
    if (threadIdx.x == 0) {
        a.mq_head[h] = running;
        __threadfence();
        s_last = atomicAdd(a.sel + kSelOffsetsDone, 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (s_last && threadIdx.x == 0) {
        __threadfence();
        int t = 0;
        for (int hh = 0; hh < a.heads; ++hh) {
            a.tile_prefix[hh] = t;
            t += (__ldcg(a.mq_head + hh) + 127) / 128;
        }
        a.tile_prefix[a.heads] = t;
    }
}

cudaError_t launch_deviation(const OutlierArgs& a, int sm_count, cudaStream_t stream) {
    CUtensorMap mq;
    if (!encode_block_map(&mq, a.src_q, a.layout, a.heads)) return cudaErrorInvalidValue;
    const int64_t n_tasks = (int64_t)a.heads * a.n_blocks;
    int64_t grid = (n_tasks + kDevWarps - 1) / kDevWarps;
    if (grid > 2ll * sm_count) grid = 2ll * sm_count;
    if (grid < 1) grid = 1;
    deviation_kernel<<<(unsigned)grid, kDevWarps * 32, kDevSmem, stream>>>(mq, a);
    return cudaGetLastError();
}
cudaError_t launch_threshold(const OutlierArgs& a, int sm_count, cudaStream_t stream) {
    const int64_t quads = ((int64_t)a.heads * a.n_tokens) >> 2;
    int64_t grid = (quads + kRefineThreads * 4 - 1) / (kRefineThreads * 4);   // about four 16-byte loads per thread
    if (grid > 2ll * sm_count) grid = 2ll * sm_count;
    if (grid < 1) grid = 1;
    refine_kernel<1><<<(unsigned)grid, kRefineThreads, 0, stream>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    refine_kernel<2><<<(unsigned)grid, kRefineThreads, 0, stream>>>(a);
    return cudaGetLastError();
}
cudaError_t launch_threshold0(const OutlierArgs& a, int sm_count, cudaStream_t stream) {
    const int64_t quads = ((int64_t)a.heads * a.n_tokens) >> 2;
    int64_t grid = (quads + kRefineThreads * 4 - 1) / (kRefineThreads * 4);
    if (grid > 2ll * sm_count) grid = 2ll * sm_count;
    if (grid < 1) grid = 1;
    refine_kernel<0><<<(unsigned)grid, kRefineThreads, 0, stream>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_threshold(a, sm_count, stream);
}
cudaError_t launch_refine_level(const OutlierArgs& a, int level, int sm_count, cudaStream_t stream) {
    const int64_t quads = ((int64_t)a.heads * a.n_tokens) >> 2;
    int64_t grid = (quads + kRefineThreads * 4 - 1) / (kRefineThreads * 4);
    if (grid > 2ll * sm_count) grid = 2ll * sm_count;
    if (grid < 1) grid = 1;
    if (level == 0)
        refine_kernel<0><<<(unsigned)grid, kRefineThreads, 0, stream>>>(a);
    else if (level == 1)
        refine_kernel<1><<<(unsigned)grid, kRefineThreads, 0, stream>>>(a);
    else
        refine_kernel<2><<<(unsigned)grid, kRefineThreads, 0, stream>>>(a);
    return cudaGetLastError();
}
cudaError_t launch_select_level(const OutlierArgs& a, int level, cudaStream_t stream) {
    select_level_kernel<<<1, 256, 0, stream>>>(a, level);
    return cudaGetLastError();
}
cudaError_t launch_offsets(const OutlierArgs& a, cudaStream_t stream) {
    offsets_kernel<<<(unsigned)a.heads, kOffsetsThreads, 0, stream>>>(a);
    return cudaGetLastError();
}
cudaError_t launch_filter(const OutlierArgs& a, cudaStream_t stream) {
    const int64_t threads = (int64_t)a.heads * a.n_blocks * 32;
    filter_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, stream>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return launch_offsets(a, stream);
}

// ------------------------------------------------------------------------------------
// a5. Head-wise unmerge + inverse reorder + head concat (Eq. 5-7): every original token
//     copies the attention output of the merged query token it went into.
//     8 threads move one 128-byte (token, head) row.  A CTA works on one head and 128
//     consecutive original tokens: the map reads of neighbouring tokens share sectors and
//     the merged rows they point to are close together.  Each thread carries four rows at
//     a time so that four independent load chains are in flight.
// ------------------------------------------------------------------------------------
constexpr int kUnmergeThreads = 256;
constexpr int kUnmergeUnroll = 4;
constexpr int kUnmergeTokensPerCta = (kUnmergeThreads / 8) * kUnmergeUnroll;

__global__ void __launch_bounds__(kUnmergeThreads) unmerge_kernel(const __grid_constant__ UnmergeArgs a) {
    const int h = blockIdx.y;
    const int chunk = threadIdx.x & 7, slot = threadIdx.x >> 3;
    const int base = blockIdx.x * kUnmergeTokensPerCta;
    const int32_t* rank = a.rank_q + (int64_t)h * a.n_tokens;
    const uint4* om = reinterpret_cast<const uint4*>(a.o_m + (int64_t)h * a.m_q * kHeadDim) + chunk;
    __nv_bfloat16* out = a.out + (int64_t)h * a.out_stride_head + chunk * 8;
    int p[kUnmergeUnroll], row[kUnmergeUnroll];
    uint4 v[kUnmergeUnroll];
#pragma unroll
    for (int u = 0; u < kUnmergeUnroll; ++u) {
        const int i = base + u * (kUnmergeThreads / 8) + slot;
        p[u] = i < a.n_tokens ? __ldg(a.pi_inv + i) : 0;
    }
#pragma unroll
    for (int u = 0; u < kUnmergeUnroll; ++u) row[u] = __ldg(rank + p[u]);
#pragma unroll
    for (int u = 0; u < kUnmergeUnroll; ++u) {
        if (row[u] < 0 || row[u] >= a.m_q) {   // corrupt map: record, copy row 0 instead of reading out of range
            atomicCAS(a.status, kDevOk, kDevBadIndex);
            row[u] = 0;
        }
        v[u] = __ldg(om + (int64_t)row[u] * 8);
    }
#pragma unroll
    for (int u = 0; u < kUnmergeUnroll; ++u) {
        const int i = base + u * (kUnmergeThreads / 8) + slot;
        if (i < a.n_tokens) *reinterpret_cast<uint4*>(out + (int64_t)i * a.out_stride_token) = v[u];
    }
}

cudaError_t launch_unmerge(const UnmergeArgs& a, cudaStream_t stream) {
    dim3 grid((a.n_tokens + kUnmergeTokensPerCta - 1) / kUnmergeTokensPerCta, a.heads);
    unmerge_kernel<<<grid, kUnmergeThreads, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t configure_kernels() {
    cudaError_t e;
#define HTTM_SET_SMEM(kern, bytes)                                                                      \
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(bytes));          \
    if (e != cudaSuccess) return e;
    HTTM_SET_SMEM((match_kernel<1, false>), match_smem_bytes(32));
    HTTM_SET_SMEM((match_kernel<1, true>), match_smem_bytes(32));
    HTTM_SET_SMEM((match_kernel<2, false>), match_smem_bytes(64));
    HTTM_SET_SMEM((match_kernel<2, true>), match_smem_bytes(64));
    HTTM_SET_SMEM((match_kernel<4, true>), match_smem_bytes(128));
    HTTM_SET_SMEM((match_kernel<8, true>), match_smem_bytes(256));
    HTTM_SET_SMEM((match_kernel<4, false>), match_smem_bytes(128));
    HTTM_SET_SMEM((match_kernel<8, false>), match_smem_bytes(256));
    HTTM_SET_SMEM(deviation_kernel, kDevSmem);
    HTTM_SET_SMEM(merge_tc_kernel<false>, kMergeTcSmem);
    HTTM_SET_SMEM(merge_tc_kernel<true>, kMergeTcSmem);
    HTTM_SET_SMEM((merge_multi_kernel<2, false>), merge_multi_smem(64));
    HTTM_SET_SMEM((merge_multi_kernel<4, false>), merge_multi_smem(128));
    HTTM_SET_SMEM((merge_multi_kernel<8, false>), merge_multi_smem(256));
    HTTM_SET_SMEM((merge_multi_kernel<2, true>), merge_multi_smem(64));
    HTTM_SET_SMEM((merge_multi_kernel<4, true>), merge_multi_smem(128));
    HTTM_SET_SMEM((merge_multi_kernel<8, true>), merge_multi_smem(256));
#undef HTTM_SET_SMEM
    return configure_attention();
}

}  // namespace httm
