// HBM-bound kernels of the HTTM path: temporal reorder (gather), per-(head, block)
// cosine matching, mean merge, and unmerge + inverse reorder.  sm_100a only.
#include "httm_internal.h"
#include "tc_sm100.cuh"   // tensor-map encoder (host)

namespace httm {

// ------------------------------------------------------------------------------------
// small device helpers
// ------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(uint32_t mbar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t mbar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t mbar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(mbar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after about two seconds, records `code` in the status word and
// returns false.  Never spins forever.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t mbar, uint32_t parity, int32_t* status, int code) {
    if (mbar_try_wait(mbar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(mbar, parity)) return true;
        if (global_timer_ns() - t0 > 2000000000ull) {
            atomicCAS(status, kDevOk, code);
            return false;
        }
    }
}
// TMA bulk copy global -> this CTA's shared memory, completion on an mbarrier.
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void* src, uint32_t bytes, uint32_t mbar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
                 "l"(src), "r"(bytes), "r"(mbar)
                 : "memory");
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
        if (p < a.n_tokens) v[u] = __ldg(reinterpret_cast<const uint4*>(src + (int64_t)__ldg(a.pi + p) * st));
    }
#pragma unroll
    for (int u = 0; u < kReorderUnroll; ++u) {
        const int p = base + u * (kReorderThreads / 8) + slot;
        if (p < a.n_tokens) *reinterpret_cast<uint4*>(dst + (int64_t)p * kHeadDim) = v[u];
    }
}

cudaError_t launch_reorder(const ReorderArgs& a, cudaStream_t stream) {
    dim3 grid((a.n_tokens + kReorderTokensPerCta - 1) / kReorderTokensPerCta, a.heads, 3);
    reorder_kernel<<<grid, kReorderThreads, 0, stream>>>(a);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------
// a2. Block-wise bipartite matching (Eq. 1; Sec. 3.2 top-r rule), one warp per
//     (tensor in {Q, K}, head, block).  The block (n x 64 bf16, contiguous after the
//     reorder) is staged in shared memory by a tiled TMA load with the 128-byte swizzle,
//     double buffered per warp, so that lane j reads its own row j without bank conflicts.
//     Every lane keeps its row in registers as fp32; the dst rows are written once, as fp32,
//     to a small per-warp table that all src lanes then read with broadcast loads.
//     Similarities are fp32 dot products of the raw bf16 values (products are exact; two
//     per instruction with packed fp32 FMAs) scaled by the inverse norms.
//     argmax ties -> lowest dst; top-r ties -> lowest src.  The r merged src are found by
//     min(r, n_src - r) rounds of a warp-wide max (or min) extraction.
// ------------------------------------------------------------------------------------
constexpr int kDstRowFloats = 68;   // 64 channels + inverse norm + local position + 2 pad (272 B: conflict-free row stores)

__host__ __device__ constexpr int match_warps_per_cta(int nmax) { return nmax <= 32 ? 8 : (nmax <= 128 ? 4 : 2); }
__host__ __device__ constexpr int match_aux_bytes(int nmax) { return (nmax / 4) * kDstRowFloats * 4 + 16; }
__host__ __device__ constexpr int match_smem_bytes(int nmax) {
    return match_warps_per_cta(nmax) * (2 * nmax * kRowBytes + match_aux_bytes(nmax)) + 1024 /*alignment slack*/;
}

__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\tmov.b64 rc, {%6, %7};\n\t"
        "fma.rn.f32x2 rd, ra, rb, rc;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}
// tiled TMA load {64 channels, rows, heads} -> this CTA's shared memory; the channel coordinate is 0
__device__ __forceinline__ void tma_rows_load(uint32_t dst_smem, const CUtensorMap* map, uint32_t mbar, int row, int head) {
    asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(
                     dst_smem),
                 "l"(reinterpret_cast<uint64_t>(map)), "r"(mbar), "r"(0), "r"(row), "r"(head)
                 : "memory");
}
// monotone map float -> uint32 (larger float <-> larger key); every real score maps to a key >= 1
__device__ __forceinline__ uint32_t score_key(float s) {
    const uint32_t b = __float_as_uint(s);
    return b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
}

template <int PASSES>
__global__ void __launch_bounds__(match_warps_per_cta(32 * PASSES) * 32)
match_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k, const MatchArgs a) {
    constexpr int NMAX = 32 * PASSES;
    constexpr int WARPS = match_warps_per_cta(NMAX);
    constexpr uint32_t STAGE_BYTES = NMAX * kRowBytes;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned char* stage = smem + (size_t)warp * 2 * STAGE_BYTES;                                     // [2][NMAX][128], 1024-aligned
    unsigned char* aux = smem + (size_t)WARPS * 2 * STAGE_BYTES + (size_t)warp * match_aux_bytes(NMAX);
    float* dstf = reinterpret_cast<float*>(aux);                                                      // [NMAX/4][68]
    uint64_t* mbar = reinterpret_cast<uint64_t*>(aux + (NMAX / 4) * kDstRowFloats * 4);               // [2]
    const uint32_t mbar0 = smem_u32(mbar), stage0 = smem_u32(stage);

    if (lane == 0) {
        mbar_init(mbar0, 1);
        mbar_init(mbar0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    const int64_t per_tensor = (int64_t)a.heads * a.n_blocks;
    const int64_t n_tasks = 2 * per_tensor;
    const int64_t stride = (int64_t)gridDim.x * WARPS;
    const int64_t first = (int64_t)blockIdx.x * WARPS + warp;

    auto issue = [&](int64_t task, int buf) {   // lane 0 only; the whole box is always transferred (rows past the head's end are zero filled)
        const int t = (int)(task / per_tensor);
        const int64_t rem = task - t * per_tensor;
        const int h = (int)(rem / a.n_blocks), b = (int)(rem - (int64_t)h * a.n_blocks);
        const int start = __ldg(&a.blocks[b].start);
        const uint32_t mb = mbar0 + 8 * buf;
        mbar_expect_tx(mb, STAGE_BYTES);
        tma_rows_load(stage0 + buf * STAGE_BYTES, t == 0 ? &map_q : &map_k, mb, start, h);
    };
    if (lane == 0) {
        if (first < n_tasks) issue(first, 0);
        if (first + stride < n_tasks) issue(first + stride, 1);
    }

    // row j of a stage buffer, as 64 fp32 values in channel order (16-byte chunk c sits at c ^ (j & 7))
    auto load_row = [&](const unsigned char* blk, int j, float* x) {
        const unsigned char* row = blk + j * kRowBytes;
        const int sw = j & 7;
#pragma unroll
        for (int c = 0; c < 8; ++c) unpack8(*reinterpret_cast<const uint4*>(row + ((c ^ sw) << 4)), x + 8 * c);
    };

    int it = 0;
    bool failed = false;
    for (int64_t task = first; task < n_tasks; task += stride, ++it) {
        const int buf = it & 1;
        const uint32_t parity = (it >> 1) & 1;
        const int t = (int)(task / per_tensor);
        const int64_t rem = task - t * per_tensor;
        const int h = (int)(rem / a.n_blocks), b = (int)(rem - (int64_t)h * a.n_blocks);
        const BlockInfo bi = a.blocks[b];
        const int n = bi.n, r = t == 0 ? bi.r_q : bi.r_k, nd = t == 0 ? bi.nd_q : bi.nd_k;
        int32_t* A = a.assign[t] + (int64_t)h * a.n_tokens + bi.start;
        const unsigned char* blk = stage + buf * STAGE_BYTES;
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
            if (lane == 0 && task + 2 * stride < n_tasks) issue(task + 2 * stride, buf);
            continue;
        }
        // floor(x / n) for x < (n + 1) * nd by multiplication: exact for n <= 256, nd <= 64
        const uint32_t magic = (1u << 23) / (uint32_t)n + 1u;
        auto div_n = [&](int x) { return (int)(((uint32_t)x * magic) >> 23); };

        // ---- phase 1: norms of every token; fp32 copy of the dst rows
        float x[64];
        float inv[PASSES];
        bool is_src[PASSES];
#pragma unroll
        for (int p = 0; p < PASSES; ++p) {
            const int j = lane + 32 * p;
            inv[p] = 0.f;
            is_src[p] = false;
            if (j < n) {
                load_row(blk, j, x);
                float2 s0 = make_float2(0.f, 0.f), s1 = s0;
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    s0 = ffma2(make_float2(x[4 * k], x[4 * k + 1]), make_float2(x[4 * k], x[4 * k + 1]), s0);
                    s1 = ffma2(make_float2(x[4 * k + 2], x[4 * k + 3]), make_float2(x[4 * k + 2], x[4 * k + 3]), s1);
                }
                inv[p] = 1.0f / fmaxf(sqrtf((s0.x + s0.y) + (s1.x + s1.y)), 1e-12f);
                const int d = div_n(j * nd);
                if (div_n((j + 1) * nd) > d) {   // dst number d
                    float4* o = reinterpret_cast<float4*>(dstf + d * kDstRowFloats);
#pragma unroll
                    for (int k = 0; k < 16; ++k) o[k] = make_float4(x[4 * k], x[4 * k + 1], x[4 * k + 2], x[4 * k + 3]);
                    o[16] = make_float4(inv[p], __int_as_float(j), 0.f, 0.f);
                } else {
                    is_src[p] = true;
                }
            }
        }
        __syncwarp();
        if (PASSES == 1) {   // the row lives in registers from here on: the stage buffer can be refilled
            if (lane == 0 && task + 2 * stride < n_tasks) issue(task + 2 * stride, buf);
        }

        // ---- phase 2: best dst of every src
        uint32_t key[PASSES];
        int best[PASSES];
#pragma unroll
        for (int p = 0; p < PASSES; ++p) {
            key[p] = 0;
            best[p] = 0;
            if (p * 32 < n) {   // warp-uniform
                if (is_src[p]) {
                    if (PASSES > 1) load_row(blk, lane + 32 * p, x);
                    float top = -INFINITY;
                    int arg = 0;
                    auto dot = [&](const float4* dr) {
                        float2 c0 = make_float2(0.f, 0.f), c1 = c0;
#pragma unroll
                        for (int k = 0; k < 16; ++k) {
                            const float4 u = dr[k];
                            c0 = ffma2(make_float2(x[4 * k], x[4 * k + 1]), make_float2(u.x, u.y), c0);
                            c1 = ffma2(make_float2(x[4 * k + 2], x[4 * k + 3]), make_float2(u.z, u.w), c1);
                        }
                        return ((c0.x + c0.y) + (c1.x + c1.y)) * dr[16].x;
                    };
                    int d = 0;
                    for (; d + 1 < nd; d += 2) {   // two dst at a time: four independent FMA chains
                        const float s0 = dot(reinterpret_cast<const float4*>(dstf + d * kDstRowFloats));
                        const float s1 = dot(reinterpret_cast<const float4*>(dstf + (d + 1) * kDstRowFloats));
                        if (s0 > top) {
                            top = s0;
                            arg = d;
                        }
                        if (s1 > top) {
                            top = s1;
                            arg = d + 1;
                        }
                    }
                    if (d < nd) {
                        const float s0 = dot(reinterpret_cast<const float4*>(dstf + d * kDstRowFloats));
                        if (s0 > top) {
                            top = s0;
                            arg = d;
                        }
                    }
                    key[p] = score_key(top * inv[p]);
                    best[p] = __float_as_int(dstf[arg * kDstRowFloats + 65]);
                }
            }
        }

        // ---- phase 3: the r src with the best scores merge (ties: lowest position first)
        const int n_src = n - nd, n_out = n_src - r;
        bool merged[PASSES];
        if (r <= n_out) {
#pragma unroll
            for (int p = 0; p < PASSES; ++p) merged[p] = false;
            for (int round = 0; round < r; ++round) {
                uint32_t loc = 0;
#pragma unroll
                for (int p = 0; p < PASSES; ++p) loc = max(loc, (is_src[p] && !merged[p]) ? key[p] : 0u);
                const uint32_t m = __reduce_max_sync(0xffffffffu, loc);
                bool done = false;
#pragma unroll
                for (int p = 0; p < PASSES; ++p) {
                    const unsigned ball = __ballot_sync(0xffffffffu, is_src[p] && !merged[p] && key[p] == m);
                    if (!done && ball) {
                        if (lane == __ffs(ball) - 1) merged[p] = true;
                        done = true;
                    }
                }
            }
        } else {
#pragma unroll
            for (int p = 0; p < PASSES; ++p) merged[p] = is_src[p];
            for (int round = 0; round < n_out; ++round) {
                uint32_t loc = 0xffffffffu;
#pragma unroll
                for (int p = 0; p < PASSES; ++p) loc = min(loc, merged[p] ? key[p] : 0xffffffffu);
                const uint32_t m = __reduce_min_sync(0xffffffffu, loc);
                bool done = false;
#pragma unroll
                for (int p = PASSES - 1; p >= 0; --p) {
                    const unsigned ball = __ballot_sync(0xffffffffu, merged[p] && key[p] == m);
                    if (!done && ball) {
                        if (lane == 31 - __clz(ball)) merged[p] = false;
                        done = true;
                    }
                }
            }
        }
#pragma unroll
        for (int p = 0; p < PASSES; ++p) {
            const int j = lane + 32 * p;
            if (j < n) A[j] = bi.start + (merged[p] ? best[p] : j);
        }
        __syncwarp();   // every lane is done with the dst table (and, with several passes, the stage buffer)
        if (PASSES > 1) {
            if (lane == 0 && task + 2 * stride < n_tasks) issue(task + 2 * stride, buf);
        }
    }
    if (failed) {
        // give copies that may still be in flight a bounded chance to land before the CTA's
        // shared memory is released
        mbar_wait_bounded(mbar0, (it >> 1) & 1, a.status, kDevTimeoutMatchLoad);
        mbar_wait_bounded(mbar0 + 8, (it >> 1) & 1, a.status, kDevTimeoutMatchLoad);
    }
}

template <int PASSES>
static cudaError_t launch_match_t(const MatchArgs& a, int sm_count, cudaStream_t stream) {
    constexpr int NMAX = 32 * PASSES;
    constexpr int WARPS = match_warps_per_cta(NMAX);
    const size_t smem = match_smem_bytes(NMAX);
    CUtensorMap mq, mk;
    const int64_t N = a.n_tokens;
    if (!encode_rows_tensor_map(&mq, a.xr[0], N, a.heads, kHeadDim, N * kHeadDim, NMAX) ||
        !encode_rows_tensor_map(&mk, a.xr[1], N, a.heads, kHeadDim, N * kHeadDim, NMAX))
        return cudaErrorInvalidValue;
    const int64_t n_tasks = 2ll * a.heads * a.n_blocks;
    const int ctas_per_sm = (int)((224 * 1024) / (smem + 1024));
    int64_t grid = (n_tasks + WARPS - 1) / WARPS;
    const int64_t cap = (int64_t)sm_count * (ctas_per_sm < 1 ? 1 : ctas_per_sm);
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    match_kernel<PASSES><<<(unsigned)grid, WARPS * 32, smem, stream>>>(mq, mk, a);
    return cudaGetLastError();
}

cudaError_t launch_match(const MatchArgs& a, int max_block_tokens, int sm_count, cudaStream_t stream) {
    if (max_block_tokens <= 32) return launch_match_t<1>(a, sm_count, stream);
    if (max_block_tokens <= 128) return launch_match_t<4>(a, sm_count, stream);
    return launch_match_t<8>(a, sm_count, stream);
}

// ------------------------------------------------------------------------------------
// a3. Merged-token aggregation (Sec. 3.2: mean of the dst token and the src tokens
//     matched to it; Algorithm 1 "BlockAggregate"), one warp per (tensor, head, block).
//     The block is staged in shared memory by a TMA bulk copy, double buffered per warp.
//     Each lane owns two channels.  For every kept token, in reordered order, the warp
//     finds its group with one ballot over the map, sums the group's rows in token order
//     in fp32 registers (deterministic), divides once and rounds once to bf16.
//     Kept tokens are compacted: merged row = moff(block) + local rank.
//     The Q tasks also write rank_q (merged row of every token) for the unmerge.
// ------------------------------------------------------------------------------------
__host__ __device__ constexpr int merge_warps_per_cta(int nmax) { return nmax <= 32 ? 8 : (nmax <= 128 ? 4 : 2); }
__host__ __device__ constexpr int merge_smem_bytes(int nmax) { return merge_warps_per_cta(nmax) * (2 * nmax * kRowBytes + 16) + 128; }

template <int PASSES>
__global__ void __launch_bounds__(merge_warps_per_cta(32 * PASSES) * 32) merge_kernel(const __grid_constant__ MergeArgs a) {
    constexpr int NMAX = 32 * PASSES;
    constexpr int WARPS = merge_warps_per_cta(NMAX);
    constexpr uint32_t STAGE_BYTES = NMAX * kRowBytes;
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned char* stage = smem_raw + (size_t)warp * 2 * STAGE_BYTES;                       // [2][NMAX][128]
    uint64_t* mbar = reinterpret_cast<uint64_t*>(smem_raw + (size_t)WARPS * 2 * STAGE_BYTES) + 2 * warp;
    const uint32_t mbar0 = smem_u32(mbar), stage0 = smem_u32(stage);

    if (lane == 0) {
        mbar_init(mbar0, 1);
        mbar_init(mbar0 + 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncwarp();

    // task -> (tensor t, head h, unit u); units 0 .. n_blocks-1 are merging blocks, the rest are
    // chunks of 32 special tokens (never merged: rows 0 .. n_special_total-1 are copied)
    const int sp_chunks = (a.n_special_total + 31) / 32;
    const int64_t per_head = (int64_t)a.n_blocks + sp_chunks;
    const int64_t per_tensor = (int64_t)a.heads * per_head;
    const int64_t n_tasks = 3 * per_tensor;
    const int64_t stride = (int64_t)gridDim.x * WARPS;
    const int64_t first = (int64_t)blockIdx.x * WARPS + warp;

    struct Unit {
        int t, h, start, n, r, moff;
        bool special;
    };
    auto decode = [&](int64_t task) {
        Unit u;
        u.t = (int)(task / per_tensor);
        const int64_t rem = task - u.t * per_tensor;
        u.h = (int)(rem / per_head);
        const int idx = (int)(rem - (int64_t)u.h * per_head);
        u.special = idx >= a.n_blocks;
        if (u.special) {
            u.start = (idx - a.n_blocks) * 32;
            u.n = min(32, a.n_special_total - u.start);
            u.r = 0;
            u.moff = u.start;
        } else {
            const BlockInfo bi = a.blocks[idx];
            u.start = bi.start;
            u.n = bi.n;
            u.r = u.t == 0 ? bi.r_q : bi.r_k;
            u.moff = u.t == 0 ? bi.moff_q : bi.moff_k;
        }
        return u;
    };
    auto issue = [&](int64_t task, int buf) {   // lane 0 only
        const Unit u = decode(task);
        const uint32_t bytes = (uint32_t)u.n * kRowBytes;
        const uint32_t mb = mbar0 + 8 * buf;
        mbar_expect_tx(mb, bytes);
        bulk_load(stage0 + buf * STAGE_BYTES, a.xr[u.t] + ((int64_t)u.h * a.n_tokens + u.start) * kHeadDim, bytes, mb);
    };
    if (lane == 0) {
        if (first < n_tasks) issue(first, 0);
        if (first + stride < n_tasks) issue(first + stride, 1);
    }

    int it = 0;
    bool failed = false;
    for (int64_t task = first; task < n_tasks; task += stride, ++it) {
        const int buf = it & 1;
        const uint32_t parity = (it >> 1) & 1;
        const Unit u = decode(task);
        const int n = u.n;
        const int m_len = u.t == 0 ? a.m_q : a.m_k;
        uint32_t* out = reinterpret_cast<uint32_t*>(a.merged[u.t] + ((int64_t)u.h * m_len + u.moff) * kHeadDim);
        const uint32_t* xs = reinterpret_cast<const uint32_t*>(stage + buf * STAGE_BYTES);   // [n][32] bf16 pairs

        // the map entries do not depend on the staged rows: fetch them before waiting
        int rep[PASSES];
        if (u.r > 0) {
            const int32_t* A = a.assign[u.t == 0 ? 0 : 1] + (int64_t)u.h * a.n_tokens + u.start;
#pragma unroll
            for (int p = 0; p < PASSES; ++p) {
                const int j = lane + 32 * p;
                rep[p] = j < n ? __ldg(A + j) - u.start : -1;
                if (j < n && (rep[p] < 0 || rep[p] >= n)) {   // corrupt map: record, treat as kept
                    atomicCAS(a.status, kDevOk, kDevBadIndex);
                    rep[p] = j;
                }
            }
        }
        if (!mbar_wait_bounded(mbar0 + 8 * buf, parity, a.status, kDevTimeoutMatchLoad)) {
            failed = true;
            break;
        }
        if (u.r == 0) {   // nothing merges here: copy the rows, 16 bytes per lane
            const uint4* s4 = reinterpret_cast<const uint4*>(xs);
            uint4* o4 = reinterpret_cast<uint4*>(out);
            for (int q = lane; q < n * 8; q += 32) o4[q] = s4[q];
            if (u.t == 0 && !u.special)
                for (int j = lane; j < n; j += 32) a.rank_q[(int64_t)u.h * a.n_tokens + u.start + j] = u.moff + j;
        } else {
            unsigned kept[PASSES];
            int kept_before[PASSES];   // kept tokens in earlier passes
            int running = 0;
#pragma unroll
            for (int p = 0; p < PASSES; ++p) {
                const int j = lane + 32 * p;
                kept[p] = __ballot_sync(0xffffffffu, j < n && rep[p] == j);
                kept_before[p] = running;
                running += __popc(kept[p]);
            }
            if (u.t == 0) {   // merged row of every token of the block
#pragma unroll
                for (int p = 0; p < PASSES; ++p) {
                    const int j = lane + 32 * p;
                    if (j < n) {
                        int row = 0;
#pragma unroll
                        for (int pp = 0; pp < PASSES; ++pp)
                            if ((rep[p] >> 5) == pp) row = kept_before[pp] + __popc(kept[pp] & ((1u << (rep[p] & 31)) - 1u));
                        a.rank_q[(int64_t)u.h * a.n_tokens + u.start + j] = u.moff + row;
                    }
                }
            }
            int row = 0;
#pragma unroll
            for (int p = 0; p < PASSES; ++p) {
                unsigned km = kept[p];
                while (km) {
                    const int j = __ffs(km) - 1 + 32 * p;   // next kept token; its group = every token mapped to it
                    km &= km - 1;
                    float2 acc = make_float2(0.f, 0.f);
                    int cnt = 0;
#pragma unroll
                    for (int pp = 0; pp < PASSES; ++pp) {
                        unsigned mm = __ballot_sync(0xffffffffu, rep[pp] == j);
                        cnt += __popc(mm);
                        const uint32_t* xp = xs + (pp * 32) * 32 + lane;
                        while (mm) {
                            const int i0 = __ffs(mm) - 1;
                            mm &= mm - 1;
                            const uint32_t w0 = xp[i0 * 32];
                            if (mm) {
                                const int i1 = __ffs(mm) - 1;
                                mm &= mm - 1;
                                const uint32_t w1 = xp[i1 * 32];
                                acc.x += __uint_as_float(w0 << 16);
                                acc.y += __uint_as_float(w0 & 0xffff0000u);
                                acc.x += __uint_as_float(w1 << 16);
                                acc.y += __uint_as_float(w1 & 0xffff0000u);
                            } else {
                                acc.x += __uint_as_float(w0 << 16);
                                acc.y += __uint_as_float(w0 & 0xffff0000u);
                            }
                        }
                    }
                    if (cnt > 1) {   // mean: quotient by reciprocal with one correction step
                        const float c = (float)cnt, rc = 1.0f / c;
                        float qx = acc.x * rc, qy = acc.y * rc;
                        qx = fmaf(fmaf(-qx, c, acc.x), rc, qx);
                        qy = fmaf(fmaf(-qy, c, acc.y), rc, qy);
                        acc = make_float2(qx, qy);
                    }
                    const __nv_bfloat162 o = __floats2bfloat162_rn(acc.x, acc.y);
                    if (row < n - u.r) out[row * 32 + lane] = *reinterpret_cast<const uint32_t*>(&o);   // (a corrupt map cannot overrun)
                    ++row;
                }
            }
        }
        __syncwarp();   // every lane is done reading this stage buffer
        if (lane == 0 && task + 2 * stride < n_tasks) issue(task + 2 * stride, buf);
    }
    if (failed) {
        mbar_wait_bounded(mbar0, (it >> 1) & 1, a.status, kDevTimeoutMatchLoad);
        mbar_wait_bounded(mbar0 + 8, (it >> 1) & 1, a.status, kDevTimeoutMatchLoad);
    }
}

template <int PASSES>
static cudaError_t launch_merge_t(const MergeArgs& a, int sm_count, cudaStream_t stream) {
    constexpr int NMAX = 32 * PASSES;
    constexpr int WARPS = merge_warps_per_cta(NMAX);
    const size_t smem = merge_smem_bytes(NMAX);
    const int64_t n_tasks = 3ll * a.heads * (a.n_blocks + (a.n_special_total + 31) / 32);
    int ctas_per_sm = (int)((224 * 1024) / (smem + 1024));
    ctas_per_sm = ctas_per_sm < 1 ? 1 : (ctas_per_sm > 64 / WARPS ? 64 / WARPS : ctas_per_sm);
    int64_t grid = (n_tasks + WARPS - 1) / WARPS;
    const int64_t cap = (int64_t)sm_count * ctas_per_sm;
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    merge_kernel<PASSES><<<(unsigned)grid, WARPS * 32, smem, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_merge(const MergeArgs& a, int max_block_tokens, int sm_count, cudaStream_t stream) {
    if (max_block_tokens <= 32) return launch_merge_t<1>(a, sm_count, stream);
    if (max_block_tokens <= 128) return launch_merge_t<4>(a, sm_count, stream);
    return launch_merge_t<8>(a, sm_count, stream);
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
    HTTM_SET_SMEM(match_kernel<1>, match_smem_bytes(32));
    HTTM_SET_SMEM(match_kernel<4>, match_smem_bytes(128));
    HTTM_SET_SMEM(match_kernel<8>, match_smem_bytes(256));
    HTTM_SET_SMEM(merge_kernel<1>, merge_smem_bytes(32));
    HTTM_SET_SMEM(merge_kernel<4>, merge_smem_bytes(128));
    HTTM_SET_SMEM(merge_kernel<8>, merge_smem_bytes(256));
#undef HTTM_SET_SMEM
    return configure_attention();
}

}  // namespace httm
