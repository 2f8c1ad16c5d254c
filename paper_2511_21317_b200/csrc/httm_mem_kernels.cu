// HBM-bound kernels of the HTTM path: temporal reorder (gather), per-(head, block)
// cosine matching, mean merge, and unmerge + inverse reorder.  sm_100a only.
#include "httm_internal.h"

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
//     reorder) is staged in shared memory by a TMA bulk copy, double buffered per warp.
//     Similarities are fp32 dot products of the raw bf16 values (products are exact)
//     scaled by the inverse norms; argmax ties -> lowest dst, top-r ties -> lowest src.
// ------------------------------------------------------------------------------------
__host__ __device__ constexpr int match_warp_smem_bytes(int nmax) {
    // 2 stage buffers + fp32 copy of up to nmax/4 dst rows + inverse norms + 2 mbarriers, 128-byte multiple
    return ((2 * nmax * kRowBytes + (nmax / 4) * kHeadDim * 4 + nmax * 4 + 16) + 127) / 128 * 128;
}
__host__ __device__ constexpr int match_warps_per_cta(int nmax) { return nmax <= 32 ? 8 : (nmax <= 128 ? 4 : 2); }

template <int PASSES>
__global__ void __launch_bounds__(match_warps_per_cta(32 * PASSES) * 32) match_kernel(const __grid_constant__ MatchArgs a) {
    constexpr int NMAX = 32 * PASSES;
    constexpr int WARPS = match_warps_per_cta(NMAX);
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned char* wbase = smem_raw + (size_t)warp * match_warp_smem_bytes(NMAX);
    unsigned char* stage = wbase;                                                   // [2][NMAX*128]
    float* dstf = reinterpret_cast<float*>(wbase + 2 * NMAX * kRowBytes);           // [NMAX/4][64]
    float* invn = dstf + (NMAX / 4) * kHeadDim;                                     // [NMAX]
    uint64_t* mbar = reinterpret_cast<uint64_t*>(invn + NMAX);                      // [2]
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

    auto issue = [&](int64_t task, int buf) {   // lane 0 only
        const int t = (int)(task / per_tensor);
        const int64_t rem = task - t * per_tensor;
        const int h = (int)(rem / a.n_blocks), b = (int)(rem - (int64_t)h * a.n_blocks);
        const BlockInfo bi = a.blocks[b];
        const uint32_t bytes = (uint32_t)bi.n * kRowBytes;
        const uint32_t mb = mbar0 + 8 * buf;
        mbar_expect_tx(mb, bytes);
        bulk_load(stage0 + buf * NMAX * kRowBytes, a.xr[t] + ((int64_t)h * a.n_tokens + bi.start) * kHeadDim, bytes, mb);
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
        if (!mbar_wait_bounded(mbar0 + 8 * buf, parity, a.status, kDevTimeoutMatchLoad)) {
            failed = true;
            break;
        }
        const int t = (int)(task / per_tensor);
        const int64_t rem = task - t * per_tensor;
        const int h = (int)(rem / a.n_blocks), b = (int)(rem - (int64_t)h * a.n_blocks);
        const BlockInfo bi = a.blocks[b];
        const int n = bi.n, r = t == 0 ? bi.r_q : bi.r_k, nd = t == 0 ? bi.nd_q : bi.nd_k;
        int32_t* A = a.assign[t] + (int64_t)h * a.n_tokens + bi.start;
        const unsigned char* blk = stage + buf * NMAX * kRowBytes;

        if (r == 0) {
#pragma unroll
            for (int p = 0; p < PASSES; ++p) {
                const int j = lane + 32 * p;
                if (j < n) A[j] = bi.start + j;
            }
        } else {
            // own rows: lane handles tokens j = lane + 32p; x[p][..] holds the row with 16-byte
            // chunk k read from chunk (k ^ (lane & 7)) so that the warp's loads spread over banks
            float score[PASSES];
            int best[PASSES];
            const int sw = lane & 7;
            // inverse norms of all tokens
#pragma unroll
            for (int p = 0; p < PASSES; ++p) {
                const int j = lane + 32 * p;
                if (j < n) {
                    float ss = 0.f;
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        float f[8];
                        unpack8(*reinterpret_cast<const uint4*>(blk + j * kRowBytes + ((k ^ sw) << 4)), f);
#pragma unroll
                        for (int e = 0; e < 8; ++e) ss = fmaf(f[e], f[e], ss);
                    }
                    invn[j] = 1.0f / fmaxf(sqrtf(ss), 1e-12f);
                }
            }
            // fp32 copy of the dst rows: d-th dst sits at local position ceil((d+1) n / nd) - 1
            for (int q = lane; q < nd * 8; q += 32) {
                const int d = q >> 3, c = q & 7;
                const int pos = ((d + 1) * n + nd - 1) / nd - 1;
                float f[8];
                unpack8(*reinterpret_cast<const uint4*>(blk + pos * kRowBytes + (c << 4)), f);
                float4* o = reinterpret_cast<float4*>(dstf + d * kHeadDim + c * 8);
                o[0] = make_float4(f[0], f[1], f[2], f[3]);
                o[1] = make_float4(f[4], f[5], f[6], f[7]);
            }
            __syncwarp();
#pragma unroll
            for (int p = 0; p < PASSES; ++p) {
                const int j = lane + 32 * p;
                score[p] = -INFINITY;
                best[p] = -1;
                const bool is_src = j < n && !(((j + 1) * nd) / n > (j * nd) / n);
                if (p * 32 < n) {   // warp-uniform
                    float x[64];
                    if (is_src) {
#pragma unroll
                        for (int k = 0; k < 8; ++k)
                            unpack8(*reinterpret_cast<const uint4*>(blk + j * kRowBytes + ((k ^ sw) << 4)), x + 8 * k);
                        float top = -INFINITY;
                        int arg = 0;
                        for (int d = 0; d < nd; ++d) {
                            const float* dr = dstf + d * kHeadDim;
                            float acc = 0.f;
#pragma unroll
                            for (int k = 0; k < 8; ++k) {
                                const float4 u0 = *reinterpret_cast<const float4*>(dr + ((k ^ sw) << 3));
                                const float4 u1 = *reinterpret_cast<const float4*>(dr + ((k ^ sw) << 3) + 4);
                                acc = fmaf(x[8 * k + 0], u0.x, acc);
                                acc = fmaf(x[8 * k + 1], u0.y, acc);
                                acc = fmaf(x[8 * k + 2], u0.z, acc);
                                acc = fmaf(x[8 * k + 3], u0.w, acc);
                                acc = fmaf(x[8 * k + 4], u1.x, acc);
                                acc = fmaf(x[8 * k + 5], u1.y, acc);
                                acc = fmaf(x[8 * k + 6], u1.z, acc);
                                acc = fmaf(x[8 * k + 7], u1.w, acc);
                            }
                            const int pos = ((d + 1) * n + nd - 1) / nd - 1;
                            const float sim = acc * invn[pos];
                            if (sim > top) {
                                top = sim;
                                arg = pos;
                            }
                        }
                        score[p] = top * invn[j];
                        best[p] = arg;
                    }
                }
            }
            // top-r by rank counting over all src of the block (warp shuffles)
#pragma unroll
            for (int p = 0; p < PASSES; ++p) {
                const int j = lane + 32 * p;
                int rank = 0;
#pragma unroll
                for (int pp = 0; pp < PASSES; ++pp) {
                    if (pp * 32 < n) {
#pragma unroll 8
                        for (int l = 0; l < 32; ++l) {
                            const float s2 = __shfl_sync(0xffffffffu, score[pp], l);
                            const int j2 = l + 32 * pp;
                            rank += (s2 > score[p]) || (s2 == score[p] && j2 < j);
                        }
                    }
                }
                if (j < n) A[j] = bi.start + ((best[p] >= 0 && rank < r) ? best[p] : j);
            }
        }
        __syncwarp();   // every lane is done reading this stage buffer
        if (lane == 0 && task + 2 * stride < n_tasks) issue(task + 2 * stride, buf);
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
    const size_t smem = (size_t)WARPS * match_warp_smem_bytes(NMAX);
    const int64_t n_tasks = 2ll * a.heads * a.n_blocks;
    const int ctas_per_sm = (int)((220 * 1024) / (smem + 1024));
    int64_t grid = (n_tasks + WARPS - 1) / WARPS;
    const int64_t cap = (int64_t)sm_count * (ctas_per_sm < 1 ? 1 : ctas_per_sm);
    if (grid > cap) grid = cap;
    if (grid < 1) grid = 1;
    match_kernel<PASSES><<<(unsigned)grid, WARPS * 32, smem, stream>>>(a);
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
//     fp32 sums in shared memory in token order (deterministic), one rounding to bf16.
//     Kept tokens are compacted in reordered order: merged row = moff(block) + local rank.
//     The Q tasks also write rank_q (merged row of every token) for the unmerge.
// ------------------------------------------------------------------------------------
__host__ __device__ constexpr int merge_warp_smem_bytes(int nmax) {
    return nmax * kHeadDim * 4 + nmax * 4 + nmax * 4;   // acc + row_of + count
}

template <int PASSES>
__global__ void __launch_bounds__(match_warps_per_cta(32 * PASSES) * 32) merge_kernel(const __grid_constant__ MergeArgs a) {
    constexpr int NMAX = 32 * PASSES;
    constexpr int WARPS = match_warps_per_cta(NMAX);
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned char* wbase = smem_raw + (size_t)warp * merge_warp_smem_bytes(NMAX);
    float2* acc = reinterpret_cast<float2*>(wbase);                                   // [NMAX][32] float2
    int32_t* row_of = reinterpret_cast<int32_t*>(wbase + NMAX * kHeadDim * 4);        // [NMAX]
    int32_t* count = row_of + NMAX;                                                   // [NMAX]

    const int sp_chunks = (a.n_special_total + 31) / 32;
    const int64_t per_head = (int64_t)a.n_blocks + sp_chunks;
    const int64_t per_tensor = (int64_t)a.heads * per_head;
    const int64_t n_tasks = 3 * per_tensor;
    const int64_t stride = (int64_t)gridDim.x * WARPS;

    for (int64_t task = (int64_t)blockIdx.x * WARPS + warp; task < n_tasks; task += stride) {
        const int t = (int)(task / per_tensor);
        const int64_t rem = task - t * per_tensor;
        const int h = (int)(rem / per_head);
        const int u = (int)(rem - (int64_t)h * per_head);
        const int m_len = t == 0 ? a.m_q : a.m_k;
        const uint32_t* x = reinterpret_cast<const uint32_t*>(a.xr[t] + (int64_t)h * a.n_tokens * kHeadDim);
        uint32_t* out = reinterpret_cast<uint32_t*>(a.merged[t] + (int64_t)h * m_len * kHeadDim);

        if (u >= a.n_blocks) {   // special tokens: never merged, rows 0 .. n_special_total-1 copied
            const int p0 = (u - a.n_blocks) * 32;
            const int cnt = min(32, a.n_special_total - p0);
            for (int j = 0; j < cnt; ++j) out[(int64_t)(p0 + j) * 32 + lane] = __ldg(x + (int64_t)(p0 + j) * 32 + lane);
            continue;
        }
        const BlockInfo bi = a.blocks[u];
        const int n = bi.n, r = t == 0 ? bi.r_q : bi.r_k, moff = t == 0 ? bi.moff_q : bi.moff_k;
        const uint32_t* xb = x + (int64_t)bi.start * 32;
        if (r == 0) {   // nothing merges in this block: straight copy
            for (int j = 0; j < n; ++j) out[(int64_t)(moff + j) * 32 + lane] = __ldg(xb + (int64_t)j * 32 + lane);
            if (t == 0)
                for (int j = lane; j < n; j += 32) a.rank_q[(int64_t)h * a.n_tokens + bi.start + j] = moff + j;
            continue;
        }
        const int32_t* A = a.assign[t == 0 ? 0 : 1] + (int64_t)h * a.n_tokens + bi.start;
        // local rank of kept tokens (ballot prefix), then row of every token
        int rep[PASSES];
        int running = 0;
#pragma unroll
        for (int p = 0; p < PASSES; ++p) {
            const int j = lane + 32 * p;
            rep[p] = j < n ? __ldg(A + j) - bi.start : -1;
            if (j < n && (rep[p] < 0 || rep[p] >= n)) {   // corrupt map: record, treat as kept
                atomicCAS(a.status, kDevOk, kDevBadIndex);
                rep[p] = j;
            }
            const bool kept = j < n && rep[p] == j;
            const unsigned mask = __ballot_sync(0xffffffffu, kept);
            if (kept) {
                row_of[j] = running + __popc(mask & ((1u << lane) - 1u));
            }
            if (j < n) count[j] = 0;
            running += __popc(mask);
        }
        const int n_kept = running;
        __syncwarp();
#pragma unroll
        for (int p = 0; p < PASSES; ++p) {
            const int j = lane + 32 * p;
            if (j < n) {
                const int row = row_of[rep[p]];   // rep is a kept token, its row is final
                if (rep[p] != j) row_of[j] = row; // merged tokens never serve as rep, no hazard
                atomicAdd(&count[row], 1);
                if (t == 0) a.rank_q[(int64_t)h * a.n_tokens + bi.start + j] = moff + row;
            }
        }
        for (int q = lane; q < n_kept * 32; q += 32) acc[q] = make_float2(0.f, 0.f);
        __syncwarp();
        // accumulate in token order, 8 rows of loads in flight
        for (int j0 = 0; j0 < n; j0 += 8) {
            uint32_t raw[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (j0 + e < n) raw[e] = __ldg(xb + (int64_t)(j0 + e) * 32 + lane);
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (j0 + e < n) {
                    float2* c = acc + row_of[j0 + e] * 32 + lane;
                    float2 v = *c;
                    v.x += __uint_as_float(raw[e] << 16);
                    v.y += __uint_as_float(raw[e] & 0xffff0000u);
                    *c = v;
                }
        }
        for (int m = 0; m < n_kept; ++m) {
            const float2 v = acc[m * 32 + lane];
            const float c = (float)count[m];
            const __nv_bfloat162 o = __floats2bfloat162_rn(v.x / c, v.y / c);
            out[(int64_t)(moff + m) * 32 + lane] = *reinterpret_cast<const uint32_t*>(&o);
        }
        __syncwarp();
    }
}

template <int PASSES>
static cudaError_t launch_merge_t(const MergeArgs& a, int sm_count, cudaStream_t stream) {
    constexpr int NMAX = 32 * PASSES;
    constexpr int WARPS = match_warps_per_cta(NMAX);
    const size_t smem = (size_t)WARPS * merge_warp_smem_bytes(NMAX);
    const int64_t n_tasks = 3ll * a.heads * (a.n_blocks + (a.n_special_total + 31) / 32);
    const int ctas_per_sm = (int)((220 * 1024) / (smem + 1024));
    int64_t grid = (n_tasks + WARPS - 1) / WARPS;
    const int64_t cap = (int64_t)sm_count * (ctas_per_sm < 1 ? 1 : (ctas_per_sm > 8 ? 8 : ctas_per_sm));
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
//     8 threads move one 128-byte (token, head) row; consecutive thread groups take
//     consecutive heads of the same token, so the writes of a CTA are contiguous.
// ------------------------------------------------------------------------------------
constexpr int kUnmergeThreads = 256;

__global__ void __launch_bounds__(kUnmergeThreads) unmerge_kernel(const UnmergeArgs a) {
    const int64_t g = ((int64_t)blockIdx.x * kUnmergeThreads + threadIdx.x) >> 3;   // (token, head) pair
    const int chunk = threadIdx.x & 7;
    const int64_t total = (int64_t)a.n_tokens * a.heads;
    if (g >= total) return;
    const int i = (int)(g / a.heads), h = (int)(g - (int64_t)i * a.heads);
    const int p = __ldg(a.pi_inv + i);
    int row = __ldg(a.rank_q + (int64_t)h * a.n_tokens + p);
    if (row < 0 || row >= a.m_q) {
        atomicCAS(a.status, kDevOk, kDevBadIndex);
        return;
    }
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(a.o_m + ((int64_t)h * a.m_q + row) * kHeadDim) + chunk);
    *reinterpret_cast<uint4*>(a.out + (int64_t)h * a.out_stride_head + (int64_t)i * a.out_stride_token + chunk * 8) = v;
}

cudaError_t launch_unmerge(const UnmergeArgs& a, cudaStream_t stream) {
    const int64_t threads = (int64_t)a.n_tokens * a.heads * 8;
    const int64_t grid = (threads + kUnmergeThreads - 1) / kUnmergeThreads;
    unmerge_kernel<<<(unsigned)grid, kUnmergeThreads, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t configure_kernels() {
    cudaError_t e;
#define HTTM_SET_SMEM(kern, bytes)                                                                      \
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(bytes));          \
    if (e != cudaSuccess) return e;
    HTTM_SET_SMEM(match_kernel<1>, match_warps_per_cta(32) * match_warp_smem_bytes(32));
    HTTM_SET_SMEM(match_kernel<4>, match_warps_per_cta(128) * match_warp_smem_bytes(128));
    HTTM_SET_SMEM(match_kernel<8>, match_warps_per_cta(256) * match_warp_smem_bytes(256));
    HTTM_SET_SMEM(merge_kernel<1>, match_warps_per_cta(32) * merge_warp_smem_bytes(32));
    HTTM_SET_SMEM(merge_kernel<4>, match_warps_per_cta(128) * merge_warp_smem_bytes(128));
    HTTM_SET_SMEM(merge_kernel<8>, match_warps_per_cta(256) * merge_warp_smem_bytes(256));
#undef HTTM_SET_SMEM
    return configure_attention();
}

}  // namespace httm
