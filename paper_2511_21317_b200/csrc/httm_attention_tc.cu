// Softmax attention (Eq. 3-4) on the 5th-generation tensor cores:
//   out[h][m] = softmax(q[h][m] . k[h]^T / sqrt(64)) v[h]
//
// One CTA owns TWO 128-row query tiles (A, B) of one head and walks the keys in 128-key tiles.
//   warp 0      TMA producer: Q tiles once, then a ring of K and V tiles (128-byte swizzle)
//   warp 1      issues every tcgen05.mma: S_X = Q_X K^T (operands in shared memory) and
//               O_X += P_X V (P_X read from tensor memory, V MN-major from shared memory)
//   warps 4-7   softmax of tile A: one thread per query row, S read from tensor memory,
//               P written back over S as bf16 pairs; warps 8-11 the same for tile B
// While one tile's softmax runs, the tensor core works on the other tile.  Accumulators live in
// tensor memory: S_A, S_B (128 columns each), O_A, O_B (64 columns each).  Running maxima are
// only raised when they grow by more than 2^8 (then the softmax threads rescale O in place), so
// rescaling is rare after the first tiles.  Every wait is bounded; on expiry the kernel records
// kDevTimeoutAttention in the status word, releases its tensor memory and returns.
#include "httm_internal.h"
#include "tc_sm100.cuh"

namespace httm {

namespace {

constexpr int BM = 128;            // rows per query tile
constexpr int BN = 128;            // keys per tile
constexpr int KV_STAGES = 3;
constexpr int TILE_BYTES = BM * kRowBytes;   // 16 KB
constexpr int NTHREADS = 384;
constexpr int TMEM_COLS = 512;
constexpr int SMEM_BYTES = (2 + 2 * KV_STAGES) * TILE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr float kRescaleThreshold = 8.0f;   // log2 units

struct Barriers {
    uint64_t q_full;
    uint64_t k_full[KV_STAGES], k_empty[KV_STAGES];
    uint64_t v_full[KV_STAGES], v_empty[KV_STAGES];
    uint64_t s_full[2], p_full[2];
    uint64_t o_final;
    uint32_t tmem_base;
    int abort_flag;
};

struct TcParams {
    __nv_bfloat16* out;
    int64_t out_stride_head, out_stride_token;
    int32_t m_q, m_k;
    float scale_log2;
    int32_t* status;
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(NTHREADS, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, const TcParams p) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t s_q = tc::smem_addr(smem);                             // 2 tiles
    const uint32_t s_k = s_q + 2 * TILE_BYTES;                            // KV_STAGES tiles
    const uint32_t s_v = s_k + KV_STAGES * TILE_BYTES;
    Barriers* bars = reinterpret_cast<Barriers*>(smem + (2 + 2 * KV_STAGES) * TILE_BYTES);
    volatile int* abort_flag = &bars->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int head = blockIdx.y;
    const int q0 = blockIdx.x * (2 * BM);
    const int n_tiles = (p.m_k + BN - 1) / BN;

    if (tid == 0) {
        bars->abort_flag = 0;
        tc::mbar_init(tc::smem_addr(&bars->q_full), 1);
        for (int i = 0; i < KV_STAGES; ++i) {
            tc::mbar_init(tc::smem_addr(&bars->k_full[i]), 1);
            tc::mbar_init(tc::smem_addr(&bars->k_empty[i]), 1);
            tc::mbar_init(tc::smem_addr(&bars->v_full[i]), 1);
            tc::mbar_init(tc::smem_addr(&bars->v_empty[i]), 1);
        }
        for (int x = 0; x < 2; ++x) {
            tc::mbar_init(tc::smem_addr(&bars->s_full[x]), 1);
            tc::mbar_init(tc::smem_addr(&bars->p_full[x]), 128);
        }
        tc::mbar_init(tc::smem_addr(&bars->o_final), 1);
        tc::fence_barrier_init();
        tc::prefetch_tensormap(&map_q);
        tc::prefetch_tensormap(&map_k);
        tc::prefetch_tensormap(&map_v);
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_addr(&bars->tmem_base), TMEM_COLS);
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem = bars->tmem_base;
    // columns: S_A [0,128)  S_B [128,256)  O_A [256,320)  O_B [320,384); P_X overlays the first 64 columns of S_X

    // Register budget: the softmax threads hold a whole 128-wide row of S; the producer, the MMA
    // issuer and the two idle warps give most of their registers to them (128*80 + 256*208 <= 64K).
    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
        if (lane == 0) {
            const uint32_t qb = tc::smem_addr(&bars->q_full);
            tc::mbar_expect_tx(qb, 2 * TILE_BYTES);
            tc::tma_load_3d(s_q, &map_q, qb, 0, q0, head);
            tc::tma_load_3d(s_q + TILE_BYTES, &map_q, qb, 0, q0 + BM, head);
            for (int j = 0; j < n_tiles; ++j) {
                const int st = j % KV_STAGES;
                const uint32_t ph = (uint32_t)(j / KV_STAGES) & 1u;
                if (j >= KV_STAGES && !tc::mbar_wait(tc::smem_addr(&bars->k_empty[st]), ph ^ 1u, abort_flag)) break;
                const uint32_t kb = tc::smem_addr(&bars->k_full[st]);
                tc::mbar_expect_tx(kb, TILE_BYTES);
                tc::tma_load_3d(s_k + st * TILE_BYTES, &map_k, kb, 0, j * BN, head);
                if (j >= KV_STAGES && !tc::mbar_wait(tc::smem_addr(&bars->v_empty[st]), ph ^ 1u, abort_flag)) break;
                const uint32_t vb = tc::smem_addr(&bars->v_full[st]);
                tc::mbar_expect_tx(vb, TILE_BYTES);
                tc::tma_load_3d(s_v + st * TILE_BYTES, &map_v, vb, 0, j * BN, head);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
        if (lane == 0) {
            constexpr uint32_t idesc_qk = tc::idesc_bf16(BM, BN, false, false);
            constexpr uint32_t idesc_pv = tc::idesc_bf16(BM, kHeadDim, false, true);
            const uint64_t dq[2] = {tc::smem_desc_sw128(s_q), tc::smem_desc_sw128(s_q + TILE_BYTES)};
            auto issue_qk = [&](int x, int st) {
                const uint64_t dk = tc::smem_desc_sw128(s_k + st * TILE_BYTES);
#pragma unroll
                for (int k = 0; k < 4; ++k) tc::mma_ss(tmem + x * BN, dq[x] + 2 * k, dk + 2 * k, idesc_qk, k > 0);
                tc::mma_commit(tc::smem_addr(&bars->s_full[x]));
            };
            auto issue_pv = [&](int x, int st, bool first) {
                const uint64_t dv = tc::smem_desc_sw128(s_v + st * TILE_BYTES);
#pragma unroll
                for (int k = 0; k < 8; ++k)
                    tc::mma_ts(tmem + 2 * BN + x * kHeadDim, tmem + x * BN + 8 * k, dv + (uint64_t)(k * 2048 >> 4), idesc_pv,
                               (!first || k > 0) ? 1u : 0u);
            };
            bool ok = tc::mbar_wait(tc::smem_addr(&bars->q_full), 0, abort_flag) &&
                      tc::mbar_wait(tc::smem_addr(&bars->k_full[0]), 0, abort_flag);
            if (ok) {
                tc::fence_after_sync();
                issue_qk(0, 0);
                issue_qk(1, 0);
                tc::mma_commit(tc::smem_addr(&bars->k_empty[0]));
            }
            for (int j = 0; ok && j < n_tiles; ++j) {
                const int st = j % KV_STAGES, st1 = (j + 1) % KV_STAGES;
                const uint32_t ph = (uint32_t)(j / KV_STAGES) & 1u, ph1 = (uint32_t)((j + 1) / KV_STAGES) & 1u;
                const bool more = j + 1 < n_tiles;
                if (!(ok = tc::mbar_wait(tc::smem_addr(&bars->v_full[st]), ph, abort_flag))) break;
                if (!(ok = tc::mbar_wait(tc::smem_addr(&bars->p_full[0]), j & 1, abort_flag))) break;
                tc::fence_after_sync();
                issue_pv(0, st, j == 0);
                if (more) {
                    if (!(ok = tc::mbar_wait(tc::smem_addr(&bars->k_full[st1]), ph1, abort_flag))) break;
                    tc::fence_after_sync();
                    issue_qk(0, st1);
                }
                if (!(ok = tc::mbar_wait(tc::smem_addr(&bars->p_full[1]), j & 1, abort_flag))) break;
                tc::fence_after_sync();
                issue_pv(1, st, j == 0);
                tc::mma_commit(tc::smem_addr(&bars->v_empty[st]));
                if (more) {
                    issue_qk(1, st1);
                    tc::mma_commit(tc::smem_addr(&bars->k_empty[st1]));
                }
            }
            if (ok) tc::mma_commit(tc::smem_addr(&bars->o_final));
        }
        __syncwarp();
    } else if (warp < 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 80;");
    } else {
        // ------------------------------------------------------------------ softmax + epilogue
        asm volatile("setmaxnreg.inc.sync.aligned.u32 208;");
        const int x = (warp - 4) >> 2;                 // 0: tile A, 1: tile B
        const int row = (warp & 3) * 32 + lane;        // row inside the tile = TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem + x * BN + lane_addr;
        const uint32_t t_o = tmem + 2 * BN + x * kHeadDim + lane_addr;
        const uint32_t sbar = tc::smem_addr(&bars->s_full[x]), pbar = tc::smem_addr(&bars->p_full[x]);
        const float c = p.scale_log2;
        float m = -INFINITY, l = 0.f;
        bool ok = true;
        for (int j = 0; j < n_tiles; ++j) {
            if (!(ok = tc::mbar_wait(sbar, j & 1, abort_flag))) break;
            tc::fence_after_sync();
            uint32_t s[BN];   // fp32 bit patterns of this row of S
#pragma unroll
            for (int cc = 0; cc < 4; ++cc) tc::tmem_ld32(t_s + cc * 32, s + cc * 32);
            tc::tmem_wait_ld();
            const int valid = p.m_k - j * BN;
            if (valid < BN) {
#pragma unroll
                for (int i = 0; i < BN; ++i)
                    if (i >= valid) s[i] = 0xff800000u;   // -inf: keys past the end
            }
            float mx = __uint_as_float(s[0]);
#pragma unroll
            for (int i = 1; i < BN; ++i) mx = fmaxf(mx, __uint_as_float(s[i]));
            const float m_new = fmaxf(m, mx * c);
            if (j == 0) {
                m = m_new;
            } else if (__any_sync(0xffffffffu, m_new - m > kRescaleThreshold)) {
                // raise the running maximum: rescale the row sum and the accumulator O in place
                // (s_full(j) was committed after PV(j-1), so O is quiescent here)
                const float f = exp2f(m - m_new);
                l *= f;
                m = m_new;
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
                    uint32_t o[32];
                    tc::tmem_ld32(t_o + cc * 32, o);
                    tc::tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                    tc::tmem_st32(t_o + cc * 32, o);
                }
            }
            const float neg_m = -m;
            float sum = 0.f;
#pragma unroll
            for (int cc = 0; cc < 8; ++cc) {
                uint32_t pk[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float a = fast_exp2(fmaf(__uint_as_float(s[cc * 16 + 2 * i]), c, neg_m));
                    const float b = fast_exp2(fmaf(__uint_as_float(s[cc * 16 + 2 * i + 1]), c, neg_m));
                    sum += a + b;
                    pk[i] = pack_bf16(a, b);
                }
                asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(t_s + cc * 8),
                             "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]), "r"(pk[4]), "r"(pk[5]), "r"(pk[6]), "r"(pk[7])
                             : "memory");
            }
            l += sum;
            tc::tmem_wait_st();
            tc::fence_before_sync();
            tc::mbar_arrive(pbar);
        }
        if (ok && (ok = tc::mbar_wait(tc::smem_addr(&bars->o_final), 0, abort_flag))) {
            tc::fence_after_sync();
            const int grow = q0 + x * BM + row;
            const float inv = 1.0f / l;
            uint32_t o[64];
            tc::tmem_ld32(t_o, o);
            tc::tmem_ld32(t_o + 32, o + 32);
            tc::tmem_wait_ld();
            if (grow < p.m_q) {
                uint4* dst = reinterpret_cast<uint4*>(p.out + (int64_t)head * p.out_stride_head + (int64_t)grow * p.out_stride_token);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    uint4 v;
                    v.x = pack_bf16(__uint_as_float(o[8 * i + 0]) * inv, __uint_as_float(o[8 * i + 1]) * inv);
                    v.y = pack_bf16(__uint_as_float(o[8 * i + 2]) * inv, __uint_as_float(o[8 * i + 3]) * inv);
                    v.z = pack_bf16(__uint_as_float(o[8 * i + 4]) * inv, __uint_as_float(o[8 * i + 5]) * inv);
                    v.w = pack_bf16(__uint_as_float(o[8 * i + 6]) * inv, __uint_as_float(o[8 * i + 7]) * inv);
                    dst[i] = v;
                }
            }
        }
    }
    tc::fence_before_sync();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem, TMEM_COLS);
    if (tid == 0 && bars->abort_flag) atomicCAS(p.status, kDevOk, kDevTimeoutAttention);
}

}  // namespace

cudaError_t configure_attention() {
    return cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
}

// Returns cudaErrorInvalidValue if a tensor map cannot be encoded.
cudaError_t launch_attention(const AttentionArgs& a, int /*sm_count*/, cudaStream_t stream) {
    CUtensorMap mq, mk, mv;
    if (!encode_rows_tensor_map(&mq, a.q.ptr, a.m_q, a.heads, a.q.stride_token, a.q.stride_head, BM) ||
        !encode_rows_tensor_map(&mk, a.k.ptr, a.m_k, a.heads, a.k.stride_token, a.k.stride_head, BN) ||
        !encode_rows_tensor_map(&mv, a.v.ptr, a.m_k, a.heads, a.v.stride_token, a.v.stride_head, BN))
        return cudaErrorInvalidValue;
    TcParams p{a.out, a.out_stride_head, a.out_stride_token, a.m_q, a.m_k, a.scale_log2, a.status};
    dim3 grid((a.m_q + 2 * BM - 1) / (2 * BM), a.heads);
    attention_tc_kernel<<<grid, NTHREADS, SMEM_BYTES, stream>>>(mq, mk, mv, p);
    return cudaGetLastError();
}

}  // namespace httm
