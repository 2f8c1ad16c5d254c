// Softmax attention (Eq. 3-4) on warp-level mma.sync tensor-core instructions:
//   out[h][m] = softmax(q[h][m] . k[h]^T / sqrt(64)) v[h]
// 64 query rows per CTA (16 per warp), 64-key tiles double buffered with cp.async, online
// softmax in registers.  Serves both the merged sets and the dense (unmerged) baseline.
#include "httm_internal.h"

namespace httm {

namespace {

constexpr int BM = 64, BN = 64, NTHREADS = 128;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid) {
    const int bytes = valid ? 16 : 0;   // 0 -> destination is zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}
// tile [64 rows][64 bf16]: 16-byte chunk c of row r lives at chunk (c ^ (r & 7))
__device__ __forceinline__ uint32_t tile_off(int row, int chunk) { return (uint32_t)(row * 128 + ((chunk ^ (row & 7)) << 4)); }

// copy a 64-row tile (rows row0.. of `src`, clipped at n_rows -> zero fill) into shared memory
__device__ __forceinline__ void load_tile(uint32_t smem, const __nv_bfloat16* src, int64_t stride_token, int row0,
                                          int n_rows, int tid) {
#pragma unroll
    for (int i = 0; i < (64 * 8) / NTHREADS; ++i) {
        const int q = tid + i * NTHREADS;
        const int r = q >> 3, c = q & 7;
        const bool ok = row0 + r < n_rows;
        const __nv_bfloat16* g = src + (int64_t)(ok ? row0 + r : 0) * stride_token + c * 8;
        cp_async16(smem + tile_off(r, c), g, ok);
    }
}

__global__ void __launch_bounds__(NTHREADS) attention_mma_kernel(const AttentionArgs a) {
    __shared__ __align__(128) unsigned char sq[BM * 128];
    __shared__ __align__(128) unsigned char sk[2][BN * 128];
    __shared__ __align__(128) unsigned char sv[2][BN * 128];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.y, q0 = blockIdx.x * BM;
    const __nv_bfloat16* qh = a.q.ptr + (int64_t)h * a.q.stride_head;
    const __nv_bfloat16* kh = a.k.ptr + (int64_t)h * a.k.stride_head;
    const __nv_bfloat16* vh = a.v.ptr + (int64_t)h * a.v.stride_head;
    const uint32_t sq_u = smem_u32(sq), sk_u = smem_u32(sk), sv_u = smem_u32(sv);
    const int n_tiles = (a.m_k + BN - 1) / BN;

    load_tile(sq_u, qh, a.q.stride_token, q0, a.m_q, tid);
    load_tile(sk_u, kh, a.k.stride_token, 0, a.m_k, tid);
    load_tile(sv_u, vh, a.v.stride_token, 0, a.m_k, tid);
    cp_async_commit();

    uint32_t qf[4][4];
    float o[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    float row_max[2] = {-INFINITY, -INFINITY}, row_sum[2] = {0.f, 0.f};

    for (int tile = 0; tile < n_tiles; ++tile) {
        const int buf = tile & 1;
        if (tile + 1 < n_tiles) {
            load_tile(sk_u + (buf ^ 1) * BN * 128, kh, a.k.stride_token, (tile + 1) * BN, a.m_k, tid);
            load_tile(sv_u + (buf ^ 1) * BN * 128, vh, a.v.stride_token, (tile + 1) * BN, a.m_k, tid);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        if (tile == 0) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
                ldsm_x4(sq_u + tile_off(warp * 16 + (lane & 15), ks * 2 + (lane >> 4)), qf[ks][0], qf[ks][1], qf[ks][2],
                        qf[ks][3]);
        }
        // S = Q K^T for this warp's 16 rows x 64 keys
        float s[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i) s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
        const uint32_t kb = sk_u + buf * BN * 128, vb = sv_u + buf * BN * 128;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
#pragma unroll
            for (int np = 0; np < 4; ++np) {   // pairs of 8-key tiles
                uint32_t b0, b1, b2, b3;
                const int mi = lane >> 3;
                ldsm_x4(kb + tile_off(np * 16 + (mi >> 1) * 8 + (lane & 7), ks * 2 + (mi & 1)), b0, b1, b2, b3);
                mma_bf16(s[np * 2], qf[ks], b0, b1);
                mma_bf16(s[np * 2 + 1], qf[ks], b2, b3);
            }
        }
        // scale to log2 units, mask keys past the end
        const int key0 = tile * BN + 2 * (lane & 3);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int key = key0 + i * 8 + (e & 1);
                s[i][e] = key < a.m_k ? s[i][e] * a.scale_log2 : -INFINITY;
            }
        }
        // online softmax; rows g = lane/4 (e 0,1) and g + 8 (e 2,3)
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            float mx = row_max[half];
#pragma unroll
            for (int i = 0; i < 8; ++i) mx = fmaxf(mx, fmaxf(s[i][2 * half], s[i][2 * half + 1]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            const float corr = exp2f(row_max[half] - mx);   // first tile: exp2(-inf) = 0
            row_max[half] = mx;
            float sum = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                s[i][2 * half] = exp2f(s[i][2 * half] - mx);
                s[i][2 * half + 1] = exp2f(s[i][2 * half + 1] - mx);
                sum += s[i][2 * half] + s[i][2 * half + 1];
            }
            row_sum[half] = row_sum[half] * corr + sum;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                o[i][2 * half] *= corr;
                o[i][2 * half + 1] *= corr;
            }
        }
        // O += P V
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {   // 16 keys per step
            uint32_t pf[4];
            pf[0] = pack_bf16(s[2 * ks][0], s[2 * ks][1]);
            pf[1] = pack_bf16(s[2 * ks][2], s[2 * ks][3]);
            pf[2] = pack_bf16(s[2 * ks + 1][0], s[2 * ks + 1][1]);
            pf[3] = pack_bf16(s[2 * ks + 1][2], s[2 * ks + 1][3]);
#pragma unroll
            for (int dp = 0; dp < 4; ++dp) {   // pairs of 8-channel tiles
                uint32_t b0, b1, b2, b3;
                const int mi = lane >> 3;
                ldsm_x4_t(vb + tile_off(ks * 16 + (mi & 1) * 8 + (lane & 7), dp * 2 + (mi >> 1)), b0, b1, b2, b3);
                mma_bf16(o[dp * 2], pf, b0, b1);
                mma_bf16(o[dp * 2 + 1], pf, b2, b3);
            }
        }
        __syncthreads();   // all warps done with this buffer before it is refilled
    }

#pragma unroll
    for (int half = 0; half < 2; ++half) {
        float sum = row_sum[half];
        sum += __shfl_xor_sync(0xffffffffu, sum, 1);
        sum += __shfl_xor_sync(0xffffffffu, sum, 2);
        const float inv = 1.0f / sum;
        const int row = q0 + warp * 16 + (lane >> 2) + 8 * half;
        if (row < a.m_q) {
            __nv_bfloat16* dst = a.out + (int64_t)h * a.out_stride_head + (int64_t)row * a.out_stride_token + 2 * (lane & 3);
#pragma unroll
            for (int i = 0; i < 8; ++i)
                *reinterpret_cast<uint32_t*>(dst + i * 8) = pack_bf16(o[i][2 * half] * inv, o[i][2 * half + 1] * inv);
        }
    }
}

}  // namespace

cudaError_t launch_attention(const AttentionArgs& a, int /*sm_count*/, cudaStream_t stream) {
    dim3 grid((a.m_q + BM - 1) / BM, a.heads);
    attention_mma_kernel<<<grid, NTHREADS, 0, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace httm
