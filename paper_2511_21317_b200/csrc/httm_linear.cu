// The projections around the path (Algorithm 1's first and last lines: Q, K, V = x W_qkv and out = Attn W_o) as a
// tcgen05 GEMM of the library's own:  y[n][out] = x[n][in] . w[out][in]^T,  bf16 operands, fp32 accumulation in tensor
// memory, bf16 result.  Weights are given as [out][in] (the layout a linear layer stores them in), so both operands are
// K-major and a 128 x 256 output tile is four tcgen05.mma M128 N256 K16 per 64 input channels.
//   warp 0      TMA producer: a ring of (x tile 128 x 64, w tile 256 x 64) stages, 128-byte swizzle
//   warp 1      issues every MMA into one of two 256-column accumulators
//   warps 2-5   epilogue: accumulator -> registers -> bf16 -> y, while the MMAs of the next tile fill the other accumulator
// Persistent: one CTA per SM; consecutive CTAs take the output tiles of the same 128 rows of x, so that x is read from
// DRAM once and the weights stay in L2.  Every wait is bounded; on expiry the status word is set and the kernel returns.
#include "../../include/httm.h"
#include "httm_internal.h"
#include "tc_sm100.cuh"

namespace httm {

namespace {

constexpr int BM = 128, BN = 256, BK = 64;
constexpr int LIN_STAGES = 4;
constexpr int A_BYTES = BM * BK * 2, B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;   // 16 + 32 KB
constexpr int LIN_THREADS = 192;
constexpr int LIN_SMEM = LIN_STAGES * STAGE_BYTES + 256 + 1024 /*alignment slack*/;

struct LinBars {
    uint64_t full[LIN_STAGES], empty[LIN_STAGES];
    uint64_t acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int abort_flag;
};

__global__ void __launch_bounds__(LIN_THREADS, 1)
linear_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, __nv_bfloat16* y, int64_t ldy,
              int64_t n_rows, int out_features, int k_blocks, int n_tiles, int64_t total_tiles, int32_t* status) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const uint32_t s0 = tc::smem_addr(smem);
    LinBars* bars = reinterpret_cast<LinBars*>(smem + LIN_STAGES * STAGE_BYTES);
    volatile int* abort_flag = &bars->abort_flag;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        bars->abort_flag = 0;
        for (int i = 0; i < LIN_STAGES; ++i) {
            tc::mbar_init(tc::smem_addr(&bars->full[i]), 1);
            tc::mbar_init(tc::smem_addr(&bars->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            tc::mbar_init(tc::smem_addr(&bars->acc_full[i]), 1);
            tc::mbar_init(tc::smem_addr(&bars->acc_empty[i]), 4);   // one arrival per epilogue warp
        }
        tc::fence_barrier_init();
        tc::prefetch_tensormap(&map_x);
        tc::prefetch_tensormap(&map_w);
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_addr(&bars->tmem_base), 512);
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem = bars->tmem_base;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (tc::elect_one()) {
            uint32_t cnt = 0;   // stages filled so far
            bool ok = true;
            for (int64_t t = blockIdx.x; ok && t < total_tiles; t += gridDim.x) {
                const int m0 = (int)(t / n_tiles) * BM, n0 = (int)(t % n_tiles) * BN;
                for (int kb = 0; kb < k_blocks; ++kb, ++cnt) {
                    const uint32_t st = cnt % LIN_STAGES, ph = (cnt / LIN_STAGES) & 1u;
                    ok = tc::mbar_wait(tc::smem_addr(&bars->empty[st]), ph ^ 1u, abort_flag);
                    if (!ok) break;
                    const uint32_t bar = tc::smem_addr(&bars->full[st]);
                    tc::mbar_expect_tx(bar, STAGE_BYTES);   // rows past the end of x or w are zero filled and still counted
                    tc::tma_load_3d(s0 + st * STAGE_BYTES, &map_x, bar, 0, m0, kb);
                    tc::tma_load_3d(s0 + st * STAGE_BYTES + A_BYTES, &map_w, bar, 0, n0, kb);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (tc::elect_one()) {
            constexpr uint32_t idesc = tc::idesc_bf16(BM, BN, false, false);
            const uint64_t d0 = tc::smem_desc_sw128(s0);
            uint32_t cnt = 0, tile_i = 0;
            bool ok = true;
            for (int64_t t = blockIdx.x; ok && t < total_tiles; t += gridDim.x, ++tile_i) {
                const uint32_t acc = tile_i & 1u;
                ok = tc::mbar_wait(tc::smem_addr(&bars->acc_empty[acc]), ((tile_i >> 1) & 1u) ^ 1u, abort_flag);
                if (!ok) break;
                tc::fence_after_sync();
                for (int kb = 0; kb < k_blocks; ++kb, ++cnt) {
                    const uint32_t st = cnt % LIN_STAGES, ph = (cnt / LIN_STAGES) & 1u;
                    ok = tc::mbar_wait(tc::smem_addr(&bars->full[st]), ph, abort_flag);
                    if (!ok) break;
                    tc::fence_after_sync();
                    const uint64_t da = d0 + (uint64_t)st * (STAGE_BYTES >> 4), db = da + (A_BYTES >> 4);
#pragma unroll
                    for (int k = 0; k < 4; ++k)   // four K = 16 steps of the 64-channel stage (32 bytes = 2 descriptor units each)
                        tc::mma_ss(tmem + acc * BN, da + 2 * k, db + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
                    tc::mma_commit(tc::smem_addr(&bars->empty[st]));   // the stage may be refilled when these MMAs are done
                }
                if (ok) tc::mma_commit(tc::smem_addr(&bars->acc_full[acc]));
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue: thread = row of the tile
        const int row = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        uint32_t tile_i = 0;
        bool ok = true;
        for (int64_t t = blockIdx.x; ok && t < total_tiles; t += gridDim.x, ++tile_i) {
            const uint32_t acc = tile_i & 1u;
            const int64_t m = (t / n_tiles) * BM + row;
            const int n0 = (int)(t % n_tiles) * BN;
            ok = __all_sync(0xffffffffu, tc::mbar_wait(tc::smem_addr(&bars->acc_full[acc]), (tile_i >> 1) & 1u, abort_flag));
            if (!ok) break;
            tc::fence_after_sync();
            __nv_bfloat16* dst = y + m * ldy + n0;
#pragma unroll 1
            for (int c = 0; c < BN; c += 32) {
                uint32_t r[32];
                tc::tmem_ld32(tmem + acc * BN + c + lane_addr, r);
                tc::tmem_wait_ld();
                if (m < n_rows) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {   // 8 columns = 16 bytes per store (out_features is a multiple of 8)
                        if (n0 + c + 8 * q < out_features) {
                            uint4 o;
                            __nv_bfloat162 p;
                            p = __floats2bfloat162_rn(__uint_as_float(r[8 * q + 0]), __uint_as_float(r[8 * q + 1]));
                            o.x = *reinterpret_cast<uint32_t*>(&p);
                            p = __floats2bfloat162_rn(__uint_as_float(r[8 * q + 2]), __uint_as_float(r[8 * q + 3]));
                            o.y = *reinterpret_cast<uint32_t*>(&p);
                            p = __floats2bfloat162_rn(__uint_as_float(r[8 * q + 4]), __uint_as_float(r[8 * q + 5]));
                            o.z = *reinterpret_cast<uint32_t*>(&p);
                            p = __floats2bfloat162_rn(__uint_as_float(r[8 * q + 6]), __uint_as_float(r[8 * q + 7]));
                            o.w = *reinterpret_cast<uint32_t*>(&p);
                            *reinterpret_cast<uint4*>(dst + c + 8 * q) = o;
                        }
                    }
                }
            }
            tc::fence_before_sync();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(tc::smem_addr(&bars->acc_empty[acc]));   // the accumulator may be overwritten
        }
    }
    tc::fence_before_sync();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem, 512);
    if (tid == 0 && bars->abort_flag) atomicCAS(status, kDevOk, kDevTimeoutLinear);
}

}  // namespace

cudaError_t configure_linear() { return cudaFuncSetAttribute(linear_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, LIN_SMEM); }

// Returns cudaErrorInvalidValue if a tensor map cannot be encoded.
cudaError_t launch_linear(const LinearArgs& a, int sm_count, cudaStream_t stream) {
    CUtensorMap mx, mw;
    // a matrix [rows][in] as {64 channels, rows, in / 64 blocks of 64 channels}: the block index is the third coordinate
    const int k_blocks = a.in_features / BK;
    if (!encode_rows_tensor_map(&mx, a.x, a.n_rows, k_blocks, a.ldx, BK, BM) ||
        !encode_rows_tensor_map(&mw, a.w, a.out_features, k_blocks, a.ldw, BK, BN))
        return cudaErrorInvalidValue;
    const int n_tiles = (a.out_features + BN - 1) / BN;
    const int64_t total = ((a.n_rows + BM - 1) / BM) * n_tiles;
    int ctas = sm_count < 1 ? 1 : sm_count;
    if (ctas > total) ctas = (int)total;
    if (ctas < 1) return cudaSuccess;   // nothing to do
    linear_kernel<<<ctas, LIN_THREADS, LIN_SMEM, stream>>>(mx, mw, a.y, a.ldy, a.n_rows, a.out_features, k_blocks, n_tiles, total, a.status);
    return cudaGetLastError();
}

}  // namespace httm
