// Softmax attention (Eq. 3-4) on the 5th-generation tensor cores:
//   out[h][m] = softmax(q[h][m] . k[h]^T / sqrt(64)) v[h]
//
// One CTA owns TWO 128-row query tiles (A, B) of one head and walks the keys in 128-key tiles.
//   warp 0      TMA producer: Q tiles once, then a ring of K and V tiles (128-byte swizzle)
//   warp 1      issues every tcgen05.mma: S = Q_X K^T (operands in shared memory) and
//               O_X += P V (P read from tensor memory, V MN-major from shared memory)
//   warps 2-5   softmax of tile A: one thread per query row, S read from tensor memory,
//               P written back over S as bf16 pairs; warps 6-9 the same for tile B
// Score tiles are numbered k = 2 j + x (key tile j, query tile x) and live in a ring of THREE
// 128-column buffers of tensor memory shared by both query tiles (tile k in buffer k mod 3); the
// accumulators O_A, O_B take the remaining 2 x 64 columns.  S(k+3) is issued right after P(k) V, into
// the buffer that P(k) V releases, so the scores of a softmax warp's next tile are ready before it
// finishes the current one: the softmax warps never wait for the tensor core in steady state.
// A row's stabiliser is the maximum of its first score tile; later tiles take their exponentials without
// looking for the maximum first and are redone (with O rescaled in place) only if their weights would
// overflow, which bounded scores never do.  Every wait is bounded; on expiry the kernel
// records kDevTimeoutAttention in the status word, releases its tensor memory and returns.
#include "httm_internal.h"
#include "tc_sm100.cuh"

#include <type_traits>

namespace httm {

namespace {

constexpr int BM = 128;            // rows per query tile
constexpr int BN = 128;            // keys per tile
constexpr int KV_STAGES = 3;
constexpr int TILE_BYTES = BM * kRowBytes;   // 16 KB
constexpr int NTHREADS = 320;   // producer warp, MMA warp, 2 x 4 softmax warps: registers are granted per four warps, so 168 per thread as with twelve
constexpr int TMEM_COLS = 512;
constexpr int kTableHeads = 256;   // head tables (per-head query lengths) of up to this many heads are kept in shared memory
constexpr int kOutRowPitch = kRowBytes + 16;             // staged output rows: the pitch keeps 16-byte stores of a quarter warp on distinct banks
constexpr int kOutStageBytes = 8 * 32 * kOutRowPitch;   // eight softmax warps x 32 output rows, staged for bulk stores
constexpr int SMEM_BYTES = (2 + 2 * KV_STAGES) * TILE_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/ + 1024 /*row exchange*/ +
                           (2 * kTableHeads + 4) * 4 /*head tables*/ + kOutStageBytes;
constexpr int kPColumn = 64;                  // P (bf16 pairs, 64 columns) lies over columns 64 .. 127 of its S
constexpr float kSumLimit = 1.2676506e30f;   // 2^100: a tile whose row sum of weights reaches it is redone with a raised maximum

struct Barriers {
    uint64_t q_full;
    uint64_t k_full[KV_STAGES], k_empty[KV_STAGES];
    uint64_t v_full[KV_STAGES], v_empty[KV_STAGES];
    uint64_t s_full[3], p_full[3];   // per score buffer
    uint64_t o_done[2];              // per query tile: one completion per P V
    uint64_t o_final;
    uint64_t q_free;                 // every S = Q K^T of the pass has been computed: the Q tiles may be replaced
    uint64_t x_full, x_done;         // single pass: tile B's (max, sum) published / tile A done reading O_B
    uint32_t tmem_base;
    int abort_flag;
};

struct TcParams {
    __nv_bfloat16* out;
    int64_t out_stride_head, out_stride_token;
    int32_t m_q, m_k;
    float scale_log2;
    int32_t* status;
    int32_t tiles_per_head, total_tiles, rounds;  // query tiles per head and in all heads; rounds of pair passes
    const int32_t* mq_head;      // optional: per-head query length (then m_q is the row stride and tile_prefix the tile table)
    const int32_t* tile_prefix;
    int32_t heads;
    const int32_t* group_start;  // optional (UNMERGE): members of every merged query row, see AttentionArgs
    const int32_t* group_member;
    int32_t n_tokens;
    const __nv_bfloat16 *q, *k;  // the rows themselves, for the tile that is redone (element strides)
    int64_t q_stride_head, q_stride_token, k_stride_head, k_stride_token;
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

// 2^t for two values without the special-function unit.  The arguments are clamped to [-125, 125] (an argument of
// 125 or more gives 2^125, which the caller's test of the tile's row sum catches; without the clamps the exponent
// arithmetic below would wrap).  Then round-to-nearest range reduction t = n + f, f in [-0.5, 0.5] (the integer lands
// in the low mantissa bits of t + 1.5 * 2^23), a cubic minimax polynomial for 2^f (relative error < 1e-4, far below
// the bf16 rounding of P) evaluated with packed fp32 FMAs, and n added to the exponent field.
__device__ __forceinline__ float2 exp2_poly2(float2 t) {
    const float kMagic = 12582912.0f;
    t.x = fminf(fmaxf(t.x, -125.0f), 125.0f);
    t.y = fminf(fmaxf(t.y, -125.0f), 125.0f);
    const float2 tt = tc::fadd2(t, make_float2(kMagic, kMagic));
    const float2 n = tc::fadd2(tt, make_float2(-kMagic, -kMagic));
    const float2 f = tc::ffma2(n, make_float2(-1.0f, -1.0f), t);
    float2 q = tc::ffma2(make_float2(0.055171460f, 0.055171460f), f, make_float2(0.24261086f, 0.24261086f));
    q = tc::ffma2(q, f, make_float2(0.69326097f, 0.69326097f));
    q = tc::ffma2(q, f, make_float2(0.99992812f, 0.99992812f));
    return make_float2(__int_as_float(__float_as_int(q.x) + (__float_as_int(tt.x) << 23)),
                       __int_as_float(__float_as_int(q.y) + (__float_as_int(tt.y) << 23)));
}
// Of every eight pairs of scores, the pairs whose bit is set here take the polynomial (FMA pipe), the
// others ex2.approx (special-function unit, 16 results per clock per SM: with every exponential there,
// the softmax of two query tiles needs 2048 cycles against 1056 of tensor-core work).  The polynomial
// costs about ten issue slots per pair against two.  Measured at 10500 x 10500 x 16 heads with the
// persistent kernel: 0/8: 545 us, 1/8: 510 us, 2/8: 481 us, 3/8: 497-504 us, 4/8: 570 us, 8/8: 790 us
// (alternating 2/8 and 3/8 over the 16-column groups: 480 us).
constexpr uint32_t kPolyPairs = 0x11;   // pairs 0 and 4 of 8

// A score tile whose weights overflowed with the stabiliser at hand is done again here, for one query row per thread:
// its 128 scores are recomputed from the rows in global memory by plain fp32 FMAs (the tile in tensor memory is
// partly overwritten by the weights, the key tile in shared memory may have been replaced), first for their maximum,
// then for the weights 2^(s c - m'), m' = max(m, c max s), written as bf16 pairs to the eight-column groups at
// `t_p`.  Returns m' and the row's sum of weights.  Only inputs whose scores differ by more than 69 (100 in base 2)
// between key tiles ever come here; it is kept out of line so that it costs the ordinary tiles no registers.
struct RedoneTile {
    float m, sum;
};
__device__ __noinline__ RedoneTile redo_score_tile(const __nv_bfloat16* q_row, const __nv_bfloat16* k_rows, int64_t k_stride_token, int valid,
                                                   float c, float m_old, uint32_t t_p) {
    float qf[kHeadDim];
    if (q_row) {
#pragma unroll
        for (int i = 0; i < kHeadDim / 8; ++i) {
            const uint4 u = __ldg(reinterpret_cast<const uint4*>(q_row) + i);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                qf[8 * i + 2 * e] = __uint_as_float(w[e] << 16);
                qf[8 * i + 2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
            }
        }
    } else {   // a row past the end of the queries (zero-filled by the tile load)
#pragma unroll
        for (int i = 0; i < kHeadDim; ++i) qf[i] = 0.f;
    }
    auto score = [&](int key) {
        const uint4* kr = reinterpret_cast<const uint4*>(k_rows + (int64_t)key * k_stride_token);
        float a0 = 0.f, a1 = 0.f;
#pragma unroll
        for (int i = 0; i < kHeadDim / 8; ++i) {
            const uint4 u = __ldg(kr + i);
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                a0 = fmaf(qf[8 * i + 2 * e], __uint_as_float(w[e] << 16), a0);
                a1 = fmaf(qf[8 * i + 2 * e + 1], __uint_as_float(w[e] & 0xffff0000u), a1);
            }
        }
        return a0 + a1;
    };
    float mx = -INFINITY;
#pragma unroll 1
    for (int key = 0; key < valid; ++key) mx = fmaxf(mx, score(key));
    RedoneTile r;
    r.m = fmaxf(m_old, mx * c);
    r.sum = 0.f;
#pragma unroll 1
    for (int cc = 0; cc < 8; ++cc) {
        uint32_t pk[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int key = cc * 16 + 2 * i;
            const float e0 = key < valid ? exp2f(fmaf(score(key), c, -r.m)) : 0.f;
            const float e1 = key + 1 < valid ? exp2f(fmaf(score(key + 1), c, -r.m)) : 0.f;
            r.sum += e0 + e1;
            pk[i] = pack_bf16(e0, e1);
        }
        tc::tmem_st8(t_p + cc * 8, pk);
    }
    return r;
}

// Work decomposition.  The query tiles of all heads form one list (head-major, T tiles).  With G CTAs
// (one per SM), round r < R = T / (2 G) gives CTA c the two tiles 2 (r G + c), +1: a PAIR pass (tiles A and B
// share the K/V stream) if they belong to the same head, else two single passes.  The remaining
// T - 2 G R < 2 G tiles are one more partial round of pairs if there are more than G of them, else they are
// dealt one per CTA as SINGLE passes: the same machinery with ONE query tile whose
// even key tiles go to softmax group A / accumulator O_A and odd ones to group B / O_B (two partial
// softmaxes over disjoint keys), combined in the epilogue; a single pass takes about half a pair pass.
// Either way score tile k is handled by group k mod 2 in buffer k mod 3.  All CTAs work on neighbouring
// tiles at any time (K/V of one or two heads stay in L2), and the SMs finish within half a pass of each
// other, whereas a grid of 672 two-tile CTAs on 148 SMs runs 4.54 waves as 5.
struct Pass {
    int head, tile;   // tile = index of query tile A inside the head
    bool pair;
};
template <bool VAR>   // VAR: the heads differ in query length (tile table in device memory)
struct PassWalker {
    int r = 0, sub = 0;
    int rounds, total, tiles_per_head;
    const int32_t* prefix;   // optional: first tile of every head (heads + 1 entries) when the heads differ in length
    int heads;
    __device__ PassWalker(int rounds_, int total_, int tph, const int32_t* prefix_, int heads_)
        : rounds(rounds_), total(total_), tiles_per_head(tph), prefix(prefix_), heads(heads_) {
        if (VAR) {
            total = prefix[heads];
            rounds = total / (2 * (int)gridDim.x);
        }
    }
    __device__ int head_of(int t) const {
        if (!VAR) return t / tiles_per_head;
        int lo = 0, hi = heads - 1;   // largest h with prefix[h] <= t
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (prefix[mid] <= t)
                lo = mid;
            else
                hi = mid - 1;
        }
        return lo;
    }
    __device__ void set(Pass* ps, int t, bool pair) {
        ps->head = head_of(t);
        ps->tile = t - (VAR ? prefix[ps->head] : ps->head * tiles_per_head);
        ps->pair = pair;
    }
    __device__ bool same_head(int t) const {   // tiles t and t + 1
        if (!VAR) return t / tiles_per_head == (t + 1) / tiles_per_head;
        return t + 1 < prefix[head_of(t) + 1];
    }
    __device__ bool next(Pass* ps) {
        const int G = gridDim.x, c = blockIdx.x;
        const int rem = total - 2 * G * rounds;               // tiles left after the full rounds, < 2 G
        const int pair_rounds = rounds + (rem > G ? 1 : 0);   // more than G left: one more (partial) round of pairs
        if (r < pair_rounds) {
            const int t = 2 * (r * G + c);
            if (t + 1 < total && same_head(t)) {
                set(ps, t, true);
                ++r;
                return true;
            }
            if (t + sub < total) {   // the two tiles straddle a head boundary (two single passes, the cost of one pair pass),
                set(ps, t + sub, false);   // or only one tile is left
                if (sub == 1) ++r;
                sub ^= 1;
                return true;
            }
            r = pair_rounds + 1;
            return false;
        }
        if (r > pair_rounds || rem > G) return false;
        const int t = 2 * G * rounds + c;                     // at most G left: one single pass each
        ++r;
        if (t >= total) return false;
        set(ps, t, false);
        return true;
    }
};
// Completions a pass adds to each barrier family, so that every role can carry the phase parities from
// pass to pass: stage st of the K/V ring completes once per key tile j with j mod 3 == st; score buffer b
// once per score tile k with k mod 3 == b (2 n tiles in a pair pass, n in a single pass).
__device__ __forceinline__ int count_mod3(int n, int r) { return (n - r + 2) / 3; }

// Where the 32 output rows of a softmax warp go.  UNMERGE (Eq. 5-7 folded into the epilogue): row `grow` is the attention
// output of a merged query and goes to every original token of its group, at the token's place in the final
// [tokens][heads x 64] tensor; the first four members are fetched ahead of the epilogue, larger groups read the rest
// of their list when they are stored.  Otherwise the row goes to row `grow` of the merged output.
struct RowTargets {
    int count;      // tokens this thread's row is written to (0: the row does not exist)
    int token[4];   // the first four of them
    int first;      // index of the group's first member in the member list
};
template <bool UNMERGE>
__device__ __forceinline__ RowTargets row_targets(const TcParams& p, int head, int grow, bool valid) {
    RowTargets t{};
    if (!valid) return t;
    if (!UNMERGE) {
        t.count = 1;
        t.token[0] = grow;
        return t;
    }
    const int32_t* gs = p.group_start + (int64_t)head * (p.m_q + 1) + grow;
    const int32_t* member = p.group_member + (int64_t)head * p.n_tokens;
    t.first = __ldg(gs);
    t.count = __ldg(gs + 1) - t.first;
#pragma unroll
    for (int i = 0; i < 4; ++i) t.token[i] = i < t.count ? __ldg(member + t.first + i) : 0;
    return t;
}
// Every lane hands in its row (eight 16-byte pieces) and its targets.  The row is staged in shared memory and leaves as
// one 128-byte bulk copy per target token (whole lines, issued by the row's own thread: no loop over the warp's rows).
// The copies are asynchronous: bulk_stores_done() must come before the stage is rewritten and before the kernel ends.
__device__ __forceinline__ void bulk_stores_done() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
template <bool UNMERGE>
__device__ __forceinline__ void store_rows(const TcParams& p, int head, const uint4 (&v)[8], const RowTargets& t, unsigned char* stage, int lane) {
    bulk_stores_done();   // (the copies of the previous pass have long left)
    unsigned char* row = stage + lane * kOutRowPitch;
#pragma unroll
    for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(row + c * 16) = v[c];
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the staged row is visible to the bulk-copy engine
    const uint32_t src = tc::smem_addr(row);
    __nv_bfloat16* base = p.out + (int64_t)head * p.out_stride_head;
    const int32_t* member = UNMERGE ? p.group_member + (int64_t)head * p.n_tokens + t.first : nullptr;
    auto send = [&](int token) {
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(base + (int64_t)token * p.out_stride_token), "r"(src),
                     "n"(kRowBytes)
                     : "memory");
    };
#pragma unroll
    for (int q = 0; q < 4; ++q)
        if (q < t.count) send(t.token[q]);
    for (int q = 4; q < t.count; ++q) send(__ldg(member + q));
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}

template <bool VAR, bool UNMERGE>
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
    const int n_tiles = (p.m_k + BN - 1) / BN;
    const int kv_cnt[3] = {count_mod3(n_tiles, 0), count_mod3(n_tiles, 1), count_mod3(n_tiles, 2)};   // per pass

    if (tid == 0) {
        bars->abort_flag = 0;
        tc::mbar_init(tc::smem_addr(&bars->q_full), 1);
        for (int i = 0; i < KV_STAGES; ++i) {
            tc::mbar_init(tc::smem_addr(&bars->k_full[i]), 1);
            tc::mbar_init(tc::smem_addr(&bars->k_empty[i]), 1);
            tc::mbar_init(tc::smem_addr(&bars->v_full[i]), 1);
            tc::mbar_init(tc::smem_addr(&bars->v_empty[i]), 1);
        }
        for (int b = 0; b < 3; ++b) {
            tc::mbar_init(tc::smem_addr(&bars->s_full[b]), 1);
            tc::mbar_init(tc::smem_addr(&bars->p_full[b]), 128);
        }
        tc::mbar_init(tc::smem_addr(&bars->o_done[0]), 1);
        tc::mbar_init(tc::smem_addr(&bars->o_done[1]), 1);
        tc::mbar_init(tc::smem_addr(&bars->o_final), 1);
        tc::mbar_init(tc::smem_addr(&bars->q_free), 1);
        tc::mbar_init(tc::smem_addr(&bars->x_full), 128);
        tc::mbar_init(tc::smem_addr(&bars->x_done), 128);
        tc::fence_barrier_init();
        tc::prefetch_tensormap(&map_q);
        tc::prefetch_tensormap(&map_k);
        tc::prefetch_tensormap(&map_v);
    }
    // per-head query lengths: every pass looks its head up (binary search over the tile table): keep the tables on chip
    int32_t* s_prefix = reinterpret_cast<int32_t*>(smem + (2 + 2 * KV_STAGES) * TILE_BYTES + 256 + 1024);   // [heads + 1]
    int32_t* s_mq = s_prefix + kTableHeads + 4;                                                               // [heads]
    const bool tables_on_chip = VAR && p.heads <= kTableHeads;
    if (tables_on_chip) {
        for (int i = tid; i <= p.heads; i += NTHREADS) {
            s_prefix[i] = p.tile_prefix[i];
            if (i < p.heads) s_mq[i] = p.mq_head[i];
        }
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_addr(&bars->tmem_base), TMEM_COLS);
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    const uint32_t tmem = bars->tmem_base;
    // columns: score buffers [0,128) [128,256) [256,384); O_A [384,448)  O_B [448,512); P overlays the last 64 columns of its S
    const int32_t* mq_table = tables_on_chip ? s_mq : p.mq_head;
    PassWalker<VAR> walker(p.rounds, p.total_tiles, p.tiles_per_head, tables_on_chip ? s_prefix : p.tile_prefix, p.heads);
    Pass ps;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (tc::elect_one()) {
            uint32_t kv_base[3] = {0, 0, 0};   // completions of each ring stage before this pass (parity bit)
            for (int pass = 0; walker.next(&ps); ++pass) {
                // The Q tiles are free once the previous pass's last S has been computed (a few key tiles before its end):
                // the next pass's Q and first K / V tiles arrive while the previous pass finishes, the ring runs on.
                if (pass > 0 && !tc::mbar_wait(tc::smem_addr(&bars->q_free), (uint32_t)(pass - 1) & 1u, abort_flag)) break;
                const uint32_t qb = tc::smem_addr(&bars->q_full);
                tc::mbar_expect_tx(qb, ps.pair ? 2 * TILE_BYTES : TILE_BYTES);
                tc::tma_load_3d(s_q, &map_q, qb, 0, ps.tile * BM, ps.head);
                if (ps.pair) tc::tma_load_3d(s_q + TILE_BYTES, &map_q, qb, 0, (ps.tile + 1) * BM, ps.head);
                bool ok = true;
                for (int j = 0; j < n_tiles; ++j) {
                    const int st = j % KV_STAGES;
                    const uint32_t fill = kv_base[st] + (uint32_t)(j / KV_STAGES);         // completion index of tile j in stage st
                    const uint32_t par = fill & 1u;
                    if (fill > 0 && !(ok = tc::mbar_wait(tc::smem_addr(&bars->k_empty[st]), par ^ 1u, abort_flag))) break;
                    const uint32_t kb = tc::smem_addr(&bars->k_full[st]);
                    tc::mbar_expect_tx(kb, TILE_BYTES);
                    tc::tma_load_3d(s_k + st * TILE_BYTES, &map_k, kb, 0, j * BN, ps.head);
                    if (fill > 0 && !(ok = tc::mbar_wait(tc::smem_addr(&bars->v_empty[st]), par ^ 1u, abort_flag))) break;
                    const uint32_t vb = tc::smem_addr(&bars->v_full[st]);
                    tc::mbar_expect_tx(vb, TILE_BYTES);
                    tc::tma_load_3d(s_v + st * TILE_BYTES, &map_v, vb, 0, j * BN, ps.head);
                }
                if (!ok) break;
#pragma unroll
                for (int st = 0; st < 3; ++st) kv_base[st] += (uint32_t)kv_cnt[st];
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // Every operand of a tcgen05.mma below is a loop-invariant base plus a compile-time offset (score
        // buffer, query tile and ring stage are template constants of the unrolled steps): operands that
        // are recomputed per instruction at run time make the issue itself cost more than the MMA.
        if (tc::elect_one()) {
            constexpr uint32_t idesc_qk = tc::idesc_bf16(BM, BN, false, false);
            constexpr uint32_t idesc_pv = tc::idesc_bf16(BM, kHeadDim, false, true);
            const uint64_t dq0 = tc::smem_desc_sw128(s_q);
            const uint64_t dk0 = tc::smem_desc_sw128(s_k), dv0 = tc::smem_desc_sw128(s_v);
            constexpr uint64_t kStageStep = TILE_BYTES >> 4;   // descriptor address field counts 16-byte units
            // S(buffer) = Q_x K(stage)^T: four K=16 steps, 32 bytes apart inside the 128-byte rows
            auto issue_qk = [&](uint32_t t_s, uint64_t dq, uint64_t dk, uint32_t bar) {
                tc::mma_ss_c<false>(t_s, dq, dk, idesc_qk);
                tc::mma_ss_c<true>(t_s, dq + 2, dk + 2, idesc_qk);
                tc::mma_ss_c<true>(t_s, dq + 4, dk + 4, idesc_qk);
                tc::mma_ss_c<true>(t_s, dq + 6, dk + 6, idesc_qk);
                tc::mma_commit(bar);
            };
            // O_x += P(buffer) V(stage): eight K=16 steps; P advances 8 columns (16 bf16), V 16 rows (2048 bytes).
            // O starts at zero (written by the softmax threads), so every step accumulates.
            auto issue_pv = [&](uint32_t t_o, uint32_t t_p, uint64_t dv) {
#pragma unroll
                for (int k = 0; k < 8; ++k) tc::mma_ts_c<true>(t_o, t_p + 8 * k, dv + (uint64_t)(k * 128), idesc_pv);
            };
            uint32_t kv_base[3] = {0, 0, 0}, sp_base[3] = {0, 0, 0};   // completions before this pass: ring stages, score buffers
            // PAIR pass, score tile k = k0 + C with k0 a multiple of 6 (round_par = parity of k0 / 6).
            auto step_pair = [&](auto c_c, int k0, uint32_t round_par, int n_score) -> bool {
                constexpr int C = decltype(c_c)::value;
                constexpr int B = C % 3, X = C % 2, ST = (C >> 1) % KV_STAGES;                 // this tile: P(k) V
                constexpr int X3 = 1 - X, J3 = (C + 3) >> 1, ST3 = J3 % KV_STAGES;            // tile k + 3: next S in the same buffer
                const uint32_t t_buf = tmem + B * BN, t_o = tmem + 3 * BN + X * kHeadDim;
                if (X == 0 && !tc::mbar_wait(tc::smem_addr(&bars->v_full[ST]), (kv_base[ST] + round_par) & 1u, abort_flag)) return false;
                if (!tc::mbar_wait(tc::smem_addr(&bars->p_full[B]), (sp_base[B] + (C / 3)) & 1u, abort_flag)) return false;
                tc::fence_after_sync();
                issue_pv(t_o, t_buf + kPColumn, dv0 + ST * kStageStep);
                tc::mma_commit(tc::smem_addr(&bars->o_done[X]));
                if (X == 1) tc::mma_commit(tc::smem_addr(&bars->v_empty[ST]));
                if (k0 + C + 3 < n_score) {
                    if (X3 == 0) {
                        if (!tc::mbar_wait(tc::smem_addr(&bars->k_full[ST3]), (kv_base[ST3] + round_par + (J3 >= 3 ? 1u : 0u)) & 1u, abort_flag)) return false;
                        tc::fence_after_sync();
                    }
                    issue_qk(t_buf, dq0 + X3 * kStageStep, dk0 + ST3 * kStageStep, tc::smem_addr(&bars->s_full[B]));
                    if (X3 == 1) tc::mma_commit(tc::smem_addr(&bars->k_empty[ST3]));
                    if (k0 + C + 4 == n_score) tc::mma_commit(tc::smem_addr(&bars->q_free));   // that was the last S of the pass
                }
                return true;
            };
            // SINGLE pass, score tile k = key tile k = k0 + C with k0 a multiple of 6: buffer and ring stage k mod 3,
            // softmax group and accumulator k mod 2.
            auto step_single = [&](auto c_c, int k0) -> bool {
                constexpr int C = decltype(c_c)::value;
                constexpr int B = C % 3, X = C % 2;
                constexpr uint32_t IDX = C / 3;   // completion index of this tile in its buffer / stage, modulo 2 (k0 / 3 is even)
                const uint32_t t_buf = tmem + B * BN, t_o = tmem + 3 * BN + X * kHeadDim;
                if (!tc::mbar_wait(tc::smem_addr(&bars->v_full[B]), (kv_base[B] + IDX) & 1u, abort_flag)) return false;
                if (!tc::mbar_wait(tc::smem_addr(&bars->p_full[B]), (sp_base[B] + IDX) & 1u, abort_flag)) return false;
                tc::fence_after_sync();
                issue_pv(t_o, t_buf + kPColumn, dv0 + B * kStageStep);
                tc::mma_commit(tc::smem_addr(&bars->o_done[X]));
                tc::mma_commit(tc::smem_addr(&bars->v_empty[B]));
                if (k0 + C + 3 < n_tiles) {
                    if (!tc::mbar_wait(tc::smem_addr(&bars->k_full[B]), (kv_base[B] + IDX + 1u) & 1u, abort_flag)) return false;
                    tc::fence_after_sync();
                    issue_qk(t_buf, dq0, dk0 + B * kStageStep, tc::smem_addr(&bars->s_full[B]));
                    tc::mma_commit(tc::smem_addr(&bars->k_empty[B]));
                    if (k0 + C + 4 == n_tiles) tc::mma_commit(tc::smem_addr(&bars->q_free));   // that was the last S of the pass
                }
                return true;
            };
            static_assert(KV_STAGES == 3, "the issue loops are unrolled over three ring stages and three score buffers");
            bool ok = true;
            for (int pass = 0; ok && walker.next(&ps); ++pass) {
                ok = tc::mbar_wait(tc::smem_addr(&bars->q_full), (uint32_t)pass & 1u, abort_flag) &&
                     tc::mbar_wait(tc::smem_addr(&bars->k_full[0]), kv_base[0] & 1u, abort_flag);
                if (!ok) break;
                tc::fence_after_sync();
                if (ps.pair) {
                    const int n_score = 2 * n_tiles;   // score tiles k = 2 j + x
                    // prologue: S(0), S(1) from key tile 0, S(2) from key tile 1
                    issue_qk(tmem, dq0, dk0, tc::smem_addr(&bars->s_full[0]));
                    issue_qk(tmem + BN, dq0 + kStageStep, dk0, tc::smem_addr(&bars->s_full[1]));
                    tc::mma_commit(tc::smem_addr(&bars->k_empty[0]));
                    if (n_score > 2) {
                        if (!(ok = tc::mbar_wait(tc::smem_addr(&bars->k_full[1]), kv_base[1] & 1u, abort_flag))) break;
                        tc::fence_after_sync();
                        issue_qk(tmem + 2 * BN, dq0, dk0 + kStageStep, tc::smem_addr(&bars->s_full[2]));
                    }
                    if (n_score <= 3) tc::mma_commit(tc::smem_addr(&bars->q_free));
                    uint32_t round_par = 0;
                    for (int k0 = 0; ok && k0 < n_score; k0 += 6, round_par ^= 1u) {
                        ok = step_pair(std::integral_constant<int, 0>{}, k0, round_par, n_score);
                        if (ok) ok = step_pair(std::integral_constant<int, 1>{}, k0, round_par, n_score);   // n_score is even
                        if (ok && k0 + 2 < n_score) ok = step_pair(std::integral_constant<int, 2>{}, k0, round_par, n_score);
                        if (ok && k0 + 2 < n_score) ok = step_pair(std::integral_constant<int, 3>{}, k0, round_par, n_score);
                        if (ok && k0 + 4 < n_score) ok = step_pair(std::integral_constant<int, 4>{}, k0, round_par, n_score);
                        if (ok && k0 + 4 < n_score) ok = step_pair(std::integral_constant<int, 5>{}, k0, round_par, n_score);
                    }
#pragma unroll
                    for (int b = 0; b < 3; ++b) sp_base[b] += (uint32_t)count_mod3(n_score, b);
                } else {
                    // prologue: S(0), S(1), S(2) from key tiles 0, 1, 2
                    issue_qk(tmem, dq0, dk0, tc::smem_addr(&bars->s_full[0]));
                    tc::mma_commit(tc::smem_addr(&bars->k_empty[0]));
                    if (n_tiles > 1) {
                        if (!(ok = tc::mbar_wait(tc::smem_addr(&bars->k_full[1]), kv_base[1] & 1u, abort_flag))) break;
                        tc::fence_after_sync();
                        issue_qk(tmem + BN, dq0, dk0 + kStageStep, tc::smem_addr(&bars->s_full[1]));
                        tc::mma_commit(tc::smem_addr(&bars->k_empty[1]));
                    }
                    if (n_tiles > 2) {
                        if (!(ok = tc::mbar_wait(tc::smem_addr(&bars->k_full[2]), kv_base[2] & 1u, abort_flag))) break;
                        tc::fence_after_sync();
                        issue_qk(tmem + 2 * BN, dq0, dk0 + 2 * kStageStep, tc::smem_addr(&bars->s_full[2]));
                        tc::mma_commit(tc::smem_addr(&bars->k_empty[2]));
                    }
                    if (n_tiles <= 3) tc::mma_commit(tc::smem_addr(&bars->q_free));
                    for (int k0 = 0; ok && k0 < n_tiles; k0 += 6) {
                        ok = step_single(std::integral_constant<int, 0>{}, k0);
                        if (ok && k0 + 1 < n_tiles) ok = step_single(std::integral_constant<int, 1>{}, k0);
                        if (ok && k0 + 2 < n_tiles) ok = step_single(std::integral_constant<int, 2>{}, k0);
                        if (ok && k0 + 3 < n_tiles) ok = step_single(std::integral_constant<int, 3>{}, k0);
                        if (ok && k0 + 4 < n_tiles) ok = step_single(std::integral_constant<int, 4>{}, k0);
                        if (ok && k0 + 5 < n_tiles) ok = step_single(std::integral_constant<int, 5>{}, k0);
                    }
#pragma unroll
                    for (int b = 0; b < 3; ++b) sp_base[b] += (uint32_t)count_mod3(n_tiles, b);
                }
                if (ok) tc::mma_commit(tc::smem_addr(&bars->o_final));
#pragma unroll
                for (int st = 0; st < 3; ++st) kv_base[st] += (uint32_t)kv_cnt[st];
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax + epilogue
        const int x = (warp - 2) >> 2;                 // 0: tile A (warps 2-5), 1: tile B (warps 6-9)
        const int row = (warp & 3) * 32 + lane;        // row inside the tile = TMEM lane
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_o = tmem + 3 * BN + x * kHeadDim + lane_addr;
        const uint32_t obar = tc::smem_addr(&bars->o_done[x]);
        const float c = p.scale_log2;
        uint32_t sp_base[3] = {0, 0, 0}, od_base = 0;   // completions before this pass: score buffers, this group's P V
        uint32_t n_single = 0;                          // single passes so far (phase of x_full / x_done)
        float2* xch = reinterpret_cast<float2*>(smem + (2 + 2 * KV_STAGES) * TILE_BYTES + 256);   // [128 rows] (max, sum) of group B
        unsigned char* out_stage = smem + (2 + 2 * KV_STAGES) * TILE_BYTES + 256 + 1024 + (2 * kTableHeads + 4) * 4 +
                                   (warp - 2) * 32 * kOutRowPitch;   // this warp's 32 output rows
        bool ok = true;
        for (int pass = 0; ok && walker.next(&ps); ++pass) {
            const int n_score = ps.pair ? 2 * n_tiles : n_tiles;
            const int mq_rows = VAR ? mq_table[ps.head] : p.m_q;   // valid query rows of this head
            // this group's score tiles are k = 2 i + x; in a pair pass they come from key tile i, in a single pass from key tile k
            const int n_own = ps.pair ? n_tiles : (n_tiles - x + 1) / 2;
            const int own_row = (ps.tile + (ps.pair ? x : 0)) * BM + row;   // this thread's query row inside the head
            const bool row_exists = own_row < mq_rows;
            const __nv_bfloat16* q_row = row_exists ? p.q + (int64_t)ps.head * p.q_stride_head + (int64_t)own_row * p.q_stride_token : nullptr;
            const __nv_bfloat16* k_head = p.k + (int64_t)ps.head * p.k_stride_head;
            {
                float m = -INFINITY, l = 0.f;
                {   // the accumulator O starts at zero: every PV step accumulates (ordered before the first p_full arrival)
                    uint32_t z[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) z[i] = 0u;
                    tc::tmem_st32(t_o, z);
                    tc::tmem_st32(t_o + 32, z);
                    if (n_own == 0) tc::tmem_wait_st();
                }
                for (int j = 0; j < n_own; ++j) {
                    const int k = 2 * j + x, buf = k % 3;                      // score tile and its buffer
                    const int key_tile = ps.pair ? j : k;
                    const uint32_t kpar = (sp_base[buf] + (uint32_t)(k / 3)) & 1u;
                    const uint32_t t_s = tmem + buf * BN + lane_addr;
                    const uint32_t sbar = tc::smem_addr(&bars->s_full[buf]), pbar = tc::smem_addr(&bars->p_full[buf]);
                    if (!(ok = tc::mbar_wait(sbar, kpar, abort_flag))) break;
                    tc::fence_after_sync();
                    uint32_t s[BN];   // fp32 bit patterns of this row of S
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) tc::tmem_ld32(t_s + cc * 32, s + cc * 32);
                    tc::tmem_wait_ld();
                    const int valid = p.m_k - key_tile * BN;
                    auto mask_tail = [&](auto first_c, auto last_c) {   // -inf for keys past the end
                        if (valid < BN) {
#pragma unroll
                            for (int i = decltype(first_c)::value; i < decltype(last_c)::value; ++i)
                                if (i >= valid) s[i] = 0xff800000u;
                        }
                    };
                    mask_tail(std::integral_constant<int, 0>{}, std::integral_constant<int, BN>{});
                    // The stabiliser m of a row is the maximum of its FIRST score tile (times c) and is raised later only if
                    // a tile would overflow: bf16 weights and the fp32 sums and accumulators do not care about a common
                    // factor, so weights of up to 2^100 are as good as weights of at most 1.  Every later tile therefore goes
                    // without a pass over its scores for the row maximum: the exponentials are taken with the m at hand,
                    // and only if some row's sum of weights reaches 2^100 (or is not a number) the tile is done again, this
                    // time with its own maximum (redo_score_tile). the sum and the accumulator O are
                    // rescaled in place once the previous P V of this query tile has completed (the next one is issued
                    // after this tile's P), and the weights are written anew.
                    auto row_max = [&]() {   // four independent chains of three-input maxima
                        float mx4[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            mx4[q] = fmaxf(__uint_as_float(s[32 * q]), __uint_as_float(s[32 * q + 1]));
#pragma unroll
                            for (int i = 2; i < 32; i += 2)
                                mx4[q] = tc::fmax3(mx4[q], __uint_as_float(s[32 * q + i]), __uint_as_float(s[32 * q + i + 1]));
                        }
                        return fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                    };
                    auto weights = [&]() {   // P = 2^(s c - m) as bf16 pairs over the LAST 64 columns of S; returns the row sum
                        const float2 c2 = make_float2(c, c), neg_m2 = make_float2(-m, -m);
                        float2 sum0 = make_float2(0.f, 0.f), sum1 = sum0;
#pragma unroll
                        for (int cc = 0; cc < 8; ++cc) {
                            uint32_t pk[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const float2 t = tc::ffma2(make_float2(__uint_as_float(s[cc * 16 + 2 * i]), __uint_as_float(s[cc * 16 + 2 * i + 1])), c2, neg_m2);
                                const float2 e = ((kPolyPairs >> i) & 1u) ? exp2_poly2(t) : make_float2(fast_exp2(t.x), fast_exp2(t.y));
                                if (i & 1)
                                    sum1 = tc::fadd2(sum1, e);
                                else
                                    sum0 = tc::fadd2(sum0, e);
                                pk[i] = pack_bf16(e.x, e.y);
                            }
                            tc::tmem_st8(t_s + kPColumn + cc * 8, pk);
                        }
                        return (sum0.x + sum0.y) + (sum1.x + sum1.y);
                    };
                    if (j == 0) m = row_max() * c;
                    float tile_sum = weights();
                    if (j > 0 && __any_sync(0xffffffffu, row_exists && !(tile_sum < kSumLimit))) {
                        if (!(ok = tc::mbar_wait(obar, (od_base + (uint32_t)(j - 1)) & 1u, abort_flag))) break;
                        tc::fence_after_sync();
                        const RedoneTile redone = redo_score_tile(q_row, k_head + (int64_t)key_tile * BN * p.k_stride_token, p.k_stride_token,
                                                                  valid < BN ? valid : BN, c, m, t_s + kPColumn);
                        const float f = exp2f(m - redone.m);
                        l *= f;
                        m = redone.m;
                        tile_sum = redone.sum;
#pragma unroll 1
                        for (int cc = 0; cc < 8; ++cc) {   // eight columns at a time: this rare path must not cost registers
                            uint32_t o[8];
                            tc::tmem_ld8(t_o + cc * 8, o);
                            tc::tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 8; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                            tc::tmem_st8(t_o + cc * 8, o);
                        }
                    }
                    l += tile_sum;
                    tc::tmem_wait_st();
                    tc::fence_before_sync();
                    tc::mbar_arrive(pbar);
                }
                if (ok && ps.pair) {
                    const int grow = (ps.tile + x) * BM + row;
                    const RowTargets targets = row_targets<UNMERGE>(p, ps.head, grow, grow < mq_rows);   // (in flight during the wait)
                    if ((ok = tc::mbar_wait(tc::smem_addr(&bars->o_final), (uint32_t)pass & 1u, abort_flag))) {
                        tc::fence_after_sync();
                        const float inv = 1.0f / l;
                        uint32_t o[64];
                        tc::tmem_ld32(t_o, o);
                        tc::tmem_ld32(t_o + 32, o + 32);
                        tc::tmem_wait_ld();
                        uint4 v[8];
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            v[i].x = pack_bf16(__uint_as_float(o[8 * i + 0]) * inv, __uint_as_float(o[8 * i + 1]) * inv);
                            v[i].y = pack_bf16(__uint_as_float(o[8 * i + 2]) * inv, __uint_as_float(o[8 * i + 3]) * inv);
                            v[i].z = pack_bf16(__uint_as_float(o[8 * i + 4]) * inv, __uint_as_float(o[8 * i + 5]) * inv);
                            v[i].w = pack_bf16(__uint_as_float(o[8 * i + 6]) * inv, __uint_as_float(o[8 * i + 7]) * inv);
                        }
                        store_rows<UNMERGE>(p, ps.head, v, targets, out_stage, lane);
                    }
                } else if (ok && x == 1) {
                    // single pass, group B: publish this row's partial (max, sum); O_B stays in tensor memory for group A.
                    // Do not touch O_B again (next pass's zero fill) before group A has read it.
                    xch[row] = make_float2(m, l);
                    tc::mbar_arrive(tc::smem_addr(&bars->x_full));
                    ok = tc::mbar_wait(tc::smem_addr(&bars->x_done), n_single & 1u, abort_flag);
                } else if (ok) {
                    // single pass, group A: combine the two partial softmaxes over disjoint keys
                    //   out = (O_A 2^(m_A - m) + O_B 2^(m_B - m)) / (l_A 2^(m_A - m) + l_B 2^(m_B - m)),  m = max(m_A, m_B)
                    const int grow = ps.tile * BM + row;
                    const RowTargets targets = row_targets<UNMERGE>(p, ps.head, grow, grow < mq_rows);   // (in flight during the waits)
                    ok = tc::mbar_wait(tc::smem_addr(&bars->o_final), (uint32_t)pass & 1u, abort_flag) &&
                         tc::mbar_wait(tc::smem_addr(&bars->x_full), n_single & 1u, abort_flag);
                    if (ok) {
                        tc::fence_after_sync();
                        const float2 pb = xch[row];
                        const float mm = fmaxf(m, pb.x);
                        const float fa = exp2f(m - mm), fb = exp2f(pb.x - mm);   // 2^(-inf) = 0 when group B had no key tile
                        const float inv = 1.0f / (l * fa + pb.y * fb);
                        const float wa = fa * inv, wb = fb * inv;
                        uint4 v[8];
#pragma unroll
                        for (int half = 0; half < 2; ++half) {
                            uint32_t oa[32], ob[32];
                            tc::tmem_ld32(t_o + half * 32, oa);
                            tc::tmem_ld32(t_o + kHeadDim + half * 32, ob);   // O_B sits right behind O_A; same TMEM lanes
                            tc::tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                uint32_t w[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    w[e] = pack_bf16(fmaf(__uint_as_float(oa[8 * i + 2 * e]), wa, __uint_as_float(ob[8 * i + 2 * e]) * wb),
                                                     fmaf(__uint_as_float(oa[8 * i + 2 * e + 1]), wa, __uint_as_float(ob[8 * i + 2 * e + 1]) * wb));
                                v[half * 4 + i] = make_uint4(w[0], w[1], w[2], w[3]);
                            }
                        }
                        store_rows<UNMERGE>(p, ps.head, v, targets, out_stage, lane);
                        tc::fence_before_sync();
                        tc::mbar_arrive(tc::smem_addr(&bars->x_done));
                    }
                }
                od_base += (uint32_t)n_own;
                if (!ps.pair) ++n_single;
            }
#pragma unroll
            for (int b = 0; b < 3; ++b) sp_base[b] += (uint32_t)count_mod3(n_score, b);
        }
        bulk_stores_done();
    }
    tc::fence_before_sync();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem, TMEM_COLS);
    if (tid == 0 && bars->abort_flag) atomicCAS(p.status, kDevOk, kDevTimeoutAttention);
}

}  // namespace

cudaError_t configure_attention() {
    cudaError_t e = cudaFuncSetAttribute(attention_tc_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attention_tc_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(attention_tc_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
}

// Returns cudaErrorInvalidValue if a tensor map cannot be encoded.
cudaError_t launch_attention(const AttentionArgs& a, int sm_count, cudaStream_t stream) {
    CUtensorMap mq, mk, mv;
    if (!encode_rows_tensor_map(&mq, a.q.ptr, a.m_q, a.heads, a.q.stride_token, a.q.stride_head, BM) ||
        !encode_rows_tensor_map(&mk, a.k.ptr, a.m_k, a.heads, a.k.stride_token, a.k.stride_head, BN) ||
        !encode_rows_tensor_map(&mv, a.v.ptr, a.m_k, a.heads, a.v.stride_token, a.v.stride_head, BN))
        return cudaErrorInvalidValue;
    const int tiles_per_head = (a.m_q + BM - 1) / BM, total = tiles_per_head * a.heads;
    // one CTA per SM (fewer when there are fewer tiles)
    int ctas = sm_count < 1 ? 1 : sm_count;
    if (ctas > total) ctas = total;
    const int rounds = total / (2 * ctas);
    TcParams p{a.out, a.out_stride_head, a.out_stride_token, a.m_q, a.m_k, a.scale_log2, a.status, tiles_per_head, total, rounds, a.mq_head, a.tile_prefix, a.heads,
               a.group_start, a.group_member, a.n_tokens, a.q.ptr, a.k.ptr, a.q.stride_head, a.q.stride_token, a.k.stride_head, a.k.stride_token};
    if (a.mq_head) {   // the tile table lives in device memory: full grid, CTAs without tiles leave at once
        if (a.group_start) return cudaErrorInvalidValue;   // (the member lists are built for equal query lengths only)
        attention_tc_kernel<true, false><<<sm_count < 1 ? 1 : sm_count, NTHREADS, SMEM_BYTES, stream>>>(mq, mk, mv, p);
        return cudaGetLastError();
    }
    if (a.group_start)
        attention_tc_kernel<false, true><<<ctas, NTHREADS, SMEM_BYTES, stream>>>(mq, mk, mv, p);
    else
        attention_tc_kernel<false, false><<<ctas, NTHREADS, SMEM_BYTES, stream>>>(mq, mk, mv, p);
    return cudaGetLastError();
}

}  // namespace httm
