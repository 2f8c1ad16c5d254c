/*
 * CPU oracle for head-wise temporal token merging (HTTM) global attention.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, double-precision
 * restatement of what the method computes.  It shares no code with the CUDA
 * library and must never be linked, imported or called by the product path:
 * only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Every function cites the passage of the paper it follows.  Where the paper is
 * silent (block shape in 2-D, clipped edge blocks, the src/dst split, the
 * integer merge budget, tie-breaks, special tokens) the reading taken is stated
 * in the comment of the function that needs it.
 *
 * Parity status: the paper prints no worked numeric example, so no function is
 * pinned by paper numbers; each is pinned by the closed forms, brute-force
 * searches, library cross-checks and invariants in tests/test_oracle_*.py.
 *
 * Conventions
 *   S frames; each frame has n_sp special tokens followed by an h x w patch grid
 *   (row-major); P = n_sp + h*w; N = S*P; original token index i = s*P + p.
 *   H heads, D channels per head.  Inputs are bf16 bit patterns (uint16),
 *   layout [H][N][D].  All arithmetic is double.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t frames, n_special, grid_h, grid_w;
    int32_t heads, head_dim;
    int32_t blk_frames, blk_h, blk_w;
} oracle_geom;

static double bf16_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

static int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

int oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

int64_t oracle_num_tokens(const oracle_geom* g) {
    return (int64_t)g->frames * (g->n_special + (int64_t)g->grid_h * g->grid_w);
}

int64_t oracle_num_blocks(const oracle_geom* g) {
    return ceil_div(g->frames, g->blk_frames) * ceil_div(g->grid_h, g->blk_h) * ceil_div(g->grid_w, g->blk_w);
}

/*
 * Temporal reordering (Sec. 3.3; Algorithm 1, TemporalReorder / Reorder).
 * The same spatial block of blk_frames consecutive frames is made contiguous so
 * that merging can work on blocks of n_b = n_s * n_t tokens.
 * Readings: a spatial block is a blk_h x blk_w patch window; windows and frame
 * groups that stick out of the grid / the sequence are clipped (never padded);
 * special tokens belong to no block and are placed first, frame-major.
 *
 *   pi[p']       original index of the token at reordered position p'   (N)
 *   blk_start[b] reordered position of block b's first token           (nb+1,
 *                last entry = N); blocks are enumerated (frame group, window
 *                row, window column); inside a block (frame, y, x) row-major.
 */
void oracle_temporal_reorder(const oracle_geom* g, int64_t* pi, int64_t* blk_start) {
    const int64_t S = g->frames, nsp = g->n_special, h = g->grid_h, w = g->grid_w;
    const int64_t P = nsp + h * w;
    int64_t pos = 0, b = 0;
    for (int64_t s = 0; s < S; ++s)
        for (int64_t j = 0; j < nsp; ++j) pi[pos++] = s * P + j;
    for (int64_t t0 = 0; t0 < S; t0 += g->blk_frames)
        for (int64_t y0 = 0; y0 < h; y0 += g->blk_h)
            for (int64_t x0 = 0; x0 < w; x0 += g->blk_w) {
                blk_start[b++] = pos;
                for (int64_t s = t0; s < t0 + g->blk_frames && s < S; ++s)
                    for (int64_t y = y0; y < y0 + g->blk_h && y < h; ++y)
                        for (int64_t x = x0; x < x0 + g->blk_w && x < w; ++x)
                            pi[pos++] = s * P + nsp + y * w + x;
            }
    blk_start[b] = pos;
}

/* Reorder(X, pi): out[hd][p'] = x[hd][pi[p']]  (Algorithm 1). */
void oracle_reorder(const oracle_geom* g, const int64_t* pi, const uint16_t* x, uint16_t* out) {
    const int64_t N = oracle_num_tokens(g), D = g->head_dim;
    for (int64_t hd = 0; hd < g->heads; ++hd)
        for (int64_t p = 0; p < N; ++p)
            memcpy(out + (hd * N + p) * D, x + (hd * N + pi[p]) * D, (size_t)D * sizeof(uint16_t));
}

/*
 * Merge budget of one block of n tokens at merge ratio rho (Sec. 3.2: r = N - M
 * src tokens are merged away).  Readings: r = floor(rho*n + 1e-9), at most n-1
 * (one token always survives); the block has n_dst = min(ceil(n/4), n - r)
 * destination tokens (the 25 % / 75 % split of Sec. 3.3's cost example, shrunk
 * when the ratio needs more than 75 % of the block as sources).
 */
void oracle_block_budget(int64_t n, double rho, int64_t* r, int64_t* n_dst) {
    int64_t rr = (int64_t)floor(rho * (double)n + 1e-9);
    if (rr > n - 1) rr = n - 1;
    if (rr < 0) rr = 0;
    int64_t nd = ceil_div(n, 4);
    if (nd > n - rr) nd = n - rr;
    *r = rr;
    *n_dst = nd;
}

/* Disjoint src/dst partition (Sec. 3.2, "following ToMeSD", made deterministic):
 * n_dst evenly spaced local positions are dst, all others src. */
int oracle_is_dst(int64_t j, int64_t n, int64_t n_dst) {
    return ((j + 1) * n_dst) / n > (j * n_dst) / n;
}

/* Closed-form merged length: M = S*n_sp + sum over blocks (n - r). */
int64_t oracle_merged_len(const oracle_geom* g, double rho) {
    const int64_t nb = oracle_num_blocks(g), N = oracle_num_tokens(g);
    int64_t* pi = (int64_t*)malloc(sizeof(int64_t) * (size_t)N);
    int64_t* bs = (int64_t*)malloc(sizeof(int64_t) * (size_t)(nb + 1));
    oracle_temporal_reorder(g, pi, bs);
    int64_t M = (int64_t)g->frames * g->n_special;
    for (int64_t b = 0; b < nb; ++b) {
        int64_t n = bs[b + 1] - bs[b], r, nd;
        oracle_block_budget(n, rho, &r, &nd);
        M += n - r;
    }
    free(pi);
    free(bs);
    return M;
}

/*
 * Block-wise bipartite matching (Eq. 1 and the paragraph after it; Algorithm 1,
 * BlockwiseToMe), independently per head and per block, on REORDERED tokens xr.
 *   Sim = RowNorm(S) RowNorm(D)^T; each src keeps its most similar dst; the r src
 *   with the highest scores are merged into that dst.
 * Tie-breaks (paper silent): equal similarities -> lowest dst position; equal
 * scores -> lowest src position.  Zero vectors: the norm is clamped at 1e-12.
 *
 *   assign[hd][p']  reordered position of the token p' is merged into (itself if
 *                   it is kept: dst, unselected src, special token)
 *   margin_best[hd][p']  for src tokens with >= 2 dst: best sim minus runner-up
 *                   sim; +inf otherwise           (may be NULL)
 *   margin_sel[hd][b]    r-th best score minus (r+1)-th best score of block b;
 *                   +inf if 0 == r or r == n_src  (may be NULL)
 */
void oracle_match(const oracle_geom* g, const int64_t* blk_start, double rho, const uint16_t* xr,
                  int64_t* assign, double* margin_best, double* margin_sel) {
    const int64_t N = oracle_num_tokens(g), D = g->head_dim, nb = oracle_num_blocks(g);
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t hd = 0; hd < g->heads; ++hd) {
        const uint16_t* x = xr + hd * N * D;
        int64_t* A = assign + hd * N;
        for (int64_t p = 0; p < N; ++p) A[p] = p;
        if (margin_best)
            for (int64_t p = 0; p < N; ++p) margin_best[hd * N + p] = INFINITY;
        for (int64_t b = 0; b < nb; ++b) {
            const int64_t base = blk_start[b], n = blk_start[b + 1] - base;
            int64_t r, nd;
            oracle_block_budget(n, rho, &r, &nd);
            if (margin_sel) margin_sel[hd * nb + b] = INFINITY;
            if (r == 0) continue;
            double* xn = (double*)malloc(sizeof(double) * (size_t)(n * D)); /* RowNorm(x) */
            for (int64_t j = 0; j < n; ++j) {
                double ss = 0.0;
                for (int64_t c = 0; c < D; ++c) {
                    double v = bf16_to_double(x[(base + j) * D + c]);
                    ss += v * v;
                }
                double nrm = sqrt(ss);
                if (nrm < 1e-12) nrm = 1e-12;
                for (int64_t c = 0; c < D; ++c) xn[j * D + c] = bf16_to_double(x[(base + j) * D + c]) / nrm;
            }
            int64_t* best = (int64_t*)malloc(sizeof(int64_t) * (size_t)n);
            double* score = (double*)malloc(sizeof(double) * (size_t)n);
            int64_t* src = (int64_t*)malloc(sizeof(int64_t) * (size_t)n);
            int64_t ns = 0;
            for (int64_t a = 0; a < n; ++a) {
                if (oracle_is_dst(a, n, nd)) continue;
                double top = -INFINITY, second = -INFINITY;
                int64_t arg = -1;
                for (int64_t d = 0; d < n; ++d) {
                    if (!oracle_is_dst(d, n, nd)) continue;
                    double sim = 0.0;
                    for (int64_t c = 0; c < D; ++c) sim += xn[a * D + c] * xn[d * D + c];
                    if (sim > top) {
                        second = top;
                        top = sim;
                        arg = d;
                    } else if (sim > second) {
                        second = sim;
                    }
                }
                best[a] = arg;
                score[a] = top;
                src[ns++] = a;
                if (margin_best && nd >= 2) margin_best[hd * N + base + a] = top - second;
            }
            /* order src by (score descending, position ascending): stable insertion sort */
            for (int64_t i = 1; i < ns; ++i) {
                int64_t a = src[i], k = i;
                while (k > 0 && score[src[k - 1]] < score[a]) {
                    src[k] = src[k - 1];
                    --k;
                }
                src[k] = a;
            }
            for (int64_t i = 0; i < r; ++i) A[base + src[i]] = base + best[src[i]];
            if (margin_sel && r < ns) margin_sel[hd * nb + b] = score[src[r - 1]] - score[src[r]];
            free(xn);
            free(best);
            free(score);
            free(src);
        }
    }
}

/*
 * Rank of every token's group among the kept tokens of its head: kept tokens
 * (assign[p'] == p') are numbered in reordered order; a merged token takes the
 * number of the token it is merged into.  Returns the number of kept tokens of
 * head 0 (all heads have the same count, see oracle_merged_len) or -1 if heads
 * disagree.
 */
int64_t oracle_merged_rank(const oracle_geom* g, const int64_t* assign, int64_t* rank) {
    const int64_t N = oracle_num_tokens(g);
    int64_t M0 = -1;
    for (int64_t hd = 0; hd < g->heads; ++hd) {
        const int64_t* A = assign + hd * N;
        int64_t* R = rank + hd * N;
        int64_t m = 0;
        for (int64_t p = 0; p < N; ++p)
            if (A[p] == p) R[p] = m++;
        for (int64_t p = 0; p < N; ++p)
            if (A[p] != p) R[p] = R[A[p]];
        if (hd == 0) M0 = m;
        else if (m != M0) return -1;
    }
    return M0;
}

/*
 * Merged-token aggregation (Sec. 3.2: a merged token is the mean of its
 * constituents, i.e. the dst token and every src token matched to it;
 * Algorithm 1, BlockAggregate).  xr: reordered tokens [H][N][D] (bf16 bits),
 * rank from oracle_merged_rank, out: [H][M][D] double.
 */
void oracle_merge(const oracle_geom* g, const int64_t* rank, int64_t M, const uint16_t* xr, double* out) {
    const int64_t N = oracle_num_tokens(g), D = g->head_dim;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t hd = 0; hd < g->heads; ++hd) {
        double* o = out + hd * M * D;
        int64_t* cnt = (int64_t*)calloc((size_t)M, sizeof(int64_t));
        memset(o, 0, sizeof(double) * (size_t)(M * D));
        for (int64_t p = 0; p < N; ++p) {
            const int64_t m = rank[hd * N + p];
            cnt[m] += 1;
            for (int64_t c = 0; c < D; ++c) o[m * D + c] += bf16_to_double(xr[(hd * N + p) * D + c]);
        }
        for (int64_t m = 0; m < M; ++m)
            for (int64_t c = 0; c < D; ++c) o[m * D + c] /= (double)cnt[m];
        free(cnt);
    }
}

/*
 * Attention on the merged sets (Eq. 3-4): per head
 *   out = softmax(Q K^T / sqrt(D)) V,   no mask, no size bias.
 * q [H][Mq][D], k, v [H][Mk][D] double.  Only the query rows listed in rows[]
 * (n_rows of them, the same list for every head; NULL = all Mq rows) are
 * computed; out is [H][n_rows][D].
 */
void oracle_attention(int64_t H, int64_t Mq, int64_t Mk, int64_t D, const double* q, const double* k,
                      const double* v, const int64_t* rows, int64_t n_rows, double* out) {
    const double scale = 1.0 / sqrt((double)D);
    if (!rows) n_rows = Mq;
#pragma omp parallel for collapse(2) schedule(dynamic, 16)
    for (int64_t hd = 0; hd < H; ++hd)
        for (int64_t ri = 0; ri < n_rows; ++ri) {
            const int64_t row = rows ? rows[ri] : ri;
            const double* qr = q + (hd * Mq + row) * D;
            double* s = (double*)malloc(sizeof(double) * (size_t)Mk);
            double mx = -INFINITY;
            for (int64_t j = 0; j < Mk; ++j) {
                const double* kr = k + (hd * Mk + j) * D;
                double acc = 0.0;
                for (int64_t c = 0; c < D; ++c) acc += qr[c] * kr[c];
                s[j] = acc * scale;
                if (s[j] > mx) mx = s[j];
            }
            double den = 0.0;
            for (int64_t j = 0; j < Mk; ++j) {
                s[j] = exp(s[j] - mx);
                den += s[j];
            }
            double* o = out + (hd * n_rows + ri) * D;
            for (int64_t c = 0; c < D; ++c) o[c] = 0.0;
            for (int64_t j = 0; j < Mk; ++j) {
                const double pj = s[j] / den;
                const double* vr = v + (hd * Mk + j) * D;
                for (int64_t c = 0; c < D; ++c) o[c] += pj * vr[c];
            }
            free(s);
        }
}

/*
 * Head-wise unmerge + inverse reorder + head concat (Eq. 5-7; Algorithm 1,
 * UnmergeByCluster / InverseReorder): every original token copies the output of
 * the merged query token it went into.
 *   om [H][Mq][D], rank_q [H][N] (reordered positions), pi (N) -> out [N][H*D].
 */
void oracle_unmerge(const oracle_geom* g, const int64_t* pi, const int64_t* rank_q, int64_t Mq,
                    const double* om, double* out) {
    const int64_t N = oracle_num_tokens(g), D = g->head_dim, H = g->heads;
    for (int64_t hd = 0; hd < H; ++hd)
        for (int64_t p = 0; p < N; ++p) {
            const int64_t m = rank_q[hd * N + p], i = pi[p];
            memcpy(out + (i * H + hd) * D, om + (hd * Mq + m) * D, sizeof(double) * (size_t)D);
        }
}

/* bf16 bit patterns -> double, elementwise (used to feed unmerged tensors to
 * oracle_attention for the dense reference). */
void oracle_bf16_to_double(const uint16_t* x, int64_t count, double* out) {
    for (int64_t i = 0; i < count; ++i) out[i] = bf16_to_double(x[i]);
}
