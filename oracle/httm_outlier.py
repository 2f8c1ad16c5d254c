"""CPU oracle of HTTM's adaptive outlier filtering for query tokens (Sec. 3.4, Algorithm 2
"BlockAggregateQuantile"): plain numpy in float64, written from the paper's steps.

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's CPU
baseline; the product path (the CUDA library) shares no code with it.

Steps, in the paper's order (Sec. 3.4, items 1-4):
  1. initial merging of the query tokens inside every block (the assignment map A_q of the matching step);
  2. deviation of every query token from the merged token it went into: the L2 distance to the mean of
     its group; tokens that were not merged with any other token have deviation 0;
  3. the tokens with the largest deviations over ALL heads, a fraction `gamma` of the H x N tokens, are
     outliers;
  4. outliers leave their groups and stay on their own; the merged tokens they left are the means of
     the remaining constituents.
Only query tokens are filtered (Sec. 3.4, last sentence before the kernel paragraph); K and V are untouched.

Readings where the paper is silent (listed in the design notes as well):
  * threshold (Alg. 2: tau = Quantile(eps, gamma), outlier iff eps > tau): with K = floor(gamma * H * N + 1e-9),
    tau is the (K+1)-th largest deviation; outlier iff eps > tau.  Without ties at the threshold that is exactly
    the top K; tokens tied with tau are not outliers.  K = 0 filters nothing.
  * a group whose destination token is an outlier keeps its other constituents together: its new
    representative (which fixes the place of the merged token in the merged order) is the remaining
    constituent with the lowest reordered position.
  * the merged length now differs from head to head; merged order stays "kept tokens in reordered order".
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from . import httm_oracle as orc


def deviations(assign_q: np.ndarray, qr_bits: np.ndarray) -> np.ndarray:
    """eps [H][N]: distance of every reordered query token to the mean of the group it was merged into
    (Sec. 3.4 item 2); 0 for tokens whose group has a single member."""
    A = np.asarray(assign_q, dtype=np.int64)
    H, N = A.shape
    x = orc.bf16_to_double(qr_bits)                       # [H][N][D]
    eps = np.zeros((H, N), dtype=np.float64)
    for h in range(H):
        cnt = np.bincount(A[h], minlength=N).astype(np.float64)
        s = np.zeros((N, x.shape[2]), dtype=np.float64)
        np.add.at(s, A[h], x[h])
        mean = s / np.maximum(cnt, 1.0)[:, None]
        d = np.sqrt(((x[h] - mean[A[h]]) ** 2).sum(axis=1))
        eps[h] = np.where(cnt[A[h]] >= 2, d, 0.0)
    return eps


def outlier_budget(n_values: int, gamma: float) -> int:
    return int(np.floor(gamma * n_values + 1e-9))


def outlier_threshold(eps: np.ndarray, gamma: float) -> float:
    """tau of Algorithm 2: the (K+1)-th largest deviation, K = floor(gamma * H * N + 1e-9); +inf when K = 0."""
    K = outlier_budget(eps.size, gamma)
    if K <= 0:
        return float("inf")
    flat = np.sort(eps.ravel())[::-1]
    return float(flat[K]) if K < flat.size else -1.0


def filter_map(assign_q: np.ndarray, outlier: np.ndarray) -> np.ndarray:
    """Assignment map after the outliers have left their groups (Sec. 3.4 item 4; Alg. 2 'C_q[j] <- -1' and
    'recompute only the centroids of clusters affected'): an outlier maps to itself; the other tokens of a
    group stay together, under the old representative if it is not an outlier, else under the remaining
    constituent with the lowest position."""
    A = np.asarray(assign_q, dtype=np.int64)
    out = np.asarray(outlier, dtype=bool)
    H, N = A.shape
    new = np.empty_like(A)
    big = np.iinfo(np.int64).max
    idx = np.arange(N, dtype=np.int64)
    for h in range(H):
        lowest = np.full(N, big, dtype=np.int64)          # lowest remaining member of every group
        keep = ~out[h]
        np.minimum.at(lowest, A[h][keep], idx[keep])
        rep = np.where(out[h][A[h]], lowest[A[h]], A[h])  # old representative unless it left
        new[h] = np.where(out[h], idx, rep)
    return new


@dataclass
class FilteredResult:
    pi: np.ndarray
    blk_start: np.ndarray
    assign_q0: np.ndarray        # [H][N] map of the initial merging
    assign_q: np.ndarray         # [H][N] map after the outliers left
    assign_k: np.ndarray
    eps: np.ndarray              # [H][N] deviations
    tau: float
    outlier: np.ndarray          # [H][N] bool
    rank_q: list                 # per head: [N] merged row of each reordered token
    M_q: list                    # per head merged query length
    M_k: int
    q_m: list                    # per head [M_q[h]][D] float64
    k_m: np.ndarray
    v_m: np.ndarray
    o_m: list | None
    out: np.ndarray | None       # [N][H*D]


def _one_head(g: orc.Geometry) -> orc.Geometry:
    return orc.Geometry(**{**g.__dict__, "heads": 1})


def merge_heads(g: orc.Geometry, assign_q: np.ndarray, qr_bits: np.ndarray):
    """Per-head merged ranks, lengths and merged query tokens for a map whose kept count differs per head."""
    g1 = _one_head(g)
    ranks, lens, qms = [], [], []
    for h in range(g.heads):
        r, M = orc.merged_rank(g1, assign_q[h:h + 1])
        ranks.append(r[0])
        lens.append(M)
        qms.append(orc.merge(g1, r, M, qr_bits[h:h + 1])[0])
    return ranks, lens, qms


def global_attention_filtered(g: orc.Geometry, ratio_q: float, ratio_kv: float, gamma: float, q, k, v,
                              attend: bool = True, assign_q_filtered=None, assign_q_initial=None,
                              assign_k=None) -> FilteredResult:
    """Algorithm 1 with the query outlier filtering of Sec. 3.4 / Algorithm 2 (no projections).
    assign_q_filtered: continue from a given filtered map (used when a map under test differs from the
    oracle's only by tokens whose deviation is within the comparison margin of tau).
    assign_q_initial, assign_k: continue from given maps of the matching step (used when a map under test
    differs from the oracle's only inside the similarity margin)."""
    pi, bs = orc.temporal_reorder(g)
    qr, kr, vr = orc.reorder(g, pi, q), orc.reorder(g, pi, k), orc.reorder(g, pi, v)
    aq0 = orc.match(g, bs, ratio_q, qr, margins=False) if assign_q_initial is None else np.asarray(assign_q_initial, dtype=np.int64)
    ak = orc.match(g, bs, ratio_kv, kr, margins=False) if assign_k is None else np.asarray(assign_k, dtype=np.int64)
    eps = deviations(aq0, qr)
    tau = outlier_threshold(eps, gamma)
    outlier = eps > tau
    aq = filter_map(aq0, outlier) if assign_q_filtered is None else np.asarray(assign_q_filtered, dtype=np.int64)
    rank_q, M_q, q_m = merge_heads(g, aq, qr)
    rk, Mk = orc.merged_rank(g, ak)
    km, vm = orc.merge(g, rk, Mk, kr), orc.merge(g, rk, Mk, vr)
    o_m = out = None
    if attend:
        g1 = _one_head(g)
        o_m = [orc.attention(q_m[h][None], km[h:h + 1], vm[h:h + 1])[0] for h in range(g.heads)]
        N, D = orc.num_tokens(g), g.head_dim
        out = np.empty((N, g.heads * D), dtype=np.float64)
        for h in range(g.heads):
            out[:, h * D:(h + 1) * D] = orc.unmerge(g1, pi, rank_q[h][None], o_m[h][None])
    return FilteredResult(pi, bs, aq0, aq, ak, eps, tau, outlier, rank_q, M_q, Mk, q_m, km, vm, o_m, out)
