"""CPU oracle of first-frame anchoring (the paper's "Error Mitigation" section of the appendix): plain numpy in
float64, written from the paper's description.

TEST INFRASTRUCTURE ONLY: imported by tests/ and by the smoke check; the product path (the CUDA library) shares no
code with it.

The paper: all tokens of the first frame are dst tokens ("reference tokens"), so that tokens of later frames which
resemble them are merged INTO them and the reference frame stays intact.  Everything else of Algorithm 1 is unchanged.

Readings where the paper is silent (listed in the design notes as well):
  * the rule applies inside every merging block that contains frame 0 (the blocks of the first frame group): there
    the dst tokens are exactly the block's tokens of frame 0 - the first rows x cols positions of the block, since a
    block is ordered (frame, row, column) - and every other token of the block is a src token; the evenly spaced dst
    choice is not used in these blocks.  Blocks of later frame groups are matched as before.
  * budget of such a block of n tokens with n0 tokens of frame 0: r = min(floor(rho n + 1e-9), n - n0) src tokens are
    merged (never more than there are src tokens; a block that lies entirely in frame 0 merges nothing).
  * best dst per src, top-r src, ties: as in the plain matching (lowest dst position, lowest src position).
"""
from __future__ import annotations

import numpy as np

from . import httm_oracle as orc


def anchored_blocks(g: orc.Geometry, blk_start: np.ndarray):
    """[(block index, n, n0)] for the blocks that contain frame 0: n tokens, of which the first n0 belong to frame 0."""
    f0 = min(g.blk_frames, g.frames)                                   # frames of the first frame group
    windows = (-(-g.grid_h // g.blk_h)) * (-(-g.grid_w // g.blk_w))     # blocks per frame group, in block order
    out = []
    for b in range(windows):
        n = int(blk_start[b + 1] - blk_start[b])
        assert n % f0 == 0
        out.append((b, n, n // f0))
    return out


def anchored_budget(n: int, n0: int, rho: float):
    """(r, n_dst) of a block that contains frame 0."""
    r = int(np.floor(rho * n + 1e-9))
    return max(0, min(r, n - n0)), n0


def merged_len(g: orc.Geometry, rho: float) -> int:
    """Closed form: specials + sum over blocks (n - r) with the anchored budgets in the first frame group."""
    pi, bs = orc.temporal_reorder(g)
    first = {b: (n, n0) for b, n, n0 in anchored_blocks(g, bs)}
    M = g.frames * g.n_special
    for b in range(len(bs) - 1):
        n = int(bs[b + 1] - bs[b])
        r = anchored_budget(n, first[b][1], rho)[0] if b in first else orc.block_budget(n, rho)[0]
        M += n - r
    return M


def match(g: orc.Geometry, blk_start: np.ndarray, rho: float, xr_bits: np.ndarray):
    """Assignment map [H][N] with first-frame anchoring, and the two margin arrays in the plain oracle's convention
    (best vs second-best dst of every src; r-th vs (r+1)-th score of every block; +inf where there is no runner-up)."""
    A, mb, ms = orc.match(g, blk_start, rho, xr_bits)                  # later frame groups: plain matching
    x = orc.bf16_to_double(xr_bits)
    for b, n, n0 in anchored_blocks(g, blk_start):
        base = int(blk_start[b])
        r, nd = anchored_budget(n, n0, rho)
        for hd in range(g.heads):
            A[hd, base:base + n] = np.arange(base, base + n)
            mb[hd, base:base + n] = np.inf
            ms[hd, b] = np.inf
            if r == 0:
                continue
            blk = x[hd, base:base + n]
            xn = blk / np.maximum(np.sqrt((blk * blk).sum(axis=1, keepdims=True)), 1e-12)
            sim = xn[nd:] @ xn[:nd].T                                  # [src][dst]
            best_d = sim.argmax(axis=1)                                # first maximum: lowest dst
            best = sim[np.arange(n - nd), best_d]
            if nd >= 2:
                part = np.partition(sim, nd - 2, axis=1)
                mb[hd, base + nd:base + n] = part[:, nd - 1] - part[:, nd - 2]
            order = np.lexsort((np.arange(n - nd), -best))             # by score descending, then position ascending
            chosen = order[:r]
            A[hd, base + nd + chosen] = base + best_d[chosen]
            if r < n - nd:
                ms[hd, b] = best[order[r - 1]] - best[order[r]]
    return A, mb, ms


def global_attention(g: orc.Geometry, ratio_q: float, ratio_kv: float, q, k, v, attend: bool = True) -> orc.Result:
    """Algorithm 1 (no projections, no outlier filtering) with first-frame anchoring in both matchings."""
    pi, bs = orc.temporal_reorder(g)
    qr, kr, vr = orc.reorder(g, pi, q), orc.reorder(g, pi, k), orc.reorder(g, pi, v)
    aq, mbq, msq = match(g, bs, ratio_q, qr)
    ak, mbk, msk = match(g, bs, ratio_kv, kr)
    rq, Mq = orc.merged_rank(g, aq)
    rk, Mk = orc.merged_rank(g, ak)
    qm, km, vm = orc.merge(g, rq, Mq, qr), orc.merge(g, rk, Mk, kr), orc.merge(g, rk, Mk, vr)
    om = out = None
    if attend:
        om = orc.attention(qm, km, vm)
        out = orc.unmerge(g, pi, rq, om)
    return orc.Result(pi, bs, aq, ak, mbq, msq, mbk, msk, rq, rk, Mq, Mk, qm, km, vm, om, out)


def global_attention_filtered(g: orc.Geometry, ratio_q: float, ratio_kv: float, gamma: float, q, k, v, attend: bool = True,
                              assign_q_filtered=None, assign_q_initial=None, assign_k=None):
    """Algorithm 1 with first-frame anchoring in both matchings AND the query outlier filtering of Sec. 3.4.
    The paper describes the two separately; the composition taken here: the filtering runs unchanged on the anchored
    query map (deviation of every token from the mean of its group, one threshold over all heads, outliers leave
    their groups).  A token of the reference frame that is an outlier leaves the group it anchors and stays on its
    own row like every other outlier, so the reference frame remains unmerged; its former group continues under its
    lowest remaining member.  The optional maps continue from maps under test, as in the plain filtered oracle."""
    from . import httm_outlier as flt
    pi, bs = orc.temporal_reorder(g)
    if assign_q_initial is None:
        assign_q_initial = match(g, bs, ratio_q, orc.reorder(g, pi, q))[0]
    if assign_k is None:
        assign_k = match(g, bs, ratio_kv, orc.reorder(g, pi, k))[0]
    return flt.global_attention_filtered(g, ratio_q, ratio_kv, gamma, q, k, v, attend=attend,
                                         assign_q_filtered=assign_q_filtered, assign_q_initial=assign_q_initial,
                                         assign_k=assign_k)
