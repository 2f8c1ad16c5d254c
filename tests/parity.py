"""Comparison of the CUDA path with the CPU oracle (used by the GPU tests, the smoke
check and the benchmark's parity sample).  The rules:

  * reorder permutation, reordered tensors: bit-exact;
  * assignment maps: bit-exact, except inside blocks where the oracle's (double)
    similarity margin to the runner-up - best vs second-best destination of a source,
    or the r-th vs (r+1)-th best score - is below 1e-5; there the map under test must
    still be a valid outcome within that margin;
  * merged tensors: the bf16 value must be one of the two bf16 neighbours of the exact mean;
  * attention output: max abs error <= 2e-2 x RMS of the oracle's output.
"""
from __future__ import annotations

import numpy as np

from oracle import httm_oracle as orc

MARGIN = 1e-5
OUT_TOL = 2e-2


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def check_maps(g, rho, blk_start, xr_bits, a_oracle, margin_best, margin_sel, a_gpu, what="", anchored=None):
    """Returns the number of (head, block) pairs where the maps differ (all justified by the
    margin rule); raises AssertionError otherwise.  anchored: {block: n0} for blocks under first-frame
    anchoring (their first n0 tokens are the dst tokens, budget min(floor(rho n), n - n0))."""
    a_gpu = np.asarray(a_gpu, dtype=np.int64)
    assert a_gpu.shape == a_oracle.shape, f"{what}: map shape {a_gpu.shape} != {a_oracle.shape}"
    diff = a_gpu != a_oracle
    if not diff.any():
        return 0
    nsp_total = int(blk_start[0])
    assert not diff[:, :nsp_total].any(), f"{what}: special tokens must map to themselves"
    n_bad_blocks = 0
    for hd in np.flatnonzero(diff.any(axis=1)):
        cols = np.flatnonzero(diff[hd])
        blocks = np.unique(np.searchsorted(blk_start, cols, side="right") - 1)
        for b in blocks:
            lo, hi = int(blk_start[b]), int(blk_start[b + 1])
            n = hi - lo
            r, nd = orc.block_budget(n, rho)
            if anchored and int(b) in anchored:
                nd = anchored[int(b)]
                r = min(int(np.floor(rho * n + 1e-9)), n - nd)
            ambiguous = margin_sel[hd, b] < MARGIN or (margin_best[hd, lo:hi] < MARGIN).any()
            assert ambiguous, (f"{what}: head {hd} block {b}: map differs from the oracle but all margins are >= {MARGIN} "
                               f"(min best-margin {margin_best[hd, lo:hi].min():.3e}, selection margin {margin_sel[hd, b]:.3e})")
            # validity within the margin, from double-precision similarities
            x = bits_to_f64(xr_bits[hd, lo:hi])
            nrm = np.maximum(np.linalg.norm(x, axis=1, keepdims=True), 1e-12)
            xn = x / nrm
            if anchored and int(b) in anchored:
                dst = np.arange(nd)
            else:
                dst = np.array([j for j in range(n) if ((j + 1) * nd) // n > (j * nd) // n])
            src = np.array([j for j in range(n) if j not in set(dst.tolist())])
            sim = xn[src] @ xn[dst].T
            best = sim.max(axis=1)
            loc = a_gpu[hd, lo:hi] - lo
            assert ((loc >= 0) & (loc < n)).all(), f"{what}: head {hd} block {b}: target outside the block"
            assert (loc[dst] == dst).all(), f"{what}: a dst token was merged away"
            merged = loc[src] != src
            assert merged.sum() == r, f"{what}: head {hd} block {b}: {merged.sum()} merged, budget {r}"
            for ai in np.flatnonzero(merged):
                tgt = loc[src[ai]]
                assert tgt in dst, f"{what}: merge target is not a dst token"
                assert sim[ai, np.flatnonzero(dst == tgt)[0]] >= best[ai] - MARGIN, f"{what}: target is not the best match"
            if 0 < r < len(src):
                assert best[merged].min() >= best[~merged].max() - MARGIN, f"{what}: selection is not top-r"
            n_bad_blocks += 1
    return n_bad_blocks


def check_merged(gpu_bits: np.ndarray, exact: np.ndarray, what=""):
    """The bf16 result must be the rounding of the exact (double) mean up to the fp32 summation
    error of the kernel: |err| <= half a bf16 step (2^-8 |exact|) + 4e-6 x the largest magnitude."""
    got = bits_to_f64(gpu_bits)
    assert got.shape == exact.shape, f"{what}: shape {got.shape} != {exact.shape}"
    assert np.isfinite(got).all(), f"{what}: non-finite merged value"
    err = np.abs(got - exact)
    bound = np.abs(exact) * 2.0 ** -8 + 4e-6 * max(float(np.abs(exact).max()), 1e-30)
    bad = err > bound
    assert not bad.any(), f"{what}: {bad.sum()} merged values off by more than one bf16 step (max err {err.max():.3e})"
    # and nearly all of them are the correctly rounded value
    return float((err <= np.abs(exact) * 2.0 ** -8).mean())


def check_output(gpu_bits: np.ndarray, expect: np.ndarray, rms: float | None = None, what="", peaky: bool = False,
                 stats: dict | None = None):
    """max |gpu - oracle| <= 2e-2 x RMS(oracle).  peaky=True (tiny adversarial geometries only, where a
    few keys dominate a row and |value| is many times the RMS) adds the representation error of the
    bf16 output itself, half a bf16 step = 2^-8 |oracle value|, element by element.  If a stats dict is
    given, the number of elements that passed only thanks to that extra term is added to
    stats["peaky_needed"] and the number of elements compared to stats["out_elements"]."""
    got = bits_to_f64(gpu_bits)
    assert got.shape == expect.shape, f"{what}: shape {got.shape} != {expect.shape}"
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    if rms is None:
        rms = float(np.sqrt(np.mean(expect ** 2)))
    err = np.abs(got - expect)
    bound = OUT_TOL * rms + (2.0 ** -8 * np.abs(expect) if peaky else 0.0)
    worst = float((err - bound).max()) if err.size else 0.0
    assert worst <= 0, f"{what}: max abs err {err.max():.4e} exceeds {OUT_TOL} x RMS {rms:.4e} by {worst:.3e}"
    if stats is not None:
        stats["peaky_needed"] = stats.get("peaky_needed", 0) + int((err > OUT_TOL * rms).sum())
        stats["out_elements"] = stats.get("out_elements", 0) + int(err.size)
    return float(err.max()) / rms if err.size else 0.0


def full_check(g, rho_q, rho_kv, q, k, v, ex, out_bits, sample_tokens=None, what="", peaky=False, anchor=False):
    """Element-by-element comparison of everything the library exposes.
    ex: dict of exports (numpy) with keys pi, blk_start, qr, kr, vr, assign_q, assign_k, rank_q, q_m, k_m, v_m, o_m.
    If sample_tokens is given, attention output is checked on those ORIGINAL tokens only."""
    anchored = None
    if anchor:   # first-frame anchoring: its own oracle, and the block rules for the margin check
        from oracle import httm_anchor as anc
        res = anc.global_attention(g, rho_q, rho_kv, q, k, v, attend=False)
        anchored = {b: n0 for b, n, n0 in anc.anchored_blocks(g, res.blk_start)}
    else:
        res = orc.global_attention(g, rho_q, rho_kv, q, k, v, attend=False)
    assert np.array_equal(ex["pi"].astype(np.int64), res.pi), f"{what}: reorder permutation differs"
    assert np.array_equal(ex["blk_start"].astype(np.int64), res.blk_start), f"{what}: block table differs"
    qr, kr, vr = orc.reorder(g, res.pi, q), orc.reorder(g, res.pi, k), orc.reorder(g, res.pi, v)
    for name, ref in (("qr", qr), ("kr", kr), ("vr", vr)):
        assert np.array_equal(ex[name], ref), f"{what}: reordered {name} is not bit-exact"
    nq = check_maps(g, rho_q, res.blk_start, qr, res.assign_q, res.margin_best_q, res.margin_sel_q, ex["assign_q"], what + " A_q", anchored)
    nk = check_maps(g, rho_kv, res.blk_start, kr, res.assign_k, res.margin_best_k, res.margin_sel_k, ex["assign_k"], what + " A_k", anchored)
    if nq or nk:   # maps differ inside the margin: the oracle continues from the validated maps
        res = orc.merged_attention_from_maps(g, res.pi, q, k, v, ex["assign_q"].astype(np.int64),
                                             ex["assign_k"].astype(np.int64), attend=False)
    assert np.array_equal(ex["rank_q"].astype(np.int64), res.rank_q), f"{what}: rank_q differs"
    fr = [check_merged(ex[n], ref, f"{what} {n}") for n, ref in (("q_m", res.q_m), ("k_m", res.k_m), ("v_m", res.v_m))]
    stats = {"ambiguous_blocks_q": nq, "ambiguous_blocks_k": nk, "merged_exactly_rounded": min(fr)}
    if sample_tokens is None:
        o_m = orc.attention(res.q_m, res.k_m, res.v_m)
        out = orc.unmerge(g, res.pi, res.rank_q, o_m)
        rms = float(np.sqrt(np.mean(out ** 2)))
        stats["o_m_err"] = check_output(ex["o_m"], o_m, rms, what + " O_m", peaky)
        stats["out_err"] = check_output(out_bits, out, rms, what + " out", peaky, stats)
    else:
        rows = orc.attention_rows_for_tokens(g, res, sample_tokens)
        rms = float(np.sqrt(np.mean(rows ** 2)))
        stats["out_err"] = check_output(out_bits[sample_tokens], rows, rms, what + " out (sampled)", peaky, stats)
        # unmerge is a pure copy of O_m rows: check that on ALL tokens, bit-exactly
        D = g.head_dim
        inv = np.empty_like(res.pi)
        inv[res.pi] = np.arange(len(res.pi))
        for hd in range(g.heads):
            assert np.array_equal(out_bits[:, hd * D:(hd + 1) * D], ex["o_m"][hd][res.rank_q[hd][inv]]), \
                f"{what}: unmerge of head {hd} is not a pure copy"
    stats["rms"] = rms
    return stats


DEV_TOL = 1e-5   # deviations: |gpu - oracle| <= DEV_TOL x (largest |q| + the deviation): fp32 means, differences and sums of 64 squares


def filtered_check(g, rho_q, rho_kv, gamma, q, k, v, ex, out_bits, n_outliers, sample_tokens=None, what="", peaky=False,
                   anchor=False):
    """Query outlier filtering (Sec. 3.4, Algorithm 2) against its oracle.
    ex: exports pi, blk_start, assign_q0 (map of the initial merging), assign_q (after the outliers left), assign_k,
    eps, tau, mq_head, rank_q, q_m, k_m, v_m, o_m (q_m, o_m with N rows per head, head h's first mq_head[h] valid).
    Rules: the matching maps as in check_maps; deviations within DEV_TOL; the threshold is the (K+1)-th largest of
    the deviations under test, within DEV_TOL of the oracle's; the outlier decision agrees with the oracle's for
    every token whose deviation is further than 2 x DEV_TOL from the oracle's threshold; the filtered map is exactly
    what the oracle's rule makes of the decisions under test; everything downstream continues from that map.
    anchor: the matching maps are those of first-frame anchoring (its oracle, its block rules in the margin check)."""
    from oracle import httm_outlier as flt
    anchored = None
    if anchor:
        from oracle import httm_anchor as anc
        res0 = anc.global_attention(g, rho_q, rho_kv, q, k, v, attend=False)
        anchored = {b: n0 for b, n, n0 in anc.anchored_blocks(g, res0.blk_start)}
    else:
        res0 = orc.global_attention(g, rho_q, rho_kv, q, k, v, attend=False)
    assert np.array_equal(ex["pi"].astype(np.int64), res0.pi), f"{what}: reorder permutation differs"
    qr, kr = orc.reorder(g, res0.pi, q), orc.reorder(g, res0.pi, k)
    nq = check_maps(g, rho_q, res0.blk_start, qr, res0.assign_q, res0.margin_best_q, res0.margin_sel_q, ex["assign_q0"], what + " A_q (initial)", anchored)
    nk = check_maps(g, rho_kv, res0.blk_start, kr, res0.assign_k, res0.margin_best_k, res0.margin_sel_k, ex["assign_k"], what + " A_k", anchored)
    aq0 = ex["assign_q0"].astype(np.int64)
    eps = flt.deviations(aq0, qr)
    eps_gpu = ex["eps"].astype(np.float64)
    tol = DEV_TOL * (float(np.abs(bits_to_f64(qr)).max()) + eps)
    err = np.abs(eps_gpu - eps)
    assert (err <= tol).all(), f"{what}: deviation off by {err.max():.3e} (tolerance {tol.flat[err.argmax()]:.3e})"
    alone = np.stack([np.bincount(aq0[hd], minlength=aq0.shape[1])[aq0[hd]] == 1 for hd in range(aq0.shape[0])])
    assert (eps_gpu[alone] == 0).all(), f"{what}: tokens on their own must have deviation exactly 0"
    K = flt.outlier_budget(eps.size, gamma)
    tau, tau_gpu = flt.outlier_threshold(eps, gamma), float(ex["tau"][0])
    outl_gpu = eps_gpu > tau_gpu
    if K <= 0:
        assert tau_gpu == float("inf") and not outl_gpu.any()
    elif K >= eps.size:
        assert outl_gpu.all()
    else:
        assert outl_gpu.sum() <= K < (eps_gpu >= tau_gpu).sum(), f"{what}: tau is not the (K+1)-th largest deviation"
        assert abs(tau_gpu - tau) <= DEV_TOL * (float(np.abs(bits_to_f64(qr)).max()) + tau), f"{what}: tau {tau_gpu} vs {tau}"
        clear = np.abs(eps - tau) > 2 * tol
        assert np.array_equal(outl_gpu[clear], (eps > tau)[clear]), f"{what}: outlier decisions differ outside the margin"
    in_blocks = int(outl_gpu[:, int(ex["blk_start"][0]):].sum())   # (special tokens are in no block and never merged)
    assert n_outliers == in_blocks, f"{what}: outlier counter {n_outliers} != {in_blocks}"
    aq = flt.filter_map(aq0, outl_gpu)
    assert np.array_equal(ex["assign_q"].astype(np.int64), aq), f"{what}: filtered map differs from the rule applied to the decisions"
    res = (anc if anchor else flt).global_attention_filtered(g, rho_q, rho_kv, gamma, q, k, v, attend=False, assign_q_filtered=aq,
                                        assign_q_initial=aq0, assign_k=ex["assign_k"].astype(np.int64))
    assert ex["mq_head"].tolist() == res.M_q, f"{what}: merged query lengths {ex['mq_head'].tolist()} != {res.M_q}"
    stats = {"ambiguous_blocks_q": nq, "ambiguous_blocks_k": nk, "outliers": int(outl_gpu.sum()), "tau": tau_gpu,
             "undecided": int((~(np.abs(eps - tau) > 2 * tol)).sum()) if 0 < K < eps.size else 0, "M_q": res.M_q}
    fr = [check_merged(ex[n], ref, f"{what} {n}") for n, ref in (("k_m", res.k_m), ("v_m", res.v_m))]
    for hd in range(g.heads):
        assert np.array_equal(ex["rank_q"][hd].astype(np.int64), res.rank_q[hd]), f"{what}: rank_q of head {hd} differs"
        fr.append(check_merged(ex["q_m"][hd][:res.M_q[hd]], res.q_m[hd], f"{what} q_m head {hd}"))
    stats["merged_exactly_rounded"] = min(fr)
    D = g.head_dim
    inv = np.empty_like(res.pi)
    inv[res.pi] = np.arange(len(res.pi))
    if sample_tokens is None:
        o_m = [orc.attention(res.q_m[hd][None], res.k_m[hd:hd + 1], res.v_m[hd:hd + 1])[0] for hd in range(g.heads)]
        out = np.concatenate([o_m[hd][res.rank_q[hd][inv]] for hd in range(g.heads)], axis=1)
        rms = float(np.sqrt(np.mean(out ** 2)))
        for hd in range(g.heads):
            check_output(ex["o_m"][hd][:res.M_q[hd]], o_m[hd], rms, f"{what} O_m head {hd}", peaky)
        stats["out_err"] = check_output(out_bits, out, rms, what + " out", peaky, stats)
    else:
        pos = inv[np.asarray(sample_tokens)]
        rows = np.concatenate([orc.attention(res.q_m[hd][res.rank_q[hd][pos]][None], res.k_m[hd:hd + 1], res.v_m[hd:hd + 1])[0]
                               for hd in range(g.heads)], axis=1)
        rms = float(np.sqrt(np.mean(rows ** 2)))
        stats["out_err"] = check_output(out_bits[sample_tokens], rows, rms, what + " out (sampled)", peaky, stats)
    for hd in range(g.heads):   # unmerge is a pure copy of O_m rows: on ALL tokens, bit-exactly
        assert np.array_equal(out_bits[:, hd * D:(hd + 1) * D], ex["o_m"][hd][res.rank_q[hd][inv]]), \
            f"{what}: unmerge of head {hd} is not a pure copy"
    stats["rms"] = rms
    return stats
