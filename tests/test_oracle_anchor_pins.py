"""Pins of the first-frame-anchoring oracle against what the paper's description and the mathematics fix."""
import numpy as np
import pytest

from oracle import httm_anchor as anc
from oracle import httm_oracle as orc
from paper_2511_21317_b200 import synth


def case(seed=0, S=5, h=5, w=6, blk=(4, 2, 4), heads=2, nsp=(1, 1)):
    wl = synth.Workload("a", S, h, w, blk[0], blk[1], blk[2], 0.7, 0.6, heads=heads, n_camera=nsp[0], n_register=nsp[1], seed=seed, sigma=0.5)
    return wl, orc.Geometry.of(wl), synth.make_qkv(wl)


def frame_of_position(g, pi):
    return pi // (g.n_special + g.grid_h * g.grid_w)


def test_first_frame_tokens_are_kept_and_collect_the_merges_of_their_blocks():
    wl, g, (q, k, v) = case()
    res = anc.global_attention(g, 0.7, 0.6, q, k, v, attend=False)
    frame = frame_of_position(g, res.pi)
    idx = np.arange(res.pi.size)
    first_group = np.zeros(res.pi.size, dtype=bool)
    for b, n, n0 in anc.anchored_blocks(g, res.blk_start):
        first_group[res.blk_start[b]:res.blk_start[b + 1]] = True
    for A in (res.assign_q, res.assign_k):
        for hd in range(g.heads):
            assert (A[hd][frame == 0] == idx[frame == 0]).all()                    # the reference frame stays intact
            merged = (A[hd] != idx) & first_group
            assert merged.any() and (frame[A[hd][merged]] == 0).all()               # merges of these blocks go into frame 0
            assert (frame[idx[merged]] > 0).all()


def test_map_against_plain_loops():
    wl, g, (q, k, v) = case(seed=3, heads=1)
    pi, bs = orc.temporal_reorder(g)
    xr = orc.reorder(g, pi, q)
    x = orc.bf16_to_double(xr)[0]
    for rho in (0.3, 0.7, 0.95):
        A, _, _ = anc.match(g, bs, rho, xr)
        plain = orc.match(g, bs, rho, xr, margins=False)
        first = {b: (n, n0) for b, n, n0 in anc.anchored_blocks(g, bs)}
        for b in range(len(bs) - 1):
            base, n = int(bs[b]), int(bs[b + 1] - bs[b])
            if b not in first:
                assert np.array_equal(A[0, base:base + n], plain[0, base:base + n])   # later frame groups: unchanged
                continue
            n0 = first[b][1]
            r = min(int(np.floor(rho * n + 1e-9)), n - n0)
            nrm = [max(float(np.sqrt((x[base + j] ** 2).sum())), 1e-12) for j in range(n)]
            cand = []
            for a in range(n0, n):
                sims = [float(x[base + a] @ x[base + d]) / (nrm[a] * nrm[d]) for d in range(n0)]
                d = max(range(n0), key=lambda t: (sims[t], -t))
                cand.append((-sims[d], a, d))
            cand.sort()
            expect = np.arange(n)
            for _, a, d in cand[:r]:
                expect[a] = d
            assert np.array_equal(A[0, base:base + n] - base, expect)


def test_budget_and_closed_form_length():
    wl, g, (q, k, v) = case(seed=5)
    for rho in (0.0, 0.5, 0.7, 0.99):
        res = anc.global_attention(g, rho, rho, q, k, v, attend=False)
        assert res.M_q == anc.merged_len(g, rho) == res.M_k
        idx = np.arange(res.pi.size)
        for b, n, n0 in anc.anchored_blocks(g, res.blk_start):
            lo, hi = int(res.blk_start[b]), int(res.blk_start[b + 1])
            r = min(int(np.floor(rho * n + 1e-9)), n - n0)
            for hd in range(g.heads):
                assert int((res.assign_q[hd, lo:hi] != idx[lo:hi]).sum()) == r
    # more src than the plain rule would merge can go: at 0.99 every later-frame token of the first group is merged
    res = anc.global_attention(g, 0.99, 0.99, q, k, v, attend=False)
    for b, n, n0 in anc.anchored_blocks(g, res.blk_start):
        lo = int(res.blk_start[b])
        assert (res.assign_q[:, lo + n0:lo + n] < lo + n0).all()


def test_blocks_inside_the_first_frame_merge_nothing_and_ratio_zero_is_dense_attention():
    wl, g, (q, k, v) = case(seed=7, S=3, blk=(1, 2, 4))
    res = anc.global_attention(g, 0.7, 0.7, q, k, v, attend=False)
    idx = np.arange(res.pi.size)
    for b, n, n0 in anc.anchored_blocks(g, res.blk_start):
        assert n0 == n
        lo, hi = int(res.blk_start[b]), int(res.blk_start[b + 1])
        assert (res.assign_q[:, lo:hi] == idx[lo:hi]).all()
    wl, g, (q, k, v) = case(seed=8)
    out = anc.global_attention(g, 0.0, 0.0, q, k, v).out
    assert np.allclose(out, orc.dense_attention(g, q, k, v), rtol=1e-9, atol=1e-12)


def test_margins_follow_the_plain_convention():
    wl, g, (q, k, v) = case(seed=9, heads=1)
    pi, bs = orc.temporal_reorder(g)
    xr = orc.reorder(g, pi, q)
    A, mb, ms = anc.match(g, bs, 0.5, xr)
    x = orc.bf16_to_double(xr)[0]
    b, n, n0 = anc.anchored_blocks(g, bs)[0]
    base = int(bs[b])
    blk = x[base:base + n]
    xn = blk / np.maximum(np.linalg.norm(blk, axis=1, keepdims=True), 1e-12)
    sim = xn[n0:] @ xn[:n0].T
    srt = np.sort(sim, axis=1)
    assert np.allclose(mb[0, base + n0:base + n], srt[:, -1] - srt[:, -2])
    best = np.sort(sim.max(axis=1))[::-1]
    r = min(int(np.floor(0.5 * n + 1e-9)), n - n0)
    assert ms[0, b] == pytest.approx(best[r - 1] - best[r])


def test_anchoring_with_outlier_filtering_against_plain_loops():
    """The composition (filtering on the anchored query map) restated with loops: deviations from the group means,
    the K largest over all heads leave, an orphaned group continues under its lowest remaining member."""
    wl, g, (q, k, v) = case(seed=11, S=6, h=4, w=6, blk=(3, 2, 3), heads=2)
    gamma = 0.08
    res = anc.global_attention_filtered(g, 0.7, 0.6, gamma, q, k, v, attend=False)
    base = anc.global_attention(g, 0.7, 0.6, q, k, v, attend=False)
    assert np.array_equal(res.assign_q0, base.assign_q) and np.array_equal(res.assign_k, base.assign_k)
    x = orc.bf16_to_double(orc.reorder(g, res.pi, q))
    H, N = base.assign_q.shape
    eps = np.zeros((H, N))
    for hd in range(H):
        for i in range(N):
            members = [j for j in range(N) if base.assign_q[hd, j] == base.assign_q[hd, i]]
            mean = sum(x[hd, j] for j in members) / len(members)
            eps[hd, i] = float(np.sqrt(((x[hd, i] - mean) ** 2).sum())) if len(members) > 1 else 0.0
    assert np.allclose(res.eps, eps, rtol=1e-12, atol=1e-14)
    K = int(np.floor(gamma * H * N + 1e-9))
    order = sorted(((-eps[hd, i], hd, i) for hd in range(H) for i in range(N)))
    assert -order[K][0] < -order[K - 1][0]                       # no tie at the threshold in this case
    out = {(hd, i) for _, hd, i in order[:K]}
    assert {(int(a), int(b)) for a, b in zip(*np.nonzero(res.outlier))} == out
    for hd in range(H):
        for i in range(N):
            if (hd, i) in out:
                expect = i
            else:
                rest = [j for j in range(N) if base.assign_q[hd, j] == base.assign_q[hd, i] and (hd, j) not in out]
                d = int(base.assign_q[hd, i])
                expect = d if (hd, d) not in out else min(rest)
            assert res.assign_q[hd, i] == expect
    frame = frame_of_position(g, res.pi)
    assert (res.assign_q[:, frame == 0] == np.arange(N)[frame == 0]).all()      # the reference frame stays unmerged
    assert any((hd, i) in out for hd in range(H) for i in np.nonzero(frame == 0)[0])   # ... although some of it are outliers
    assert res.M_q == [len(set(res.assign_q[hd].tolist())) for hd in range(H)] and min(res.M_q) > anc.merged_len(g, 0.7)


def test_anchoring_with_an_outlier_budget_of_zero_or_all_tokens():
    wl, g, (q, k, v) = case(seed=12)
    plain = anc.global_attention(g, 0.7, 0.6, q, k, v)
    res = anc.global_attention_filtered(g, 0.7, 0.6, 0.0, q, k, v)
    assert np.array_equal(res.assign_q, plain.assign_q) and np.allclose(res.out, plain.out, rtol=1e-12, atol=1e-14)
    res = anc.global_attention_filtered(g, 0.7, 0.6, 1.0, q, k, v)                  # every query on its own: K/V merging only
    assert res.M_q == [res.pi.size] * g.heads
    ref = orc.merged_attention_from_maps(g, res.pi, q, k, v, np.tile(np.arange(res.pi.size), (g.heads, 1)), plain.assign_k)
    assert np.allclose(res.out, ref.out, rtol=1e-12, atol=1e-14)
