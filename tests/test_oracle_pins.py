"""Pins of the CPU oracle against things other than itself: closed forms,
brute-force searches, library routines, and invariants the paper's definitions fix.
CPU only."""
import itertools
import math

import numpy as np
import pytest

from oracle import httm_oracle as orc
from paper_2511_21317_b200 import synth


def geom(S=3, nsp=2, h=5, w=6, H=2, D=8, blk=(2, 2, 4)):
    return orc.Geometry(S, nsp, h, w, H, D, *blk)


def rand_bf16(shape, seed):
    rng = np.random.default_rng(seed)
    return synth.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))


def as_f64(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def naive_mha(q, k, v):
    """Independent textbook attention, float64: q,k,v [H][N][D] -> [N][H*D]."""
    H, N, D = q.shape
    out = np.empty((N, H * D))
    for hd in range(H):
        s = q[hd] @ k[hd].T / math.sqrt(D)
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        p /= p.sum(axis=1, keepdims=True)
        out[:, hd * D:(hd + 1) * D] = p @ v[hd]
    return out


# ---------------------------------------------------------------- geometry / reorder


def block_key(g, i):
    """Independent statement of which block an ORIGINAL token index belongs to."""
    P = g.n_special + g.grid_h * g.grid_w
    s, p = divmod(i, P)
    if p < g.n_special:
        return None
    y, x = divmod(p - g.n_special, g.grid_w)
    return (s // g.blk_frames, y // g.blk_h, x // g.blk_w)


@pytest.mark.parametrize("g", [geom(), geom(S=4, nsp=5, h=16, w=16, blk=(2, 4, 4)), geom(S=5, nsp=0, h=7, w=3, blk=(4, 8, 8)),
                               geom(S=1, nsp=1, h=1, w=1, blk=(1, 1, 1)), geom(S=8, nsp=5, h=37, w=37, blk=(2, 4, 4))])
def test_reorder_is_block_contiguous_permutation(g):
    pi, bs = orc.temporal_reorder(g)
    N = orc.num_tokens(g)
    assert N == g.frames * (g.n_special + g.grid_h * g.grid_w)
    assert sorted(pi.tolist()) == list(range(N))                      # a permutation
    inv = np.empty(N, dtype=np.int64)
    inv[pi] = np.arange(N)
    assert np.array_equal(pi[inv], np.arange(N)) and np.array_equal(inv[pi], np.arange(N))
    nsp_total = g.frames * g.n_special
    assert bs[0] == nsp_total and bs[-1] == N
    # segment A: specials, frame-major, in order
    P = g.n_special + g.grid_h * g.grid_w
    assert pi[:nsp_total].tolist() == [s * P + j for s in range(g.frames) for j in range(g.n_special)]
    # every block holds exactly the tokens of one (frame group, window) key, all of them
    keys = [block_key(g, int(i)) for i in pi]
    seen = []
    for b in range(len(bs) - 1):
        ks = set(keys[bs[b]:bs[b + 1]])
        assert len(ks) == 1 and None not in ks
        seen.append(ks.pop())
    assert seen == sorted(set(seen)) and len(seen) == len(set(seen))   # lexicographic, no block split in two
    assert sum(bs[b + 1] - bs[b] for b in range(len(bs) - 1)) == g.frames * g.grid_h * g.grid_w
    # inside a block: (frame, y, x) row-major == increasing original index
    for b in range(len(bs) - 1):
        blk = pi[bs[b]:bs[b + 1]]
        assert np.all(np.diff(blk) > 0)


def test_reorder_then_inverse_is_identity_on_data():
    g = geom()
    pi, _ = orc.temporal_reorder(g)
    x = rand_bf16((g.heads, orc.num_tokens(g), g.head_dim), 1)
    xr = orc.reorder(g, pi, x)
    assert np.array_equal(xr, x[:, pi, :])
    back = np.empty_like(x)
    back[:, pi, :] = xr
    assert np.array_equal(back, x)


# ---------------------------------------------------------------- budget / closed-form M


def closed_form_M(S, nsp, h, w, blk, rho):
    """Independent formula: block sizes are products of clipped extents."""
    def extents(total, b):
        return [min(b, total - o) for o in range(0, total, b)]
    M = S * nsp
    for f in extents(S, blk[0]):
        for hh in extents(h, blk[1]):
            for ww in extents(w, blk[2]):
                n = f * hh * ww
                M += n - min(int(math.floor(rho * n + 1e-9)), n - 1)
    return M


@pytest.mark.parametrize("name,blk,rho,expect", [
    ("tiny", (2, 4, 4), 0.5, 532), ("small", (2, 4, 4), 0.7, 3500),
    ("medium", (2, 4, 4), 0.5, 16548), ("medium", (2, 4, 4), 0.7, 10500), ("medium", (2, 4, 4), 0.9, 4236),
    ("medium", (4, 4, 4), 0.7, 10392), ("medium", (4, 4, 4), 0.9, 3744),
    ("medium", (2, 8, 8), 0.7, 10092), ("medium", (2, 8, 8), 0.9, 3444),
    ("large", (4, 4, 4), 0.8, 28650), ("stack_layer", (2, 4, 4), 0.7, 21000)])
def test_merged_length_closed_form(name, blk, rho, expect):
    wl = synth.WORKLOADS[name].replace(blk_frames=blk[0], blk_h=blk[1], blk_w=blk[2])
    g = orc.Geometry.of(wl)
    assert closed_form_M(wl.frames, wl.n_special, wl.grid_h, wl.grid_w, blk, rho) == expect
    assert orc.merged_len(g, rho) == expect


@pytest.mark.parametrize("rho", [0.0, 0.1, 0.25, 0.5, 0.7, 0.75, 0.8, 0.9, 0.99])
def test_block_budget_and_split(rho):
    for n in list(range(1, 40)) + [50, 64, 80, 128]:
        r, nd = orc.block_budget(n, rho)
        assert r == min(int(math.floor(rho * n + 1e-9)), n - 1)
        assert nd == min(-(-n // 4), n - r) and nd >= 1
        dst = [j for j in range(n) if orc.is_dst(j, n, nd)]
        assert len(dst) == nd and dst[-1] == n - 1          # exactly n_dst, last position is dst
        assert n - nd >= r                                   # enough src to merge r of them
        if nd > 1:                                           # evenly spaced: gaps differ by at most 1
            gaps = np.diff(dst)
            assert gaps.max() - gaps.min() <= 1
    assert orc.block_budget(10, 0.7) == (7, 3)              # 70 % of 10 tokens is 7
    assert 0.58 * 50 < 29 and orc.block_budget(50, 0.58)[0] == 29   # binary 0.58*50 falls just short of 29
    assert 0.29 * 100 < 29 and orc.block_budget(100, 0.29)[0] == 29
    assert orc.block_budget(32, 0.9)[1] == 4                # dst shrink when more than 75 % are merged


def test_merged_count_matches_closed_form_on_data():
    wl = synth.WORKLOADS["tiny"]
    g = orc.Geometry.of(wl)
    q, k, v = synth.make_qkv(wl)
    res = orc.global_attention(g, 0.5, 0.7, q, k, v, attend=False)
    assert res.M_q == 532 == closed_form_M(4, 5, 16, 16, (2, 4, 4), 0.5)
    assert res.M_k == closed_form_M(4, 5, 16, 16, (2, 4, 4), 0.7)
    for A, M in ((res.assign_q, res.M_q), (res.assign_k, res.M_k)):
        for hd in range(g.heads):
            assert int((A[hd] == np.arange(A.shape[1])).sum()) == M


# ---------------------------------------------------------------- matching


def cosine_matrix(x):
    n = np.linalg.norm(x, axis=1, keepdims=True)
    xn = x / np.maximum(n, 1e-12)
    return xn @ xn.T


def test_match_equals_selection_from_global_cosine_matrix():
    """Appendix B, Prop. 1: block similarities are entries of the global matrix. An
    independent numpy matcher working from the global N x N cosine matrix must give
    the same assignment (inputs are random, margins are far above rounding)."""
    g = geom(S=3, nsp=2, h=5, w=6, H=2, D=8, blk=(2, 2, 4))
    pi, bs = orc.temporal_reorder(g)
    x = rand_bf16((g.heads, orc.num_tokens(g), g.head_dim), 3)
    xr = orc.reorder(g, pi, x)
    for rho in (0.3, 0.5, 0.8):
        A, mb, ms = orc.match(g, bs, rho, xr)
        for hd in range(g.heads):
            W = cosine_matrix(as_f64(x[hd]))                 # ORIGINAL order, global
            expect = np.arange(A.shape[1])
            for b in range(len(bs) - 1):
                base, n = int(bs[b]), int(bs[b + 1] - bs[b])
                r, nd = orc.block_budget(n, rho)
                dst = [j for j in range(n) if ((j + 1) * nd) // n > (j * nd) // n]
                src = [j for j in range(n) if j not in dst]
                cand = []
                for a in src:
                    sims = [W[pi[base + a], pi[base + d]] for d in dst]
                    bd = int(np.argmax(sims))
                    cand.append((-sims[bd], a, dst[bd]))
                cand.sort()
                for _, a, d in cand[:r]:
                    expect[base + a] = base + d
            assert np.array_equal(A[hd], expect)
            assert np.all(mb[hd][np.isfinite(mb[hd])] > 1e-9) and np.all(ms[hd][np.isfinite(ms[hd])] > 1e-9)


def test_match_is_optimal_by_brute_force():
    """Appendix B: the rule picks the r pairs (one per src) of maximum mean similarity
    Q(M). Enumerate every r-subset of src and every src->dst map on tiny blocks."""
    g = orc.Geometry(2, 1, 2, 4, 3, 8, 2, 2, 2)              # blocks of 2*2*2 = 8 tokens
    pi, bs = orc.temporal_reorder(g)
    x = rand_bf16((g.heads, orc.num_tokens(g), g.head_dim), 5)
    xr = orc.reorder(g, pi, x)
    for rho in (0.25, 0.5, 0.8):
        A = orc.match(g, bs, rho, xr, margins=False)
        for hd in range(g.heads):
            for b in range(len(bs) - 1):
                base, n = int(bs[b]), int(bs[b + 1] - bs[b])
                r, nd = orc.block_budget(n, rho)
                W = cosine_matrix(as_f64(xr[hd, base:base + n]))
                dst = [j for j in range(n) if orc.is_dst(j, n, nd)]
                src = [j for j in range(n) if j not in dst]
                best_q, best_sets = -np.inf, []
                for subset in itertools.combinations(src, r):
                    for targets in itertools.product(dst, repeat=r):
                        qv = sum(W[a, d] for a, d in zip(subset, targets))
                        if qv > best_q + 1e-12:
                            best_q, best_sets = qv, [dict(zip(subset, targets))]
                        elif abs(qv - best_q) <= 1e-12:
                            best_sets.append(dict(zip(subset, targets)))
                got = {a: int(A[hd, base + a] - base) for a in range(n) if A[hd, base + a] != base + a}
                assert len(got) == r and all(a in src and d in dst for a, d in got.items())
                assert len(best_sets) == 1 and got == best_sets[0]


def test_match_tie_breaks_and_zero_vectors():
    g = orc.Geometry(1, 0, 2, 4, 1, 4, 1, 2, 4)              # one block of 8 tokens: dst = {3, 7}
    _, bs = orc.temporal_reorder(g)
    one = np.zeros((1, 8, 4), dtype=np.float32)
    one[0, :, 0] = 1.0                                       # all tokens identical: every sim is 1
    A = orc.match(g, bs, 0.5, synth.f32_to_bf16_bits(one), margins=False)[0]
    # ties: lowest dst (3) and lowest src positions (0,1,2,4) win
    assert A.tolist() == [3, 3, 3, 3, 3, 5, 6, 7]
    z = one.copy()
    z[0, 0] = 0.0                                            # a zero vector has sim 0 to everything: ranked last
    A = orc.match(g, bs, 0.5, synth.f32_to_bf16_bits(z), margins=False)[0]
    assert A.tolist() == [0, 3, 3, 3, 3, 3, 6, 7]


def test_value_follows_key_matches():
    """Sec. 3.2: V is merged with K's matches; K's matches do not look at V."""
    wl = synth.WORKLOADS["tiny"].replace(heads=2)
    g = orc.Geometry.of(wl)
    q, k, v = synth.make_qkv(wl)
    r1 = orc.global_attention(g, 0.5, 0.5, q, k, v, attend=False)
    r2 = orc.global_attention(g, 0.5, 0.5, q, k, q, attend=False)   # another V
    assert np.array_equal(r1.assign_k, r2.assign_k) and np.array_equal(r1.rank_k, r2.rank_k)
    assert not np.array_equal(r1.assign_k, r1.assign_q)              # head-wise, tensor-wise independent
    assert np.allclose(r2.v_m, orc.merge(g, r1.rank_k, r1.M_k, orc.reorder(g, r1.pi, q)))


# ---------------------------------------------------------------- merge


def test_merge_is_group_mean_and_conserves_mass():
    wl = synth.WORKLOADS["tiny"].replace(heads=3)
    g = orc.Geometry.of(wl)
    q, k, v = synth.make_qkv(wl)
    res = orc.global_attention(g, 0.5, 0.7, q, k, v, attend=False)
    for x, A, R, M, xm in ((q, res.assign_q, res.rank_q, res.M_q, res.q_m), (v, res.assign_k, res.rank_k, res.M_k, res.v_m)):
        xr = as_f64(x[:, res.pi, :])
        for hd in range(g.heads):
            kept = np.flatnonzero(A[hd] == np.arange(A.shape[1]))
            assert len(kept) == M and np.array_equal(R[hd, kept], np.arange(M))   # kept tokens in reordered order
            cnt = np.bincount(R[hd], minlength=M)
            for m in (0, 7, 100, M // 2, M - 1):
                members = np.flatnonzero(A[hd] == kept[m])
                assert kept[m] in members and len(members) == cnt[m]
                assert np.allclose(xm[hd, m], xr[hd, members].mean(axis=0), rtol=0, atol=1e-12)
            # sum_m c_m * x_m == sum_i x_i per block; members stay inside the block; convex hull
            for b in (0, 5, len(res.blk_start) - 2):
                lo, hi = int(res.blk_start[b]), int(res.blk_start[b + 1])
                rows = np.unique(R[hd, lo:hi])
                assert np.all(A[hd, lo:hi] >= lo) and np.all(A[hd, lo:hi] < hi)
                assert cnt[rows].sum() == hi - lo
                assert np.allclose((cnt[rows, None] * xm[hd, rows]).sum(0), xr[hd, lo:hi].sum(0), atol=1e-9)
                assert np.all(xm[hd, rows] <= xr[hd, lo:hi].max(0) + 1e-12)
                assert np.all(xm[hd, rows] >= xr[hd, lo:hi].min(0) - 1e-12)


# ---------------------------------------------------------------- attention


def test_attention_matches_torch_sdpa_and_naive():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(11)
    H, Mq, Mk, D = 3, 37, 53, 16
    q, k, v = rng.standard_normal((H, Mq, D)), rng.standard_normal((H, Mk, D)), rng.standard_normal((H, Mk, D))
    got = orc.attention(q, k, v)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(k)[None], torch.from_numpy(v)[None])[0].numpy()
    assert np.allclose(got, ref, rtol=0, atol=1e-12)
    s = np.einsum("hqd,hkd->hqk", q, k) / math.sqrt(D)
    p = np.exp(s - s.max(-1, keepdims=True))
    p /= p.sum(-1, keepdims=True)
    assert np.allclose(got, np.einsum("hqk,hkd->hqd", p, v), rtol=0, atol=1e-12)
    rows = np.array([5, 0, 36, 5])
    assert np.array_equal(orc.attention(q, k, v, rows), got[:, rows])
    # each output row is a convex combination of V rows
    assert np.all(got <= v.max(1, keepdims=True) + 1e-12) and np.all(got >= v.min(1, keepdims=True) - 1e-12)
    # closed form: identical keys -> output is the mean of V
    k0 = np.broadcast_to(k[:, :1], k.shape)
    assert np.allclose(orc.attention(q, k0, v), np.broadcast_to(v.mean(1, keepdims=True), (H, Mq, D)), atol=1e-12)


def test_ratio_zero_is_exact_dense_attention():
    """With merge ratio 0 nothing merges, so reorder -> attention -> inverse reorder
    must be textbook multi-head attention over all N tokens."""
    torch = pytest.importorskip("torch")
    g = geom(S=3, nsp=2, h=5, w=6, H=2, D=8, blk=(2, 2, 4))
    N = orc.num_tokens(g)
    q, k, v = (rand_bf16((g.heads, N, g.head_dim), s) for s in (21, 22, 23))
    res = orc.global_attention(g, 0.0, 0.0, q, k, v)
    assert res.M_q == N and res.M_k == N
    assert np.array_equal(res.assign_q, np.broadcast_to(np.arange(N), (g.heads, N)))
    ref = naive_mha(as_f64(q), as_f64(k), as_f64(v))
    assert np.allclose(res.out, ref, rtol=0, atol=1e-12)
    assert np.allclose(orc.dense_attention(g, q, k, v), ref, rtol=0, atol=1e-12)
    t = lambda b: torch.from_numpy(as_f64(b))[None]
    sd = torch.nn.functional.scaled_dot_product_attention(t(q), t(k), t(v))[0]          # [H][N][D]
    assert np.allclose(res.out, sd.permute(1, 0, 2).reshape(N, -1).numpy(), rtol=0, atol=1e-12)
    toks = np.array([0, 17, N - 1])
    assert np.allclose(orc.dense_attention(g, q, k, v, toks), ref[toks], atol=1e-12)


# ---------------------------------------------------------------- whole pipeline


def python_pipeline(g, rho_q, rho_kv, q, k, v):
    """Independent restatement of the whole path with python sets / dicts, tiny sizes only."""
    P = g.n_special + g.grid_h * g.grid_w
    N = g.frames * P
    blocks = {}
    for i in range(N):
        key = block_key(g, i)
        if key is not None:
            blocks.setdefault(key, []).append(i)          # original indices, increasing

    def groups(x, rho):                                   # x [N][D] float64 -> list of member lists
        rep = {i: i for i in range(N)}
        for key in sorted(blocks):
            idx = blocks[key]
            n = len(idx)
            r = min(int(math.floor(rho * n + 1e-9)), n - 1)
            nd = min(-(-n // 4), n - r)
            dst = [idx[j] for j in range(n) if ((j + 1) * nd) // n > (j * nd) // n]
            src = [i for i in idx if i not in dst]
            unit = {i: x[i] / max(np.linalg.norm(x[i]), 1e-12) for i in idx}
            cand = []
            for a in src:
                sims = [float(unit[a] @ unit[d]) for d in dst]
                j = max(range(len(dst)), key=lambda t: (sims[t], -t))
                cand.append((-sims[j], a, dst[j]))
            for _, a, d in sorted(cand)[:r]:
                rep[a] = d
        out = {}
        for i in range(N):
            out.setdefault(rep[i], []).append(i)
        return rep, out

    res = np.empty((N, g.heads * g.head_dim))
    for hd in range(g.heads):
        Q, K, V = as_f64(q[hd]), as_f64(k[hd]), as_f64(v[hd])
        rep_q, gq = groups(Q, rho_q)
        _, gk = groups(K, rho_kv)
        qk = sorted(gq)
        kk = sorted(gk)
        Qm = np.stack([Q[gq[m]].mean(0) for m in qk])
        Km = np.stack([K[gk[m]].mean(0) for m in kk])
        Vm = np.stack([V[gk[m]].mean(0) for m in kk])
        Om = naive_mha(Qm[None], Km[None], Vm[None])
        row = {m: j for j, m in enumerate(qk)}
        for i in range(N):
            res[i, hd * g.head_dim:(hd + 1) * g.head_dim] = Om[row[rep_q[i]]]
    return res


@pytest.mark.parametrize("rho_q,rho_kv", [(0.5, 0.5), (0.9, 0.3), (0.0, 0.7), (0.6, 0.0)])
def test_pipeline_equals_independent_python_statement(rho_q, rho_kv):
    g = geom(S=3, nsp=2, h=5, w=6, H=2, D=8, blk=(2, 2, 4))
    N = orc.num_tokens(g)
    q, k, v = (rand_bf16((g.heads, N, g.head_dim), s) for s in (31, 32, 33))
    res = orc.global_attention(g, rho_q, rho_kv, q, k, v)
    assert np.allclose(res.out, python_pipeline(g, rho_q, rho_kv, q, k, v), rtol=0, atol=1e-11)
    again = orc.merged_attention_from_maps(g, res.pi, q, k, v, res.assign_q, res.assign_k)
    assert np.array_equal(again.out, res.out)
    toks = np.array([0, 3, 40, N - 1])
    assert np.allclose(orc.attention_rows_for_tokens(g, res, toks), res.out[toks], atol=1e-13)


def test_unmerge_is_a_pure_copy_decided_by_query_matches_only():
    """Eq. 5: merged-away query tokens copy their group's output; the tie pattern
    depends on Q's matches only (end of Sec. 3.2)."""
    wl = synth.WORKLOADS["tiny"].replace(heads=2)
    g = orc.Geometry.of(wl)
    q, k, v = synth.make_qkv(wl)
    a = orc.global_attention(g, 0.5, 0.5, q, k, v)
    b = orc.global_attention(g, 0.5, 0.0, q, k, v)
    assert np.array_equal(a.assign_q, b.assign_q) and np.array_equal(a.rank_q, b.rank_q)
    N, D = orc.num_tokens(g), g.head_dim
    for res in (a, b):
        for hd in range(g.heads):
            o = res.out[:, hd * D:(hd + 1) * D][res.pi]     # reordered order
            assert np.array_equal(o, res.o_m[hd][res.rank_q[hd]])
            merged = np.flatnonzero(res.assign_q[hd] != np.arange(N))
            assert len(merged) == N - res.M_q
            assert np.array_equal(o[merged], o[res.assign_q[hd][merged]])
    assert not np.allclose(a.out, b.out)                    # K/V merging does change values


def test_identical_tokens_in_blocks():
    """Merging identical tokens: Q-side merging never changes the output. K/V-side
    merging preserves it only when every block keeps the same fraction of its tokens
    and there are no special tokens (Eq. 3 has no size term, so otherwise the softmax
    mass of the blocks is re-weighted)."""
    # (a) Q-side only, general geometry with specials and clipped blocks: exact
    wl = synth.WORKLOADS["tiny"].replace(heads=2, frames=3, grid_h=6, grid_w=7)
    g = orc.Geometry.of(wl)
    x = synth.make_identical_block_tokens(wl, seed=1)
    _, k, v = synth.make_qkv(wl)
    dense = orc.dense_attention(g, x, k, v)
    res = orc.global_attention(g, 0.6, 0.0, x, k, v)
    assert res.M_q < orc.num_tokens(g)
    assert np.allclose(res.out, dense, rtol=0, atol=1e-12)
    # (b) K/V-side, uniform blocks (all of size 32, same kept fraction), no specials: exact
    wl2 = synth.WORKLOADS["tiny"].replace(heads=2, n_camera=0, n_register=0, grid_h=8, grid_w=8)
    g2 = orc.Geometry.of(wl2)
    kk = synth.make_identical_block_tokens(wl2, seed=2)
    vv = synth.make_identical_block_tokens(wl2, seed=3)
    q2, _, _ = synth.make_qkv(wl2)
    dense2 = orc.dense_attention(g2, q2, kk, vv)
    res2 = orc.global_attention(g2, 0.0, 0.5, q2, kk, vv)
    assert res2.M_k == orc.num_tokens(g2) // 2
    assert np.allclose(res2.out, dense2, rtol=0, atol=1e-12)
    # (c) negative control: with special tokens present the K/V-side result differs
    kk3 = synth.make_identical_block_tokens(wl, seed=2)
    vv3 = synth.make_identical_block_tokens(wl, seed=3)
    q3, _, _ = synth.make_qkv(wl)
    d3 = orc.dense_attention(g, q3, kk3, vv3)
    r3 = orc.global_attention(g, 0.0, 0.5, q3, kk3, vv3)
    assert np.abs(r3.out - d3).max() > 1e-6


def test_similarity_cost_model():
    """Appendix B (ii): sum over blocks of n_src*n_dst*D is about alpha(1-alpha) N n_b D."""
    wl = synth.WORKLOADS["medium"]
    g = orc.Geometry.of(wl)
    _, bs = orc.temporal_reorder(g)
    macs = full = 0
    for b in range(len(bs) - 1):
        n = int(bs[b + 1] - bs[b])
        r, nd = orc.block_budget(n, 0.7)
        macs += (n - nd) * nd * g.head_dim
        full += n == 32
    assert full == 972
    model = 0.25 * 0.75 * (full * 32) * 32 * g.head_dim     # full blocks only
    rest = macs - full * 24 * 8 * g.head_dim
    assert full * 24 * 8 * g.head_dim == model and 0 < rest < 0.05 * model


def test_merged_length_golden_table():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "merged_lengths.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 13
    for S, grid, bt, bh, bw, rho, M in rows:
        g = orc.Geometry(int(S), 5, int(grid), int(grid), 16, 64, int(bt), int(bh), int(bw))
        assert orc.merged_len(g, float(rho)) == int(M)


# ---------------------------------------------------------------- the paper's 1-D block regime (Sec. 3.3 / 4.1)


def test_runs_of_one_grid_row_equal_row_windows():
    """Sec. 3.3 defines spatial blocks as runs of n_s consecutive tokens of a frame.  Handing the frame over as a
    1 x (h w) grid with 1 x n_s windows is that definition; for n_s = w the runs are the rows of the h x w grid, so
    both geometries must give the same permutation, maps and output."""
    h, w, S = 4, 6, 5
    g2 = geom(S=S, nsp=2, h=h, w=w, H=2, D=8, blk=(3, 1, w))
    g1 = geom(S=S, nsp=2, h=1, w=h * w, H=2, D=8, blk=(3, 1, w))
    N = orc.num_tokens(g2)
    q, k, v = (rand_bf16((2, N, 8), s) for s in (71, 72, 73))
    a = orc.global_attention(g2, 0.6, 0.4, q, k, v)
    b = orc.global_attention(g1, 0.6, 0.4, q, k, v)
    assert np.array_equal(a.pi, b.pi) and np.array_equal(a.blk_start, b.blk_start)
    assert np.array_equal(a.assign_q, b.assign_q) and np.array_equal(a.assign_k, b.assign_k)
    assert np.array_equal(a.out, b.out)


def test_large_run_blocks_match_by_brute_force():
    """Blocks of several hundred tokens (runs of 100 tokens over 4 frames, the last run ragged): the map equals a plain
    loop over src x dst cosines with the top-r rule, at the budgets of the paper's configuration (0.9 / 0.7)."""
    g = geom(S=4, nsp=1, h=1, w=230, H=1, D=16, blk=(4, 1, 100))
    pi, bs = orc.temporal_reorder(g)
    assert np.diff(bs).tolist() == [400, 400, 120]
    x = rand_bf16((1, orc.num_tokens(g), 16), 9)
    xr = as_f64(orc.reorder(g, pi, x))[0]
    for rho in (0.9, 0.7):
        A = orc.match(g, bs, rho, orc.reorder(g, pi, x), margins=False)[0]
        for b in range(len(bs) - 1):
            base, n = int(bs[b]), int(bs[b + 1] - bs[b])
            r = min(int(np.floor(rho * n + 1e-9)), n - 1)
            nd = min(-(-n // 4), n - r)
            dst = [j for j in range(n) if ((j + 1) * nd) // n > (j * nd) // n]
            assert len(dst) == nd
            blk = xr[base:base + n]
            nrm = np.maximum(np.sqrt((blk * blk).sum(1)), 1e-12)
            best = []
            for a in range(n):
                if a in dst:
                    continue
                sims = [float(blk[a] @ blk[d]) / (nrm[a] * nrm[d]) for d in dst]
                j = max(range(nd), key=lambda t: (sims[t], -t))
                best.append((-sims[j], a, dst[j]))
            best.sort()
            expect = np.arange(n)
            for _, a, d in best[:r]:
                expect[a] = d
            assert np.array_equal(A[base:base + n] - base, expect)
