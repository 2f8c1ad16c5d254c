"""Pins of the outlier-filtering oracle (Sec. 3.4, Algorithm 2) against what the paper and the mathematics fix:
the no-filtering limit, a brute-force restatement on small inputs, the budget, singleton tokens against
exact attention, mass conservation, the everything-is-an-outlier limit, and the re-rooting rule."""
import numpy as np
import pytest

from oracle import httm_oracle as orc
from oracle import httm_outlier as out
from paper_2511_21317_b200 import synth


def small_case(seed=0, heads=3, ratio_q=0.7, ratio_kv=0.5, sigma=0.6):
    wl = synth.Workload("o", 3, 7, 9, 2, 4, 4, ratio_q, ratio_kv, heads=heads, seed=seed, sigma=sigma)
    return wl, orc.Geometry.of(wl), synth.make_qkv(wl)


def test_no_budget_filters_nothing():
    wl, g, (q, k, v) = small_case()
    ref = orc.global_attention(g, wl.ratio_q, wl.ratio_kv, q, k, v)
    res = out.global_attention_filtered(g, wl.ratio_q, wl.ratio_kv, 0.0, q, k, v)
    assert res.tau == float("inf") and not res.outlier.any()
    assert np.array_equal(res.assign_q, ref.assign_q)
    assert res.M_q == [ref.M_q] * g.heads
    assert np.array_equal(res.out, ref.out)


def test_deviation_threshold_and_map_against_brute_force():
    """Plain loops over tokens and groups, no vectorised indexing: same deviations, same threshold, same map."""
    wl, g, (q, k, v) = small_case(seed=3, heads=2)
    gamma = 0.08
    res = out.global_attention_filtered(g, wl.ratio_q, wl.ratio_kv, gamma, q, k, v, attend=False)
    qr = orc.bf16_to_double(orc.reorder(g, res.pi, q))
    H, N, D = qr.shape
    eps = np.zeros((H, N))
    for h in range(H):
        for r in range(N):
            members = [i for i in range(N) if res.assign_q0[h, i] == r]
            if len(members) >= 2:
                mean = [sum(qr[h, i, c] for i in members) / len(members) for c in range(D)]
                for i in members:
                    eps[h, i] = sum((qr[h, i, c] - mean[c]) ** 2 for c in range(D)) ** 0.5
    assert np.allclose(res.eps, eps, rtol=1e-12, atol=1e-12)
    K = int(np.floor(gamma * H * N + 1e-9))
    tau = sorted(eps.ravel().tolist(), reverse=True)[K]
    assert res.tau == pytest.approx(tau, rel=1e-12)
    for h in range(H):
        for r in set(res.assign_q0[h].tolist()):
            members = [i for i in range(N) if res.assign_q0[h, i] == r]
            stay = [i for i in members if not eps[h, i] > tau]
            for i in members:
                if eps[h, i] > tau:
                    assert res.assign_q[h, i] == i                       # an outlier stands alone
                else:
                    want = r if r in stay else min(stay)                 # old representative, else lowest remaining member
                    assert res.assign_q[h, i] == want


def test_budget_is_the_requested_fraction_of_all_heads_tokens():
    wl, g, (q, k, v) = small_case(seed=5, heads=4)
    for gamma in (0.01, 0.05, 0.2):
        res = out.global_attention_filtered(g, wl.ratio_q, wl.ratio_kv, gamma, q, k, v, attend=False)
        K = out.outlier_budget(res.eps.size, gamma)
        merged = int((res.eps > 0).sum())
        assert res.outlier.sum() == min(K, merged)          # continuous data: no ties at the threshold
        assert (res.eps[res.outlier] > res.eps[~res.outlier].max()).all()
        # one global budget (Sec. 3.4 item 3): heads take unequal shares
        assert sum(res.M_q) == g.heads * orc.merged_len(g, wl.ratio_q) + _extra_kept(res)
    assert len(set(res.outlier.sum(axis=1).tolist())) > 1


def _extra_kept(res):
    """Kept tokens added by the filtering = kept after - kept before, counted from the two maps."""
    idx = np.arange(res.assign_q.shape[1])
    return int((res.assign_q == idx).sum() - (res.assign_q0 == idx).sum())


def test_singleton_queries_reproduce_exact_attention_rows():
    """With unmerged keys (ratio_kv = 0) a query that stands alone - every outlier among them - must get the
    textbook softmax-attention row of the dense oracle."""
    wl, g, (q, k, v) = small_case(seed=7, heads=2, ratio_kv=0.0)
    res = out.global_attention_filtered(g, wl.ratio_q, 0.0, 0.1, q, k, v)
    dense = orc.dense_attention(g, q, k, v)
    D = g.head_dim
    checked = 0
    for h in range(g.heads):
        A = res.assign_q[h]
        alone = np.flatnonzero((A == np.arange(A.size)) & (np.bincount(A, minlength=A.size) == 1))
        assert res.outlier[h].sum() > 0 and np.isin(np.flatnonzero(res.outlier[h]), alone).all()
        toks = res.pi[alone]
        assert np.allclose(res.out[toks, h * D:(h + 1) * D], dense[toks, h * D:(h + 1) * D], rtol=1e-9, atol=1e-12)
        checked += alone.size
    assert checked > 0


def test_mass_is_conserved_and_merged_tokens_are_means_of_the_remaining_constituents():
    wl, g, (q, k, v) = small_case(seed=9, heads=2)
    res = out.global_attention_filtered(g, wl.ratio_q, wl.ratio_kv, 0.15, q, k, v, attend=False)
    qr = orc.bf16_to_double(orc.reorder(g, res.pi, q))
    for h in range(g.heads):
        A, rank = res.assign_q[h], res.rank_q[h]
        cnt = np.bincount(rank, minlength=res.M_q[h])
        assert cnt.sum() == A.size and res.M_q[h] == np.unique(A).size
        assert np.allclose((res.q_m[h] * cnt[:, None]).sum(axis=0), qr[h].sum(axis=0), rtol=1e-10)
        for m in np.flatnonzero(cnt >= 2)[:20]:
            assert np.allclose(res.q_m[h][m], qr[h][rank == m].mean(axis=0), rtol=1e-12, atol=1e-14)


def test_everything_an_outlier_equals_no_query_merging():
    wl, g, (q, k, v) = small_case(seed=11, heads=2)
    res = out.global_attention_filtered(g, wl.ratio_q, wl.ratio_kv, 1.0, q, k, v)
    ref = orc.global_attention(g, 0.0, wl.ratio_kv, q, k, v)
    assert res.M_q == [orc.num_tokens(g)] * g.heads
    assert np.allclose(res.out, ref.out, rtol=1e-12, atol=1e-14)


def test_group_survives_the_loss_of_its_destination_token():
    """Hand-made map: group {2 (dst), 0, 5}, token 2 an outlier -> 0 and 5 stay together under 0, 2 alone."""
    A = np.array([[2, 1, 2, 3, 4, 2, 6]])
    outl = np.array([[False, False, True, False, False, False, False]])
    assert out.filter_map(A, outl).tolist() == [[0, 1, 2, 3, 4, 0, 6]]
    outl2 = np.array([[True, False, True, False, False, False, False]])          # 0 and 2 leave: 5 is what remains
    assert out.filter_map(A, outl2).tolist() == [[0, 1, 2, 3, 4, 5, 6]]
    outl3 = np.array([[False, False, False, False, False, True, False]])         # a src leaves: the rest is untouched
    assert out.filter_map(A, outl3).tolist() == [[2, 1, 2, 3, 4, 5, 6]]
