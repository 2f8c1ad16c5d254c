"""Pins of the two margin arrays the matching oracle returns (Eq. 1 and the top-r rule of
Sec. 3.2): `margin_best` (best minus runner-up similarity of every src token) and `margin_sel`
(r-th minus (r+1)-th best score of a block).  They decide where a map under test may differ from
the oracle's, so their VALUES are compared element by element with an independent numpy
statement that works by sorting, and on hand-made inputs whose margins are known in closed form.
CPU only."""
import numpy as np
import pytest

from oracle import httm_oracle as orc
from paper_2511_21317_b200 import synth


def rand_bf16(shape, seed):
    rng = np.random.default_rng(seed)
    return synth.f32_to_bf16_bits(rng.standard_normal(shape).astype(np.float32))


def as_f64(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def closed_form_budget(n, rho):
    r = min(int(np.floor(rho * n + 1e-9)), n - 1)
    return r, min(-(-n // 4), n - r)


def margins_by_sorting(g, bs, rho, xr):
    """Independent statement: per block, the full src x dst cosine table from one matrix product,
    each row SORTED (best - second), then the row maxima sorted (r-th - (r+1)-th)."""
    H, N = xr.shape[0], xr.shape[1]
    nb = len(bs) - 1
    mb = np.full((H, N), np.inf)
    ms = np.full((H, nb), np.inf)
    for hd in range(H):
        x = as_f64(xr[hd])
        xn = x / np.maximum(np.sqrt((x * x).sum(axis=1, keepdims=True)), 1e-12)
        for b in range(nb):
            lo, n = int(bs[b]), int(bs[b + 1] - bs[b])
            r, nd = closed_form_budget(n, rho)
            if r == 0:
                continue
            is_dst = np.array([((j + 1) * nd) // n > (j * nd) // n for j in range(n)])
            src, dst = np.flatnonzero(~is_dst), np.flatnonzero(is_dst)
            table = np.sort(xn[lo + src] @ xn[lo + dst].T, axis=1)      # ascending along dst
            if nd >= 2:
                mb[hd, lo + src] = table[:, -1] - table[:, -2]
            scores = np.sort(table[:, -1])[::-1]                         # descending
            if r < len(src):
                ms[hd, b] = scores[r - 1] - scores[r]
    return mb, ms


@pytest.mark.parametrize("blk,rho", [((2, 2, 4), 0.3), ((2, 2, 4), 0.5), ((2, 2, 4), 0.8), ((2, 4, 4), 0.7),
                                     ((3, 3, 5), 0.9), ((1, 3, 3), 0.5)])
def test_margins_equal_independent_sorting_statement(blk, rho):
    """A 5 x 6 grid over 3 frames: every block shape above leaves clipped windows and a short last
    frame group, so full, clipped, tiny (n = 1, 2) blocks and both budget regimes all occur."""
    g = orc.Geometry(3, 2, 5, 6, 3, 8, *blk)
    pi, bs = orc.temporal_reorder(g)
    xr = orc.reorder(g, pi, rand_bf16((g.heads, orc.num_tokens(g), g.head_dim), 11))
    _, mb, ms = orc.match(g, bs, rho, xr)
    mb_ref, ms_ref = margins_by_sorting(g, bs, rho, xr)
    assert np.array_equal(np.isinf(mb), np.isinf(mb_ref)) and np.array_equal(np.isinf(ms), np.isinf(ms_ref))
    fin = np.isfinite(mb_ref)
    assert fin.any() and (np.isfinite(ms_ref).any() or rho > 0.75)   # above 0.75 every src merges: no (r+1)-th score
    assert np.allclose(mb[fin], mb_ref[fin], rtol=0, atol=1e-14)
    fin = np.isfinite(ms_ref)
    assert np.allclose(ms[fin], ms_ref[fin], rtol=0, atol=1e-14)
    assert (mb[np.isfinite(mb)] >= 0).all() and (ms[np.isfinite(ms)] >= 0).all()
    # special tokens and dst tokens have no margin
    assert np.isinf(mb[:, :int(bs[0])]).all()


def unit(angle_deg):
    a = np.deg2rad(angle_deg)
    return np.array([np.cos(a), np.sin(a)])


def one_block(tokens, rho):
    """One head, one frame, a 1 x n grid with one 1 x n window: the block is `tokens` in order."""
    tokens = np.asarray(tokens, dtype=np.float32)
    n, D = tokens.shape
    g = orc.Geometry(1, 0, 1, n, 1, D, 1, 1, n)
    pi, bs = orc.temporal_reorder(g)
    assert pi.tolist() == list(range(n))
    A, mb, ms = orc.match(g, bs, rho, synth.f32_to_bf16_bits(tokens)[None])
    return A[0], mb[0], ms[0]


def test_margins_of_a_hand_made_block():
    """n = 8 at ratio 0.5: r = 4, dst = positions 3 and 7 (evenly spaced, last position dst).
    Values are exactly representable in bf16 and the cosines are known: dst e1 and e2; src tokens
    (1,0): cos 1 / 0; (3,4): .6 / .8; (4,3): .8 / .6; (0,2): 0 / 1; (1,1): both 1/sqrt 2 (tie);
    (-1,0): -1 / 0."""
    tok = [[1, 0], [3, 4], [4, 3], [2, 0], [0, 2], [1, 1], [-1, 0], [0, 5]]
    A, mb, ms = one_block(tok, 0.5)
    s = 1 / np.sqrt(2)
    expect_mb = [1.0, 0.2, 0.2, np.inf, 1.0, 0.0, 1.0, np.inf]
    assert np.allclose(mb[[0, 1, 2, 4, 5, 6]], np.array(expect_mb)[[0, 1, 2, 4, 5, 6]], atol=1e-15)
    assert np.isinf(mb[[3, 7]]).all()
    # scores: 1, .8, .8, 1, .7071, 0  ->  sorted 1, 1, .8, .8 | .7071, 0 : margin .8 - .7071
    assert ms[0] == pytest.approx(0.8 - s, abs=1e-15)
    assert A.tolist() == [3, 7, 3, 3, 7, 5, 6, 7]


def test_selection_margin_is_zero_on_an_exact_tie():
    """Two src tokens with the same score on either side of the budget: margin exactly 0, and the
    lower position is the one merged."""
    tok = [[3, 4], [4, 3], [1, 0], [0, 0], [0, 0], [0, 0], [0, 0], [0, 1]]   # n = 8, dst = 3 (zero vector) and 7
    # src scores vs dst e2 (the zero dst gives 0): .8, .6, 0, 0, 0, 0 -> r = 2 takes .8, .6 ; margin .6 - 0
    A, mb, ms = one_block(tok, 0.25)
    assert ms[0] == pytest.approx(0.6, abs=1e-15) and A.tolist() == [7, 7, 2, 3, 4, 5, 6, 7]
    tok = [[3, 4], [3, 4], [3, 4], [1, 0], [0, 0], [0, 0], [0, 0], [0, 1]]   # three equal scores, r = 2
    A, mb, ms = one_block(tok, 0.25)
    assert ms[0] == 0.0 and A.tolist() == [7, 7, 2, 3, 4, 5, 6, 7]
    assert mb[0] == pytest.approx(0.8 - 0.6, abs=1e-15)                       # vs dst (1,0): .6


def test_margins_are_infinite_where_nothing_is_decided():
    rng = np.random.default_rng(5)
    tok = rng.standard_normal((8, 4))
    # ratio 0: r = 0 -> nothing is chosen, both margins +inf
    A, mb, ms = one_block(tok, 0.0)
    assert np.isinf(mb).all() and np.isinf(ms).all() and A.tolist() == list(range(8))
    # ratio 0.9 on 8 tokens: r = 7, n_dst = min(2, 1) = 1 -> one dst (no runner-up), r = n_src (no (r+1)-th score)
    A, mb, ms = one_block(tok, 0.9)
    assert np.isinf(mb).all() and np.isinf(ms).all() and A.tolist() == [7] * 8
    # ratio 0.75 on 8 tokens: r = 6 = n_src with two dst: selection margin +inf, best margins finite
    A, mb, ms = one_block(tok, 0.75)
    assert np.isinf(ms).all() and np.isfinite(mb[[0, 1, 2, 4, 5, 6]]).all() and np.isinf(mb[[3, 7]]).all()
    # a block of one token
    A, mb, ms = one_block(tok[:1], 0.9)
    assert np.isinf(mb).all() and np.isinf(ms).all() and A.tolist() == [0]


def test_best_margin_uses_the_runner_up_not_the_first_loser():
    """The runner-up must be tracked through a rising sequence (a new best demotes the old best)
    and through values that fall between second and best: four dst at 16 tokens, ratio 0.25."""
    dst_angles = [10.0, 20.0, 40.0, 30.0]        # dst positions 3, 7, 11, 15
    tok = np.zeros((16, 2))
    for j, a in zip((3, 7, 11, 15), dst_angles):
        tok[j] = unit(a)
    src_pos = [j for j in range(16) if j not in (3, 7, 11, 15)]
    src_angles = [41.0, 9.0, 26.0, 33.0, 100.0, 0.0, 19.0, 38.0, 29.0, 45.0, 15.0, 24.0]
    for j, a in zip(src_pos, src_angles):
        tok[j] = unit(a)
    bits = synth.f32_to_bf16_bits(tok.astype(np.float32))
    x = as_f64(bits)
    xn = x / np.linalg.norm(x, axis=1, keepdims=True)
    A, mb, ms = one_block(synth.bf16_bits_to_f32(bits), 0.25)
    for j in src_pos:
        sims = np.sort(xn[j] @ xn[[3, 7, 11, 15]].T)
        assert mb[j] == pytest.approx(sims[-1] - sims[-2], abs=1e-15)
