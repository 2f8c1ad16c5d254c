"""Parity of the large-block path (merging blocks of 257 .. 4096 tokens: the paper's runs of 128 tokens over 30
frames, Sec. 3.3 / 4.1) with the CPU oracle.  All tests here need a B200."""
import numpy as np
import pytest
import torch

from oracle import httm_oracle as orc
from paper_2511_21317_b200 import binding as hb
from paper_2511_21317_b200 import synth
from tests import parity
from tests.test_gpu_parity import exports

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_big(wl, q=None, k=None, v=None, sample=None, peaky=False):
    if q is None:
        q, k, v = synth.make_qkv(wl)
    g = orc.Geometry.of(wl)
    with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
        assert ctx.query(hb.Q_MAX_BLOCK_TOKENS) > 256
        assert ctx.m_q == orc.merged_len(g, wl.ratio_q) and ctx.m_k == orc.merged_len(g, wl.ratio_kv)
        dq, dk, dv = (hb.bf16_from_bits(x, DEV) for x in (q, k, v))
        before = ctx.launch_count()
        out = ctx.global_attention(dq, dk, dv)
        torch.cuda.synchronize()
        assert ctx.launch_count() - before == 6          # reorder, scores, select, merge, attention, unmerge
        assert ctx.query(hb.Q_DEVICE_STATUS) == 0
        ex = exports(ctx)
        stats = parity.full_check(g, wl.ratio_q, wl.ratio_kv, q, k, v, ex, hb.bits_from_bf16(out), sample, wl.name, peaky)
        out2 = ctx.global_attention(dq, dk, dv)
        torch.cuda.synchronize()
        assert torch.equal(out, out2)
        ex2 = exports(ctx)
        for name in ex:
            assert np.array_equal(ex[name], ex2[name]), f"{name} differs between two identical calls"
        # the stages one by one give the same result
        out3 = ctx.new_output()
        for st in (hb.STAGE_REORDER, hb.STAGE_BIG_SCORES, hb.STAGE_BIG_SELECT, hb.STAGE_MERGE, hb.STAGE_ATTENTION, hb.STAGE_UNMERGE):
            ctx.launch_stage(st, dq, dk, dv, out3)
        torch.cuda.synchronize()
        assert torch.equal(out, out3)
        for st in (hb.STAGE_MATCH, hb.STAGE_MATCH_DIRECT, hb.STAGE_MERGE_DIRECT):
            with pytest.raises(hb.HttmError) as e:
                ctx.launch_stage(st, dq, dk, dv, out3)
            assert e.value.code == hb.ERR_UNSUPPORTED
    return stats


GEOMS = [
    # name, frames, grid_h, grid_w, blk, ratio_q, ratio_kv, n_camera, n_register, heads
    ("runs_ragged", 4, 1, 230, (4, 1, 100), 0.9, 0.7, 1, 0, 2),            # blocks of 400, 400, 120 tokens
    ("windows_512", 5, 17, 19, (4, 8, 16), 0.7, 0.5, 1, 4, 2),             # 2-D windows, clipped in every direction
    ("just_above_256", 3, 10, 30, (3, 9, 10), 0.6, 0.8, 1, 4, 2),          # 270-token blocks
    ("runs_3840", 30, 1, 300, (30, 1, 128), 0.9, 0.7, 1, 4, 2),            # the paper's block: 3840, 3840, 1320 tokens
    ("max_4096", 32, 1, 140, (32, 1, 128), 0.75, 0.9, 1, 0, 1),            # 4096-token block + a ragged one
    ("ratio_zero_q", 4, 1, 300, (4, 1, 128), 0.0, 0.7, 1, 4, 2),
    ("ratio_099", 4, 1, 300, (4, 1, 128), 0.99, 0.99, 1, 4, 2),
    ("odd_dst_counts", 7, 1, 211, (7, 1, 97), 0.83, 0.41, 0, 0, 3),        # n = 679, 679, 119: n_dst not a multiple of anything
]


@pytest.mark.parametrize("case", GEOMS, ids=[c[0] for c in GEOMS])
def test_large_block_geometries(case):
    name, S, h, w, blk, rq, rkv, ncam, nreg, H = case
    wl = synth.Workload(name, S, h, w, blk[0], blk[1], blk[2], rq, rkv, n_camera=ncam, n_register=nreg, heads=H, seed=5)
    run_big(wl, peaky=True)


def test_large_blocks_random_uncorrelated_inputs():
    wl = synth.Workload("gauss_big", 8, 1, 200, 8, 1, 128, 0.8, 0.6, heads=3)
    rng = np.random.default_rng(11)
    q, k, v = (synth.f32_to_bf16_bits(rng.standard_normal((wl.heads, wl.n_tokens, 64)).astype(np.float32)) for _ in range(3))
    run_big(wl, q, k, v, peaky=True)


def test_large_blocks_ties_and_zero_vectors():
    """Identical tokens in a block: every cosine ties, all src go to the first dst (one group of hundreds of tokens)."""
    wl = synth.Workload("ties_big", 4, 1, 150, 4, 1, 100, 0.5, 0.5, heads=2, n_camera=1, n_register=1)
    x = synth.make_identical_block_tokens(wl, seed=4)
    q, k, v = synth.make_qkv(wl)
    z = q.copy()
    z[:, 10:400, :] = 0
    run_big(wl, x, k, v, peaky=True)
    run_big(wl, q, x, v, peaky=True)
    run_big(wl, z, z, v, peaky=True)


def test_paper_block_regime_full_size_sampled():
    """Runs of 128 tokens x 30 frames on 60 frames of 37 x 37 patches, 90 % / 70 % merged (Sec. 4.1), all 16 heads (the
    configuration the benchmark times): maps and merged tensors on all tokens, attention output on sampled tokens."""
    wl = synth.WORKLOADS["paper_1d"]
    rng = np.random.default_rng(2)
    toks = np.unique(np.concatenate([rng.integers(0, wl.n_tokens, 24), [0, 4, 5, wl.n_tokens - 1]]))
    stats = run_big(wl, sample=toks)
    assert stats["out_err"] <= parity.OUT_TOL and stats["peaky_needed"] == 0
