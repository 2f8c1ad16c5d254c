"""Head-sharded layers on one GPU: two contexts with half of the heads each, whose threshold histograms are summed the
way an all-reduce over two GPUs would sum them, must arrive at exactly the threshold, the maps and the merged
tensors of one context with all the heads (Sec. 3.4 item 3: one outlier budget across all heads).  Needs a B200."""
import numpy as np
import pytest
import torch

from paper_2511_21317_b200 import binding as hb
from paper_2511_21317_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


class Exchange:
    """Stands in for the all-reduce of one shard: remembers the local histogram of every level and, where the sum over
    the shards is already known, puts it in place."""

    def __init__(self):
        self.level = 0
        self.local = {}
        self.summed = {}

    def __call__(self, counts):
        self.local[self.level] = counts.clone()
        if self.level in self.summed:
            counts.copy_(self.summed[self.level])
        self.level += 1


@pytest.mark.parametrize("blk,gamma", [((2, 4, 4), 0.05), ((4, 4, 4), 0.1)])   # warp-per-block filter kernels / sorted-group kernels
def test_two_head_shards_reproduce_the_whole_layer(blk, gamma):
    wl = synth.Workload("shards", 6, 9, 10, blk[0], blk[1], blk[2], 0.7, 0.5, heads=8, seed=21)
    q, k, v = (hb.bf16_from_bits(x, DEV) for x in synth.make_qkv(wl))
    with hb.Httm(hb.HttmConfig.of(wl)) as whole:
        whole.set_outlier_fraction(gamma)
        out = whole.global_attention(q, k, v)
        torch.cuda.synchronize()
        ref = {n: whole.export(w) for n, w in (("tau", hb.X_THRESHOLD), ("aq", hb.X_ASSIGN_Q), ("mq", hb.X_MERGED_Q_HEAD),
                                               ("rank", hb.X_RANK_Q), ("qm", hb.X_Q_MERGED), ("km", hb.X_K_MERGED))}
        n_out = whole.query(hb.Q_OUTLIERS)
    half = wl.replace(heads=4)
    shards = [hb.Httm(hb.HttmConfig.of(half)) for _ in range(2)]
    try:
        full_out = torch.zeros_like(out)
        xs = [Exchange(), Exchange()]
        for c, x in zip(shards, xs):
            c.set_outlier_fraction(gamma)
            c.set_head_shard(8, x)
        # Each level's histogram depends on the bins chosen before it: one round per level makes that level's sum
        # known (the histograms are deterministic), the last round runs with all three in place.
        for rnd in range(4):
            for g, (c, x) in enumerate(zip(shards, xs)):
                x.level = 0
                hs = slice(4 * g, 4 * g + 4)
                c.global_attention(q[hs], k[hs], v[hs], full_out[:, 256 * g:256 * (g + 1)])
            torch.cuda.synchronize()
            if rnd < 3:
                total = xs[0].local[rnd] + xs[1].local[rnd]
                xs[0].summed[rnd] = xs[1].summed[rnd] = total
        for g, c in enumerate(shards):
            assert c.query(hb.Q_DEVICE_STATUS) == 0
            hs = slice(4 * g, 4 * g + 4)
            assert c.export(hb.X_THRESHOLD)[0] == ref["tau"][0]
            assert np.array_equal(c.export(hb.X_ASSIGN_Q), ref["aq"][hs])
            assert np.array_equal(c.export(hb.X_MERGED_Q_HEAD), ref["mq"][hs])
            assert np.array_equal(c.export(hb.X_RANK_Q), ref["rank"][hs])
            assert np.array_equal(c.export(hb.X_K_MERGED), ref["km"][hs])
            for hd in range(4):
                rows = int(ref["mq"][4 * g + hd])
                assert np.array_equal(c.export(hb.X_Q_MERGED)[hd][:rows], ref["qm"][4 * g + hd][:rows])
        assert shards[0].query(hb.Q_OUTLIERS) + shards[1].query(hb.Q_OUTLIERS) == n_out
        # same merged tensors per head; the attention kernel deals its query tiles differently for 4 and for 8 heads, so the
        # outputs agree to rounding, not bit by bit
        a, b = parity.bits_to_f64(hb.bits_from_bf16(full_out)), parity.bits_to_f64(hb.bits_from_bf16(out))
        assert np.abs(a - b).max() <= 1e-2 * np.sqrt((b ** 2).mean())
    finally:
        for c in shards:
            c.close()


def test_head_shard_argument_errors():
    wl = synth.Workload("shard_args", 2, 8, 8, 2, 4, 4, 0.5, 0.5, heads=4)
    with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
        with pytest.raises(hb.HttmError) as e:
            ctx.set_head_shard(2, lambda counts: None)          # the layer cannot have fewer heads than the shard
        assert e.value.code == hb.ERR_INVALID_ARG
        with pytest.raises(hb.HttmError) as e:
            ctx.set_head_shard(8, None)                          # other shards hold heads: their counts must come from somewhere
        assert e.value.code == hb.ERR_INVALID_ARG
        ctx.set_head_shard(8, lambda counts: None)
        ctx.set_head_shard(0, None)
        # a failing exchange surfaces as an error of the attention call
        q, k, v = (hb.bf16_from_bits(x, DEV) for x in synth.make_qkv(wl))
        ctx.set_outlier_fraction(0.1)

        def broken(counts):
            raise RuntimeError("link down")
        ctx.set_head_shard(8, broken)
        with pytest.raises(hb.HttmError) as e:
            ctx.global_attention(q, k, v)
        assert e.value.code == hb.ERR_CUDA
        torch.cuda.synchronize()
