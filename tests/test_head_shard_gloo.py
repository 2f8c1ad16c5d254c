"""Head-sharded layers, host side, as two gloo ranks on the CPU: the shard bookkeeping of bench.py, and the fact the
sharded threshold selection rests on: summing the shards' radix histograms level by level (an all-reduce) selects
exactly the threshold the oracle finds over all heads (Sec. 3.4 item 3)."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def radix_threshold(bits_local, budget, allreduce):
    """(K+1)-th largest of the non-negative floats whose bit patterns the shards hold, by the 11 + 11 + 10 bit radix
    select with one histogram sum per level.  Zeros are never counted at the first level (they cannot be outliers)."""
    prefix, rank, mask = 0, budget, 0
    for nb, shift in ((2048, 21), (2048, 10), (1024, 0)):
        sel = bits_local[(bits_local & mask) == prefix]
        hist = np.bincount((sel >> shift) & (nb - 1), minlength=nb).astype(np.int64)
        hist = allreduce(hist)
        above, b = 0, nb - 1
        while b > 0 and above + hist[b] <= rank:
            above += hist[b]
            b -= 1
        prefix |= b << shift
        rank -= above
        mask |= (nb - 1) << shift
    return np.array([prefix], dtype=np.uint32).view(np.float32)[0]


def worker(rank, world, port, results):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        from oracle import httm_oracle as orc
        from oracle import httm_outlier as flt
        from paper_2511_21317_b200 import synth

        wl = synth.Workload("shards", 4, 9, 10, 2, 4, 4, 0.7, 0.5, heads=6, seed=3)
        first, count = bench.head_shard(rank, world, wl.heads)
        assert count == 3 and first == 3 * rank
        spans = [bench.head_shard(r, world, wl.heads) for r in range(world)]
        assert sorted(h for f, c in spans for h in range(f, f + c)) == list(range(wl.heads))
        q, k, v = synth.make_qkv(wl)
        g = orc.Geometry.of(wl)
        res = orc.global_attention(g, wl.ratio_q, wl.ratio_kv, q, k, v, attend=False)
        eps = flt.deviations(res.assign_q, orc.reorder(g, res.pi, q)).astype(np.float32)   # the kernels keep deviations in fp32
        gamma = 0.07
        K = flt.outlier_budget(eps.size, gamma)
        expect = np.sort(eps.ravel())[::-1][K]                         # the (K+1)-th largest over ALL heads

        def allreduce(h):
            t = torch.from_numpy(h)
            dist.all_reduce(t)
            return t.numpy()
        mine = eps[first:first + count].ravel().view(np.uint32)
        tau = radix_threshold(mine, K, allreduce)
        # the summed level-0 histogram is the histogram of all heads
        h_all = np.bincount(eps.ravel().view(np.uint32) >> 21, minlength=2048)
        h_sum = allreduce(np.bincount(mine >> 21, minlength=2048).astype(np.int64))
        results[rank] = (float(tau), float(expect), bool(np.array_equal(h_all, h_sum)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_select_the_threshold_of_all_heads():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    with mp.Manager() as m:
        results = m.dict()
        mp.spawn(worker, args=(2, port, results), nprocs=2, join=True)
        assert len(results) == 2
        for rank in range(2):
            tau, expect, same = results[rank]
            assert tau == expect and same, (rank, tau, expect, same)
