"""Run a few HTTM global-attention layers of a named synthetic workload and nothing else.

    python -m paper_2511_21317_b200.run_layer --workload medium --calls 2 [--dense 1] [--stages 1] [--ratio 0.9] [--block 4x4x4]
                                              [--outlier-fraction 0.01]

A profiler is pointed at this command (the ncu summaries under profiles/ name it): few launches, no timing loops,
no CPU work besides the input generator.  It is not needed to use the library.  It prints the merged lengths and the device status word, and exits
non-zero if the status word is set.
"""
from __future__ import annotations

import argparse
import sys

import torch

from . import binding as hb
from . import synth


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="medium", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--calls", type=int, default=2, help="httm_global_attention calls")
    ap.add_argument("--dense", type=int, default=0, help="httm_dense_attention calls")
    ap.add_argument("--stages", type=int, default=0, help="rounds of every kernel launched on its own (reorder, match, merge, "
                    "match and merge with direct block loads, attention, unmerge, and - blocks of at most 32 tokens - attention "
                    "with the unmerge in its epilogue; for large blocks reorder, scores, select, merge, attention, unmerge)")
    ap.add_argument("--heads", type=int, default=None, help="override the number of heads")
    ap.add_argument("--ratio", type=float, default=None, help="override both merge ratios")
    ap.add_argument("--block", default=None, help="override the block shape, e.g. 4x4x4")
    ap.add_argument("--outlier-fraction", type=float, default=0.0, help="query outlier filtering (Sec. 3.4) in the public calls")
    args = ap.parse_args()
    wl = synth.WORKLOADS[args.workload]
    if args.heads is not None:
        wl = wl.replace(heads=args.heads)
    if args.ratio is not None:
        wl = wl.replace(ratio_q=args.ratio, ratio_kv=args.ratio)
    if args.block:
        bt, bh, bw = (int(x) for x in args.block.lower().split("x"))
        wl = wl.replace(blk_frames=bt, blk_h=bh, blk_w=bw)
    if not torch.cuda.is_available():
        raise SystemExit("run_layer: no CUDA device; the HTTM path has no CPU fallback")
    q, k, v = synth.make_qkv(wl)
    with hb.Httm(hb.HttmConfig.of(wl, device=0)) as ctx:
        dq, dk, dv = (hb.bf16_from_bits(x, "cuda:0") for x in (q, k, v))
        out = ctx.new_output()
        if args.outlier_fraction > 0:
            ctx.set_outlier_fraction(args.outlier_fraction)
        for _ in range(args.calls):
            ctx.global_attention(dq, dk, dv, out)
        for _ in range(args.dense):
            ctx.dense_attention(dq, dk, dv, out)
        ctx.set_outlier_fraction(0.0)
        max_block = ctx.query(hb.Q_MAX_BLOCK_TOKENS)
        big = max_block > 256   # large blocks: reorder (+ norms), scores, select, merge, attention, unmerge
        order = [0, 8, 9, 2, 3, 4] if big else [0, 1, 2, 5, 6, 3, 4]
        if max_block <= 32:
            order.append(hb.STAGE_ATTENTION_UNMERGE)   # attention with the unmerge in its epilogue (what the public call runs)
        for _ in range(args.stages):
            for st in order:
                ctx.launch_stage(st, dq, dk, dv, out)
        torch.cuda.synchronize()
        status = ctx.query(hb.Q_DEVICE_STATUS)
        print(f"run_layer: {wl.name} N={wl.n_tokens} M_q={ctx.m_q} M_k={ctx.m_k} calls={args.calls} dense={args.dense} "
              f"launches={ctx.launch_count()} device_status={status}")
    return 0 if status == 0 else 1


if __name__ == "__main__":
    sys.exit(main())
