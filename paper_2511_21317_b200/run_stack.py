"""A stack of global-attention layers around the HTTM path: end-to-end latency against the dense kernel.

    python -m paper_2511_21317_b200.run_stack [--workload stack_layer] [--layers 24] [--steps 3] [--ratio 0.7]

Every layer is  x <- x + W_o . Attn(split(W_qkv . rmsnorm(x)))  with random-init bf16 projections (N(0, 0.02)) on a
correlated-field input.  The norm and the residual are torch elementwise kernels; the projections are torch.matmul or,
with --own-gemm, the library's own tcgen05 GEMM (httm_linear).  They run identically in both arms and are reported
separately.  Q, K, V are strided views of the fused projection output [N][3 * heads * 64] (no copies); the attention
output lands in [N][heads * 64], the layout the output projection reads.  The two arms:
    httm   httm_global_attention in every layer (merge ratios of the workload)
    dense  httm_dense_attention in every layer (the same attention kernel on all tokens)
Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import sys

import torch

from . import binding as hb
from . import synth


def rmsnorm(x: torch.Tensor) -> torch.Tensor:
    xf = x.float()
    return (xf * torch.rsqrt(xf.pow(2).mean(dim=-1, keepdim=True) + 1e-6)).to(torch.bfloat16)


class Stack:
    def __init__(self, wl, layers: int, device: str = "cuda:0", seed: int = 0, own_gemm: bool = False):
        self.wl, self.layers, self.device, self.own_gemm = wl, layers, device, own_gemm
        self.H, self.D, self.N = wl.heads, wl.head_dim, wl.n_tokens
        dim = self.H * self.D
        g = torch.Generator(device=device).manual_seed(seed)
        # weights as [out][in], the layout a linear layer stores
        self.w_qkv = [(torch.randn(3 * dim, dim, generator=g, device=device) * 0.02).to(torch.bfloat16) for _ in range(layers)]
        self.w_o = [(torch.randn(dim, dim, generator=g, device=device) * 0.02).to(torch.bfloat16) for _ in range(layers)]
        self.proj = torch.empty(self.N, dim, dtype=torch.bfloat16, device=device)
        q, _, _ = synth.make_qkv(wl)                                   # [H][N][64] correlated field, one tensor is enough
        self.x0 = hb.bf16_from_bits(q, device).permute(1, 0, 2).reshape(self.N, dim).contiguous()
        self.ctx = hb.Httm(hb.HttmConfig.of(wl))
        self.qkv = torch.empty(self.N, 3 * dim, dtype=torch.bfloat16, device=device)
        self.attn = torch.empty(self.N, dim, dtype=torch.bfloat16, device=device)

    def close(self):
        self.ctx.close()

    def views(self):
        """Q, K, V as [H][N][64] views of the fused projection output (token stride 3 * dim, head stride 64)."""
        v = self.qkv.view(self.N, 3, self.H, self.D)
        return [v[:, i].permute(1, 0, 2) for i in range(3)]

    def forward(self, dense: bool, attention: bool = True) -> torch.Tensor:
        x = self.x0.clone()
        q, k, v = self.views()
        for layer in range(self.layers):
            if self.own_gemm:
                self.ctx.linear(rmsnorm(x), self.w_qkv[layer], self.qkv)
            else:
                torch.matmul(rmsnorm(x), self.w_qkv[layer].t(), out=self.qkv)
            if attention:
                if dense:
                    self.ctx.dense_attention(q, k, v, self.attn)
                else:
                    self.ctx.global_attention(q, k, v, self.attn)
            if self.own_gemm:
                x = x + self.ctx.linear(self.attn, self.w_o[layer], self.proj)
            else:
                x = x + torch.matmul(self.attn, self.w_o[layer].t())
        return x


def timed(fn, steps: int) -> float:
    fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="stack_layer", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--layers", type=int, default=24)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--ratio", type=float, default=None, help="override both merge ratios")
    ap.add_argument("--own-gemm", action="store_true", help="projections by the library's own tcgen05 GEMM (httm_linear) instead of torch.matmul")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("run_stack: no CUDA device; the HTTM path has no CPU fallback")
    wl = synth.WORKLOADS[args.workload]
    if args.ratio is not None:
        wl = wl.replace(ratio_q=args.ratio, ratio_kv=args.ratio)
    st = Stack(wl, args.layers, own_gemm=args.own_gemm)
    try:
        st.attn.zero_()
        ms_lib = timed(lambda: st.forward(False, attention=False), args.steps)      # projections, norm, residual only
        ms_httm = timed(lambda: st.forward(False), args.steps)
        ms_dense = timed(lambda: st.forward(True), max(1, min(args.steps, 2)))
        y_h, y_d = st.forward(False).float(), st.forward(True).float()
        torch.cuda.synchronize()
        rel = float((y_h - y_d).norm() / y_d.norm())
        status = st.ctx.query(hb.Q_DEVICE_STATUS)
        print(json.dumps({
            "workload": wl.name, "layers": args.layers, "tokens": wl.n_tokens, "heads": wl.heads, "ratio_q": wl.ratio_q,
            "ratio_kv": wl.ratio_kv, "merged_tokens": {"M_q": st.ctx.m_q, "M_k": st.ctx.m_k},
            "ms_stack_httm": ms_httm, "ms_stack_dense": ms_dense, "speedup_end_to_end": ms_dense / ms_httm,
            "ms_library_ops_only": ms_lib, "ms_attention_path_httm": ms_httm - ms_lib, "ms_attention_path_dense": ms_dense - ms_lib,
            "speedup_attention_path": (ms_dense - ms_lib) / (ms_httm - ms_lib),
            "relative_l2_difference_of_the_outputs": rel, "finite": bool(torch.isfinite(y_h).all()), "device_status": status,
            "projections": "httm_linear (tcgen05 GEMM of this library)" if args.own_gemm else "torch.matmul",
            "note": "projections, rmsnorm and residual are identical in both arms; rmsnorm and residual are torch kernels"}))
    finally:
        st.close()
    return 0 if status == 0 else 1


if __name__ == "__main__":
    sys.exit(main())
