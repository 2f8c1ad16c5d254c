"""Parity of the projection GEMM (tcgen05) with its CPU oracle.  Needs a B200."""
import numpy as np
import pytest
import torch

from oracle import httm_linear as lin
from paper_2511_21317_b200 import binding as hb
from paper_2511_21317_b200 import run_stack, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    with hb.Httm(hb.HttmConfig.of(synth.WORKLOADS["tiny"])) as c:
        yield c


def check(ctx, n, k, o, seed=0, ldx=None, ldw=None, ldy=None, scale=1.0):
    rng = np.random.default_rng(seed)
    xb = synth.f32_to_bf16_bits((rng.standard_normal((n, k)) * scale).astype(np.float32))
    wb = synth.f32_to_bf16_bits((rng.standard_normal((o, k)) * 0.05).astype(np.float32))
    x = torch.zeros(n, ldx or k, dtype=torch.bfloat16, device=DEV)
    w = torch.zeros(o, ldw or k, dtype=torch.bfloat16, device=DEV)
    x[:, :k] = hb.bf16_from_bits(xb, DEV)
    w[:, :k] = hb.bf16_from_bits(wb, DEV)
    ybuf = torch.full((n, ldy or o), 7.0, dtype=torch.bfloat16, device=DEV)
    y = ctx.linear(x[:, :k], w[:, :k], ybuf[:, :o])
    torch.cuda.synchronize()
    assert ctx.query(hb.Q_DEVICE_STATUS) == 0
    got = parity.bits_to_f64(hb.bits_from_bf16(y.contiguous()))
    exact = lin.linear(xb, wb)
    # one rounding to bf16 (half a step = 2^-9 |y|, written as 2^-8 like the merged tensors) + fp32 accumulation of k products
    bound = np.abs(exact) * 2.0 ** -8 + 2.0 ** -22 * lin.magnitude(xb, wb)
    err = np.abs(got - exact)
    assert (err <= bound).all(), f"n={n} k={k} o={o}: max err {err.max():.3e}, worst excess {(err - bound).max():.3e}"
    if ldy and ldy > o:
        assert (ybuf[:, o:].float() == 7.0).all()          # nothing is written past a row's end
    return float((err / np.maximum(np.abs(exact), 1e-30)).mean())


@pytest.mark.parametrize("n,k,o", [(128, 64, 256), (300, 128, 264), (1, 64, 8), (129, 1024, 3072), (777, 1024, 1024), (2000, 192, 40)])
def test_shapes_with_ragged_tiles(ctx, n, k, o):
    check(ctx, n, k, o, seed=n + k + o)


def test_strided_rows_and_large_values(ctx):
    check(ctx, 260, 128, 520, seed=5, ldx=136, ldw=200, ldy=528)
    check(ctx, 260, 64, 256, seed=6, scale=100.0)


def test_argument_errors(ctx):
    x = torch.zeros(16, 64, dtype=torch.bfloat16, device=DEV)
    w = torch.zeros(8, 64, dtype=torch.bfloat16, device=DEV)
    for bad_x, bad_w, code in ((x[:, :32], w[:, :32], hb.ERR_UNSUPPORTED),            # in_features not a multiple of 64
                               (x, torch.zeros(4, 64, dtype=torch.bfloat16, device=DEV), hb.ERR_UNSUPPORTED)):   # out not a multiple of 8
        with pytest.raises(hb.HttmError) as e:
            ctx.linear(bad_x, bad_w)
        assert e.value.code == code
    with pytest.raises(hb.HttmError) as e:
        ctx.linear(x, w, out=x[:, :8])                                                  # y overlaps x
    assert e.value.code == hb.ERR_INVALID_ARG
    assert ctx.linear(x[:0], w).shape == (0, 8)


def test_stack_with_own_projections_matches_the_library_projections():
    wl = synth.WORKLOADS["tiny"]
    a, b = run_stack.Stack(wl, layers=2), run_stack.Stack(wl, layers=2, own_gemm=True)
    try:
        ya, yb = a.forward(False).float(), b.forward(False).float()
        torch.cuda.synchronize()
        assert float((ya - yb).norm() / ya.norm()) < 2e-2
    finally:
        a.close()
        b.close()
