"""One-tile check of the tcgen05 / TMEM / TMA building blocks against plain fp64 matmuls."""
import numpy as np
import pytest
import torch

from paper_2511_21317_b200 import binding as hb

pytestmark = pytest.mark.gpu


def test_single_tile_qk_and_pv():
    g = torch.Generator().manual_seed(0)
    q, k, v = (torch.randn(128, 64, generator=g).to(torch.bfloat16).cuda() for _ in range(3))
    s, o = hb.selftest_tensor_core(q, k, v)
    qd, kd, vd = (t.double().cpu().numpy() for t in (q, k, v))
    s_ref = qd @ kd.T
    assert np.abs(s.cpu().numpy() - s_ref).max() <= 1e-4 * np.abs(s_ref).max()
    p = s.to(torch.bfloat16).double().cpu().numpy()          # the kernel rounds its own S to bf16
    o_ref = p @ vd
    assert np.abs(o.cpu().numpy() - o_ref).max() <= 1e-4 * np.abs(o_ref).max()
    # structured input: catches transposed / permuted operands that random data could hide less clearly
    qi = torch.zeros(128, 64); qi[:, 0] = torch.arange(128) / 64.0; qi[:, 1] = 1.0
    ki = torch.zeros(128, 64); ki[:, 0] = 1.0; ki[:, 1] = torch.arange(128) / 128.0
    vi = torch.zeros(128, 64); vi[torch.arange(128), torch.arange(128) % 64] = 1.0
    qi, ki, vi = (t.to(torch.bfloat16).cuda() for t in (qi, ki, vi))
    s2, o2 = hb.selftest_tensor_core(qi, ki, vi)
    s2_ref = qi.double().cpu().numpy() @ ki.double().cpu().numpy().T
    assert np.allclose(s2.cpu().numpy(), s2_ref, atol=1e-5)
    o2_ref = s2.to(torch.bfloat16).double().cpu().numpy() @ vi.double().cpu().numpy()
    assert np.allclose(o2.cpu().numpy(), o2_ref, rtol=1e-5, atol=1e-5)
