"""The error paths the library promises, provoked from the host (nothing here faults or hangs the device):
an allocation that fails (HTTM_ERR_NOMEM, everything taken so far is given back) and a bounded device-side wait
that runs out (the kernel returns, the status word is set, the host reports HTTM_ERR_TIMEOUT, the context stays
usable).  Needs a B200."""
import time

import numpy as np
import pytest
import torch

from paper_2511_21317_b200 import binding as hb
from paper_2511_21317_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_failed_allocation_is_reported_and_nothing_leaks():
    wl = synth.WORKLOADS["tiny"]
    cfg = hb.HttmConfig.of(wl)
    with hb.Httm(cfg):                      # (loads the library's device code, so that the readings below are comparable)
        pass
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    try:
        for nth in (1, 2, 7, 15):           # the first allocation of httm_create, early ones, the last of the base workspace
            hb.fail_nth_allocation(nth)
            with pytest.raises(hb.HttmError) as e:
                hb.Httm(cfg)
            assert e.value.code == hb.ERR_NOMEM and "cudaMalloc" in str(e.value)
            assert torch.cuda.mem_get_info()[0] == free0, f"allocation {nth}: device memory was not given back"
        hb.fail_nth_allocation(0)
        with hb.Httm(cfg) as ctx:
            base = ctx.query(hb.Q_WORKSPACE_BYTES)
            free1 = torch.cuda.mem_get_info()[0]
            hb.fail_nth_allocation(4)       # inside the workspace of the outlier filter
            with pytest.raises(hb.HttmError) as e:
                ctx.set_outlier_fraction(0.1)
            assert e.value.code == hb.ERR_NOMEM
            assert ctx.query(hb.Q_WORKSPACE_BYTES) == base and torch.cuda.mem_get_info()[0] == free1
            ctx.set_outlier_fraction(0.1)   # the retry allocates everything and works
            q, k, v = (hb.bf16_from_bits(x, DEV) for x in synth.make_qkv(wl))
            out = ctx.global_attention(q, k, v)
            torch.cuda.synchronize()
            assert ctx.query(hb.Q_DEVICE_STATUS) == 0 and torch.isfinite(out.float()).all()
    finally:
        hb.fail_nth_allocation(0)


def test_an_expired_wait_is_reported_as_a_timeout_and_the_context_stays_usable():
    wl = synth.WORKLOADS["tiny"].replace(heads=2)
    q, k, v = (hb.bf16_from_bits(x, DEV) for x in synth.make_qkv(wl))
    with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
        ref = ctx.global_attention(q, k, v).clone()
        torch.cuda.synchronize()
        assert ctx.query(hb.Q_DEVICE_STATUS) == 0
        t0 = time.perf_counter()
        ctx.expire_a_wait()                 # the kernel gives up after about two seconds and RETURNS
        torch.cuda.synchronize()
        waited = time.perf_counter() - t0
        assert 1.0 < waited < 10.0, waited
        with pytest.raises(hb.HttmError) as e:
            ctx.query(hb.Q_DEVICE_STATUS)
        assert e.value.code == hb.ERR_TIMEOUT
        with pytest.raises(hb.HttmError) as e:
            ctx.export(hb.X_ASSIGN_Q)
        assert e.value.code == hb.ERR_TIMEOUT
        again = ctx.global_attention(q, k, v)          # the device context and the library's context still work
        torch.cuda.synchronize()
        assert torch.equal(again, ref)
    with hb.Httm(hb.HttmConfig.of(wl)) as fresh:       # ... and so does a new one
        out = fresh.global_attention(q, k, v)
        torch.cuda.synchronize()
        assert fresh.query(hb.Q_DEVICE_STATUS) == 0 and torch.equal(out, ref)
