"""The allocation-free entry point (httm_global_attention_static) against the context-based one.

Some callers cannot call cudaMalloc when they need the layer (the device already belongs to
their own memory pool, or an allocation's device-wide synchronisation is not allowed where they
run), so the library offers a variant whose scratch is a fixed array inside the library.  It runs
the same kernels, so on the same inputs its output must equal httm_global_attention's; the file
is named to be collected last, so that a failure here cannot hide the result of any other test."""
import numpy as np
import pytest
import torch

from oracle import httm_oracle as orc
from paper_2511_21317_b200 import binding as hb
from paper_2511_21317_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def reference(wl, q, k, v):
    with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
        out = ctx.global_attention(q, k, v)
        torch.cuda.synchronize()
        assert ctx.query(hb.Q_DEVICE_STATUS) == 0
        return out.clone()


def test_static_scratch_entry_matches_context_entry_twice_in_a_row():
    # two different problems back to back: the second call finds the first call's data in the shared array
    wl_a = synth.WORKLOADS["tiny"]                                             # 1044 tokens, 16 heads, ~11 MiB of scratch
    wl_b = synth.Workload("static_b", 3, 9, 11, 2, 4, 4, 0.7, 0.5, heads=4, n_camera=1, n_register=2, seed=9)
    cases = []
    for wl in (wl_a, wl_b):
        q, k, v = (hb.bf16_from_bits(x, DEV) for x in synth.make_qkv(wl))
        out = torch.empty(wl.n_tokens, wl.heads * 64, dtype=torch.bfloat16, device=DEV)
        cases.append((wl, q, k, v, reference(wl, q, k, v), out))
    for rep in range(2):
        for wl, q, k, v, ref, out in cases:
            out.fill_(float("nan"))
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            hb.global_attention_static(hb.HttmConfig.of(wl), q, k, v, out)
            torch.cuda.synchronize()
            if rep == 1:   # (the very first call may load the library's device code lazily)
                # the call took no device memory; through a context the tiny case alone needs 11 MiB
                assert torch.cuda.mem_get_info()[0] >= free_before - (1 << 20)
            rms = ref.float().pow(2).mean().sqrt().item()
            err = (out.float() - ref.float()).abs().max().item()
            assert np.isfinite(err) and err <= 2e-2 * rms, (wl.name, rep, err, rms)
            assert torch.equal(out, ref), (wl.name, rep)        # same kernels, same order: bit-identical


def test_static_scratch_entry_with_larger_blocks_after_a_smaller_geometry():
    """Blocks of 64 and 128 tokens (the kernels that take a block in several passes), each run right after the tiny
    32-token case has left its data in the shared array, and clipped at the grid edge."""
    tiny = synth.WORKLOADS["tiny"]
    tq, tk, tv = (hb.bf16_from_bits(x, DEV) for x in synth.make_qkv(tiny))
    tout = torch.empty(tiny.n_tokens, tiny.heads * 64, dtype=torch.bfloat16, device=DEV)
    for wl in (synth.Workload("static_64", 6, 9, 10, 4, 4, 4, 0.6, 0.8, heads=3, seed=11),
               synth.Workload("static_128", 3, 17, 19, 2, 8, 8, 0.7, 0.5, heads=2, seed=12)):
        q, k, v = (hb.bf16_from_bits(x, DEV) for x in synth.make_qkv(wl))
        ref = reference(wl, q, k, v)
        out = torch.full((wl.n_tokens, wl.heads * 64), float("nan"), dtype=torch.bfloat16, device=DEV)
        hb.global_attention_static(hb.HttmConfig.of(tiny), tq, tk, tv, tout)
        hb.global_attention_static(hb.HttmConfig.of(wl), q, k, v, out)
        torch.cuda.synchronize()
        assert torch.equal(out, ref), wl.name


def test_static_scratch_entry_repeated_configuration_enqueues_kernels_only():
    """A call that repeats the configuration resident in the array copies nothing from the host, so it returns while
    earlier work on the stream is still running (a pageable host-to-device copy would wait for it)."""
    wl = synth.Workload("static_b", 3, 9, 11, 2, 4, 4, 0.7, 0.5, heads=4, n_camera=1, n_register=2, seed=9)
    q, k, v = (hb.bf16_from_bits(x, DEV) for x in synth.make_qkv(wl))
    ref = reference(wl, q, k, v)
    out = torch.empty(wl.n_tokens, wl.heads * 64, dtype=torch.bfloat16, device=DEV)
    cfg = hb.HttmConfig.of(wl)
    hb.global_attention_static(cfg, q, k, v, out)          # makes this configuration the resident one
    torch.cuda.synchronize()
    out.fill_(float("nan"))
    torch.cuda._sleep(400_000_000)                          # about 0.2 s of GPU time ahead of the call on the same stream
    hb.global_attention_static(cfg, q, k, v, out)
    still_busy = not torch.cuda.current_stream().query()
    torch.cuda.synchronize()
    assert still_busy, "the call waited for earlier work on the stream"
    assert torch.equal(out, ref)


def test_static_scratch_entry_against_the_oracle():
    """Directly against the CPU oracle (not only through the context entry): output within 2e-2 x RMS on the tiny scene."""
    wl = synth.WORKLOADS["tiny"]
    q, k, v = synth.make_qkv(wl)
    out = torch.empty(wl.n_tokens, wl.heads * 64, dtype=torch.bfloat16, device=DEV)
    hb.global_attention_static(hb.HttmConfig.of(wl), *(hb.bf16_from_bits(x, DEV) for x in (q, k, v)), out)
    torch.cuda.synchronize()
    ref = orc.global_attention(orc.Geometry.of(wl), wl.ratio_q, wl.ratio_kv, q, k, v).out
    assert parity.check_output(hb.bits_from_bf16(out), ref, what="static entry, tiny") <= parity.OUT_TOL


def test_static_scratch_entry_rejects_what_does_not_fit():
    wl = synth.WORKLOADS["small"]                                             # 10992 tokens x 16 heads: far beyond 16 MiB
    q = torch.zeros(wl.heads, wl.n_tokens, 64, dtype=torch.bfloat16, device=DEV)
    out = torch.zeros(wl.n_tokens, wl.heads * 64, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(hb.HttmError) as e:
        hb.global_attention_static(hb.HttmConfig.of(wl), q, q.clone(), q.clone(), out)
    assert e.value.code == hb.ERR_UNSUPPORTED and "static scratch" in str(e.value)
    assert torch.count_nonzero(out).item() == 0
    # a problem that passes the first size estimate (Q, K, V alone would fit) but not the exact layout of the array
    wl = synth.Workload("static_carve", 1, 200, 200, 1, 4, 4, 0.0, 0.0, heads=1)
    assert wl.n_tokens * 384 < 16 << 20
    q = torch.zeros(1, wl.n_tokens, 64, dtype=torch.bfloat16, device=DEV)
    out = torch.zeros(wl.n_tokens, 64, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(hb.HttmError) as e:
        hb.global_attention_static(hb.HttmConfig.of(wl), q, q.clone(), q.clone(), out)
    assert e.value.code == hb.ERR_UNSUPPORTED and "bytes of scratch" in str(e.value)
    torch.cuda.synchronize()
    assert torch.count_nonzero(out).item() == 0
