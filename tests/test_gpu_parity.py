"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element.
All tests here need a B200."""
import numpy as np
import pytest
import torch

from oracle import httm_oracle as orc
from paper_2511_21317_b200 import binding as hb
from paper_2511_21317_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def exports(ctx):
    names = {"pi": hb.X_PI, "blk_start": hb.X_BLOCK_START, "qr": hb.X_Q_REORDERED, "kr": hb.X_K_REORDERED,
             "vr": hb.X_V_REORDERED, "assign_q": hb.X_ASSIGN_Q, "assign_k": hb.X_ASSIGN_K, "rank_q": hb.X_RANK_Q,
             "q_m": hb.X_Q_MERGED, "k_m": hb.X_K_MERGED, "v_m": hb.X_V_MERGED, "o_m": hb.X_O_MERGED}
    return {k: ctx.export(v) for k, v in names.items()}


def run_case(wl, q=None, k=None, v=None, sample=None, peaky=False):
    if q is None:
        q, k, v = synth.make_qkv(wl)
    g = orc.Geometry.of(wl)
    with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
        assert ctx.n_tokens == wl.n_tokens
        assert ctx.m_q == orc.merged_len(g, wl.ratio_q) and ctx.m_k == orc.merged_len(g, wl.ratio_kv)
        dq, dk, dv = (hb.bf16_from_bits(x, DEV) for x in (q, k, v))
        out = ctx.global_attention(dq, dk, dv)
        torch.cuda.synchronize()
        assert ctx.query(hb.Q_DEVICE_STATUS) == 0
        # the public call reads small blocks straight from Q/K/V; the reorder kernel runs on request
        ctx.launch_stage(hb.STAGE_REORDER, dq, dk, dv)
        ex = exports(ctx)
        out_bits = hb.bits_from_bf16(out)
        stats = parity.full_check(g, wl.ratio_q, wl.ratio_kv, q, k, v, ex, out_bits, sample, wl.name, peaky)
        # determinism: a second call gives bit-identical results (catches races)
        out2 = ctx.global_attention(dq, dk, dv)
        torch.cuda.synchronize()
        assert torch.equal(out, out2)
        ctx.launch_stage(hb.STAGE_REORDER, dq, dk, dv)
        ex2 = exports(ctx)
        for name in ex:
            assert np.array_equal(ex[name], ex2[name]), f"{name} differs between two identical calls"
    return stats


def test_tiny_config_full_parity():
    stats = run_case(synth.WORKLOADS["tiny"])
    assert stats["out_err"] <= parity.OUT_TOL and stats["peaky_needed"] == 0


def report_peaky(name, stats):
    """The adversarial cases are checked with the extra bf16-representation term; say how many elements used it."""
    print(f"[peaky] {name}: {stats['peaky_needed']} of {stats['out_elements']} output elements beyond "
          f"{parity.OUT_TOL} x RMS (max err / RMS {stats['out_err']:.4f})")
    assert stats["peaky_needed"] <= 0.001 * stats["out_elements"]   # (at most 5 elements in any case when this was written)


GEOMS = [
    # name, frames, grid_h, grid_w, blk, ratio_q, ratio_kv, n_camera, n_register, heads
    ("clipped_all_dims", 3, 5, 6, (2, 2, 4), 0.5, 0.7, 1, 1, 2),
    ("window_1x1", 3, 3, 3, (2, 1, 1), 0.5, 0.5, 1, 4, 2),
    ("single_token_blocks", 2, 2, 2, (1, 1, 1), 0.9, 0.9, 1, 0, 1),
    ("no_specials", 4, 8, 8, (2, 4, 4), 0.5, 0.75, 0, 0, 3),
    ("frames_not_divisible", 5, 9, 9, (4, 4, 4), 0.7, 0.8, 1, 4, 2),
    ("ratio_zero_q", 4, 8, 8, (2, 4, 4), 0.0, 0.6, 1, 4, 2),
    ("ratio_zero_kv", 4, 8, 8, (2, 4, 4), 0.6, 0.0, 1, 4, 2),
    ("ratio_099", 4, 9, 9, (2, 4, 4), 0.99, 0.99, 1, 4, 2),
    ("block_128", 4, 17, 19, (2, 8, 8), 0.7, 0.9, 1, 4, 2),
    ("block_64", 9, 10, 10, (4, 4, 4), 0.5, 0.9, 1, 4, 2),
    ("block_256_max", 5, 9, 8, (4, 8, 8), 0.8, 0.3, 1, 4, 1),
    ("one_frame", 1, 12, 12, (2, 4, 4), 0.5, 0.5, 1, 4, 2),
    ("many_specials", 3, 6, 6, (2, 4, 4), 0.5, 0.5, 1, 44, 2),      # 45 special tokens per frame: the path over the reordered copies
    ("many_specials_64", 3, 8, 8, (4, 4, 4), 0.6, 0.6, 3, 67, 2),
]


@pytest.mark.parametrize("case", GEOMS, ids=[c[0] for c in GEOMS])
def test_adversarial_geometries(case):
    name, S, h, w, blk, rq, rkv, ncam, nreg, H = case
    wl = synth.Workload(name, S, h, w, blk[0], blk[1], blk[2], rq, rkv, n_camera=ncam, n_register=nreg, heads=H, seed=3)
    report_peaky(name, run_case(wl, peaky=True))


def test_random_uncorrelated_inputs():
    wl = synth.Workload("gauss", 4, 11, 13, 2, 4, 4, 0.6, 0.6, heads=4)
    rng = np.random.default_rng(5)
    q, k, v = (synth.f32_to_bf16_bits(rng.standard_normal((wl.heads, wl.n_tokens, 64)).astype(np.float32)) for _ in range(3))
    report_peaky("gauss", run_case(wl, q, k, v, peaky=True))


def test_ties_and_zero_vectors():
    wl = synth.Workload("ties", 2, 8, 8, 2, 4, 4, 0.5, 0.5, heads=2, n_camera=1, n_register=1)
    x = synth.make_identical_block_tokens(wl, seed=4)       # every similarity inside a block is a tie
    q, k, v = synth.make_qkv(wl)
    z = q.copy()
    z[:, 10:40, :] = 0                                         # zero vectors: norm clamp
    report_peaky("ties q", run_case(wl, x, k, v, peaky=True))
    report_peaky("ties k", run_case(wl, q, x, v, peaky=True))
    report_peaky("zero vectors", run_case(wl, z, z, v, peaky=True))


def test_ratio_zero_equals_dense_and_textbook():
    wl = synth.Workload("r0", 3, 7, 9, 2, 4, 4, 0.0, 0.0, heads=3)
    q, k, v = synth.make_qkv(wl)
    g = orc.Geometry.of(wl)
    ref = orc.dense_attention(g, q, k, v)
    with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
        assert ctx.m_q == wl.n_tokens == ctx.m_k
        dq, dk, dv = (hb.bf16_from_bits(x, DEV) for x in (q, k, v))
        o_h = ctx.global_attention(dq, dk, dv)
        o_d = ctx.dense_attention(dq, dk, dv)
        torch.cuda.synchronize()
        parity.check_output(hb.bits_from_bf16(o_d), ref, what="dense")
        parity.check_output(hb.bits_from_bf16(o_h), ref, what="httm ratio 0")
        # same kernel, same rows, same key order up to the permutation -> very close
        d = (o_h.float() - o_d.float()).abs().max().item()
        assert d <= 2e-2 * float(np.sqrt(np.mean(ref ** 2)))


@pytest.mark.parametrize("heads", [2, 26])
def test_scores_far_above_those_of_the_first_key_tile(heads):
    """Keys whose scores exceed everything in a row's first key tile by 2^80 .. 2^320: the kernel takes its stabiliser
    from the first tile and redoes a tile whose weights would overflow (even heads: two such jumps; odd heads stay just
    below the limit, with weights of up to 2^90); rows with the opposite sign see scores that only fall.  Two heads
    are dealt as single passes (one query tile per CTA), 26 heads as pair passes."""
    wl = synth.Workload("grow", 2, 18, 20, 2, 4, 4, 0.0, 0.0, heads=heads)
    N = wl.n_tokens                                              # 730 tokens: six key tiles, pair passes and single passes
    rng = np.random.default_rng(21)
    w = rng.standard_normal(64)
    w /= np.linalg.norm(w)
    tile = np.arange(N) // 128
    a = np.stack([np.where(tile == 0, 0.1, np.where(tile <= 2, 25.0, 60.0)),     # q.k/8*log2(e): 0.5, 135, 325
                  np.where(tile == 0, 0.1, 15.0)] * (heads // 2))                 # 0.5, 81
    b = np.where(rng.random(N) < 0.5, 30.0, -30.0)
    b[::7] = 0.01                                                # rows that see almost flat scores
    k = a[:, :, None] * w + 0.3 * rng.standard_normal((heads, N, 64))
    q = b[None, :, None] * w + 0.05 * rng.standard_normal((heads, N, 64))
    v = rng.standard_normal((heads, N, 64))
    q, k, v = (synth.f32_to_bf16_bits(x.astype(np.float32)) for x in (q, k, v))
    ref = orc.dense_attention(orc.Geometry.of(wl), q, k, v)
    with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
        dq, dk, dv = (hb.bf16_from_bits(x, DEV) for x in (q, k, v))
        o_d = ctx.dense_attention(dq, dk, dv)
        o_h = ctx.global_attention(dq, dk, dv)                  # ratio 0: the same rows through the epilogue that unmerges
        torch.cuda.synchronize()
        assert ctx.query(hb.Q_DEVICE_STATUS) == 0
        for name, o in (("dense", o_d), ("ratio 0", o_h)):
            bits = hb.bits_from_bf16(o)
            assert np.isfinite(parity.bits_to_f64(bits)).all(), name
            stats = {}
            stats["out_err"] = parity.check_output(bits, ref, what=f"growing scores, {name}", peaky=True, stats=stats)
            report_peaky(f"growing scores, {name}", stats)


def test_dense_attention_small_config_sampled():
    wl = synth.WORKLOADS["small"].replace(heads=4)
    q, k, v = synth.make_qkv(wl)
    g = orc.Geometry.of(wl)
    rng = np.random.default_rng(0)
    toks = np.unique(np.concatenate([rng.integers(0, wl.n_tokens, 96), [0, 1, 4, wl.n_tokens - 1, 10944, 10943]]))
    ref = orc.dense_attention(g, q, k, v, toks)
    with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
        out = ctx.dense_attention(*(hb.bf16_from_bits(x, DEV) for x in (q, k, v)))
        torch.cuda.synchronize()
        bits = hb.bits_from_bf16(out)
        assert np.isfinite(parity.bits_to_f64(bits)).all()
        parity.check_output(bits[toks], ref, what="dense small")


def test_strided_layouts_fused_qkv_and_head_major_output():
    """Q/K/V as slices of one [N][3][H][D] projection output; output written as [H][N][D]."""
    wl = synth.Workload("strided", 4, 9, 9, 2, 4, 4, 0.5, 0.7, heads=4)
    q, k, v = synth.make_qkv(wl)
    H, N, D = wl.heads, wl.n_tokens, 64
    fused = torch.empty(N, 3, H, D, dtype=torch.bfloat16, device=DEV)
    for i, x in enumerate((q, k, v)):
        fused[:, i] = hb.bf16_from_bits(x, DEV).permute(1, 0, 2)
    with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
        ref = ctx.global_attention(*(hb.bf16_from_bits(x, DEV) for x in (q, k, v)))
        views = [fused[:, i].permute(1, 0, 2) for i in range(3)]      # [H][N][D] views, token stride 3*H*D
        assert not views[0].is_contiguous()
        got = ctx.global_attention(*views)
        out_hm = torch.zeros(H, N, D, dtype=torch.bfloat16, device=DEV)
        lib_out = hb._Tensor(out_hm.data_ptr(), N * D, D)
        rc = ctx._lib.httm_global_attention(ctx._h, ctx._tensor(views[0], "q"), ctx._tensor(views[1], "k"),
                                            ctx._tensor(views[2], "v"), lib_out, ctx._stream(None))
        assert rc == 0
        torch.cuda.synchronize()
        assert torch.equal(ref, got)
        assert torch.equal(out_hm.permute(1, 0, 2).reshape(N, H * D), ref)
        d_ref = ctx.dense_attention(*(hb.bf16_from_bits(x, DEV) for x in (q, k, v)))
        d_got = ctx.dense_attention(*views)
        torch.cuda.synchronize()
        assert torch.equal(d_ref, d_got)


def test_stage_calls_equal_the_fused_call_and_host_entry_point():
    wl = synth.WORKLOADS["tiny"].replace(heads=4)
    q, k, v = synth.make_qkv(wl)
    with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
        dq, dk, dv = (hb.bf16_from_bits(x, DEV) for x in (q, k, v))
        ref = ctx.global_attention(dq, dk, dv)
        n0 = ctx.launch_count()
        out = ctx.new_output().zero_()
        for st in range(5):
            ctx.launch_stage(st, dq, dk, dv, out)
        torch.cuda.synchronize()
        assert ctx.launch_count() == n0 + 5
        assert torch.equal(ref, out)
        hq, hk, hv = (hb.bf16_from_bits(x, pin=True) for x in (q, k, v))
        hout = torch.empty(wl.n_tokens, wl.heads * 64, dtype=torch.bfloat16).pin_memory()
        ctx.attention_host(hq, hk, hv, hout)
        torch.cuda.synchronize()
        assert torch.equal(hout, ref.cpu())
        dref = ctx.dense_attention(dq, dk, dv)
        ctx.attention_host(hq, hk, hv, hout, dense=True)
        torch.cuda.synchronize()
        assert torch.equal(hout, dref.cpu())


def test_unmerge_in_the_attention_epilogue_equals_the_separate_kernels():
    """With blocks of at most 32 tokens the public call is three kernels: the attention epilogue writes every merged query
    row to its member tokens (Eq. 5-7).  Same bits as attention -> O_m -> unmerge kernel, for clipped blocks, scenes that go
    over the reordered copies (many special tokens), single-token blocks, ratio 0, and a head-major output."""
    cases = [synth.WORKLOADS["tiny"].replace(heads=3),
             synth.Workload("fused_clipped", 5, 9, 10, 2, 4, 4, 0.6, 0.7, heads=3, seed=7),
             synth.Workload("fused_specials", 3, 6, 6, 2, 4, 4, 0.5, 0.5, heads=2, n_camera=1, n_register=44, seed=8),
             synth.Workload("fused_single_tokens", 2, 3, 3, 1, 1, 1, 0.9, 0.9, heads=2, n_camera=1, n_register=0, seed=9),
             synth.Workload("fused_ratio_zero", 3, 7, 9, 2, 4, 4, 0.0, 0.5, heads=2, seed=10),
             synth.WORKLOADS["small"].replace(heads=2)]
    for wl in cases:
        q, k, v = synth.make_qkv(wl)
        H, N = wl.heads, wl.n_tokens
        with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
            dq, dk, dv = (hb.bf16_from_bits(x, DEV) for x in (q, k, v))
            direct = wl.n_camera + wl.n_register <= 32
            n0 = ctx.launch_count()
            fused = ctx.global_attention(dq, dk, dv)
            torch.cuda.synchronize()
            assert ctx.launch_count() - n0 == (3 if direct else 4), wl.name
            with pytest.raises(hb.HttmError) as e:      # O_m of that call was never written
                ctx.launch_stage(hb.STAGE_UNMERGE, dq, dk, dv, ctx.new_output())
            assert e.value.code == hb.ERR_INVALID_ARG
            o_m = ctx.export(hb.X_O_MERGED)              # ... and is computed on request
            rank_q, pi_inv = ctx.export(hb.X_RANK_Q), ctx.export(hb.X_PI_INV)
            bits = hb.bits_from_bf16(fused)
            for hd in range(H):
                assert np.array_equal(bits[:, hd * 64:(hd + 1) * 64], o_m[hd][rank_q[hd][pi_inv]]), f"{wl.name}: head {hd}"
            sep = ctx.new_output().fill_(float("nan"))
            stages = (hb.STAGE_MATCH_DIRECT, hb.STAGE_MERGE_DIRECT) if direct else (hb.STAGE_REORDER, hb.STAGE_MATCH, hb.STAGE_MERGE)
            for st in stages + (hb.STAGE_ATTENTION, hb.STAGE_UNMERGE):
                ctx.launch_stage(st, dq, dk, dv, sep)
            again = ctx.new_output().fill_(float("nan"))
            ctx.launch_stage(hb.STAGE_ATTENTION_UNMERGE, dq, dk, dv, again)
            out_hm = torch.full((H, N, 64), float("nan"), dtype=torch.bfloat16, device=DEV)    # head-major output
            rc = ctx._lib.httm_global_attention(ctx._h, ctx._tensor(dq, "q"), ctx._tensor(dk, "k"), ctx._tensor(dv, "v"),
                                                hb._Tensor(out_hm.data_ptr(), N * 64, 64), ctx._stream(None))
            assert rc == 0
            torch.cuda.synchronize()
            assert ctx.query(hb.Q_DEVICE_STATUS) == 0
            assert torch.equal(fused, sep) and torch.equal(fused, again), wl.name
            assert torch.equal(out_hm.permute(1, 0, 2).reshape(N, H * 64), fused), wl.name


def test_call_timing_names_the_kernels_of_the_public_call():
    """Events between the kernels of httm_global_attention: the parts are the kernels the call runs, in order, their
    times are positive and add up to no more than the whole call, and the results do not change."""
    wl = synth.WORKLOADS["tiny"]
    q, k, v = (hb.bf16_from_bits(x, DEV) for x in synth.make_qkv(wl))
    with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
        ref = ctx.global_attention(q, k, v).clone()
        with pytest.raises(hb.HttmError) as e:
            ctx.call_times()
        assert e.value.code == hb.ERR_INVALID_ARG
        ctx.set_call_timing(True)
        assert ctx.call_times() == []                                  # no call yet
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        before = ctx.launch_count()
        e0.record()
        out = ctx.global_attention(q, k, v)
        e1.record()
        parts = ctx.call_times()
        torch.cuda.synchronize()
        assert ctx.launch_count() - before == 3 and torch.equal(out, ref)
        assert [n for n, _ in parts] == ["match_direct", "merge_direct", "attention_unmerge"]
        assert all(ms > 0 for _, ms in parts) and sum(ms for _, ms in parts) <= e0.elapsed_time(e1) * 1.001
        ctx.set_outlier_fraction(0.05)
        ctx.global_attention(q, k, v)
        assert [n for n, _ in ctx.call_times()] == ["match_direct", "outlier_filter", "merge_direct", "attention", "unmerge"]
        ctx.set_outlier_fraction(0.0)
        ctx.set_call_timing(False)
        assert torch.equal(ctx.global_attention(q, k, v), ref)
    big = synth.Workload("timing_big", 4, 1, 230, 4, 1, 100, 0.9, 0.7, heads=2)
    q, k, v = (hb.bf16_from_bits(x, DEV) for x in synth.make_qkv(big))
    with hb.Httm(hb.HttmConfig.of(big)) as ctx:
        ctx.set_call_timing(True)
        ctx.global_attention(q, k, v)
        assert [n for n, _ in ctx.call_times()] == ["reorder", "big_scores", "big_select", "merge", "attention", "unmerge"]


def test_argument_errors_are_reported_before_any_launch():
    wl = synth.WORKLOADS["tiny"].replace(heads=2)
    with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
        H, N, D = wl.heads, wl.n_tokens, 64
        good = [torch.zeros(H, N, D, dtype=torch.bfloat16, device=DEV) for _ in range(3)]
        out = ctx.new_output()
        n0 = ctx.launch_count()
        T = hb._Tensor
        t = lambda x: ctx._tensor(x, "x")
        o = ctx._tensor(out, "out", True)
        call = lambda q, k, v, oo: ctx._lib.httm_global_attention(ctx._h, q, k, v, oo, ctx._stream(None))
        assert call(T(None, N * D, D), t(good[1]), t(good[2]), o) == hb.ERR_INVALID_ARG
        assert call(T(good[0].data_ptr() + 2, N * D, D), t(good[1]), t(good[2]), o) == hb.ERR_ALIGNMENT
        assert call(T(good[0].data_ptr(), N * D, D + 4), t(good[1]), t(good[2]), o) == hb.ERR_ALIGNMENT
        assert call(T(good[0].data_ptr(), N * D, 32), t(good[1]), t(good[2]), o) == hb.ERR_INVALID_ARG
        assert call(t(good[0]), t(good[1]), t(good[2]), T(good[0].data_ptr(), D, H * D)) == hb.ERR_INVALID_ARG   # aliasing
        assert ctx._lib.httm_dense_attention(ctx._h, t(good[0]), t(good[1]), T(None, 0, 0), o, ctx._stream(None)) == hb.ERR_INVALID_ARG
        assert b"null" in ctx._lib.httm_last_error(ctx._h)
        assert ctx._lib.httm_launch_stage(ctx._h, 99, t(good[0]), t(good[1]), t(good[2]), o, ctx._stream(None)) == hb.ERR_INVALID_ARG
        buf = np.empty(3, dtype=np.int32)
        assert ctx._lib.httm_export(ctx._h, hb.X_PI, buf.ctypes.data, buf.nbytes, None) == hb.ERR_INVALID_ARG
        assert ctx.launch_count() == n0
        with pytest.raises(hb.HttmError):
            ctx.global_attention(good[0].float(), good[1], good[2])
        torch.cuda.synchronize()
        assert ctx.query(hb.Q_DEVICE_STATUS) == 0


def test_small_config_full_size_sampled():
    """VGGT-shaped small scene at full size: maps and merged tensors in full, attention on sampled tokens."""
    wl = synth.WORKLOADS["small"]
    rng = np.random.default_rng(1)
    toks = np.unique(np.concatenate([rng.integers(0, wl.n_tokens, 64), np.arange(5), [wl.n_tokens - 1]]))
    stats = run_case(wl, sample=toks)
    assert stats["merged_exactly_rounded"] > 0.99 and stats["peaky_needed"] == 0


def test_medium_config_full_size_sampled():
    """The benchmark's workload at full size (33k tokens, 16 heads), in the launch configuration the benchmark
    times: permutation, reordered tensors, maps, rank and merged tensors in full; attention on sampled tokens;
    unmerge as a pure copy on every token."""
    wl = synth.WORKLOADS["medium"]
    rng = np.random.default_rng(2)
    toks = np.unique(np.concatenate([rng.integers(0, wl.n_tokens, 48), np.arange(5), [wl.n_tokens - 1]]))
    stats = run_case(wl, sample=toks)
    assert stats["merged_exactly_rounded"] > 0.99 and stats["peaky_needed"] == 0


SWEEP = [(ratio, blk) for blk in ((2, 4, 4), (4, 4, 4), (2, 8, 8)) for ratio in (0.5, 0.7, 0.9)]


@pytest.mark.parametrize("ratio,blk", SWEEP, ids=[f"{b[0]}x{b[1]}x{b[2]}-{r}" for r, b in SWEEP])
def test_medium_sweep_full_size_sampled(ratio, blk):
    """Every point of the medium scene's sweep (merge ratio 0.5 / 0.7 / 0.9, blocks 2x4x4 / 4x4x4 / 2x8x8) at full size:
    permutation, maps, ranks and merged tensors on all tokens, attention on sampled tokens, plain 2e-2 x RMS bound."""
    wl = synth.WORKLOADS["medium"].replace(name=f"medium-{blk}-{ratio}", blk_frames=blk[0], blk_h=blk[1], blk_w=blk[2],
                                           ratio_q=ratio, ratio_kv=ratio)
    rng = np.random.default_rng(20)
    toks = np.unique(np.concatenate([rng.integers(0, wl.n_tokens, 24), np.arange(5), [wl.n_tokens - 1]]))
    stats = run_case(wl, sample=toks)
    assert stats["merged_exactly_rounded"] > 0.99 and stats["peaky_needed"] == 0


def test_stack_layer_full_size_sampled():
    """One layer of the 24-layer configuration at full size (S = 48, 65 952 tokens, 2x4x4 blocks, ratio 0.7)."""
    wl = synth.WORKLOADS["stack_layer"]
    rng = np.random.default_rng(21)
    toks = np.unique(np.concatenate([rng.integers(0, wl.n_tokens, 16), np.arange(5), [wl.n_tokens - 1]]))
    stats = run_case(wl, sample=toks)
    assert stats["merged_exactly_rounded"] > 0.99 and stats["peaky_needed"] == 0


def test_dense_attention_medium_config_sampled():
    """The dense in-run reference at the benchmark's size, on sampled tokens."""
    wl = synth.WORKLOADS["medium"]
    q, k, v = synth.make_qkv(wl)
    g = orc.Geometry.of(wl)
    rng = np.random.default_rng(3)
    toks = np.unique(np.concatenate([rng.integers(0, wl.n_tokens, 24), [0, 4, 5, wl.n_tokens - 1, 32768, 32767]]))
    ref = orc.dense_attention(g, q, k, v, toks)
    with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
        out = ctx.dense_attention(*(hb.bf16_from_bits(x, DEV) for x in (q, k, v)))
        torch.cuda.synchronize()
        assert ctx.query(hb.Q_DEVICE_STATUS) == 0
        bits = hb.bits_from_bf16(out)
        assert np.isfinite(parity.bits_to_f64(bits)).all()
        parity.check_output(bits[toks], ref, what="dense medium")


def test_direct_block_loads_equal_the_reordered_copies():
    """Match and merge reading their blocks straight from Q/K/V (what the public call does) against the same kernels reading the reorder kernel's copies: identical maps and
    ranks; merged values identical where no block is clipped, within one bf16 step elsewhere (the order
    in which a clipped block's tokens enter the fp32 sums differs)."""
    for wl in (synth.WORKLOADS["tiny"].replace(heads=3),
               synth.Workload("clipped", 5, 9, 10, 2, 4, 4, 0.6, 0.7, heads=3, seed=7),
               synth.Workload("clipped", 9, 10, 11, 4, 4, 4, 0.5, 0.8, heads=2, seed=8),     # 64-token blocks
               synth.Workload("clipped", 5, 17, 19, 2, 8, 8, 0.7, 0.9, heads=2, seed=9),     # 128
               synth.Workload("clipped", 5, 9, 11, 4, 8, 8, 0.8, 0.3, heads=1, seed=10)):    # 256
        q, k, v = synth.make_qkv(wl)
        with hb.Httm(hb.HttmConfig.of(wl)) as ctx:
            dq, dk, dv = (hb.bf16_from_bits(x, DEV) for x in (q, k, v))
            names = {"assign_q": hb.X_ASSIGN_Q, "assign_k": hb.X_ASSIGN_K, "rank_q": hb.X_RANK_Q,
                     "q_m": hb.X_Q_MERGED, "k_m": hb.X_K_MERGED, "v_m": hb.X_V_MERGED}
            for st in (hb.STAGE_REORDER, hb.STAGE_MATCH, hb.STAGE_MERGE):
                ctx.launch_stage(st, dq, dk, dv)
            sep = {n: ctx.export(w).copy() for n, w in names.items()}
            # other inputs through the separate kernels: nothing of the first run is left in the buffers
            for st in (hb.STAGE_REORDER, hb.STAGE_MATCH, hb.STAGE_MERGE):
                ctx.launch_stage(st, dv, dq, dk)
            for st in (hb.STAGE_MATCH_DIRECT, hb.STAGE_MERGE_DIRECT):
                ctx.launch_stage(st, dq, dk, dv)
            direct = {n: ctx.export(w) for n, w in names.items()}
            for n in ("assign_q", "assign_k", "rank_q"):
                assert np.array_equal(sep[n], direct[n]), f"{wl.name}: {n} differs between the two ways of loading a block"
            for n in ("q_m", "k_m", "v_m"):
                a, b = parity.bits_to_f64(sep[n]), parity.bits_to_f64(direct[n])
                if wl.name != "clipped":
                    assert np.array_equal(sep[n], direct[n]), f"{wl.name}: {n} differs"
                else:
                    assert (np.abs(a - b) <= 2.0 ** -7 * np.abs(a) + 1e-30).all(), f"{wl.name}: {n} differs by more than a bf16 step"


def test_large_config_full_size_sampled():
    """S=100 frames (137k tokens), 64-token blocks, weaker redundancy: the kernels for blocks of more than 32 tokens at
    full size - maps, ranks and merged tensors in full, attention on sampled tokens."""
    wl = synth.WORKLOADS["large"]
    rng = np.random.default_rng(4)
    toks = np.unique(np.concatenate([rng.integers(0, wl.n_tokens, 16), np.arange(5), [wl.n_tokens - 1]]))
    stats = run_case(wl, sample=toks)
    assert stats["merged_exactly_rounded"] > 0.99 and stats["peaky_needed"] == 0
