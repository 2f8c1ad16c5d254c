"""Thin ctypes binding of libhttm.so (the C ABI declared in include/httm.h).

Argument marshalling only: every step of the path runs in the library's CUDA kernels.
torch is used for device memory and streams.  There is no CPU fallback: if the shared
library is missing or fails to load, importing a symbol from it raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhttm.so")

# selectors (mirror include/httm.h)
(Q_TOKENS, Q_MERGED_Q, Q_MERGED_K, Q_BLOCKS, Q_WORKSPACE_BYTES, Q_MAX_BLOCK_TOKENS, Q_DEVICE_STATUS, Q_MERGED_Q_ROWS,
 Q_OUTLIERS) = range(9)
(X_PI, X_PI_INV, X_BLOCK_START, X_ASSIGN_Q, X_ASSIGN_K, X_RANK_Q, X_Q_REORDERED, X_K_REORDERED, X_V_REORDERED,
 X_Q_MERGED, X_K_MERGED, X_V_MERGED, X_O_MERGED, X_DEVIATION, X_THRESHOLD, X_MERGED_Q_HEAD, X_ASSIGN_Q_INITIAL) = range(17)
(STAGE_REORDER, STAGE_MATCH, STAGE_MERGE, STAGE_ATTENTION, STAGE_UNMERGE, STAGE_MATCH_DIRECT, STAGE_MERGE_DIRECT,
 STAGE_OUTLIER_FILTER, STAGE_BIG_SCORES, STAGE_BIG_SELECT, STAGE_ATTENTION_UNMERGE) = range(11)
STAGE_NAMES = ("reorder", "match", "merge", "attention", "unmerge", "match_direct", "merge_direct", "outlier_filter",
               "big_scores", "big_select", "attention_unmerge")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_NOMEM, ERR_CUDA, ERR_TIMEOUT = 0, -1, -2, -3, -4, -5, -6
_STATUS_NAMES = {0: "HTTM_OK", -1: "HTTM_ERR_INVALID_ARG", -2: "HTTM_ERR_UNSUPPORTED", -3: "HTTM_ERR_ALIGNMENT",
                 -4: "HTTM_ERR_NOMEM", -5: "HTTM_ERR_CUDA", -6: "HTTM_ERR_TIMEOUT"}

EXPORTED_SYMBOLS = (
    "httm_create", "httm_global_attention", "httm_dense_attention", "httm_attention_host", "httm_launch_stage",
    "httm_query", "httm_export", "httm_last_error", "httm_launch_count", "httm_destroy",
    "httm_global_attention_static", "httm_selftest_tensor_core", "httm_set_outlier_fraction", "httm_linear",
    "httm_set_head_shard", "httm_fail_nth_allocation", "httm_expire_a_wait", "httm_set_call_timing", "httm_call_times",
)
_EXCHANGE_FN = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p)


class HttmError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"{_STATUS_NAMES.get(code, code)}: {message}")
        self.code = code


class _Config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("frames", "n_camera", "n_register", "grid_h", "grid_w", "heads", "head_dim",
                                               "blk_frames", "blk_h", "blk_w")] + [
        ("ratio_q", ctypes.c_double), ("ratio_kv", ctypes.c_double), ("device", ctypes.c_int32), ("anchor_first_frame", ctypes.c_int32)]


class _Tensor(ctypes.Structure):
    _fields_ = [("ptr", ctypes.c_void_p), ("stride_head", ctypes.c_int64), ("stride_token", ctypes.c_int64)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Load libhttm.so and declare the prototypes.  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2511_21317_b200.build` "
                          "(there is no CPU fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i64 = ctypes.c_void_p, ctypes.c_int64
    L.httm_create.argtypes = [ctypes.POINTER(_Config), ctypes.POINTER(vp)]
    L.httm_global_attention.argtypes = [vp, _Tensor, _Tensor, _Tensor, _Tensor, vp]
    L.httm_dense_attention.argtypes = [vp, _Tensor, _Tensor, _Tensor, _Tensor, vp]
    L.httm_set_outlier_fraction.argtypes = [vp, ctypes.c_double]
    L.httm_set_head_shard.argtypes = [vp, ctypes.c_int32, _EXCHANGE_FN, vp]
    L.httm_fail_nth_allocation.argtypes = [ctypes.c_int32]
    L.httm_expire_a_wait.argtypes = [vp, vp]
    L.httm_linear.argtypes = [vp, vp, i64, vp, i64, vp, i64, i64, ctypes.c_int32, ctypes.c_int32, vp]
    L.httm_attention_host.argtypes = [vp, vp, vp, vp, vp, ctypes.c_int, vp]
    L.httm_launch_stage.argtypes = [vp, ctypes.c_int, _Tensor, _Tensor, _Tensor, _Tensor, vp]
    L.httm_query.argtypes = [vp, ctypes.c_int, ctypes.POINTER(i64)]
    L.httm_export.argtypes = [vp, ctypes.c_int, vp, ctypes.c_size_t, vp]
    L.httm_last_error.argtypes = [vp]
    L.httm_last_error.restype = ctypes.c_char_p
    L.httm_launch_count.argtypes = [vp]
    L.httm_launch_count.restype = i64
    L.httm_destroy.argtypes = [vp]
    L.httm_global_attention_static.argtypes = [ctypes.POINTER(_Config), _Tensor, _Tensor, _Tensor, _Tensor, vp]
    L.httm_selftest_tensor_core.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    for name in EXPORTED_SYMBOLS:
        if name not in ("httm_last_error", "httm_launch_count"):
            getattr(L, name).restype = ctypes.c_int
    _lib = L
    return L


@dataclass(frozen=True)
class HttmConfig:
    frames: int
    grid_h: int
    grid_w: int
    blk_frames: int
    blk_h: int
    blk_w: int
    ratio_q: float
    ratio_kv: float
    n_camera: int = 1
    n_register: int = 4
    heads: int = 16
    head_dim: int = 64
    device: int = 0
    anchor_first_frame: int = 0   # 1: the tokens of frame 0 are the dst tokens of their blocks (first-frame anchoring)

    @staticmethod
    def of(obj, device: int = 0) -> "HttmConfig":
        """Build from any record with the same attribute names (e.g. a synthetic workload)."""
        names = ("frames", "grid_h", "grid_w", "blk_frames", "blk_h", "blk_w", "ratio_q", "ratio_kv", "n_camera",
                 "n_register", "heads", "head_dim")
        return HttmConfig(**{n: getattr(obj, n) for n in names}, device=device,
                          anchor_first_frame=int(getattr(obj, "anchor_first_frame", 0)))


def _null_tensor() -> _Tensor:
    return _Tensor(None, 0, 0)


class Httm:
    """One context of the library: a geometry, its plan and its device workspace."""

    def __init__(self, cfg: HttmConfig):
        self._lib = load_library()
        self.cfg = cfg
        c = _Config(cfg.frames, cfg.n_camera, cfg.n_register, cfg.grid_h, cfg.grid_w, cfg.heads, cfg.head_dim,
                    cfg.blk_frames, cfg.blk_h, cfg.blk_w, float(cfg.ratio_q), float(cfg.ratio_kv), cfg.device,
                    int(cfg.anchor_first_frame))
        h = ctypes.c_void_p()
        rc = self._lib.httm_create(ctypes.byref(c), ctypes.byref(h))
        if rc != OK:
            raise HttmError(rc, (self._lib.httm_last_error(None) or b"").decode())
        self._h = h
        self.n_tokens = self.query(Q_TOKENS)
        self.m_q = self.query(Q_MERGED_Q)
        self.m_k = self.query(Q_MERGED_K)
        self.n_blocks = self.query(Q_BLOCKS)

    # ---- lifetime
    def close(self):
        if getattr(self, "_h", None):
            self._lib.httm_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    # ---- helpers
    def _check(self, rc: int):
        if rc != OK:
            raise HttmError(rc, (self._lib.httm_last_error(self._h) or b"").decode())

    def _stream(self, stream):
        if stream is None:
            stream = torch.cuda.current_stream(self.cfg.device)
        return ctypes.c_void_p(stream.cuda_stream)

    def _tensor(self, t: torch.Tensor, name: str, out_layout: bool = False) -> _Tensor:
        H, N, D = self.cfg.heads, self.n_tokens, self.cfg.head_dim
        if t.dtype != torch.bfloat16 or not t.is_cuda:
            raise HttmError(ERR_INVALID_ARG, f"{name}: expected a CUDA bfloat16 tensor")
        if out_layout:  # [N][H*D] or [N][H][D]
            t = t.view(N, H, D)
            if t.stride(2) != 1:
                raise HttmError(ERR_INVALID_ARG, f"{name}: channels must be contiguous")
            return _Tensor(t.data_ptr(), t.stride(1), t.stride(0))
        if tuple(t.shape) != (H, N, D) or t.stride(2) != 1:
            raise HttmError(ERR_INVALID_ARG, f"{name}: expected shape [heads][tokens][head_dim] with contiguous channels")
        return _Tensor(t.data_ptr(), t.stride(0), t.stride(1))

    def new_output(self) -> torch.Tensor:
        return torch.empty(self.n_tokens, self.cfg.heads * self.cfg.head_dim, dtype=torch.bfloat16,
                           device=f"cuda:{self.cfg.device}")

    # ---- the calls of the ABI
    def global_attention(self, q, k, v, out=None, stream=None) -> torch.Tensor:
        out = self.new_output() if out is None else out
        self._check(self._lib.httm_global_attention(self._h, self._tensor(q, "q"), self._tensor(k, "k"),
                                                    self._tensor(v, "v"), self._tensor(out, "out", True),
                                                    self._stream(stream)))
        return out

    def dense_attention(self, q, k, v, out=None, stream=None) -> torch.Tensor:
        out = self.new_output() if out is None else out
        self._check(self._lib.httm_dense_attention(self._h, self._tensor(q, "q"), self._tensor(k, "k"),
                                                   self._tensor(v, "v"), self._tensor(out, "out", True),
                                                   self._stream(stream)))
        return out

    def attention_host(self, q, k, v, out, dense: bool = False, stream=None):
        """q, k, v, out: CPU bf16 tensors (pinned for asynchronous copies), contiguous."""
        for t, name in ((q, "q"), (k, "k"), (v, "v"), (out, "out")):
            if t.is_cuda or t.dtype != torch.bfloat16 or not t.is_contiguous():
                raise HttmError(ERR_INVALID_ARG, f"{name}: expected a contiguous CPU bfloat16 tensor")
        if q.numel() != out.numel() or k.numel() != q.numel() or v.numel() != q.numel() or \
                q.numel() != self.cfg.heads * self.n_tokens * self.cfg.head_dim:
            raise HttmError(ERR_INVALID_ARG, "host tensors have the wrong number of elements")
        self._check(self._lib.httm_attention_host(self._h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                                  int(dense), self._stream(stream)))
        return out

    def set_outlier_fraction(self, fraction: float):
        """Query outlier filtering (Sec. 3.4) for the later calls; 0 switches it off."""
        self._check(self._lib.httm_set_outlier_fraction(self._h, float(fraction)))

    def set_call_timing(self, enable: bool):
        """Events between the kernels of global_attention (see httm_set_call_timing)."""
        self._check(self._lib.httm_set_call_timing(self._h, 1 if enable else 0))

    def call_times(self):
        """[(part name, milliseconds)] of the last global_attention call, in launch order (waits for the call to finish)."""
        cap = 16
        ms = (ctypes.c_float * cap)()
        names = (ctypes.c_char_p * cap)()
        n = ctypes.c_int32(0)
        self._check(self._lib.httm_call_times(self._h, ms, names, cap, ctypes.byref(n)))
        return [(names[i].decode(), float(ms[i])) for i in range(min(n.value, cap))]

    def expire_a_wait(self, stream=None):
        """Error-path test aid: a kernel whose bounded wait runs out (see httm_expire_a_wait)."""
        self._check(self._lib.httm_expire_a_wait(self._h, self._stream(stream)))

    def set_head_shard(self, total_heads: int, exchange=None):
        """This context holds some of the heads of a layer with `total_heads` heads (see httm_set_head_shard).
        exchange(counts) gets a CUDA int32 tensor that aliases the library's histogram and must sum it in place over all
        shards on the current stream (e.g. torch.distributed.all_reduce); None with total_heads = 0 switches sharding off."""
        if exchange is None:
            cb = ctypes.cast(None, _EXCHANGE_FN)
        else:
            device = f"cuda:{self.cfg.device}"

            def trampoline(_user, ptr, n, _stream):
                try:
                    exchange(device_int32_view(int(ptr), int(n), device))
                    return 0
                except Exception:   # the C side turns this into HTTM_ERR_CUDA; keep the reason
                    import traceback
                    traceback.print_exc()
                    return 1
            cb = _EXCHANGE_FN(trampoline)
        self._check(self._lib.httm_set_head_shard(self._h, int(total_heads), cb, None))
        self._exchange_cb = cb   # the library keeps the pointer: keep the object alive

    def linear(self, x: torch.Tensor, w: torch.Tensor, out: torch.Tensor = None, stream=None) -> torch.Tensor:
        """y = x . w^T with x [n][in], w [out][in] (rows may be strided), bf16 CUDA tensors; returns y [n][out]."""
        for t, name in ((x, "x"), (w, "w")):
            if t.dtype != torch.bfloat16 or not t.is_cuda or t.dim() != 2 or t.stride(1) != 1:
                raise HttmError(ERR_INVALID_ARG, f"{name}: expected a CUDA bfloat16 matrix with contiguous rows")
        if w.shape[1] != x.shape[1]:
            raise HttmError(ERR_INVALID_ARG, "w: expected [out_features][in_features]")
        if out is None:
            out = torch.empty(x.shape[0], w.shape[0], dtype=torch.bfloat16, device=x.device)
        elif out.dtype != torch.bfloat16 or not out.is_cuda or out.shape != (x.shape[0], w.shape[0]) or out.stride(1) != 1:
            raise HttmError(ERR_INVALID_ARG, "out: expected a CUDA bfloat16 matrix [n][out_features] with contiguous rows")
        self._check(self._lib.httm_linear(self._h, x.data_ptr(), x.stride(0), w.data_ptr(), w.stride(0), out.data_ptr(), out.stride(0),
                                          x.shape[0], x.shape[1], w.shape[0], self._stream(stream)))
        return out

    def launch_stage(self, stage: int, q=None, k=None, v=None, out=None, stream=None):
        tq = self._tensor(q, "q") if q is not None else _null_tensor()
        tk = self._tensor(k, "k") if k is not None else _null_tensor()
        tv = self._tensor(v, "v") if v is not None else _null_tensor()
        to = self._tensor(out, "out", True) if out is not None else _null_tensor()
        self._check(self._lib.httm_launch_stage(self._h, stage, tq, tk, tv, to, self._stream(stream)))

    def query(self, what: int) -> int:
        v = ctypes.c_int64()
        self._check(self._lib.httm_query(self._h, what, ctypes.byref(v)))
        return int(v.value)

    def launch_count(self) -> int:
        return int(self._lib.httm_launch_count(self._h))

    def export(self, what: int, stream=None) -> np.ndarray:
        """Intermediate of the last call as a numpy array (int32 indices or uint16 bf16 bits)."""
        H, N, D = self.cfg.heads, self.n_tokens, self.cfg.head_dim
        q_rows = self.query(Q_MERGED_Q_ROWS)
        shapes = {
            X_PI: ((N,), np.int32), X_PI_INV: ((N,), np.int32), X_BLOCK_START: ((self.n_blocks + 1,), np.int32),
            X_ASSIGN_Q: ((H, N), np.int32), X_ASSIGN_K: ((H, N), np.int32), X_RANK_Q: ((H, N), np.int32),
            X_Q_REORDERED: ((H, N, D), np.uint16), X_K_REORDERED: ((H, N, D), np.uint16),
            X_V_REORDERED: ((H, N, D), np.uint16), X_Q_MERGED: ((H, q_rows, D), np.uint16),
            X_K_MERGED: ((H, self.m_k, D), np.uint16), X_V_MERGED: ((H, self.m_k, D), np.uint16),
            X_O_MERGED: ((H, q_rows, D), np.uint16), X_DEVIATION: ((H, N), np.float32), X_THRESHOLD: ((1,), np.float32),
            X_MERGED_Q_HEAD: ((H,), np.int32), X_ASSIGN_Q_INITIAL: ((H, N), np.int32),
        }
        shape, dt = shapes[what]
        arr = np.empty(shape, dtype=dt)
        self._check(self._lib.httm_export(self._h, what, arr.ctypes.data_as(ctypes.c_void_p), arr.nbytes,
                                          self._stream(stream)))
        return arr


class _DeviceInt32:
    def __init__(self, ptr: int, n: int):
        self.__cuda_array_interface__ = {"shape": (n,), "typestr": "<i4", "data": (ptr, False), "version": 2}


def device_int32_view(ptr: int, n: int, device) -> torch.Tensor:
    """A CUDA int32 tensor over n counters at a raw device address (no copy)."""
    return torch.as_tensor(_DeviceInt32(ptr, n), device=device)


def fail_nth_allocation(n: int):
    """Error-path test aid: the n-th device allocation of the library from now on fails (0: off)."""
    load_library().httm_fail_nth_allocation(int(n))


def selftest_tensor_core(q, k, v):
    """One 128 x 64 tile: returns (Q K^T [128][128], bf16(Q K^T) V [128][64]) as fp32 CUDA tensors."""
    lib = load_library()
    for t in (q, k, v):
        if not t.is_cuda or t.dtype != torch.bfloat16 or tuple(t.shape) != (128, 64) or not t.is_contiguous():
            raise HttmError(ERR_INVALID_ARG, "expected contiguous CUDA bfloat16 [128][64]")
    s = torch.zeros(128, 128, dtype=torch.float32, device=q.device)
    o = torch.zeros(128, 64, dtype=torch.float32, device=q.device)
    st = torch.zeros(1, dtype=torch.int32, device=q.device)
    rc = lib.httm_selftest_tensor_core(q.data_ptr(), k.data_ptr(), v.data_ptr(), s.data_ptr(), o.data_ptr(), st.data_ptr(),
                                       ctypes.c_void_p(torch.cuda.current_stream(q.device).cuda_stream))
    if rc != OK:
        raise HttmError(rc, "tensor-core self test could not be launched")
    torch.cuda.synchronize(q.device)
    if int(st.item()) != 0:
        raise HttmError(ERR_TIMEOUT, "tensor-core self test: a bounded wait gave up")
    return s, o


STATIC_SCRATCH_BYTES = 16 << 20


def global_attention_static(cfg: HttmConfig, q, k, v, out, stream=None):
    """HTTM global attention without any device allocation (see httm_global_attention_static in
    include/httm.h): q, k, v are CUDA bf16 [heads][tokens][64], out is CUDA bf16 [tokens][heads*64],
    all owned by the caller.  Only problems whose intermediates fit the library's built-in
    16 MiB scratch array are accepted."""
    lib = load_library()
    H, D = cfg.heads, cfg.head_dim
    N = cfg.frames * (cfg.n_camera + cfg.n_register + cfg.grid_h * cfg.grid_w)
    for t, name in ((q, "q"), (k, "k"), (v, "v")):
        if not t.is_cuda or t.dtype != torch.bfloat16 or tuple(t.shape) != (H, N, D) or t.stride(2) != 1:
            raise HttmError(ERR_INVALID_ARG, f"{name}: expected CUDA bfloat16 [heads][tokens][head_dim]")
    if not out.is_cuda or out.dtype != torch.bfloat16 or out.numel() != N * H * D:
        raise HttmError(ERR_INVALID_ARG, "out: expected CUDA bfloat16 [tokens][heads*head_dim]")
    o = out.view(N, H, D)
    c = _Config(cfg.frames, cfg.n_camera, cfg.n_register, cfg.grid_h, cfg.grid_w, H, D, cfg.blk_frames, cfg.blk_h,
                cfg.blk_w, float(cfg.ratio_q), float(cfg.ratio_kv), cfg.device, int(cfg.anchor_first_frame))
    if stream is None:
        stream = torch.cuda.current_stream(cfg.device)
    rc = lib.httm_global_attention_static(
        ctypes.byref(c), _Tensor(q.data_ptr(), q.stride(0), q.stride(1)), _Tensor(k.data_ptr(), k.stride(0), k.stride(1)),
        _Tensor(v.data_ptr(), v.stride(0), v.stride(1)), _Tensor(o.data_ptr(), o.stride(1), o.stride(0)),
        ctypes.c_void_p(stream.cuda_stream))
    if rc != OK:
        raise HttmError(rc, (lib.httm_last_error(None) or b"").decode())
    return out


def bf16_from_bits(bits: np.ndarray, device=None, pin: bool = False) -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 tensor (same bytes)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    if device is not None:
        return t.to(device)
    return t.pin_memory() if pin else t


def bits_from_bf16(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
