"""ctypes front end of the CPU oracle (oracle/httm_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg, never by the CUDA library or its Python binding.
It shares no code with them and imports nothing from the package.

The functions mirror the steps of Algorithm 1 of the paper in its order:
temporal_reorder -> reorder -> match -> merged_rank/merge -> attention -> unmerge.
All floating point is double; inputs are bf16 bit patterns (numpy uint16),
layout [heads][tokens][head_dim].
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "httm_oracle.c")
_LIB = os.path.join(_HERE, "libhttm_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2 -fopenmp) if the library is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Geom(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "frames", "n_special", "grid_h", "grid_w", "heads", "head_dim", "blk_frames", "blk_h", "blk_w")]


@dataclass(frozen=True)
class Geometry:
    frames: int
    n_special: int
    grid_h: int
    grid_w: int
    heads: int
    head_dim: int
    blk_frames: int
    blk_h: int
    blk_w: int

    @staticmethod
    def of(obj) -> "Geometry":
        """Build from any object with the same attribute names (e.g. a workload record)."""
        return Geometry(*(int(getattr(obj, f)) for f in (
            "frames", "n_special", "grid_h", "grid_w", "heads", "head_dim", "blk_frames", "blk_h", "blk_w")))

    def _c(self) -> _Geom:
        return _Geom(self.frames, self.n_special, self.grid_h, self.grid_w, self.heads, self.head_dim,
                     self.blk_frames, self.blk_h, self.blk_w)


def _load():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        p = ctypes.c_void_p
        i64, f64 = ctypes.c_int64, ctypes.c_double
        G = ctypes.POINTER(_Geom)
        L.oracle_threads.restype = ctypes.c_int
        L.oracle_num_tokens.restype = i64
        L.oracle_num_tokens.argtypes = [G]
        L.oracle_num_blocks.restype = i64
        L.oracle_num_blocks.argtypes = [G]
        L.oracle_temporal_reorder.argtypes = [G, p, p]
        L.oracle_reorder.argtypes = [G, p, p, p]
        L.oracle_block_budget.argtypes = [i64, f64, ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.oracle_is_dst.restype = ctypes.c_int
        L.oracle_is_dst.argtypes = [i64, i64, i64]
        L.oracle_merged_len.restype = i64
        L.oracle_merged_len.argtypes = [G, f64]
        L.oracle_match.argtypes = [G, p, f64, p, p, p, p]
        L.oracle_merged_rank.restype = i64
        L.oracle_merged_rank.argtypes = [G, p, p]
        L.oracle_merge.argtypes = [G, p, i64, p, p]
        L.oracle_attention.argtypes = [i64, i64, i64, i64, p, p, p, p, i64, p]
        L.oracle_unmerge.argtypes = [G, p, p, i64, p, p]
        L.oracle_bf16_to_double.argtypes = [p, i64, p]
        for f in ("oracle_temporal_reorder", "oracle_reorder", "oracle_block_budget", "oracle_match",
                  "oracle_merge", "oracle_attention", "oracle_unmerge", "oracle_bf16_to_double"):
            getattr(L, f).restype = None
        _lib = L
    return _lib


def _ptr(a: np.ndarray):
    assert a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.c_void_p)


def threads() -> int:
    return int(_load().oracle_threads())


def num_tokens(g: Geometry) -> int:
    return int(_load().oracle_num_tokens(ctypes.byref(g._c())))


def num_blocks(g: Geometry) -> int:
    return int(_load().oracle_num_blocks(ctypes.byref(g._c())))


def temporal_reorder(g: Geometry):
    """(pi, blk_start): pi[p'] = original index at reordered position p'; blk_start has nb+1 entries."""
    N, nb = num_tokens(g), num_blocks(g)
    pi = np.empty(N, dtype=np.int64)
    bs = np.empty(nb + 1, dtype=np.int64)
    _load().oracle_temporal_reorder(ctypes.byref(g._c()), _ptr(pi), _ptr(bs))
    return pi, bs


def reorder(g: Geometry, pi: np.ndarray, x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.uint16)
    out = np.empty_like(x)
    _load().oracle_reorder(ctypes.byref(g._c()), _ptr(pi), _ptr(x), _ptr(out))
    return out


def block_budget(n: int, rho: float):
    r, nd = ctypes.c_int64(), ctypes.c_int64()
    _load().oracle_block_budget(n, float(rho), ctypes.byref(r), ctypes.byref(nd))
    return int(r.value), int(nd.value)


def is_dst(j: int, n: int, n_dst: int) -> bool:
    return bool(_load().oracle_is_dst(j, n, n_dst))


def merged_len(g: Geometry, rho: float) -> int:
    return int(_load().oracle_merged_len(ctypes.byref(g._c()), float(rho)))


def match(g: Geometry, blk_start: np.ndarray, rho: float, xr: np.ndarray, margins: bool = True):
    """Assignment map [H][N] (reordered positions) and, optionally, the two margin arrays."""
    N, nb = num_tokens(g), num_blocks(g)
    xr = np.ascontiguousarray(xr, dtype=np.uint16)
    assert xr.shape == (g.heads, N, g.head_dim)
    A = np.empty((g.heads, N), dtype=np.int64)
    mb = np.empty((g.heads, N), dtype=np.float64) if margins else None
    ms = np.empty((g.heads, nb), dtype=np.float64) if margins else None
    _load().oracle_match(ctypes.byref(g._c()), _ptr(blk_start), float(rho), _ptr(xr), _ptr(A),
                         _ptr(mb) if margins else None, _ptr(ms) if margins else None)
    return (A, mb, ms) if margins else A


def merged_rank(g: Geometry, assign: np.ndarray):
    """(rank [H][N], M): merged row index of every reordered token, and the merged length."""
    assign = np.ascontiguousarray(assign, dtype=np.int64)
    R = np.empty_like(assign)
    M = int(_load().oracle_merged_rank(ctypes.byref(g._c()), _ptr(assign), _ptr(R)))
    if M < 0:
        raise ValueError("heads disagree on the number of kept tokens")
    return R, M


def merge(g: Geometry, rank: np.ndarray, M: int, xr: np.ndarray) -> np.ndarray:
    xr = np.ascontiguousarray(xr, dtype=np.uint16)
    rank = np.ascontiguousarray(rank, dtype=np.int64)
    out = np.empty((g.heads, M, g.head_dim), dtype=np.float64)
    _load().oracle_merge(ctypes.byref(g._c()), _ptr(rank), M, _ptr(xr), _ptr(out))
    return out


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, rows=None) -> np.ndarray:
    """softmax(q k^T / sqrt(D)) v per head; q [H][Mq][D], k/v [H][Mk][D] float64.
    rows: optional list of query rows (same for every head) -> out [H][len(rows)][D]."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    k = np.ascontiguousarray(k, dtype=np.float64)
    v = np.ascontiguousarray(v, dtype=np.float64)
    H, Mq, D = q.shape
    Mk = k.shape[1]
    assert k.shape == (H, Mk, D) and v.shape == (H, Mk, D)
    if rows is None:
        rp, nr = None, Mq
    else:
        rows = np.ascontiguousarray(rows, dtype=np.int64)
        assert rows.ndim == 1 and (rows.size == 0 or (rows.min() >= 0 and rows.max() < Mq))
        rp, nr = _ptr(rows), rows.size
    out = np.empty((H, nr, D), dtype=np.float64)
    if nr:
        _load().oracle_attention(H, Mq, Mk, D, _ptr(q), _ptr(k), _ptr(v), rp, nr, _ptr(out))
    return out


def unmerge(g: Geometry, pi: np.ndarray, rank_q: np.ndarray, om: np.ndarray) -> np.ndarray:
    om = np.ascontiguousarray(om, dtype=np.float64)
    rank_q = np.ascontiguousarray(rank_q, dtype=np.int64)
    N = num_tokens(g)
    out = np.empty((N, g.heads * g.head_dim), dtype=np.float64)
    _load().oracle_unmerge(ctypes.byref(g._c()), _ptr(pi), _ptr(rank_q), om.shape[1], _ptr(om), _ptr(out))
    return out


def bf16_to_double(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.uint16)
    out = np.empty(x.shape, dtype=np.float64)
    _load().oracle_bf16_to_double(_ptr(x), x.size, _ptr(out))
    return out


# --------------------------------------------------------------------------- pipelines


@dataclass
class Result:
    pi: np.ndarray          # [N]   reordered position -> original index
    blk_start: np.ndarray   # [nb+1]
    assign_q: np.ndarray    # [H][N] reordered positions
    assign_k: np.ndarray
    margin_best_q: np.ndarray | None
    margin_sel_q: np.ndarray | None
    margin_best_k: np.ndarray | None
    margin_sel_k: np.ndarray | None
    rank_q: np.ndarray      # [H][N] merged row of each reordered token
    rank_k: np.ndarray
    M_q: int
    M_k: int
    q_m: np.ndarray         # [H][M_q][D] float64
    k_m: np.ndarray
    v_m: np.ndarray
    o_m: np.ndarray | None  # [H][M_q][D]
    out: np.ndarray | None  # [N][H*D]


def merged_attention_from_maps(g: Geometry, pi, q, k, v, assign_q, assign_k, attend: bool = True) -> Result:
    """Steps 'merge -> attention -> unmerge -> inverse reorder' for GIVEN assignment
    maps (used when a map under test differs from the oracle's only inside the
    allowed similarity margin)."""
    qr, kr, vr = reorder(g, pi, q), reorder(g, pi, k), reorder(g, pi, v)
    rq, Mq = merged_rank(g, assign_q)
    rk, Mk = merged_rank(g, assign_k)
    qm, km, vm = merge(g, rq, Mq, qr), merge(g, rk, Mk, kr), merge(g, rk, Mk, vr)
    om = out = None
    if attend:
        om = attention(qm, km, vm)
        out = unmerge(g, pi, rq, om)
    return Result(pi, None, assign_q, assign_k, None, None, None, None, rq, rk, Mq, Mk, qm, km, vm, om, out)


def global_attention(g: Geometry, ratio_q: float, ratio_kv: float, q, k, v, attend: bool = True) -> Result:
    """Algorithm 1 without outlier filtering and without the projections:
    reorder, match Q and K per head and block, merge Q / K / V (V follows K),
    attention on the merged sets, head-wise unmerge, inverse reorder."""
    pi, bs = temporal_reorder(g)
    qr, kr, vr = reorder(g, pi, q), reorder(g, pi, k), reorder(g, pi, v)
    aq, mbq, msq = match(g, bs, ratio_q, qr)
    ak, mbk, msk = match(g, bs, ratio_kv, kr)
    rq, Mq = merged_rank(g, aq)
    rk, Mk = merged_rank(g, ak)
    qm, km, vm = merge(g, rq, Mq, qr), merge(g, rk, Mk, kr), merge(g, rk, Mk, vr)
    om = out = None
    if attend:
        om = attention(qm, km, vm)
        out = unmerge(g, pi, rq, om)
    return Result(pi, bs, aq, ak, mbq, msq, mbk, msk, rq, rk, Mq, Mk, qm, km, vm, om, out)


def attention_rows_for_tokens(g: Geometry, res: Result, tokens: np.ndarray) -> np.ndarray:
    """Final output rows [len(tokens)][H*D] for the given ORIGINAL token indices,
    computing only the merged query rows those tokens need."""
    tokens = np.asarray(tokens, dtype=np.int64)
    N = num_tokens(g)
    inv = np.empty(N, dtype=np.int64)
    inv[res.pi] = np.arange(N)
    out = np.empty((tokens.size, g.heads * g.head_dim), dtype=np.float64)
    for hd in range(g.heads):
        rows = res.rank_q[hd, inv[tokens]]
        uniq, back = np.unique(rows, return_inverse=True)
        o = attention(res.q_m[hd:hd + 1], res.k_m[hd:hd + 1], res.v_m[hd:hd + 1], uniq)[0]
        out[:, hd * g.head_dim:(hd + 1) * g.head_dim] = o[back]
    return out


def dense_attention(g: Geometry, q, k, v, tokens=None) -> np.ndarray:
    """Exact multi-head attention over all N tokens; out [N][H*D] (or the listed tokens' rows)."""
    qd, kd, vd = bf16_to_double(q), bf16_to_double(k), bf16_to_double(v)
    o = attention(qd, kd, vd, tokens)  # [H][n][D]
    return np.ascontiguousarray(o.transpose(1, 0, 2)).reshape(o.shape[1], g.heads * g.head_dim)
