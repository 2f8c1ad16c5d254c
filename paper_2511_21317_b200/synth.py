"""Seeded synthetic Q/K/V for a VGGT-style global-attention layer.

This module holds NO arithmetic of the merging method: it only draws inputs.
It is the one module that both the CPU oracle's tests and the CUDA path's
tests / benchmark use, so that both sides see the same bytes.

Recipe (stand-in for real VGGT activations, which show spatial locality and
temporal correspondence, Sec. 3.1 of the paper):
  * per (tensor, head, channel) an 8x8 lattice of N(0,1) values is bilinearly
    upsampled, with periodic wrap, to the h x w patch grid;
  * frame s sees that field shifted by s patches along x (wrap);
  * every patch token adds sigma * N(0,1) noise;
  * the special tokens (camera + register) of every frame are N(0,1);
  * values are rounded to bf16 (round-to-nearest-even) and returned as uint16
    bit patterns in the layout [heads][tokens][head_dim], tokens frame-major,
    inside a frame: specials first, then patches row-major.

Random numbers are counter based (a 64-bit mix of seed, tensor, head and the
element counter), so any element is reproducible on its own.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_LATTICE = 8
_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)


@dataclasses.dataclass(frozen=True)
class Workload:
    """Geometry + merge parameters of one global-attention problem."""

    name: str
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
    sigma: float = 0.1
    seed: int = 0
    # Shape of the patch grid the synthetic field is drawn on, when it differs from (grid_h, grid_w): the 1-D block
    # regime hands the library a frame's patch tokens as one run (grid 1 x P) of a field_h x field_w image.
    field_h: int = 0
    field_w: int = 0

    @property
    def n_special(self) -> int:
        return self.n_camera + self.n_register

    @property
    def tokens_per_frame(self) -> int:
        return self.n_special + self.grid_h * self.grid_w

    @property
    def n_tokens(self) -> int:
        return self.frames * self.tokens_per_frame

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def _wl(name, frames, grid, blk, ratio, **kw) -> Workload:
    return Workload(name, frames, grid, grid, blk[0], blk[1], blk[2], ratio, ratio, **kw)


#: The five benchmark configurations (tiny / small / medium / large / stack layer).
WORKLOADS = {
    "tiny": _wl("tiny", 4, 16, (2, 4, 4), 0.5),
    "small": _wl("small", 8, 37, (2, 4, 4), 0.7),
    "medium": _wl("medium", 24, 37, (2, 4, 4), 0.7),
    "large": _wl("large", 100, 37, (4, 4, 4), 0.8, sigma=0.3),
    "stack_layer": _wl("stack_layer", 48, 37, (2, 4, 4), 0.7),
    # The paper's own block regime (Sec. 4.1): runs of n_s = 128 patch tokens in raster order over n_t = 30 frames
    # (blocks of 3840 tokens), 90 % of the queries and 70 % of the keys / values merged.
    "paper_1d": Workload("paper_1d", 60, 1, 37 * 37, 30, 1, 128, 0.9, 0.7, field_h=37, field_w=37),
}


def _mix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser, vectorised on uint64 (wrap-around arithmetic)."""
    with np.errstate(over="ignore"):
        x = (x + np.uint64(0x9E3779B97F4A7C15)) & _M64
        x = ((x ^ (x >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)) & _M64
        x = ((x ^ (x >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)) & _M64
        return x ^ (x >> np.uint64(31))


def _stream_key(seed: int, tensor: int, head: int, stream: int) -> np.uint64:
    k = np.array([(seed * 0x1000193 + 0x243F6A88) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64)
    for v in (tensor, head, stream):
        k = _mix64(k ^ np.uint64(v + 1))
    return k[0]


def _normals(key: np.uint64, counters: np.ndarray) -> np.ndarray:
    """One N(0,1) float64 per counter (Box-Muller on the two halves of one hash)."""
    with np.errstate(over="ignore"):
        h = _mix64(counters.astype(np.uint64) * np.uint64(0xD1342543DE82EF95) ^ key)
    u1 = ((h >> np.uint64(32)).astype(np.float64) + 0.5) * (1.0 / 4294967296.0)
    u2 = ((h & np.uint64(0xFFFFFFFF)).astype(np.float64) + 0.5) * (1.0 / 4294967296.0)
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _one_head(wl: Workload, tensor: int, head: int) -> np.ndarray:
    S, D, nsp = wl.frames, wl.head_dim, wl.n_special
    h, w = (wl.field_h, wl.field_w) if wl.field_h > 0 else (wl.grid_h, wl.grid_w)
    if h * w != wl.grid_h * wl.grid_w:
        raise ValueError("field_h x field_w must hold as many patches as grid_h x grid_w")
    P = wl.tokens_per_frame
    # lattice [D][8][8]
    lat = _normals(_stream_key(wl.seed, tensor, head, 0), np.arange(D * _LATTICE * _LATTICE)).reshape(
        D, _LATTICE, _LATTICE
    )
    # bilinear, periodic upsample to [D][h][w]
    v = np.arange(h, dtype=np.float64) * (_LATTICE / h)
    u = np.arange(w, dtype=np.float64) * (_LATTICE / w)
    y0 = np.floor(v).astype(np.int64)
    x0 = np.floor(u).astype(np.int64)
    fy = (v - y0)[None, :, None]
    fx = (u - x0)[None, None, :]
    y0 %= _LATTICE
    x0 %= _LATTICE
    y1 = (y0 + 1) % _LATTICE
    x1 = (x0 + 1) % _LATTICE
    field = (
        lat[:, y0][:, :, x0] * (1 - fy) * (1 - fx)
        + lat[:, y0][:, :, x1] * (1 - fy) * fx
        + lat[:, y1][:, :, x0] * fy * (1 - fx)
        + lat[:, y1][:, :, x1] * fy * fx
    )  # [D][h][w]
    out = np.empty((S, P, D), dtype=np.float32)
    key_noise = _stream_key(wl.seed, tensor, head, 1)
    xs = np.arange(w)
    for s in range(S):
        cnt = (np.arange(P * D, dtype=np.uint64) + np.uint64(s * P * D))
        nz = _normals(key_noise, cnt).reshape(P, D)
        out[s, :nsp, :] = nz[:nsp]
        shifted = field[:, :, (xs + s) % w]  # frame s sees the field moved by s patches along x
        out[s, nsp:, :] = (shifted.reshape(D, h * w).T + wl.sigma * nz[nsp:]).astype(np.float32)
    return f32_to_bf16_bits(out.reshape(S * P, D))


def make_qkv(wl: Workload, threads: int = 8):
    """Return (q, k, v): uint16 bf16 bit patterns, each [heads][tokens][head_dim]."""
    outs = [np.empty((wl.heads, wl.n_tokens, wl.head_dim), dtype=np.uint16) for _ in range(3)]

    def job(th):
        t, a = th
        outs[t][a] = _one_head(wl, t, a)

    jobs = [(t, a) for t in range(3) for a in range(wl.heads)]
    if threads > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(job, jobs))
    else:
        for j in jobs:
            job(j)
    return tuple(outs)


def make_identical_block_tokens(wl: Workload, seed: int = 0) -> np.ndarray:
    """One tensor [heads][tokens][head_dim] (bf16 bits) in which all patch tokens of
    one spatio-temporal block carry the same vector (a different one per block and
    head); special tokens are N(0,1). Used by property tests."""
    S, h, w, D, nsp, P = wl.frames, wl.grid_h, wl.grid_w, wl.head_dim, wl.n_special, wl.tokens_per_frame
    gb = -(-S // wl.blk_frames)
    hb = -(-h // wl.blk_h)
    wb = -(-w // wl.blk_w)
    out = np.empty((wl.heads, S, P, D), dtype=np.float32)
    for a in range(wl.heads):
        key = _stream_key(seed, 7, a, 2)
        vec = _normals(key, np.arange(gb * hb * wb * D)).reshape(gb, hb, wb, D)
        sp = _normals(_stream_key(seed, 7, a, 3), np.arange(S * max(nsp, 1) * D)).reshape(S, max(nsp, 1), D)
        out[a, :, :nsp, :] = sp[:, :nsp]
        g = np.arange(S) // wl.blk_frames
        by = np.arange(h) // wl.blk_h
        bx = np.arange(w) // wl.blk_w
        out[a, :, nsp:, :] = vec[g][:, by][:, :, bx].reshape(S, h * w, D)
    return f32_to_bf16_bits(out.reshape(wl.heads, S * P, D))
