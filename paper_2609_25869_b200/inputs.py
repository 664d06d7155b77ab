"""Seeded synthetic inputs for dynamic block-sparse attention requests.

This module only *generates* inputs (bf16 Q/K/V bit patterns and logical block
masks).  It holds none of the method's arithmetic: no attention, no softmax, no
tile planning, no mask statistics.  Both the CUDA path and the CPU oracle's
tests consume what it returns; neither depends on the other.

The masks stand in for the video-diffusion masks the paper evaluates on
(Section 7.1, Table 3): same token counts, block geometries, densities and
3-D locality, but drawn from an integer-only counter-based generator so they
are reproducible bit for bit on any machine.

Conventions: ``H`` heads, ``N`` tokens, ``d`` head dim, ``B = (B_Q, B_KV)``
logical block geometry, ``nQb = ceil(N / B_Q)``, ``nKb = ceil(N / B_KV)``,
mask ``M`` is ``uint8 [H, nQb, nKb]`` with 1 = active.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Tuple

import numpy as np

_U64 = np.uint64
_MASK64 = (1 << 64) - 1


def cdiv(a: int, b: int) -> int:
    return -(-a // b)


# --------------------------------------------------------------------------
# counter-based integer generator (splitmix64 finaliser over a mixed key)
# --------------------------------------------------------------------------
def _mix64(x: np.ndarray) -> np.ndarray:
    x = x.astype(_U64, copy=True)
    with np.errstate(over="ignore"):
        x ^= x >> _U64(30)
        x *= _U64(0xBF58476D1CE4E5B9)
        x ^= x >> _U64(27)
        x *= _U64(0x94D049BB133111EB)
        x ^= x >> _U64(31)
    return x


def hash_u32(seed: int, stream: int, *idx: np.ndarray) -> np.ndarray:
    """Deterministic uint32 per index tuple; ``idx`` arrays broadcast together."""
    with np.errstate(over="ignore"):
        h = _mix64(np.asarray((seed * 0x9E3779B97F4A7C15 + stream * 0xD1B54A32D192ED03 + 0x2545F4914F6CDD1D) & _MASK64,
                              dtype=_U64))
        for a in idx:
            a = np.asarray(a).astype(_U64)
            h = _mix64((h + _U64(0x9E3779B97F4A7C15)) ^ (a * _U64(0xC2B2AE3D27D4EB4F) + _U64(0x165667B19E3779F9)))
    return (h >> _U64(32)).astype(np.uint32)


def bernoulli(p: float, seed: int, stream: int, *idx: np.ndarray) -> np.ndarray:
    """Integer-only Bernoulli(p): ``u32 < floor(p * 2**32)``."""
    thr = min(int(p * 4294967296.0), 4294967295)
    return hash_u32(seed, stream, *idx) < np.uint32(thr)


def uniform01(seed: int, stream: int, *idx: np.ndarray) -> np.ndarray:
    return (hash_u32(seed, stream, *idx).astype(np.float64) + 0.5) / 4294967296.0


# --------------------------------------------------------------------------
# Q / K / V
# --------------------------------------------------------------------------
def make_qkv(seed: int, H: int, N: int, d: int, dtype: str = "bf16"):
    """i.i.d. N(0,1) rounded to bf16 (round-to-nearest-even), or to IEEE half with ``dtype="fp16"``.

    Returns three ``torch.bfloat16`` (``torch.float16``) CPU tensors of shape ``[H, N, d]``.  The
    oracle always consumes these same rounded values (as raw 16-bit patterns).
    """
    import torch
    tdt = {"bf16": torch.bfloat16, "fp16": torch.float16}[dtype]

    out = []
    for t in range(3):
        g = torch.Generator(device="cpu")
        g.manual_seed((seed * 1000003 + t * 7919 + 12345) & 0x7FFFFFFFFFFFFFFF)
        x = torch.empty((H, N, d), dtype=torch.float32)
        x.normal_(0.0, 1.0, generator=g)
        out.append(x.to(tdt))
    return tuple(out)


def bf16_bits(t) -> np.ndarray:
    """torch.bfloat16 (or float16) CPU tensor -> numpy uint16 view of the same bytes."""
    import torch

    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


# --------------------------------------------------------------------------
# request description
# --------------------------------------------------------------------------
@dataclasses.dataclass
class Request:
    name: str
    H: int
    N: int
    d: int
    B_Q: int
    B_KV: int
    mask: np.ndarray  # uint8 [H, nQb, nKb]
    qkv_seed: int
    note: str = ""
    N_kv: int = 0  # key/value tokens per head; 0 = N (self-attention, every workload of the paper)
    dtype: str = "bf16"  # element type of Q, K, V, O ("fp16": IEEE half)

    @property
    def n_kv(self) -> int:
        return self.N_kv if self.N_kv > 0 else self.N

    @property
    def nQb(self) -> int:
        return cdiv(self.N, self.B_Q)

    @property
    def nKb(self) -> int:
        return cdiv(self.n_kv, self.B_KV)

    def qkv(self):
        if self.n_kv == self.N:
            return make_qkv(self.qkv_seed, self.H, self.N, self.d, self.dtype)
        q, _, _ = make_qkv(self.qkv_seed, self.H, self.N, self.d, self.dtype)
        _, k, v = make_qkv(self.qkv_seed + 7777, self.H, self.n_kv, self.d, self.dtype)
        return q, k, v


# --------------------------------------------------------------------------
# 3-D latent helpers: tokens flattened tile-major, one tile = contiguous tokens
# --------------------------------------------------------------------------
def _tile_coords(nt: int, nh: int, nw: int) -> np.ndarray:
    """[ntiles, 3] coordinates of tile id b = (bt*nh + bh)*nw + bw."""
    b = np.arange(nt * nh * nw)
    return np.stack([b // (nh * nw), (b // nw) % nh, b % nw], axis=1)


def window_mask(grid: Tuple[int, int, int], win: Tuple[int, int, int]) -> np.ndarray:
    """Block (i, j) active iff the tile offsets are within ``win`` per axis."""
    c = _tile_coords(*grid)
    diff = np.abs(c[:, None, :] - c[None, :, :])
    return ((diff[..., 0] <= win[0]) & (diff[..., 1] <= win[1]) & (diff[..., 2] <= win[2])).astype(np.uint8)


# --------------------------------------------------------------------------
# the five evaluation configurations
# --------------------------------------------------------------------------
def config_tiny(seed: int = 0, H: int = 2, N: int = 2048, d: int = 64, B: int = 64, p: float = 0.25) -> Request:
    nb = cdiv(N, B)
    h, i, j = np.meshgrid(np.arange(H), np.arange(nb), np.arange(nb), indexing="ij")
    M = bernoulli(p, seed, 1, h, i, j).astype(np.uint8)
    M[:, np.arange(nb), np.arange(nb)] = 1
    return Request("tiny", H, N, d, B, B, M, qkv_seed=seed, note=f"Bernoulli({p}) + diagonal")


def config_mid(seed: int = 1, H: int = 8, extra: float = 0.02, win: Tuple[int, int, int] = (1, 1, 1)) -> Request:
    grid = (8, 4, 4)  # 16x32x32 latent in 2x8x8-token tiles -> 128 blocks of 128 tokens
    nb = 128
    W = window_mask(grid, win)
    h, i, j = np.meshgrid(np.arange(H), np.arange(nb), np.arange(nb), indexing="ij")
    M = (W[None] | bernoulli(extra, seed, 2, h, i, j)).astype(np.uint8)
    return Request("mid", H, 16384, 128, 128, 128, M, qkv_seed=seed,
                   note=f"3-D window({win[0]},{win[1]},{win[2]}) + Bernoulli({extra})")


def config_hunyuan(seed: int = 2, H: int = 24, extra: float = 0.03, win: Tuple[int, int, int] = (1, 1, 2)) -> Request:
    grid = (15, 6, 10)  # 30x48x80 latent in 2x8x8-token tiles -> 900 blocks of 128 tokens
    nb = 900
    W = window_mask(grid, win)
    M = np.empty((H, nb, nb), dtype=np.uint8)
    i, j = np.meshgrid(np.arange(nb), np.arange(nb), indexing="ij")
    for h in range(H):
        M[h] = W | bernoulli(extra, seed * 1000 + h, 3, i, j)
    return Request("hunyuan", H, 115200, 128, 128, 128, M, qkv_seed=seed,
                   note=f"3-D window({win[0]},{win[1]},{win[2]}) + per-head Bernoulli({extra})")


def _runs_row(nKb: int, target: int, seed: int, h: int, i: int) -> np.ndarray:
    """One row of the clustered mask: R ~ U{4..12} runs, lengths ~ Geom(0.3)
    rescaled to sum to ``target``, placed with at least one gap between runs."""
    R = min(4 + int(hash_u32(seed, 10, h, i)) % 9, max(1, target), max(1, (nKb - target + 1)))
    u = uniform01(seed, 11, np.full(R, h), np.full(R, i), np.arange(R))
    lens = np.floor(np.log(u) / np.log(0.7)).astype(np.int64) + 1  # geometric(p=0.3), support >= 1
    # rescale to the density target, keeping every run >= 1
    scaled = np.maximum(1, np.floor(lens * (target / lens.sum())).astype(np.int64))
    k = 0
    while scaled.sum() < target:
        scaled[k % R] += 1
        k += 1
    while scaled.sum() > target:
        c = k % R
        if scaled[c] > 1:
            scaled[c] -= 1
        k += 1
    free = nKb - target - (R - 1)  # slack after the R-1 mandatory single gaps
    w = uniform01(seed, 12, np.full(R + 1, h), np.full(R + 1, i), np.arange(R + 1))
    gaps = np.floor(w / w.sum() * free).astype(np.int64)
    gaps[0] += free - gaps.sum()
    row = np.zeros(nKb, dtype=np.uint8)
    pos = int(gaps[0])
    for r in range(R):
        row[pos:pos + scaled[r]] = 1
        pos += int(scaled[r]) + 1 + int(gaps[r + 1])
    return row


def config_stress_a(seed: int = 3, H: int = 16, N: int = 32768, density: float = 0.15) -> Request:
    B_Q, B_KV = 16, 64
    nQb, nKb = cdiv(N, B_Q), cdiv(N, B_KV)
    target = max(1, int(round(density * nKb)))
    M = np.zeros((H, nQb, nKb), dtype=np.uint8)
    for h in range(H):
        for i in range(nQb):
            M[h, i] = _runs_row(nKb, target, seed, h, i)
    return Request("stress_a", H, N, 64, B_Q, B_KV, M, qkv_seed=3,
                   note=f"4-12 contiguous runs per row, geometric lengths rescaled to {density:.0%} density")


def config_stress_b(seed: int = 4, H: int = 16, N: int = 32768, p: float = 0.2) -> Request:
    B = 256
    nb = cdiv(N, B)
    h, i, j = np.meshgrid(np.arange(H), np.arange(nb), np.arange(nb), indexing="ij")
    M = bernoulli(p, seed, 4, h, i, j).astype(np.uint8)
    M[:, np.arange(nb), np.arange(nb)] = 1
    return Request("stress_b", H, N, 64, B, B, M, qkv_seed=3, note=f"Bernoulli({p}) + diagonal")


SWEEP_GEOMETRIES: List[Tuple[int, int]] = [(32, 32), (64, 128), (128, 64), (128, 128), (256, 256)]
SWEEP_DENSITIES: List[float] = [0.03, 0.10, 0.30, 0.60]


def _sweep_block_coords(N: int, Bsz: int) -> np.ndarray:
    """Tile coordinate (5x9x14 grid of 120-token tiles) of each block's centre token."""
    nb = cdiv(N, Bsz)
    centre = np.minimum(np.arange(nb) * Bsz + Bsz // 2, N - 1)
    tile = centre // 120
    return np.stack([tile // (9 * 14), (tile // 14) % 9, tile % 14], axis=1)


def config_sweep(r: int, H: int = 24, N: int = 75600, d: int = 128,
                 B: Tuple[int, int] | None = None, rho: float | None = None) -> Request:
    """Request ``r`` of the dynamic-request sweep (seed 5 + r).

    Mixes a 3-D window, per-head column stripes (every 8th KV block) and random
    fill up to a per-row budget; ceil(H/8) heads are 10x heavier than the rest.
    """
    seed = 5 + r
    if B is None:
        B = SWEEP_GEOMETRIES[int(hash_u32(seed, 20, 0)) % len(SWEEP_GEOMETRIES)]
    if rho is None:
        rho = SWEEP_DENSITIES[int(hash_u32(seed, 21, 0)) % len(SWEEP_DENSITIES)]
    B_Q, B_KV = B
    nQb, nKb = cdiv(N, B_Q), cdiv(N, B_KV)
    # head weights: ceil(H/8) seeded heavy heads (weight 10), others 1; water-fill to keep the mean at rho
    order = np.argsort(hash_u32(seed, 22, np.arange(H)), kind="stable")
    w = np.ones(H)
    w[order[: cdiv(H, 8)]] = 10.0
    rho_h = rho * w / w.mean()
    for _ in range(8):
        over = rho_h > 0.95
        if not over.any():
            break
        excess = (rho_h[over] - 0.95).sum()
        rho_h[over] = 0.95
        free = ~over
        if free.any():
            rho_h[free] += excess * w[free] / w[free].sum()
    rho_h = np.minimum(rho_h, 0.95)
    cq = _sweep_block_coords(N, B_Q)
    ck = _sweep_block_coords(N, B_KV)
    M = np.zeros((H, nQb, nKb), dtype=np.uint8)
    cols = np.arange(nKb)
    for h in range(H):
        z = uniform01(seed, 23, np.full(nQb, h), np.arange(nQb))
        z2 = uniform01(seed, 24, np.full(nQb, h), np.arange(nQb))
        gauss = np.sqrt(-2.0 * np.log(z)) * np.cos(2.0 * np.pi * z2)
        g = np.exp(0.5 * gauss - 0.125)  # lognormal(sigma=0.5), mean 1
        budget = np.maximum(1, np.rint(np.minimum(1.0, rho_h[h] * g) * nKb).astype(np.int64))
        budget = np.minimum(budget, nKb)
        phi = int(hash_u32(seed, 25, h)) % 8
        stripe = (cols % 8) == phi
        step = max(1, (1 << 22) // nKb)
        for i0 in range(0, nQb, step):
            rows = np.arange(i0, min(nQb, i0 + step))
            cheb = np.abs(ck[None, :, :] - cq[rows][:, None, :]).max(axis=2)
            # priority class: 0 = same tile, 1 = neighbouring tile, 2 = stripe column, 3 = the rest
            cls = np.where(cheb == 0, 0, np.where(cheb == 1, 1, np.where(stripe[None, :], 2, 3)))
            key = cls.astype(np.uint64) * np.uint64(1 << 32) + hash_u32(seed, 26, h, rows[:, None], cols[None, :]).astype(np.uint64)
            srt = np.sort(key, axis=1)
            thr = srt[np.arange(len(rows)), budget[rows] - 1]
            M[h, rows] = key <= thr[:, None]  # hash ties inside a class are kept (at most a few blocks)
    return Request(f"sweep{r}", H, N, d, B_Q, B_KV, M, qkv_seed=seed,
                   note=f"B={B} target density {rho}")


# --------------------------------------------------------------------------
# small seeded masks for parity and property tests
# --------------------------------------------------------------------------
def random_mask(seed: int, H: int, nQb: int, nKb: int, p: float, diag: bool = False,
                empty_rows: float = 0.0) -> np.ndarray:
    h, i, j = np.meshgrid(np.arange(H), np.arange(nQb), np.arange(nKb), indexing="ij")
    M = bernoulli(p, seed, 30, h, i, j).astype(np.uint8)
    if diag:
        ii = np.arange(nQb)
        M[:, ii, np.minimum(ii * nKb // nQb, nKb - 1)] = 1
    if empty_rows > 0:
        hh, ii = np.meshgrid(np.arange(H), np.arange(nQb), indexing="ij")
        kill = bernoulli(empty_rows, seed, 31, hh, ii)
        M[kill] = 0
    return M


def sample_query_blocks(seed: int, H: int, nQb: int, k: int = 64) -> Dict[int, np.ndarray]:
    """Seeded sample of ``k`` distinct query blocks per head (all of them if nQb <= k)."""
    out = {}
    for h in range(H):
        if nQb <= k:
            out[h] = np.arange(nQb)
        else:
            key = hash_u32(seed, 40, h, np.arange(nQb))
            out[h] = np.sort(np.argsort(key, kind="stable")[:k])
    return out


CONFIGS = {
    "tiny": config_tiny,
    "mid": config_mid,
    "hunyuan": config_hunyuan,
    "stress_a": config_stress_a,
    "stress_b": config_stress_b,
}
