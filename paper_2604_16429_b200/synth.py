"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no arithmetic of the attention method: it only draws numbers.
Both the CUDA path and the test oracle are fed the arrays it returns, bit for bit.

The real activations (ERA5 / HRES-derived fields pushed through trained
projection weights) are not available, so two stand-ins are used:

* ``iid``    -- Q, K, V i.i.d. N(0,1);
* ``smooth`` -- per tensor, head and channel a sum of 8 random low-wavenumber
  waves a_w * sin(2*pi*kx_w*lon/nlon + phi_w) * cos(pi*ky_w*lat/nlat + psi_w),
  kx, ky integers in [0, 6], a_w ~ N(0,1)/sqrt(8), phases uniform in [0, 2*pi)
  (periodic in longitude, like fields on the sphere), plus 0.1 * N(0,1) noise per
  element.  The smooth part is shared by all ensemble members of a batch, the noise
  is independent per member.  Smooth fields make neighbouring query blocks choose
  overlapping key blocks and make some key blocks popular, which is what decides
  cache reuse in the forward and load imbalance in the backward.

Everything is rounded to bf16 (round to nearest even) and returned as ``uint16``
bit patterns of shape ``[B, H, N, d]``; generator: numpy PCG64, seed
``1000 * config + {0: Q, 1: K, 2: V, 3: dO}``.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    cfg: int
    B: int
    H: int
    nlat: int
    nlon: int
    bh: int
    bw: int
    topk: int
    kind: str          # "iid" or "smooth"
    backward: bool = False
    d: int = 64
    rlat: int = 1
    rlon: int = 1
    local_groups: bool = False   # local set = aligned group of rlat x rlon blocks (the paper's large local blocks)
    Hkv: int = 0                 # heads of K and V (grouped-query attention); 0 = H
    f16: bool = False            # 16-bit tensors are IEEE binary16 instead of bf16 (the same values, rounded to that type)

    @property
    def N(self): return self.nlat * self.nlon
    @property
    def m(self): return (self.nlat // self.bh) * (self.nlon // self.bw)
    @property
    def b(self): return self.bh * self.bw
    @property
    def U(self): return self.B * self.H
    @property
    def kv_heads(self): return self.Hkv or self.H


WORKLOADS = {
    "c1_tiny": Workload("c1_tiny", 1, 1, 4, 32, 64, 8, 8, 4, "iid"),
    "c2_1p5deg": Workload("c2_1p5deg", 2, 1, 8, 120, 240, 8, 8, 8, "smooth"),
    "c3_1p5deg_ens24": Workload("c3_1p5deg_ens24", 3, 24, 8, 120, 240, 8, 8, 8, "smooth"),
    "c4_1p5deg_train": Workload("c4_1p5deg_train", 4, 4, 16, 120, 240, 8, 8, 8, "smooth", True),
    "c5_0p25deg": Workload("c5_0p25deg", 5, 1, 8, 720, 1440, 16, 16, 16, "smooth"),
    # The paper's own layout and shapes (architecture table): HEALPix NESTED sequence of 12 * nside^2 tokens, sparse
    # blocks of 128 contiguous tokens (8 rows of a 16-wide view of the sequence), local attention inside aligned
    # 1024-token blocks (8 sparse blocks), 24 / 12 / 4 selected blocks, d = 64 per head.
    "hp_nside64": Workload("hp_nside64", 6, 1, 12, 3072, 16, 8, 16, 24, "smooth", rlat=8, rlon=1, local_groups=True),
    "hp_nside32": Workload("hp_nside32", 7, 1, 16, 768, 16, 8, 16, 12, "smooth", rlat=8, rlon=1, local_groups=True),
    "hp_nside16": Workload("hp_nside16", 8, 1, 20, 192, 16, 8, 16, 4, "smooth", rlat=8, rlon=1, local_groups=True),
    # stage 1 with the paper's grouped-query attention (ratio 4): 12 query heads on 3 key/value heads
    "hp_nside64_gqa": Workload("hp_nside64_gqa", 9, 1, 12, 3072, 16, 8, 16, 24, "smooth", rlat=8, rlon=1, local_groups=True, Hkv=3),
}


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns, round to nearest even (finite inputs)."""
    u = np.ascontiguousarray(x, np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    return (h.astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_f16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> IEEE binary16 bit patterns, round to nearest even."""
    return np.ascontiguousarray(x, np.float32).astype(np.float16).view(np.uint16)


def f16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    return np.ascontiguousarray(h, np.uint16).view(np.float16).astype(np.float32)


def iid_normal(B, H, N, d, seed) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(seed))
    return to_bf16_bits(rng.standard_normal((B, H, N, d), dtype=np.float32))


def smooth_plus_noise(B, H, nlat, nlon, d, seed, noise=0.1, waves=8) -> np.ndarray:
    rng = np.random.Generator(np.random.PCG64(seed))
    kx = rng.integers(0, 7, size=(H, d, waves))
    ky = rng.integers(0, 7, size=(H, d, waves))
    a = (rng.standard_normal((H, d, waves)) / np.sqrt(waves)).astype(np.float32)
    phi = rng.uniform(0.0, 2 * np.pi, size=(H, d, waves))
    psi = rng.uniform(0.0, 2 * np.pi, size=(H, d, waves))
    lon = np.arange(nlon)
    lat = np.arange(nlat)
    out = np.empty((B, H, nlat * nlon, d), np.uint16)
    for h in range(H):
        s_lon = np.sin(2 * np.pi * kx[h][..., None] * lon / nlon + phi[h][..., None]).astype(np.float32)
        c_lat = (a[h][..., None] * np.cos(np.pi * ky[h][..., None] * lat / nlat + psi[h][..., None])).astype(np.float32)
        # f[c, lat, lon] = sum_w c_lat[c, w, lat] * s_lon[c, w, lon]
        f = np.einsum("cwl,cwo->loc", c_lat, s_lon, optimize=True).reshape(nlat * nlon, d)
        for b in range(B):
            eps = rng.standard_normal((nlat * nlon, d), dtype=np.float32)
            out[b, h] = to_bf16_bits(f + np.float32(noise) * eps)
    return out


def make_inputs(w: Workload, with_do: bool | None = None) -> dict:
    """Q, K, V (and dO when the workload trains) as uint16 bf16 bits [B,H,N,d]."""
    base = 1000 * w.cfg
    if w.kind == "iid":
        gen = lambda s, h=w.H: iid_normal(w.B, h, w.N, w.d, s)
    else:
        gen = lambda s, h=w.H: smooth_plus_noise(w.B, h, w.nlat, w.nlon, w.d, s)
    out = {"q": gen(base + 0), "k": gen(base + 1, w.kv_heads), "v": gen(base + 2, w.kv_heads)}   # K, V: [B, Hkv, N, d]
    if w.backward if with_do is None else with_do:
        out["do"] = iid_normal(w.B, w.H, w.N, w.d, base + 3)
    if w.f16:   # the same draws, stored as binary16 (a bf16 value of this range is exact in binary16 bar underflow)
        out = {k: to_f16_bits(bf16_bits_to_f32(v)) for k, v in out.items()}
    return out


def small_case(nlat, nlon, bh, bw, topk, B=1, H=1, d=64, kind="iid", seed=7, rlat=1, rlon=1, backward=False,
               local_groups=False, Hkv=0, f16=False):
    """A free-form small workload for tests (cfg number = seed)."""
    return Workload(f"small_{nlat}x{nlon}_{bh}x{bw}_k{topk}" + ("_groups" if local_groups else "") + (f"_kv{Hkv}" if Hkv else "")
                    + ("_f16" if f16 else ""),
                    seed, B, H, nlat, nlon, bh, bw, topk, kind, backward, d, rlat, rlon, local_groups, Hkv, f16)
