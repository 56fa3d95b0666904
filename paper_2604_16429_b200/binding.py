"""Thin ctypes binding of the C ABI in ``include/mosaic_bsa.h``.

Argument marshalling only: every step of the path runs in the CUDA library.  torch is
used for device memory and streams.  There is no CPU fallback: if the library is missing
or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import math
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmosaic_bsa.so")
_lib = None

OP_SELECT, OP_FWD, OP_BWD, OP_FWD_BRANCHES, OP_BWD_BRANCHES = 0, 1, 2, 3, 4
EXPORTS = ("mosaic_bsa_workspace_bytes", "mosaic_bsa_select", "mosaic_bsa_fwd", "mosaic_bsa_bwd",
           "mosaic_bsa_last_status", "mosaic_bsa_strerror", "mosaic_bsa_select_static",
           "mosaic_bsa_descriptor_encodes", "mosaic_bsa_fwd_branches", "mosaic_bsa_bwd_branches", "mosaic_bsa_rope")
STATIC_SCRATCH_BYTES = 4 << 20
FLAG_LOCAL_GROUPS = 1
FLAG_FP16 = 2


class MosaicError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} ({code})")


class _Params(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("H", ctypes.c_int32), ("nlat", ctypes.c_int32), ("nlon", ctypes.c_int32),
                ("d", ctypes.c_int32), ("bh", ctypes.c_int32), ("bw", ctypes.c_int32),
                ("rlat", ctypes.c_int32), ("rlon", ctypes.c_int32), ("topk", ctypes.c_int32),
                ("scale", ctypes.c_float), ("flags", ctypes.c_uint32), ("Hkv", ctypes.c_int32)]


@dataclass(frozen=True)
class Params:
    B: int
    H: int
    nlat: int
    nlon: int
    d: int = 64
    bh: int = 8
    bw: int = 8
    rlat: int = 1
    rlon: int = 1
    topk: int = 8
    scale: float = 0.0
    flags: int = 0
    Hkv: int = 0          # heads of K and V (grouped-query attention); 0 = H

    @property
    def kv_heads(self): return self.Hkv or self.H
    @property
    def N(self): return self.nlat * self.nlon
    @property
    def m(self): return (self.nlat // self.bh) * (self.nlon // self.bw)
    @property
    def U(self): return self.B * self.H

    def c(self):
        return _Params(self.B, self.H, self.nlat, self.nlon, self.d, self.bh, self.bw, self.rlat, self.rlon,
                       self.topk, self.scale, self.flags, self.Hkv)

    @staticmethod
    def from_workload(w, **over):
        kw = dict(B=w.B, H=w.H, nlat=w.nlat, nlon=w.nlon, d=w.d, bh=w.bh, bw=w.bw, rlat=w.rlat, rlon=w.rlon,
                  topk=w.topk, flags=(FLAG_LOCAL_GROUPS if getattr(w, "local_groups", False) else 0)
                  | (FLAG_FP16 if getattr(w, "f16", False) else 0),
                  Hkv=getattr(w, "Hkv", 0))
        kw.update(over)
        return Params(**kw)


def lib():
    """Load the CUDA library; fails loudly if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2604_16429_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32p, fp = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
        pp = ctypes.POINTER(_Params)
        L.mosaic_bsa_workspace_bytes.restype = ctypes.c_size_t
        L.mosaic_bsa_workspace_bytes.argtypes = [pp, ctypes.c_int]
        L.mosaic_bsa_select.restype = ctypes.c_int
        L.mosaic_bsa_select.argtypes = [pp, vp, vp, i32p, vp, ctypes.c_size_t, vp]
        L.mosaic_bsa_select_static.restype = ctypes.c_int
        L.mosaic_bsa_select_static.argtypes = [pp, vp, vp, i32p, vp]
        L.mosaic_bsa_fwd.restype = ctypes.c_int
        L.mosaic_bsa_fwd.argtypes = [pp, vp, vp, vp, i32p, vp, fp, vp, ctypes.c_size_t, vp]
        L.mosaic_bsa_fwd_branches.restype = ctypes.c_int
        L.mosaic_bsa_fwd_branches.argtypes = [pp, vp, vp, vp, i32p, fp, vp, fp, fp, vp, ctypes.c_size_t, vp]
        L.mosaic_bsa_bwd_branches.restype = ctypes.c_int
        L.mosaic_bsa_bwd_branches.argtypes = [pp, vp, vp, vp, i32p, fp, vp, vp, vp, vp, fp, vp, ctypes.c_size_t, vp]
        L.mosaic_bsa_rope.restype = ctypes.c_int
        L.mosaic_bsa_rope.argtypes = [pp, vp, vp, fp, ctypes.c_float, vp, vp, vp]
        L.mosaic_bsa_bwd.restype = ctypes.c_int
        L.mosaic_bsa_bwd.argtypes = [pp, vp, vp, vp, vp, fp, vp, i32p, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.mosaic_bsa_last_status.restype = ctypes.c_int
        L.mosaic_bsa_last_status.argtypes = [vp, vp]
        L.mosaic_bsa_descriptor_encodes.restype = ctypes.c_longlong
        L.mosaic_bsa_descriptor_encodes.argtypes = []
        L.mosaic_bsa_strerror.restype = ctypes.c_char_p
        L.mosaic_bsa_strerror.argtypes = [ctypes.c_int]
        _lib = L
    return _lib


def strerror(code: int) -> str:
    return lib().mosaic_bsa_strerror(int(code)).decode()


def workspace_bytes(p: Params, op: int) -> int:
    pc = p.c()
    return int(lib().mosaic_bsa_workspace_bytes(ctypes.byref(pc), op))


def _stream(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _chk_qkv(p: Params, *ts, heads=None):
    h = p.H if heads is None else heads
    dt = torch.float16 if p.flags & FLAG_FP16 else torch.bfloat16
    for t in ts:
        if t.dtype != dt or not t.is_cuda or not t.is_contiguous() or tuple(t.shape) != (p.B, h, p.N, p.d):
            raise ValueError(f"expected contiguous cuda {dt} [{p.B},{h},{p.N},{p.d}], got {t.dtype} {tuple(t.shape)}")


def alloc_workspace(p: Params, op: int, device="cuda") -> torch.Tensor:
    n = workspace_bytes(p, op)
    if n == 0:
        raise MosaicError(-1, "mosaic_bsa_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def mosaic_bsa_select(p: Params, q, k, block_idx=None, ws=None, stream=None):
    _chk_qkv(p, q)
    _chk_qkv(p, k, heads=p.kv_heads)
    if block_idx is None:
        block_idx = torch.empty((p.B, p.H, p.m, p.topk), dtype=torch.int32, device=q.device)
    if ws is None:
        ws = alloc_workspace(p, OP_SELECT, q.device)
    pc = p.c()
    rc = lib().mosaic_bsa_select(ctypes.byref(pc), _ptr(q), _ptr(k), _ptr(block_idx), _ptr(ws), ws.numel(),
                                 _stream(stream))
    if rc:
        raise MosaicError(rc, "mosaic_bsa_select")
    return block_idx


def mosaic_bsa_select_static(p: Params, q, k, block_idx=None, stream=None):
    """Selection through the entry point that allocates nothing (scratch inside the library image).
    Only `block_idx` is created here when the caller passes none."""
    _chk_qkv(p, q)
    _chk_qkv(p, k, heads=p.kv_heads)
    if block_idx is None:
        block_idx = torch.empty((p.B, p.H, p.m, p.topk), dtype=torch.int32, device=q.device)
    pc = p.c()
    rc = lib().mosaic_bsa_select_static(ctypes.byref(pc), _ptr(q), _ptr(k), _ptr(block_idx), _stream(stream))
    if rc:
        raise MosaicError(rc, "mosaic_bsa_select_static")
    return block_idx


def mosaic_bsa_fwd(p: Params, q, k, v, block_idx, o=None, lse=None, ws=None, stream=None):
    _chk_qkv(p, q)
    _chk_qkv(p, k, v, heads=p.kv_heads)
    if o is None:
        o = torch.empty_like(q)
    if lse is None:
        lse = torch.empty((p.B, p.H, p.N), dtype=torch.float32, device=q.device)
    if ws is None:
        ws = alloc_workspace(p, OP_FWD, q.device)
    pc = p.c()
    rc = lib().mosaic_bsa_fwd(ctypes.byref(pc), _ptr(q), _ptr(k), _ptr(v), _ptr(block_idx), _ptr(o), _ptr(lse),
                              _ptr(ws), ws.numel(), _stream(stream))
    if rc:
        raise MosaicError(rc, "mosaic_bsa_fwd")
    return o, lse


def mosaic_bsa_fwd_branches(p: Params, q, k, v, block_idx, gates, o=None, lse_fg=None, lse_l=None, ws=None, stream=None):
    """Three-branch form: gated sum of the compression, selection and local branches.  `gates` is
    [B, H, N, 3] fp32 (compression, selection, local).  Returns (o, lse_fg, lse_l)."""
    _chk_qkv(p, q)
    _chk_qkv(p, k, v, heads=p.kv_heads)
    if gates.dtype != torch.float32 or not gates.is_contiguous() or tuple(gates.shape) != (p.B, p.H, p.N, 3):
        raise ValueError(f"expected contiguous cuda fp32 gates [{p.B},{p.H},{p.N},3]")
    o = torch.empty_like(q) if o is None else o
    lse_fg = torch.empty((p.B, p.H, p.N), dtype=torch.float32, device=q.device) if lse_fg is None else lse_fg
    lse_l = torch.empty((p.B, p.H, p.N), dtype=torch.float32, device=q.device) if lse_l is None else lse_l
    if ws is None:
        ws = alloc_workspace(p, OP_FWD_BRANCHES, q.device)
    pc = p.c()
    rc = lib().mosaic_bsa_fwd_branches(ctypes.byref(pc), _ptr(q), _ptr(k), _ptr(v), _ptr(block_idx), _ptr(gates), _ptr(o),
                                       _ptr(lse_fg), _ptr(lse_l), _ptr(ws), ws.numel(), _stream(stream))
    if rc:
        raise MosaicError(rc, "mosaic_bsa_fwd_branches")
    return o, lse_fg, lse_l


def mosaic_bsa_bwd(p: Params, q, k, v, o, lse, d_o, block_idx, dq=None, dk=None, dv=None, ws=None, stream=None):
    _chk_qkv(p, q, o, d_o)
    _chk_qkv(p, k, v, heads=p.kv_heads)
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(k) if dv is None else dv
    if ws is None:
        ws = alloc_workspace(p, OP_BWD, q.device)
    pc = p.c()
    rc = lib().mosaic_bsa_bwd(ctypes.byref(pc), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(d_o),
                              _ptr(block_idx), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(ws), ws.numel(), _stream(stream))
    if rc:
        raise MosaicError(rc, "mosaic_bsa_bwd")
    return dq, dk, dv


def mosaic_bsa_bwd_branches(p: Params, q, k, v, block_idx, gates, d_o, dq=None, dk=None, dv=None, dgates=None, ws=None,
                            stream=None):
    """Backward of the three-branch form.  Returns (dq, dk, dv, dgates); dgates is [B, H, N, 3] fp32."""
    _chk_qkv(p, q, d_o)
    _chk_qkv(p, k, v, heads=p.kv_heads)
    if gates.dtype != torch.float32 or not gates.is_contiguous() or tuple(gates.shape) != (p.B, p.H, p.N, 3):
        raise ValueError(f"expected contiguous cuda fp32 gates [{p.B},{p.H},{p.N},3]")
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(k) if dk is None else dk
    dv = torch.empty_like(k) if dv is None else dv
    dgates = torch.empty_like(gates) if dgates is None else dgates
    if ws is None:
        ws = alloc_workspace(p, OP_BWD_BRANCHES, q.device)
    pc = p.c()
    rc = lib().mosaic_bsa_bwd_branches(ctypes.byref(pc), _ptr(q), _ptr(k), _ptr(v), _ptr(block_idx), _ptr(gates), _ptr(d_o),
                                       _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dgates), _ptr(ws), ws.numel(), _stream(stream))
    if rc:
        raise MosaicError(rc, "mosaic_bsa_bwd_branches")
    return dq, dk, dv, dgates


def mosaic_bsa_rope(p: Params, q, k, pos, theta=10000.0, q_out=None, k_out=None, stream=None):
    """2-D rotary position embedding of q and k; pos is [N, 2] fp32 (longitude, latitude in radians).
    Returns (q_out, k_out)."""
    _chk_qkv(p, q)
    _chk_qkv(p, k, heads=p.kv_heads)
    if pos.dtype != torch.float32 or not pos.is_cuda or not pos.is_contiguous() or tuple(pos.shape) != (p.N, 2):
        raise ValueError(f"expected contiguous cuda fp32 positions [{p.N},2]")
    q_out = torch.empty_like(q) if q_out is None else q_out
    k_out = torch.empty_like(k) if k_out is None else k_out
    pc = p.c()
    rc = lib().mosaic_bsa_rope(ctypes.byref(pc), _ptr(q), _ptr(k), _ptr(pos), float(theta), _ptr(q_out), _ptr(k_out),
                               _stream(stream))
    if rc:
        raise MosaicError(rc, "mosaic_bsa_rope")
    return q_out, k_out


def mosaic_bsa_last_status(ws, stream=None) -> int:
    return int(lib().mosaic_bsa_last_status(_ptr(ws), _stream(stream)))


def descriptor_encodes() -> int:
    return int(lib().mosaic_bsa_descriptor_encodes())


def check_status(ws, where: str, stream=None):
    st = mosaic_bsa_last_status(ws, stream)
    if st:
        raise MosaicError(st, where + " (device status)")


def from_bits(bits, device="cuda", f16=False) -> torch.Tensor:
    """uint16 bit patterns (numpy) -> bf16 (or, with f16, float16) tensor on `device`, bit for bit."""
    import numpy as np
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.float16 if f16 else torch.bfloat16)


def default_scale(d: int) -> float:
    return 1.0 / math.sqrt(d)
