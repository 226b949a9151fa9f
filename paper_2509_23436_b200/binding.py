"""Thin ctypes binding over liblot.so: argument marshalling only.

Each function has the name and argument order of its C entry point (include/lot.h) and
takes torch CUDA tensors where the C call takes device pointers.  torch is used for
device memory and streams; every step of the path runs inside the library's kernels.
There is no fallback: if the library cannot be loaded the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

LOT_F32, LOT_BF16 = 0, 1
LOT_OK = 0
LOT_DEV_NONFINITE, LOT_DEV_EMPTY, LOT_DEV_TIMEOUT, LOT_DEV_RECOMPUTED, LOT_DEV_BOUNDS = 1, 2, 4, 8, 16

# LOT_LIBRARY selects another build of the same library (the bounds-check build liblot_debug.so)
_LIB_PATH = os.environ.get("LOT_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "liblot.so")
_lib = None

_vp, _i, _f, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t

# name -> (restype, argtypes); the list of symbols include/lot.h declares
SIGNATURES = {
    "lot_version": (_i, []),
    "lot_status_string": (ctypes.c_char_p, [_i]),
    "lot_cost": (_i, [_vp, _vp, _i, _i, _i, _i, _i, _i, _vp, _vp]),
    "lot_sinkhorn_workspace_bytes": (_sz, [_i, _i, _i, _i]),
    "lot_sinkhorn": (_i, [_vp, _vp, _vp, _i, _i, _i, _i, _f, _i, _vp, _vp, _vp, _vp, _sz, _vp]),
    "lot_sinkhorn_static": (_i, [_vp, _vp, _vp, _i, _i, _i, _i, _f, _i, _vp, _vp, _vp, _vp, _vp]),
    "lot_workspace_bytes": (_sz, [_i, _i, _i, _i, _i, _i]),
    "lot_debug_hook": (_i, [_i, ctypes.c_longlong]),
    "lot_path": (_i, [_i, _i, _i, _i, _i, _i, _i]),
    "lot_launch_count": (_i, [_i, _i, _i, _i, _i, _i, _i]),
    "lot_attention_fwd_ex": (_i, [_vp, _vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _f, _i,
                                  _vp, _vp, _vp, _vp, _sz, _vp]),
    "lot_var_workspace_bytes": (_sz, [_i, _i, _i, _i, _i, _i, _i]),
    "lot_attention_fwd_var": (_i, [_vp] * 10 + [_i, _f] + [_i] * 7 + [_f, _i] + [_vp, _vp, _vp, _vp, _sz, _vp]),
    "lot_attention_fwd": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _f, _i, _vp, _vp]),
    "lot_bwd_workspace_bytes": (_sz, [_i, _i, _i, _i, _i, _i, _i]),
    "lot_attention_bwd": (_i, [_vp] * 7 + [_i] * 6 + [_f, _i] + [_vp] * 6 + [_sz, _vp]),
    "lot_device_status": (_i, [_vp, _vp, ctypes.POINTER(_i)]),
}


class LotError(RuntimeError):
    pass


def lib():
    """Load liblot.so (once).  Raises if it has not been built: there is no other path."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise LotError(f"{_LIB_PATH} is missing: build it with `python -m paper_2509_23436_b200.build`")
        L = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(status: int, what: str):
    if status != LOT_OK:
        raise LotError(f"{what}: {lib().lot_status_string(status).decode()}")


def _dev(t: Optional[torch.Tensor], name: str, dtype=None):
    if t is None:
        return None
    if not t.is_cuda:
        raise LotError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise LotError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise LotError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return LOT_F32
    if t.dtype == torch.bfloat16:
        return LOT_BF16
    raise LotError(f"unsupported tensor dtype {t.dtype}")


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def lot_version() -> int:
    return lib().lot_version()


def lot_cost(x: torch.Tensor, z: torch.Tensor, cost: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    B, H, n, d = x.shape
    r = z.shape[1]
    if tuple(z.shape) != (H, r, d):
        raise LotError("z must be [H,r,d]")
    if cost is None:
        cost = torch.empty(B, H, n, r, device=x.device, dtype=torch.float32)
    st = lib().lot_cost(_dev(x, "x"), _dev(z, "z", torch.float32), _dtype_code(x), B, H, n, d, r,
                        _dev(cost, "cost", torch.float32), _stream(stream))
    _check(st, "lot_cost")
    return cost


def lot_sinkhorn_workspace_bytes(B, H, n, r) -> int:
    return lib().lot_sinkhorn_workspace_bytes(B, H, n, r)


def lot_sinkhorn(cost, beta, length, eps, iters, *, want_f=False, want_plan=False, ws=None, stream=None):
    """Returns (g, f or None, plan or None, ws)."""
    B, H, n, r = cost.shape
    dev = cost.device
    g = torch.empty(B, H, r, device=dev, dtype=torch.float32)
    f = torch.empty(B, H, n, device=dev, dtype=torch.float32) if want_f else None
    plan = torch.empty(B, H, n, r, device=dev, dtype=torch.float32) if want_plan else None
    need = lot_sinkhorn_workspace_bytes(B, H, n, r)
    if ws is None:
        ws = torch.empty(max(need, 256), device=dev, dtype=torch.uint8)
    st = lib().lot_sinkhorn(_dev(cost, "cost", torch.float32), _dev(beta, "beta", torch.float32),
                            _dev(length, "len", torch.int32), B, H, n, r, float(eps), int(iters),
                            _dev(g, "g"), _dev(f, "f"), _dev(plan, "plan"),
                            _dev(ws, "ws"), ws.numel(), _stream(stream))
    _check(st, "lot_sinkhorn")
    return g, f, plan, ws


LOT_STATIC_SCRATCH_BYTES = 4 << 20


def lot_sinkhorn_static(cost, beta, length, eps, iters, g, f=None, plan=None, status_out=None, stream=None):
    """lot_sinkhorn on the library's built-in scratch array: allocates nothing, so every output
    (g, and f / plan / status_out if wanted) is a tensor the caller passes in.  Returns g."""
    B, H, n, r = cost.shape
    st = lib().lot_sinkhorn_static(_dev(cost, "cost", torch.float32), _dev(beta, "beta", torch.float32),
                                   _dev(length, "len", torch.int32), B, H, n, r, float(eps), int(iters),
                                   _dev(g, "g", torch.float32), _dev(f, "f", torch.float32),
                                   _dev(plan, "plan", torch.float32), _dev(status_out, "status_out", torch.int32),
                                   _stream(stream))
    _check(st, "lot_sinkhorn_static")
    return g


def lot_workspace_bytes(B, H, n, d, r, dtype_code) -> int:
    return lib().lot_workspace_bytes(B, H, n, d, r, dtype_code)


def lot_debug_hook(what: int, value: int) -> None:
    _check(lib().lot_debug_hook(int(what), int(value)), "lot_debug_hook")


def lot_path(dtype_code: int, B: int, H: int, n: int, d: int, r: int, iters: int) -> int:
    return lib().lot_path(dtype_code, B, H, n, d, r, iters)


def lot_launch_count(dtype_code: int, B: int, H: int, n: int, d: int, r: int, iters: int) -> int:
    return lib().lot_launch_count(dtype_code, B, H, n, d, r, iters)


def lot_attention_fwd_ex(q, k, v, z, beta, key_len, eps, iters, *, out=None, g1_out=None, g2_out=None,
                         ws=None, stream=None):
    """Returns (out, ws).  dtype is taken from q; k, v, out must match."""
    B, H, n, d = q.shape
    r = z.shape[1]
    code = _dtype_code(q)
    if k.shape != q.shape or v.shape != q.shape or k.dtype != q.dtype or v.dtype != q.dtype:
        raise LotError("q, k, v must share shape and dtype")
    if tuple(z.shape) != (H, r, d) or tuple(beta.shape) != (H, r):
        raise LotError("z must be [H,r,d] and beta [H,r]")
    if out is None:
        out = torch.empty_like(q)
    need = lot_workspace_bytes(B, H, n, d, r, code)
    if ws is None:
        ws = torch.empty(max(need, 256), device=q.device, dtype=torch.uint8)
    st = lib().lot_attention_fwd_ex(_dev(q, "q"), _dev(k, "k"), _dev(v, "v"), _dev(z, "z", torch.float32),
                                    _dev(beta, "beta", torch.float32), _dev(key_len, "key_len", torch.int32),
                                    code, B, H, n, d, r, float(eps), int(iters),
                                    _dev(out, "out", q.dtype), _dev(g1_out, "g1_out", torch.float32),
                                    _dev(g2_out, "g2_out", torch.float32),
                                    _dev(ws, "ws"), ws.numel(), _stream(stream))
    _check(st, "lot_attention_fwd_ex")
    return out, ws


def lot_var_workspace_bytes(B, H, nq, nk, d, r, dtype_code) -> int:
    return lib().lot_var_workspace_bytes(B, H, nq, nk, d, r, dtype_code)


def lot_attention_fwd_var(q, k, v, z, beta, eps, iters, *, a=None, b=None, key_len=None, g1_in=None, g2_in=None,
                          cls=False, cls_tau=1.0, out=None, g1_out=None, g2_out=None, ws=None, stream=None):
    """Forward variants (cross-attention, token weights, warm start, [CLS] row).  Returns (out, ws)."""
    B, H, nq, d = q.shape
    nk = k.shape[2]
    r = z.shape[1]
    code = _dtype_code(q)
    if k.shape != (B, H, nk, d) or v.shape != k.shape or k.dtype != q.dtype or v.dtype != q.dtype:
        raise LotError("k, v must be [B,H,nk,d] in q's dtype")
    if tuple(z.shape) != (H, r, d) or tuple(beta.shape) != (H, r):
        raise LotError("z must be [H,r,d] and beta [H,r]")
    if out is None:
        out = torch.empty_like(q)
    need = lot_var_workspace_bytes(B, H, nq, nk, d, r, code)
    if ws is None:
        ws = torch.empty(max(need, 256), device=q.device, dtype=torch.uint8)
    f32 = torch.float32
    st = lib().lot_attention_fwd_var(_dev(q, "q"), _dev(k, "k"), _dev(v, "v"), _dev(z, "z", f32), _dev(beta, "beta", f32),
                                     _dev(a, "a", f32), _dev(b, "b", f32), _dev(key_len, "key_len", torch.int32),
                                     _dev(g1_in, "g1_in", f32), _dev(g2_in, "g2_in", f32), int(bool(cls)), float(cls_tau),
                                     code, B, H, nq, nk, d, r, float(eps), int(iters),
                                     _dev(out, "out", q.dtype), _dev(g1_out, "g1_out", f32), _dev(g2_out, "g2_out", f32),
                                     _dev(ws, "ws"), ws.numel(), _stream(stream))
    _check(st, "lot_attention_fwd_var")
    return out, ws


def lot_attention_fwd(q, k, v, z, beta, eps, iters, out=None, stream=None):
    """float32 tensors, uniform marginals, library-managed scratch."""
    B, H, n, d = q.shape
    r = z.shape[1]
    if out is None:
        out = torch.empty_like(q)
    f32 = torch.float32
    st = lib().lot_attention_fwd(_dev(q, "q", f32), _dev(k, "k", f32), _dev(v, "v", f32), _dev(z, "z", f32),
                                 _dev(beta, "beta", f32), B, H, n, d, r, float(eps), int(iters),
                                 _dev(out, "out", f32), _stream(stream))
    _check(st, "lot_attention_fwd")
    return out


def lot_device_status(ws: Optional[torch.Tensor], stream=None) -> int:
    val = ctypes.c_int(0)
    st = lib().lot_device_status(_dev(ws, "ws"), _stream(stream), ctypes.byref(val))
    _check(st, "lot_device_status")
    return val.value


def lot_bwd_workspace_bytes(B, H, n, d, r, dtype_code, iters) -> int:
    return lib().lot_bwd_workspace_bytes(B, H, n, d, r, dtype_code, iters)


def lot_attention_bwd(q, k, v, z, beta, key_len, dout, eps, iters, *, ws=None, stream=None):
    """Gradients of the forward with respect to q, k, v, z, beta.  Returns (dq, dk, dv, dz, dbeta, ws)."""
    B, H, n, d = q.shape
    r = z.shape[1]
    code = _dtype_code(q)
    for name, t in (("k", k), ("v", v), ("dout", dout)):
        if t.shape != q.shape or t.dtype != q.dtype:
            raise LotError(f"{name} must have q's shape and dtype")
    if tuple(z.shape) != (H, r, d) or tuple(beta.shape) != (H, r):
        raise LotError("z must be [H,r,d] and beta [H,r]")
    f32 = torch.float32
    dq, dk, dv = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
    dz = torch.empty((H, r, d), device=q.device, dtype=f32)
    dbeta = torch.empty((H, r), device=q.device, dtype=f32)
    need = lot_bwd_workspace_bytes(B, H, n, d, r, code, int(iters))
    if ws is None:
        ws = torch.empty(max(need, 256), device=q.device, dtype=torch.uint8)
    st = lib().lot_attention_bwd(_dev(q, "q"), _dev(k, "k"), _dev(v, "v"), _dev(z, "z", f32), _dev(beta, "beta", f32),
                                 _dev(key_len, "key_len", torch.int32), _dev(dout, "dout", q.dtype),
                                 code, B, H, n, d, r, float(eps), int(iters),
                                 _dev(dq, "dq"), _dev(dk, "dk"), _dev(dv, "dv"), _dev(dz, "dz", f32),
                                 _dev(dbeta, "dbeta", f32), _dev(ws, "ws"), ws.numel(), _stream(stream))
    _check(st, "lot_attention_bwd")
    return dq, dk, dv, dz, dbeta, ws
