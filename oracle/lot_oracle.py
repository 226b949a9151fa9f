"""ctypes access to the float64 CPU oracle (lot_oracle.c).  TEST INFRASTRUCTURE.

Only tests, the smoke check and the bench's CPU-baseline / reference arm may
import this module.  It knows nothing about the CUDA library.  Every function
takes numpy arrays (any float dtype; they are upcast to float64, so a caller
that wants "bf16 inputs" passes the bf16-rounded values) and returns float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lot_oracle.c")
_LIB = os.path.join(_HERE, "liblot_oracle.so")
_lib = None

_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(ctypes.c_int)


def build(force: bool = False) -> str:
    """Compile lot_oracle.c into liblot_oracle.so beside it (gcc, -O2, OpenMP)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-fno-fast-math",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.lot_oracle_cost.argtypes = [_dp, _dp, ctypes.c_int, ctypes.c_int, ctypes.c_int, _dp]
        lib.lot_oracle_cost.restype = None
        lib.lot_oracle_sinkhorn.argtypes = [_dp, _dp, _dp, ctypes.c_int, ctypes.c_int,
                                            ctypes.c_double, ctypes.c_int, _dp, _dp, _dp]
        lib.lot_oracle_sinkhorn.restype = None
        lib.lot_oracle_coupling.argtypes = [_dp, _dp, _dp, ctypes.c_int, ctypes.c_int, ctypes.c_int, _dp]
        lib.lot_oracle_coupling.restype = None
        lib.lot_oracle_apply.argtypes = [_dp, _dp, _dp, _dp, _dp, ctypes.c_int, ctypes.c_int,
                                         ctypes.c_int, ctypes.c_int, _dp]
        lib.lot_oracle_apply.restype = None
        lib.lot_oracle_head.argtypes = [_dp] * 7 + [ctypes.c_int] * 3 + [ctypes.c_double, ctypes.c_int] + [_dp] * 5
        lib.lot_oracle_head.restype = None
        lib.lot_oracle_sinkhorn_from.argtypes = [_dp, _dp, _dp, ctypes.c_int, ctypes.c_int,
                                                 ctypes.c_double, ctypes.c_int, _dp, _dp, _dp, _dp]
        lib.lot_oracle_sinkhorn_from.restype = None
        lib.lot_oracle_head_x.argtypes = ([_dp] * 7 + [ctypes.c_int] * 5 + [ctypes.c_double, ctypes.c_int] + [_dp] * 7)
        lib.lot_oracle_head_x.restype = None
        lib.lot_oracle_cls_row.argtypes = [_dp, _dp, _dp, ctypes.c_char_p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                           ctypes.c_double, _dp]
        lib.lot_oracle_cls_row.restype = None
        lib.lot_oracle_attention_fwd.argtypes = ([_dp] * 5 + [_ip] + [ctypes.c_int] * 5 +
                                                 [ctypes.c_double, ctypes.c_int] + [_dp] * 3 + [ctypes.c_int])
        lib.lot_oracle_attention_fwd.restype = ctypes.c_int
        _lib = lib
    return _lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _p(a):
    return None if a is None else a.ctypes.data_as(_dp)


def cost(x, z) -> np.ndarray:
    """C[i,t] = <x_i, z_t>; x [n,d], z [r,d] -> [n,r]."""
    x, z = _f64(x), _f64(z)
    n, d = x.shape
    r = z.shape[0]
    assert z.shape[1] == d
    C = np.empty((n, r), dtype=np.float64)
    _load().lot_oracle_cost(_p(x), _p(z), n, d, r, _p(C))
    return C


def sinkhorn(C, beta, m, eps: float, iters: int):
    """Entropic plan in U(beta, m) for similarity C [n,r]; returns (g [r], f [n], P [n,r])."""
    C, beta, m = _f64(C), _f64(beta), _f64(m)
    n, r = C.shape
    assert beta.shape == (r,) and m.shape == (n,)
    g = np.empty(r)
    f = np.empty(n)
    P = np.empty((n, r))
    _load().lot_oracle_sinkhorn(_p(C), _p(beta), _p(m), n, r, float(eps), int(iters), _p(g), _p(f), _p(P))
    return g, f, P


def sinkhorn_from(C, beta, m, eps: float, iters: int, g0):
    """sinkhorn() started from the pivot potential g0 [r] instead of zeros."""
    C, beta, m, g0 = _f64(C), _f64(beta), _f64(m), _f64(g0)
    n, r = C.shape
    assert beta.shape == (r,) and m.shape == (n,) and g0.shape == (r,)
    g, f, P = np.empty(r), np.empty(n), np.empty((n, r))
    _load().lot_oracle_sinkhorn_from(_p(C), _p(beta), _p(m), n, r, float(eps), int(iters), _p(g0), _p(g), _p(f), _p(P))
    return g, f, P


def head_x(q, k, v, z, beta, a, b, eps: float, iters: int, g1_0=None, g2_0=None):
    """One head with nq queries, nk keys, marginals a [nq], b [nk], optional starting potentials.
    Returns dict(out [nq,dv], g1, g2, P1 [nq,r], P2 [nk,r])."""
    q, k, v, z, beta, a, b = map(_f64, (q, k, v, z, beta, a, b))
    nq, d = q.shape
    nk, dv = v.shape
    r = z.shape[0]
    assert k.shape == (nk, d) and z.shape == (r, d) and a.shape == (nq,) and b.shape == (nk,)
    g10 = None if g1_0 is None else _f64(g1_0)
    g20 = None if g2_0 is None else _f64(g2_0)
    out = np.empty((nq, dv))
    g1, g2 = np.empty(r), np.empty(r)
    P1, P2 = np.empty((nq, r)), np.empty((nk, r))
    _load().lot_oracle_head_x(_p(q), _p(k), _p(v), _p(z), _p(beta), _p(a), _p(b), nq, nk, d, dv, r,
                              float(eps), int(iters), _p(g10), _p(g20), _p(out), _p(g1), _p(g2), _p(P1), _p(P2))
    return dict(out=out, g1=g1, g2=g2, P1=P1, P2=P2)


def cls_row(q0, k, v, tau: float, alive=None) -> np.ndarray:
    """Eq. (5): softmax_j(tau <q0, k_j>) over the (alive) keys, applied to v; returns [dv]."""
    q0, k, v = map(_f64, (q0, k, v))
    nk, d = k.shape
    dv = v.shape[1]
    mask = None if alive is None else np.ascontiguousarray(np.asarray(alive, dtype=np.uint8)).tobytes()
    out0 = np.empty(dv)
    _load().lot_oracle_cls_row(_p(q0), _p(k), _p(v), mask, nk, d, dv, float(tau), _p(out0))
    return out0


def head_cls(q, k, v, z, beta, eps: float, iters: int, tau: float, key_len=None):
    """One head with the [CLS] treatment of Eq. (5): token 0 is [CLS]; its row is a softmax over all (valid) keys,
    every other row follows the doubly stochastic rule among the remaining tokens (queries and keys 1..n-1, uniform
    marginals over them).  Returns out [n,dv]."""
    q, k, v = map(_f64, (q, k, v))
    n = q.shape[0]
    nk = k.shape[0] if key_len is None else int(key_len)
    out = np.zeros((n, v.shape[1]))
    alive = np.zeros(k.shape[0], dtype=np.uint8)
    alive[:nk] = 1
    out[0] = cls_row(q[0], k, v, tau, alive)
    if n > 1 and nk > 1:
        a = np.full(n - 1, 1.0 / (n - 1))
        b = np.zeros(k.shape[0] - 1)
        b[:nk - 1] = 1.0 / (nk - 1)
        out[1:] = head_x(q[1:], k[1:], v[1:], z, beta, a, b, eps, iters)["out"]
    return out


def coupling(P1, P2, beta) -> np.ndarray:
    """Glued coupling P1 Diag(1/beta) P2^T, explicit [nq,nk] (brute force)."""
    P1, P2, beta = _f64(P1), _f64(P2), _f64(beta)
    nq, r = P1.shape
    nk = P2.shape[0]
    G = np.empty((nq, nk))
    _load().lot_oracle_coupling(_p(P1), _p(P2), _p(beta), nq, nk, r, _p(G))
    return G


def apply(P1, P2, beta, a, V) -> np.ndarray:
    """Factorised head output: (P1 (Diag(1/beta) (P2^T V)))_i / a_i."""
    P1, P2, beta, a, V = _f64(P1), _f64(P2), _f64(beta), _f64(a), _f64(V)
    nq, r = P1.shape
    nk, dv = V.shape
    out = np.empty((nq, dv))
    _load().lot_oracle_apply(_p(P1), _p(P2), _p(beta), _p(a), _p(V), nq, nk, r, dv, _p(out))
    return out


def head(q, k, v, z, beta, a, b, eps: float, iters: int):
    """One head.  Returns dict(out, g1, g2, P1, P2)."""
    q, k, v, z, beta, a, b = map(_f64, (q, k, v, z, beta, a, b))
    n, d = q.shape
    r = z.shape[0]
    out = np.empty((n, d))
    g1, g2 = np.empty(r), np.empty(r)
    P1, P2 = np.empty((n, r)), np.empty((n, r))
    _load().lot_oracle_head(_p(q), _p(k), _p(v), _p(z), _p(beta), _p(a), _p(b), n, d, r,
                            float(eps), int(iters), _p(out), _p(g1), _p(g2), _p(P1), _p(P2))
    return dict(out=out, g1=g1, g2=g2, P1=P1, P2=P2)


def attention_fwd(q, k, v, z, beta, eps: float, iters: int, key_len=None, threads: int = 0,
                  return_potentials: bool = False):
    """All heads.  q,k,v [B,H,n,d]; z [H,r,d]; beta [H,r]; key_len [B] ints or None."""
    q, k, v, z, beta = map(_f64, (q, k, v, z, beta))
    B, H, n, d = q.shape
    r = z.shape[1]
    assert z.shape == (H, r, d) and beta.shape == (H, r)
    out = np.empty_like(q)
    g1 = np.empty((B, H, r))
    g2 = np.empty((B, H, r))
    kl = None
    if key_len is not None:
        kl = np.ascontiguousarray(np.asarray(key_len, dtype=np.int32))
        assert kl.shape == (B,)
    used = _load().lot_oracle_attention_fwd(
        _p(q), _p(k), _p(v), _p(z), _p(beta),
        None if kl is None else kl.ctypes.data_as(_ip),
        B, H, n, d, r, float(eps), int(iters), _p(out), _p(g1), _p(g2), int(threads))
    if return_potentials:
        return out, g1, g2, used
    return out


if __name__ == "__main__":
    print(build(force=True))
