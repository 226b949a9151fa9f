"""Float64 gradient of the LOT attention head, by reverse differentiation of the unrolled iteration.
TEST INFRASTRUCTURE (same rules as lot_oracle.py): plain numpy, no blocking, no shortcuts.

Section "Learning" trains Z, the pivot masses and the projections by back-propagating through the two shared-eps
Sinkhorn problems, Eq. (1)-(2), and the glued composition, Eq. (3)-(4).  The forward map differentiated here is the
one lot_oracle.c states (its iteration order is the documented reading: g0 given or zero, `iters` times a token
update followed by a pivot update, one closing token update):

    C = X Z^T;   repeat: f = eps (log m - LSE_t((C + g)/eps)),  g = eps (log beta - LSE_i((C + f)/eps));
    closing f;   P = exp((C + f + g)/eps);      out = Diag(1/a) P1 Diag(1/beta) P2^T V.

`head_forward` recomputes that map in numpy and keeps what the reverse sweep needs; `head_backward` returns the
gradients of sum(out * dout) with respect to q, k, v, z, beta (beta taken as free positive numbers, no simplex
constraint: a softmax parametrisation is the caller's chain rule) and the starting potentials.
"""
from __future__ import annotations

import numpy as np


def _lse(x, axis):
    m = np.max(x, axis=axis, keepdims=True)
    return np.squeeze(m, axis) + np.log(np.sum(np.exp(x - m), axis=axis))


def _solve_forward(C, beta, m, eps, iters, g0):
    """The iteration of lot_oracle_sinkhorn_from for strictly positive marginals; returns (g, f, P, trace)."""
    g = np.zeros(C.shape[1]) if g0 is None else np.asarray(g0, dtype=np.float64).copy()
    trace = []
    for _ in range(iters):
        f = eps * (np.log(m) - _lse((C + g[None, :]) / eps, 1))
        trace.append((g.copy(), f.copy()))
        g = eps * (np.log(beta) - _lse((C + f[:, None]) / eps, 0))
    f = eps * (np.log(m) - _lse((C + g[None, :]) / eps, 1))
    P = np.exp((C + f[:, None] + g[None, :]) / eps)
    return g, f, P, trace


def _solve_backward(C, beta, m, eps, g, P, trace, dP):
    """Reverse sweep of _solve_forward: gradients with respect to C, beta and the starting potential."""
    # P = m_i softmax_t(y), y = (C + g)/eps  (closing token update folded in)
    sm = P / m[:, None]
    dsm = dP * m[:, None]
    dy = sm * (dsm - np.sum(dsm * sm, axis=1, keepdims=True))
    dC = dy / eps
    dg = np.sum(dy, axis=0) / eps
    dbeta = np.zeros_like(beta)
    for g_prev, f in reversed(trace):
        # g = eps (log beta - LSE_i((C + f)/eps)): Q = softmax over tokens, per pivot
        x = (C + f[:, None]) / eps
        Q = np.exp(x - _lse(x, 0)[None, :])
        dbeta += eps * dg / beta
        dC -= Q * dg[None, :]
        df = -Q @ dg
        # f = eps (log m - LSE_t((C + g_prev)/eps)): R = softmax over pivots, per token
        y = (C + g_prev[None, :]) / eps
        R = np.exp(y - _lse(y, 1)[:, None])
        dC -= R * df[:, None]
        dg = -R.T @ df
    return dC, dbeta, dg


def head_forward(q, k, v, z, beta, a, b, eps, iters, g1_0=None, g2_0=None):
    q, k, v, z, beta, a, b = (np.asarray(t, dtype=np.float64) for t in (q, k, v, z, beta, a, b))
    C1, C2 = q @ z.T, k @ z.T
    g1, _, P1, tr1 = _solve_forward(C1, beta, a, eps, iters, g1_0)
    g2, _, P2, tr2 = _solve_forward(C2, beta, b, eps, iters, g2_0)
    W = P2.T @ v
    out = (P1 / a[:, None]) @ (W / beta[:, None])
    return dict(out=out, g1=g1, g2=g2, P1=P1, P2=P2, C1=C1, C2=C2, W=W, tr1=tr1, tr2=tr2,
                q=q, k=k, v=v, z=z, beta=beta, a=a, b=b, eps=eps)


def head_backward(fw, dout):
    """Gradients of sum(out * dout): dict(dq, dk, dv, dz, dbeta, dg1_0, dg2_0)."""
    q, k, v, z, beta, a, b, eps = (fw[n] for n in ("q", "k", "v", "z", "beta", "a", "b", "eps"))
    P1, P2, W = fw["P1"], fw["P2"], fw["W"]
    dout = np.asarray(dout, dtype=np.float64)
    S1 = P1 / a[:, None]
    Wp = W / beta[:, None]
    dS1 = dout @ Wp.T
    dWp = S1.T @ dout
    dW = dWp / beta[:, None]
    dbeta = -np.sum(dWp * W, axis=1) / beta ** 2
    dP2 = v @ dW.T
    dv = P2 @ dW
    dP1 = dS1 / a[:, None]
    dC1, db1, dg10 = _solve_backward(fw["C1"], beta, a, eps, fw["g1"], P1, fw["tr1"], dP1)
    dC2, db2, dg20 = _solve_backward(fw["C2"], beta, b, eps, fw["g2"], P2, fw["tr2"], dP2)
    return dict(dq=dC1 @ z, dk=dC2 @ z, dv=dv, dz=dC1.T @ q + dC2.T @ k, dbeta=dbeta + db1 + db2,
                dg1_0=dg10, dg2_0=dg20)
