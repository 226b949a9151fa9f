"""Pins for the float64 CPU oracle: what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each states which passage or
which piece of mathematics it holds the oracle to.
"""
import itertools
import os

import numpy as np
import pytest
from scipy.special import logsumexp, softmax

from oracle import lot_oracle as O
from paper_2509_23436_b200 import synth

RNG = np.random.default_rng(12345)


def _rand_problem(n=12, d=5, r=4, seed=0, nk=None):
    g = np.random.default_rng(seed)
    nk = nk or n
    q = g.normal(size=(n, d)) / np.sqrt(d)
    k = g.normal(size=(nk, d)) / np.sqrt(d)
    v = g.normal(size=(nk, d))
    z = g.normal(size=(r, d))
    beta = softmax(g.normal(size=r))
    return q, k, v, z, beta


def _uniform(n):
    return np.full(n, 1.0 / n)


# ---------------------------------------------------------------- cost (Section "Method", display defining C^(1), C^(2))
def test_cost_is_plain_dot_product_no_scaling():
    q, _, _, z, _ = _rand_problem(n=7, d=6, r=3, seed=1)
    C = O.cost(q, z)
    assert C.shape == (7, 3)
    np.testing.assert_allclose(C, q @ z.T, rtol=0, atol=1e-14)          # library routine
    brute = np.array([[sum(q[i, c] * z[t, c] for c in range(6)) for t in range(3)] for i in range(7)])
    np.testing.assert_allclose(C, brute, rtol=0, atol=1e-14)
    # orientation: C[i,t] pairs token i with pivot t (a transposed operand would fail here)
    assert abs(C[2, 1] - float(q[2] @ z[1])) < 1e-14


# ---------------------------------------------------------------- Eq. (1)-(2): 2x2 closed forms
@pytest.mark.parametrize("C,eps", [
    (np.array([[1.0, 0.2], [0.3, 0.9]]), 0.5),
    (np.array([[0.1, 0.8], [0.7, -0.4]]), 0.25),       # anti-diagonal favoured: pins the sign of C
    (np.array([[2.0, -1.0], [0.0, 0.5]]), 0.4),
])
def test_sinkhorn_2x2_uniform_closed_form(C, eps):
    """n=r=2, uniform marginals: P11 = P22 = s/(2(1+s)), s = exp((c11+c22-c12-c21)/(2 eps))."""
    _, _, P = O.sinkhorn(C, [0.5, 0.5], [0.5, 0.5], eps, 5000)
    s = np.exp((C[0, 0] + C[1, 1] - C[0, 1] - C[1, 0]) / (2 * eps))
    p = 0.5 * s / (1 + s)
    np.testing.assert_allclose(P, [[p, 0.5 - p], [0.5 - p, p]], rtol=0, atol=1e-12)


def test_sinkhorn_2x2_general_marginals_quadratic():
    """Rows carry the token marginal m, columns the pivot masses beta (a swapped role fails).

    With P = [[p, m1-p], [b1-p, 1-m1-b1+p]] the stationarity condition is
    p (1-m1-b1+p) / ((m1-p)(b1-p)) = exp(Delta/eps): a quadratic in p."""
    C = np.array([[0.3, -0.2], [0.1, 0.6]]); eps = 0.3
    m = np.array([0.3, 0.7]); beta = np.array([0.6, 0.4])
    _, _, P = O.sinkhorn(C, beta, m, eps, 5000)
    K = np.exp((C[0, 0] + C[1, 1] - C[0, 1] - C[1, 0]) / eps)
    m1, b1 = m[0], beta[0]
    # p(1-m1-b1+p) = K (m1-p)(b1-p)
    a2 = 1 - K; a1 = (1 - m1 - b1) + K * (m1 + b1); a0 = -K * m1 * b1
    roots = np.roots([a2, a1, a0])
    ok = [x.real for x in roots if abs(x.imag) < 1e-12 and max(0, m1 + b1 - 1) <= x.real <= min(m1, b1)]
    assert len(ok) == 1
    p = ok[0]
    np.testing.assert_allclose(P, [[p, m1 - p], [b1 - p, 1 - m1 - b1 + p]], atol=1e-12)
    np.testing.assert_allclose(P.sum(1), m, atol=1e-13)
    np.testing.assert_allclose(P.sum(0), beta, atol=1e-12)


# ---------------------------------------------------------------- scaling form, any T
@pytest.mark.parametrize("iters", [0, 1, 3, 17])
def test_scaling_form_cross_ratios_and_token_marginal_any_T(iters):
    """Gamma = Diag(u) exp(C/eps) Diag(v): every 2x2 cross ratio of P equals that of exp(C/eps),
    whatever T; and the closing token update makes the token marginal exact."""
    q, _, _, z, beta = _rand_problem(n=9, d=4, r=5, seed=3)
    C = q @ z.T; eps = 0.2
    m = softmax(np.random.default_rng(5).normal(size=9))
    g, f, P = O.sinkhorn(C, beta, m, eps, iters)
    for (i, k_), (t, l) in itertools.product(itertools.combinations(range(9), 2), itertools.combinations(range(5), 2)):
        lhs = np.log(P[i, t] * P[k_, l] / (P[i, l] * P[k_, t]))
        rhs = (C[i, t] + C[k_, l] - C[i, l] - C[k_, t]) / eps
        assert abs(lhs - rhs) < 1e-9
    np.testing.assert_allclose(P.sum(1), m, rtol=0, atol=1e-14)
    np.testing.assert_allclose(P, np.exp((C + f[:, None] + g[None, :]) / eps), rtol=1e-12)


def test_iters0_and_iters1_from_library_softmax():
    """T=0: P = m_i softmax_t(C_i/eps).  T=1: g_t = eps (log beta_t - log sum_i m_i softmax_t(C_i/eps))."""
    q, _, _, z, beta = _rand_problem(n=10, d=4, r=6, seed=7)
    C = q @ z.T; eps = 0.15; m = _uniform(10)
    g0, _, P0 = O.sinkhorn(C, beta, m, eps, 0)
    np.testing.assert_allclose(g0, 0.0, atol=0)
    np.testing.assert_allclose(P0, m[:, None] * softmax(C / eps, axis=1), atol=1e-15)
    g1, _, P1 = O.sinkhorn(C, beta, m, eps, 1)
    col = (m[:, None] * softmax(C / eps, axis=1)).sum(0)
    np.testing.assert_allclose(g1, eps * (np.log(beta) - np.log(col)), atol=1e-13)
    np.testing.assert_allclose(P1, m[:, None] * softmax((C + g1) / eps, axis=1), atol=1e-15)


@pytest.mark.parametrize("iters", [1, 2, 5, 11])
def test_equal_T_matches_scaling_domain_matvec_iteration(iters):
    """Second statement of the same T-step map as matrix-vector scalings (u, v) on K = exp(C/eps)."""
    q, _, _, z, beta = _rand_problem(n=14, d=4, r=5, seed=11)
    C = q @ z.T; eps = 0.3; m = softmax(np.random.default_rng(2).normal(size=14))
    K = np.exp(C / eps)
    v = np.ones(5)
    for _ in range(iters):
        u = m / (K @ v)
        v = beta / (K.T @ u)
    u = m / (K @ v)
    g, f, P = O.sinkhorn(C, beta, m, eps, iters)
    np.testing.assert_allclose(P, u[:, None] * K * v[None, :], rtol=1e-11, atol=1e-15)
    np.testing.assert_allclose(g, eps * np.log(v), atol=1e-11)


def test_converged_plan_is_feasible_and_maximises_objective():
    """Eq. (1): the converged plan lies in U(beta, m) and no feasible move raises <C,G> + eps H(G)."""
    q, _, _, z, beta = _rand_problem(n=8, d=4, r=4, seed=13)
    C = q @ z.T; eps = 0.25; m = _uniform(8)
    _, _, P = O.sinkhorn(C, beta, m, eps, 20000)
    np.testing.assert_allclose(P.sum(1), m, atol=1e-12)
    np.testing.assert_allclose(P.sum(0), beta, atol=1e-10)

    def obj(G):
        return float((C * G).sum() - eps * (G * (np.log(G) - 1)).sum())
    base = obj(P)
    rng = np.random.default_rng(0)
    for _ in range(200):
        i, k_ = rng.choice(8, 2, replace=False); t, l = rng.choice(4, 2, replace=False)
        for delta in (1e-4, -1e-4):
            G = P.copy(); G[i, t] += delta; G[k_, l] += delta; G[i, l] -= delta; G[k_, t] -= delta
            if G.min() <= 0:
                continue
            assert obj(G) <= base + 1e-14


# ---------------------------------------------------------------- Eq. (3), rank paragraph, soft-clustering identity
def test_bruteforce_coupling_config1():
    """Config 1 run to convergence: Gamma 1 = mu, Gamma^T 1 = nu to 1e-9, rank <= r,
    Gamma = sum_t (1/beta_t) P1[:,t] (x) P2[:,t], and n Gamma V = factorised output."""
    x = synth.config(1); d = x.f64()
    q, k, v, z, beta = d["q"][0, 0], d["k"][0, 0], d["v"][0, 0], d["z"][0], d["beta"][0]
    n, r = 64, 8
    a = _uniform(n)
    res = O.head(q, k, v, z, beta, a, a, x.eps, 100000)
    G = O.coupling(res["P1"], res["P2"], beta)
    assert G.shape == (n, n) and G.min() > 0
    assert np.abs(G.sum(1) - 1 / n).max() < 1e-9
    assert np.abs(G.sum(0) - 1 / n).max() < 1e-9
    sv = np.linalg.svd(G, compute_uv=False)
    assert sv[r] / sv[0] < 1e-12 and sv[r - 1] / sv[0] > 1e-9
    outer = sum(np.outer(res["P1"][:, t], res["P2"][:, t]) / beta[t] for t in range(r))
    np.testing.assert_allclose(G, outer, rtol=1e-12, atol=1e-18)
    np.testing.assert_allclose(G, res["P1"] @ np.diag(1 / beta) @ res["P2"].T, rtol=1e-12, atol=1e-18)
    np.testing.assert_allclose(n * G @ v, res["out"], rtol=0, atol=1e-12)
    # doubly stochastic A = n Gamma; V = 1 gives 1; mass conservation
    A = n * G
    assert np.abs(A.sum(1) - 1).max() < 1e-7 and np.abs(A.sum(0) - 1).max() < 1e-7
    np.testing.assert_allclose(res["out"].mean(0), v.mean(0), atol=1e-9)


def test_finite_T_composition_still_has_exact_row_sums_and_rank():
    """At the configured finite T the query marginal is exact and rank <= r; the key marginal is not."""
    x = synth.config(1, iters=3); d = x.f64()
    q, k, v, z, beta = d["q"][0, 0], d["k"][0, 0], d["v"][0, 0], d["z"][0], d["beta"][0]
    a = _uniform(64)
    res = O.head(q, k, v, z, beta, a, a, x.eps, 3)
    G = O.coupling(res["P1"], res["P2"], beta)
    sv = np.linalg.svd(G, compute_uv=False)
    assert sv[8] / sv[0] < 1e-12
    np.testing.assert_allclose(64 * G @ v, res["out"], atol=1e-12)
    np.testing.assert_allclose(res["P1"].sum(1), a, atol=1e-15)
    np.testing.assert_allclose(res["P2"].sum(1), a, atol=1e-15)


# ---------------------------------------------------------------- Eq. (4) special cases
@pytest.mark.parametrize("iters,eps", [(0, 0.1), (4, 0.1), (9, 2.0)])
def test_r1_gives_key_mean_of_V(iters, eps):
    q, k, v, z, _ = _rand_problem(n=11, d=3, r=1, seed=17)
    b = softmax(np.random.default_rng(1).normal(size=11))
    res = O.head(q, k, v, z, [1.0], _uniform(11), b, eps, iters)
    np.testing.assert_allclose(res["out"], np.tile(b @ v, (11, 1)), atol=1e-13)


def test_identical_pivots_give_key_mean_of_V():
    q, k, v, z, beta = _rand_problem(n=10, d=3, r=4, seed=19)
    z = np.tile(z[:1], (4, 1))
    res = O.head(q, k, v, z, beta, _uniform(10), _uniform(10), 0.1, 200)
    np.testing.assert_allclose(res["out"], np.tile(v.mean(0), (10, 1)), atol=1e-10)


def test_large_eps_tends_to_product_coupling():
    q, k, v, z, beta = _rand_problem(n=10, d=3, r=4, seed=23)
    res = O.head(q, k, v, z, beta, _uniform(10), _uniform(10), 1e7, 50)
    np.testing.assert_allclose(res["out"], np.tile(v.mean(0), (10, 1)), atol=1e-5)
    G = O.coupling(res["P1"], res["P2"], beta)
    np.testing.assert_allclose(G, np.full((10, 10), 1e-2), atol=1e-7)


def test_rows_are_convex_weights_any_T():
    """out_i = sum_t w_it W'_t with w_i on the simplex: V = const c at convergence gives c;
    at any T each output lies in the convex hull scaled by the pivot-marginal ratio colmass_t/beta_t."""
    q, k, v, z, beta = _rand_problem(n=16, d=4, r=3, seed=29)
    a = _uniform(16)
    res = O.head(q, k, np.ones_like(v), z, beta, a, a, 0.2, 4)
    ratio = res["P2"].sum(0) / beta
    w = res["P1"] / a[:, None]
    np.testing.assert_allclose(w.sum(1), 1.0, atol=1e-14)
    np.testing.assert_allclose(res["out"][:, 0], w @ ratio, atol=1e-13)


# ---------------------------------------------------------------- metamorphic invariances (any T)
def _fwd(q, k, v, z, beta, eps=0.2, iters=4):
    n = q.shape[0]; nk = k.shape[0]
    return O.head(q, k, v, z, beta, _uniform(n), _uniform(nk), eps, iters)["out"]


def test_metamorphic_invariances():
    q, k, v, z, beta = _rand_problem(n=13, d=5, r=4, seed=31)
    base = _fwd(q, k, v, z, beta)
    rng = np.random.default_rng(3)
    pq, pk, pz = rng.permutation(13), rng.permutation(13), rng.permutation(4)
    np.testing.assert_allclose(_fwd(q[pq], k, v, z, beta), base[pq], atol=1e-13)
    np.testing.assert_allclose(_fwd(q, k[pk], v[pk], z, beta), base, atol=1e-13)
    np.testing.assert_allclose(_fwd(q, k, v, z[pz], beta[pz]), base, atol=1e-13)
    w = rng.normal(size=5)
    np.testing.assert_allclose(_fwd(q, k, v, z + w, beta), base, atol=1e-12)
    lam = 3.7
    np.testing.assert_allclose(_fwd(lam * q, lam * k, v, z, beta, eps=lam * 0.2), base, atol=1e-12)
    # a different V column does not change the weights: linear in V
    np.testing.assert_allclose(_fwd(q, k, 2 * v + 1, z, beta),
                               2 * base + _fwd(q, k, np.ones_like(v), z, beta), atol=1e-12)


# ---------------------------------------------------------------- padding mask reading
def test_key_mask_equals_truncated_problem():
    """Keys beyond key_len carry no mass: same result as the cross-attention problem with nk = L."""
    B, H, n, d, r, L = 1, 2, 12, 4, 3, 7
    g = np.random.default_rng(37)
    q = g.normal(size=(B, H, n, d)); k = g.normal(size=(B, H, n, d)); v = g.normal(size=(B, H, n, d))
    z = g.normal(size=(H, r, d)); beta = softmax(g.normal(size=(H, r)), axis=1)
    out = O.attention_fwd(q, k, v, z, beta, 0.3, 5, key_len=[L])
    k2, v2 = k.copy(), v.copy(); k2[:, :, L:] = 99.0; v2[:, :, L:] = -99.0
    np.testing.assert_allclose(O.attention_fwd(q, k2, v2, z, beta, 0.3, 5, key_len=[L]), out, atol=0)
    for h in range(H):
        C1 = q[0, h] @ z[h].T; C2 = k[0, h, :L] @ z[h].T
        _, _, P1 = O.sinkhorn(C1, beta[h], _uniform(n), 0.3, 5)
        _, _, P2 = O.sinkhorn(C2, beta[h], _uniform(L), 0.3, 5)
        ref = O.apply(P1, P2, beta[h], _uniform(n), v[0, h, :L])
        np.testing.assert_allclose(out[0, h], ref, atol=1e-13)
        assert np.abs((P1 / (1 / n)).sum(1) - 1).max() < 1e-13        # rows of A still sum to 1


def test_batched_wrapper_uses_per_head_pivots_shared_over_batch():
    B, H, n, d, r = 2, 3, 9, 4, 3
    g = np.random.default_rng(41)
    q = g.normal(size=(B, H, n, d)); k = g.normal(size=(B, H, n, d)); v = g.normal(size=(B, H, n, d))
    z = g.normal(size=(H, r, d)); beta = softmax(g.normal(size=(H, r)), axis=1)
    out, g1, g2, _ = O.attention_fwd(q, k, v, z, beta, 0.25, 6, return_potentials=True, threads=2)
    for b in range(B):
        for h in range(H):
            res = O.head(q[b, h], k[b, h], v[b, h], z[h], beta[h], _uniform(n), _uniform(n), 0.25, 6)
            np.testing.assert_allclose(out[b, h], res["out"], atol=0)
            np.testing.assert_allclose(g1[b, h], res["g1"], atol=0)
            np.testing.assert_allclose(g2[b, h], res["g2"], atol=0)


# ---------------------------------------------------------------- log-domain stability (config-5 style)
def test_peaked_costs_small_eps_stay_finite_and_converge():
    x = synth.make(1, 1, 256, 128, 16, seed=5001, eps=0.01, iters=50, qk="mixture")
    d = x.f64()
    C = O.cost(d["q"][0, 0], d["z"][0])
    assert np.abs(C / 0.01).max() > 200                      # naive exp(C/eps) would overflow float32
    g, f, P = O.sinkhorn(C, d["beta"][0], _uniform(256), 0.01, 20000)
    assert np.isfinite(g).all() and np.isfinite(f).all() and np.isfinite(P).all()
    np.testing.assert_allclose(P.sum(0), d["beta"][0], rtol=1e-6)
    np.testing.assert_allclose(P.sum(1), 1 / 256, rtol=1e-12)
    # agrees with a scipy logsumexp statement of one pivot update from the final f
    g_chk = 0.01 * (np.log(d["beta"][0]) - logsumexp((C + f[:, None]) / 0.01, axis=0))
    np.testing.assert_allclose(g, g_chk, atol=1e-8)


# ---------------------------------------------------------------- stored values written by tests/golden/make_golden.py
def test_golden_config1_matches_stored_oracle_values():
    path = os.path.join(os.path.dirname(__file__), "golden", "cfg1_oracle_out.txt")
    stored = np.loadtxt(path)
    x = synth.config(1); d = x.f64()
    out = O.attention_fwd(d["q"], d["k"], d["v"], d["z"], d["beta"], x.eps, x.iters)
    np.testing.assert_allclose(out[0, 0, ::8, :], stored, rtol=0, atol=1e-13)


# ================================================================ forward variants and the gradient
# (Section "Empirical measures and pivot": arbitrary weights; Appendix "Bidirectional scope": cross-attention;
#  Eq. (5): the [CLS] row; Section "Learning": back-propagation through the two solves and the composition)
from oracle import lot_oracle_grad as OG


def _rand_head(rng, nq, nk, d, dv, r):
    q, k, v, z = rng.normal(size=(nq, d)) * 0.6, rng.normal(size=(nk, d)) * 0.6, rng.normal(size=(nk, dv)), rng.normal(size=(r, d))
    beta = rng.random(r) + 0.2; beta /= beta.sum()
    a = rng.random(nq) + 0.1; a /= a.sum()
    b = rng.random(nk) + 0.1; b /= b.sum()
    return q, k, v, z, beta, a, b


def test_warm_start_continues_the_iteration():
    """T1 iterations, then T2 more from the exported pivot potential, are T1 + T2 iterations: the potential is the
    whole state between two passes."""
    rng = np.random.default_rng(3)
    C = rng.normal(size=(37, 5)); beta = np.full(5, 0.2); m = np.full(37, 1 / 37)
    g_a, _, _ = O.sinkhorn(C, beta, m, 0.3, 4)
    g_b, f_b, P_b = O.sinkhorn_from(C, beta, m, 0.3, 7, g_a)
    g_c, f_c, P_c = O.sinkhorn(C, beta, m, 0.3, 11)
    np.testing.assert_allclose(g_b, g_c, rtol=0, atol=1e-13)
    np.testing.assert_allclose(P_b, P_c, rtol=0, atol=1e-15)
    # and a start at the fixed point stays there
    g_inf, _, P_inf = O.sinkhorn(C, beta, m, 0.3, 3000)
    g_again, _, P_again = O.sinkhorn_from(C, beta, m, 0.3, 1, g_inf)
    np.testing.assert_allclose(P_again, P_inf, rtol=0, atol=1e-14)


def test_cross_attention_and_general_marginals_by_brute_force():
    """nq != nk with arbitrary weights: at convergence the explicit nq x nk coupling has row sums a and column sums b
    to 1e-9 and rank <= r; the factorised output equals Diag(1/a) Gamma V; equal sizes and uniform weights reduce to
    the square routine."""
    rng = np.random.default_rng(11)
    q, k, v, z, beta, a, b = _rand_head(rng, 23, 31, 6, 4, 5)
    h = O.head_x(q, k, v, z, beta, a, b, 0.4, 5000)
    G = O.coupling(h["P1"], h["P2"], beta)
    assert np.abs(G.sum(1) - a).max() < 1e-9 and np.abs(G.sum(0) - b).max() < 1e-9
    sv = np.linalg.svd(G, compute_uv=False)
    assert sv[5] / sv[0] < 1e-12
    np.testing.assert_allclose(h["out"], (G / a[:, None]) @ v, atol=1e-12)
    # a key with zero weight is out of the problem: the same as deleting it
    b0 = b.copy(); b0[7] = 0; b0 /= b0.sum()
    h0 = O.head_x(q, k, v, z, beta, a, b0, 0.4, 50)
    keep = np.arange(31) != 7
    h1 = O.head_x(q, k[keep], v[keep], z, beta, a, b0[keep], 0.4, 50)
    np.testing.assert_allclose(h0["out"], h1["out"], atol=1e-13)
    # square and uniform: the routine the configurations use
    n = 19
    q2, k2, v2 = rng.normal(size=(n, 6)), rng.normal(size=(n, 6)), rng.normal(size=(n, 6))
    u = np.full(n, 1 / n)
    np.testing.assert_allclose(O.head_x(q2, k2, v2, z, beta, u, u, 0.4, 9)["out"], O.head(q2, k2, v2, z, beta, u, u, 0.4, 9)["out"],
                               atol=1e-14)


def test_cls_row_is_a_library_softmax_and_the_rest_is_the_smaller_problem():
    from scipy.special import softmax
    rng = np.random.default_rng(5)
    n, d, r, tau = 17, 8, 4, 1.7
    q, k, v, z = rng.normal(size=(n, d)), rng.normal(size=(n, d)), rng.normal(size=(n, d)), rng.normal(size=(r, d))
    beta = np.array([0.1, 0.2, 0.3, 0.4])
    out = O.head_cls(q, k, v, z, beta, 0.5, 12, tau)
    np.testing.assert_allclose(out[0], softmax(tau * (k @ q[0])) @ v, atol=1e-13)
    u = np.full(n - 1, 1 / (n - 1))
    np.testing.assert_allclose(out[1:], O.head(q[1:], k[1:], v[1:], z, beta, u, u, 0.5, 12)["out"], atol=1e-13)
    # a constant value vector comes back unchanged in every row: each row of the implied attention matrix sums to 1
    ones = O.head_cls(q, k, np.ones((n, 3)), z, beta, 0.5, 400, tau)
    np.testing.assert_allclose(ones, 1.0, atol=1e-9)
    # key mask: the softmax row and the transport problem both leave the padded keys out
    outm = O.head_cls(q, k, v, z, beta, 0.5, 12, tau, key_len=11)
    np.testing.assert_allclose(outm[0], softmax(tau * (k[:11] @ q[0])) @ v[:11], atol=1e-13)


def test_gradient_forward_agrees_with_the_c_oracle():
    rng = np.random.default_rng(2)
    q, k, v, z, beta, a, b = _rand_head(rng, 11, 13, 5, 3, 4)
    g10, g20 = rng.normal(size=4) * 0.1, rng.normal(size=4) * 0.1
    fw = OG.head_forward(q, k, v, z, beta, a, b, 0.35, 6, g10, g20)
    ref = O.head_x(q, k, v, z, beta, a, b, 0.35, 6, g10, g20)
    np.testing.assert_allclose(fw["out"], ref["out"], atol=1e-13)
    np.testing.assert_allclose(fw["g1"], ref["g1"], atol=1e-13)
    np.testing.assert_allclose(fw["P2"], ref["P2"], atol=1e-14)


@pytest.mark.parametrize("iters", [0, 1, 5])
def test_gradient_matches_central_differences(iters):
    """Every input's gradient against central finite differences of the C oracle's forward (a dropped term, a wrong
    sign or a transposed factor in the reverse sweep fails here)."""
    rng = np.random.default_rng(7 + iters)
    q, k, v, z, beta, a, b = _rand_head(rng, 7, 9, 4, 3, 3)
    dout = rng.normal(size=(7, 3))
    eps = 0.45
    g10, g20 = rng.normal(size=3) * 0.2, rng.normal(size=3) * 0.2
    grads = OG.head_backward(OG.head_forward(q, k, v, z, beta, a, b, eps, iters, g10, g20), dout)

    def loss(**kw):
        args = dict(q=q, k=k, v=v, z=z, beta=beta, g1_0=g10, g2_0=g20)
        args.update(kw)
        return float(np.sum(O.head_x(args["q"], args["k"], args["v"], args["z"], args["beta"], a, b, eps, iters,
                                     args["g1_0"], args["g2_0"])["out"] * dout))

    h = 1e-6
    for name, x0 in (("q", q), ("k", k), ("v", v), ("z", z), ("beta", beta), ("g1_0", g10), ("g2_0", g20)):
        fd = np.zeros_like(x0)
        it = np.nditer(x0, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            xp, xm = x0.copy(), x0.copy()
            xp[idx] += h; xm[idx] -= h
            fd[idx] = (loss(**{name: xp}) - loss(**{name: xm})) / (2 * h)
        got = grads["d" + name]
        assert np.abs(got - fd).max() <= 2e-6 * max(1.0, np.abs(fd).max()), name


def test_gradient_at_convergence_forgets_the_starting_potential():
    """At the fixed point the result no longer depends on where the iteration started: the gradient with respect to
    the starting potentials vanishes, and the other gradients agree for two different starts."""
    rng = np.random.default_rng(19)
    q, k, v, z, beta, a, b = _rand_head(rng, 8, 8, 4, 3, 3)
    dout = rng.normal(size=(8, 3))
    g_a = OG.head_backward(OG.head_forward(q, k, v, z, beta, a, b, 0.5, 400), dout)
    g_b = OG.head_backward(OG.head_forward(q, k, v, z, beta, a, b, 0.5, 400, rng.normal(size=3), rng.normal(size=3)), dout)
    assert np.abs(g_a["dg1_0"]).max() < 1e-12 and np.abs(g_b["dg2_0"]).max() < 1e-12
    for name in ("dq", "dk", "dv", "dz", "dbeta"):
        np.testing.assert_allclose(g_a[name], g_b[name], atol=1e-10)
