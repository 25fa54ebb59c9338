"""Pins for the fp64 oracle: every check here compares the oracle with something that is NOT
the oracle -- a closed form, a limit, an invariant of the mathematics, an independent solver,
a library routine, or values the paper prints.  All CPU.

Coverage map (what a mistake would break):
  rank-1 closed form ........ dropped term / wrong sign in K, transposed operand (x != y),
                              u-then-v order, <P,C>
  large-eps limit ........... scaling of the exponent by eps
  scaling == log ............ the log-domain formulas (sign of C, eps factors, log a term)
  protocol == centralized ... Algorithm 1 block indexing, Allgather, column-block access (Prop. 1)
  fixed point / duality ..... marginals, objective values, gauge/shift invariance
  half-step invariants ...... each pass alone; dual ascent; Hilbert-metric contraction
  2x2 quadratic ............. converged plan against an explicit root
  Newton on the dual ........ converged plan and cost against an independent convex solve
  scipy logsumexp ........... LSE rows vs columns (a transposed LSE fails here)
"""
import itertools
import os

import numpy as np
import pytest
from scipy.special import logsumexp

import oracle
from paper_2502_07021_b200 import workloads

K_, C_ = oracle.KIND_KERNEL, oracle.KIND_COST
SC, LG = oracle.DOMAIN_SCALING, oracle.DOMAIN_LOG


def dyadic_additive(n, seed):
    """C_il = x_i + y_l with x, y on a 1/64 grid, so C is exact in fp32 and K is exactly rank one."""
    rng = np.random.default_rng(seed)
    x = rng.integers(0, 64, n) / 64.0
    y = rng.integers(0, 64, n) / 64.0
    C = (x[:, None] + y[None, :]).astype(np.float32)
    assert np.array_equal(C.astype(np.float64), x[:, None] + y[None, :])
    return C, x, y


def dirichlet_pair(n, seed):
    a = workloads.dirichlet1(np.random.default_rng(seed), n).astype(np.float32)
    b = workloads.dirichlet1(np.random.default_rng(seed + 1), n).astype(np.float32)
    return a, b


def random_cost(n, seed, scale=1.0):
    rng = np.random.default_rng(seed)
    return (scale * rng.random((n, n))).astype(np.float32)


def hilbert(x, y):
    r = np.asarray(x) / np.asarray(y)
    return float(np.log(r.max()) - np.log(r.min()))


# ------------------------------------------------------------------ P1 rank-1 closed form

@pytest.mark.parametrize("n,eps", [(5, 0.3), (37, 0.11), (64, 1.0)])
def test_rank1_closed_form_scaling(n, eps):
    C, x, y = dyadic_additive(n, 11 + n)
    a, b = dirichlet_pair(n, 100 + n)
    a64, b64 = a.astype(np.float64), b.astype(np.float64)
    p, q = np.exp(-x / eps), np.exp(-y / eps)
    s = q.sum()
    # one full iteration from u = v = 1:  u_i = a_i/(p_i s),  v_l = b_l / (q_l * sum_i p_i u_i)
    u, v = oracle.sinkhorn_scaling(C, C_, eps, a, b, 1)
    u_ref = a64 / (p * s)
    v_ref = b64 / (q * (p * u_ref).sum())
    np.testing.assert_allclose(u, u_ref, rtol=1e-13)
    np.testing.assert_allclose(v, v_ref, rtol=1e-13)
    P = oracle.plan(C, C_, eps, SC, u, v)
    # P = a b^T / mass(a): rows scaled so that columns are exact after the v update
    np.testing.assert_allclose(P, np.outer(a64, b64) / a64.sum(), rtol=1e-12)
    obj = oracle.objectives(C, C_, eps, SC, u, v, C)
    cost_ref = (np.outer(a64, b64) / a64.sum() * (x[:, None] + y[None, :])).sum()
    assert obj["cost"] == pytest.approx(cost_ref, rel=1e-12)
    # with a stored kernel instead of a stored cost: same iterates up to fp32 rounding of K
    K32 = np.exp(-(x[:, None] + y[None, :]) / eps).astype(np.float32)
    uk, vk = oracle.sinkhorn_scaling(K32, K_, eps, a, b, 1)
    np.testing.assert_allclose(uk, u_ref, rtol=5e-7)
    np.testing.assert_allclose(vk, v_ref, rtol=5e-7)
    # the column error is zero from iteration 1 on, the row error too when masses agree
    e = oracle.marginal_errors(C, C_, eps, SC, u, v, a, b)
    assert e["col_l1"] < 1e-14
    mass_gap = abs(a64.sum() - b64.sum())
    assert e["row_l1"] <= mass_gap + 1e-14


@pytest.mark.parametrize("n,eps", [(6, 0.25), (33, 0.07)])
def test_rank1_closed_form_log(n, eps):
    C, x, y = dyadic_additive(n, 21 + n)
    a, b = dirichlet_pair(n, 200 + n)
    a64, b64 = a.astype(np.float64), b.astype(np.float64)
    f, g = oracle.sinkhorn_log(C, eps, a, b, 1)
    # f_i = eps log a_i + x_i - eps log sum_l exp(-y_l/eps)   (from g = 0)
    s = np.exp(-y / eps).sum()
    f_ref = eps * np.log(a64) + x - eps * np.log(s)
    # g_l = eps log b_l + y_l - eps log sum_i exp((f_i - x_i)/eps) = eps log b_l + y_l - eps log(sum a / s)
    g_ref = eps * np.log(b64) + y - eps * np.log(a64.sum() / s)
    np.testing.assert_allclose(f, f_ref, rtol=0, atol=1e-13)
    np.testing.assert_allclose(g, g_ref, rtol=0, atol=1e-13)
    P = oracle.plan(C, C_, eps, LG, f, g)
    np.testing.assert_allclose(P, np.outer(a64, b64) / a64.sum(), rtol=1e-11)


def test_rank1_nonsymmetric_catches_transpose():
    # x != y makes K non-symmetric: using K^T in the row pass would give p and q swapped
    n, eps = 9, 0.2
    C, x, y = dyadic_additive(n, 5)
    assert not np.allclose(C, C.T)
    a, b = dirichlet_pair(n, 55)
    v0 = np.random.default_rng(3).random(n) + 0.5
    u, qv = oracle.row_pass(C, C_, eps, a, v0)
    np.testing.assert_allclose(qv, np.exp(-x / eps) * (np.exp(-y / eps) * v0).sum(), rtol=1e-13)
    v, r = oracle.col_pass(C, C_, eps, b, u)
    np.testing.assert_allclose(r, np.exp(-y / eps) * (np.exp(-x / eps) * u).sum(), rtol=1e-13)
    np.testing.assert_allclose(u * qv, a, rtol=1e-15)
    np.testing.assert_allclose(v * r, b, rtol=1e-15)


# ------------------------------------------------------------------ relaxed (damped) update

def test_damped_update_closed_form_fixed_point_and_eta_one():
    n, eps, eta = 21, 0.3, 0.4
    C, x, y = dyadic_additive(n, 77)
    a, b = dirichlet_pair(n, 78)
    a64, b64 = a.astype(np.float64), b.astype(np.float64)
    p, q = np.exp(-x / eps), np.exp(-y / eps)
    # one relaxed iteration on the rank-one kernel, from u = v = 1
    u, v = oracle.sinkhorn_damped(C, C_, eps, a, b, eta, 1)
    u_ref = (1 - eta) + eta * a64 / (p * q.sum())
    v_ref = (1 - eta) + eta * b64 / (q * (p * u_ref).sum())
    np.testing.assert_allclose(u, u_ref, rtol=1e-13)
    np.testing.assert_allclose(v, v_ref, rtol=1e-13)
    # eta = 1 is the plain iteration, bit for bit
    Cr = random_cost(n, 79)
    u1, v1 = oracle.sinkhorn_damped(Cr, C_, eps, a, b, 1.0, 7)
    u0, v0 = oracle.sinkhorn_scaling(Cr, C_, eps, a, b, 7)
    assert np.array_equal(u1, u0) and np.array_equal(v1, v0)
    # the relaxed map has the same fixed point: same plan as plain Sinkhorn
    ud, vd = oracle.sinkhorn_damped(Cr, C_, eps, a, b, eta, 4000)
    us, vs = oracle.sinkhorn_scaling(Cr, C_, eps, a, b, 4000)
    np.testing.assert_allclose(oracle.plan(Cr, C_, eps, SC, ud, vd), oracle.plan(Cr, C_, eps, SC, us, vs), rtol=1e-9)
    # and it really is a convex combination of the old value and the plain update
    u_half, _ = oracle.sinkhorn_damped(Cr, C_, eps, a, b, 0.5, 1)
    u_full, _ = oracle.sinkhorn_scaling(Cr, C_, eps, a, b, 1)
    np.testing.assert_allclose(u_half, 0.5 + 0.5 * u_full, rtol=1e-15)


# ------------------------------------------------------------------ P2 large-eps limit

def test_large_eps_limit():
    n = 24
    C = random_cost(n, 31)
    a, b = dirichlet_pair(n, 32)
    ab = np.outer(a.astype(np.float64), b.astype(np.float64))
    prev = None
    for eps in (1e2, 1e4, 1e6):
        u, v = oracle.sinkhorn_scaling(C, C_, eps, a, b, 50)
        P = oracle.plan(C, C_, eps, SC, u, v)
        dev = np.abs(P - ab).max() / ab.max()
        assert dev < 3.0 * float(C.max()) / eps
        f, g = oracle.sinkhorn_log(C, eps, a, b, 50)
        Pl = oracle.plan(C, C_, eps, LG, f, g)
        assert np.abs(Pl - ab).max() / ab.max() < 3.0 * float(C.max()) / eps
        if prev is not None:
            assert dev < prev / 50       # first order in 1/eps
        prev = dev


# ------------------------------------------------------------------ P3 scaling == log

@pytest.mark.parametrize("n,eps,seed", [(17, 0.05, 1), (40, 0.02, 2), (8, 1.0, 3)])
def test_domain_equivalence_every_iteration(n, eps, seed):
    C = random_cost(n, seed)
    a, b = dirichlet_pair(n, 40 + seed)
    for t in (1, 2, 5, 13):
        u, v = oracle.sinkhorn_scaling(C, C_, eps, a, b, t)
        f, g = oracle.sinkhorn_log(C, eps, a, b, t)
        np.testing.assert_allclose(f, eps * np.log(u), rtol=0, atol=1e-12)
        np.testing.assert_allclose(g, eps * np.log(v), rtol=0, atol=1e-12)


def test_log_domain_survives_underflow():
    # exp(-C/eps) underflows fp64 for most entries here, the log form must not care
    n, eps = 12, 1e-3
    C = random_cost(n, 8, scale=4.0)
    a, b = dirichlet_pair(n, 9)
    assert (np.exp(-C.astype(np.float64) / eps) == 0).mean() > 0.5
    f, g = oracle.sinkhorn_log(C, eps, a, b, 3000)
    assert np.all(np.isfinite(f)) and np.all(np.isfinite(g))
    e = oracle.marginal_errors(C, C_, eps, LG, f, g, a, b)
    assert e["col_l1"] < 1e-12
    # convergence is slow this close to the unregularised problem; it must still be monotone
    f1, g1 = oracle.sinkhorn_log(C, eps, a, b, 300)
    assert e["row_l1"] < oracle.marginal_errors(C, C_, eps, LG, f1, g1, a, b)["row_l1"] < 1.0


# ------------------------------------------------------------------ P4 / P9 protocol == centralized

def compositions(n, c):
    for cuts in itertools.combinations(range(1, n), c - 1):
        yield np.array((0,) + cuts + (n,), dtype=np.int64)


def test_protocol_bit_identical_all_compositions():
    n, eps = 7, 0.3
    C = random_cost(n, 77)
    assert not np.allclose(C, C.T)
    a, b = dirichlet_pair(n, 78)
    u0, v0 = oracle.sinkhorn_scaling(C, C_, eps, a, b, 4)
    count = 0
    for c in range(1, n + 1):
        for off in compositions(n, c):
            u, v, agree = oracle.sinkhorn_protocol(C, C_, eps, a, b, off, 4)
            assert agree
            assert np.array_equal(u, u0) and np.array_equal(v, v0), off
            count += 1
    assert count == 2 ** (n - 1)


@pytest.mark.parametrize("offsets", [[0, 100, 101, 300, 512], [0, 512], list(range(0, 513, 64))])
def test_protocol_bit_identical_config1(offsets):
    w = workloads.make(1)
    u0, v0 = oracle.sinkhorn_scaling(w.K, K_, w.eps, w.a, w.b, 3)
    u, v, agree = oracle.sinkhorn_protocol(w.K, K_, w.eps, w.a, w.b, offsets, 3)
    assert agree and np.array_equal(u, u0) and np.array_equal(v, v0)


def test_rowpartition_equals_centralized_to_rounding():
    w = workloads.make(2, n=300)
    u0, v0 = oracle.sinkhorn_scaling(w.K, K_, w.eps, w.a, w.b, 6)
    u, v = oracle.sinkhorn_rowpartition(w.K, K_, w.eps, w.a, w.b, [0, 7, 150, 151, 300], 6)
    np.testing.assert_allclose(u, u0, rtol=1e-12)
    np.testing.assert_allclose(v, v0, rtol=1e-12)
    # a single block is the same association as the centralized sum
    u1, v1 = oracle.sinkhorn_rowpartition(w.K, K_, w.eps, w.a, w.b, [0, 300], 6)
    assert np.array_equal(u1, u0) and np.array_equal(v1, v0)


def test_batched_is_loop_of_singles():
    w = workloads.make(5, n=48, nbatch=5)
    U, V = oracle.sinkhorn_batched(w.K, K_, w.eps, w.a, w.b, 7)
    for p in range(5):
        u, v = oracle.sinkhorn_scaling(w.K, K_, w.eps, w.a[p], w.b[p], 7)
        assert np.array_equal(U[p], u) and np.array_equal(V[p], v)
    # problems do not interact: permuting the batch permutes the answers
    U2, V2 = oracle.sinkhorn_batched(w.K, K_, w.eps, w.a[::-1], w.b[::-1], 7)
    assert np.array_equal(U2[::-1], U) and np.array_equal(V2[::-1], V)


# ------------------------------------------------------------------ P5 fixed point, duality, invariance

def test_fixed_point_marginals_and_strong_duality():
    n, eps = 30, 0.08
    C = random_cost(n, 91)
    a, b = dirichlet_pair(n, 92)
    # equal masses are needed for an exact fixed point: renormalise in fp64, round once
    a = (a.astype(np.float64) / a.astype(np.float64).sum()).astype(np.float32)
    b64 = b.astype(np.float64)
    b = (b64 * (a.astype(np.float64).sum() / b64.sum())).astype(np.float32)
    mass_gap = abs(a.astype(np.float64).sum() - b.astype(np.float64).sum())
    u, v = oracle.sinkhorn_scaling(C, C_, eps, a, b, 4000)
    e = oracle.marginal_errors(C, C_, eps, SC, u, v, a, b)
    assert e["col_l1"] < 1e-13
    assert e["row_l1"] < 1e-13 + 2 * mass_gap
    f, g = eps * np.log(u), eps * np.log(v)
    obj = oracle.objectives(C, C_, eps, SC, u, v, C)
    D = oracle.dual_value(eps, f, g, a, b, obj["mass"])
    assert obj["primal"] == pytest.approx(D, abs=1e-10 + 10 * mass_gap)
    # log-domain run reaches the same plan
    fl, gl = oracle.sinkhorn_log(C, eps, a, b, 4000)
    np.testing.assert_allclose(oracle.plan(C, C_, eps, LG, fl, gl), oracle.plan(C, C_, eps, SC, u, v),
                               rtol=1e-9, atol=1e-16)


def test_plan_invariant_under_row_column_shifts():
    # C_il -> C_il + alpha_i + beta_l only changes the duals, never P* (shifts on a dyadic grid so
    # the shifted cost is exact in fp32)
    n, eps = 16, 0.25
    rng = np.random.default_rng(5)
    C = (rng.integers(0, 256, (n, n)) / 256.0).astype(np.float32)
    al = rng.integers(0, 32, n) / 32.0
    be = rng.integers(0, 32, n) / 32.0
    C2 = (C.astype(np.float64) + al[:, None] + be[None, :]).astype(np.float32)
    assert np.array_equal(C2.astype(np.float64), C.astype(np.float64) + al[:, None] + be[None, :])
    a, b = dirichlet_pair(n, 6)
    u, v = oracle.sinkhorn_scaling(C, C_, eps, a, b, 3000)
    u2, v2 = oracle.sinkhorn_scaling(C2, C_, eps, a, b, 3000)
    np.testing.assert_allclose(oracle.plan(C2, C_, eps, SC, u2, v2), oracle.plan(C, C_, eps, SC, u, v), rtol=1e-10)


# ------------------------------------------------------------------ P6 half-step invariants

def test_half_step_invariants_dual_ascent_and_contraction():
    n, eps = 25, 0.1
    C = random_cost(n, 123)
    a, b = dirichlet_pair(n, 124)
    a64, b64 = a.astype(np.float64), b.astype(np.float64)
    u, v = np.ones(n), np.ones(n)

    def dual(u, v):
        mass = oracle.objectives(C, C_, eps, SC, u, v, C)["mass"]
        return oracle.dual_value(eps, eps * np.log(u), eps * np.log(v), a, b, mass)

    last_D = dual(u, v)
    last_dh = None
    for t in range(12):
        u_new, q = oracle.row_pass(C, C_, eps, a, v)
        row, _ = oracle.marginals(C, C_, eps, SC, u_new, v)
        np.testing.assert_allclose(row, a64, rtol=1e-14)            # after the u update P1 = a
        D = dual(u_new, v)
        assert D >= last_D - 1e-13
        last_D = D
        v_new, r = oracle.col_pass(C, C_, eps, b, u_new)
        _, col = oracle.marginals(C, C_, eps, SC, u_new, v_new)
        np.testing.assert_allclose(col, b64, rtol=1e-14)            # after the v update P^T 1 = b
        D = dual(u_new, v_new)
        assert D >= last_D - 1e-13
        last_D = D
        if t > 0:
            dh = hilbert(u_new, u)
            if last_dh is not None and last_dh > 1e-12:
                assert dh < last_dh                                  # Birkhoff contraction
            last_dh = dh
        u, v = u_new, v_new


def test_divide_is_hilbert_isometry():
    n, eps = 10, 0.4
    C = random_cost(n, 1)
    a, _ = dirichlet_pair(n, 2)
    rng = np.random.default_rng(3)
    v1, v2 = rng.random(n) + 0.1, rng.random(n) + 0.1
    u1, q1 = oracle.row_pass(C, C_, eps, a, v1)
    u2, q2 = oracle.row_pass(C, C_, eps, a, v2)
    assert hilbert(u1, u2) == pytest.approx(hilbert(q1, q2), rel=1e-12)
    assert hilbert(q1, q2) < hilbert(v1, v2)


# ------------------------------------------------------------------ P7 2x2 closed form

@pytest.mark.parametrize("a1,b1,eps", [(0.3, 0.6, 0.5), (0.5, 0.5, 0.2), (0.85, 0.25, 1.5)])
def test_two_by_two_closed_form(a1, b1, eps):
    C = np.array([[0.0, 1.0], [0.75, 0.25]], dtype=np.float32)
    a = np.array([a1, 1 - a1], dtype=np.float32)
    b = np.array([b1, 1 - b1], dtype=np.float32)
    a1, b1 = float(a[0]), float(b[0])
    a2, b2 = float(a[1]), float(b[1])
    m = 0.5 * ((a1 + a2) + (b1 + b2))
    K = np.exp(-C.astype(np.float64) / eps)
    theta = K[0, 0] * K[1, 1] / (K[0, 1] * K[1, 0])
    # P11 = p, P12 = a1-p, P21 = b1-p, P22 = m-a1-b1+p ; cross ratio p*P22 = theta*P12*P21
    A = 1 - theta
    B = (m - a1 - b1) + theta * (a1 + b1)
    Cq = -theta * a1 * b1
    roots = np.roots([A, B, Cq]) if abs(A) > 1e-14 else np.array([-Cq / B])
    lo, hi = max(0.0, a1 + b1 - m), min(a1, b1)
    p = [float(r.real) for r in roots if abs(r.imag) < 1e-12 and lo - 1e-12 <= r.real <= hi + 1e-12]
    assert len(p) == 1
    u, v = oracle.sinkhorn_scaling(C, C_, eps, a, b, 2000)
    P = oracle.plan(C, C_, eps, SC, u, v)
    assert P[0, 0] == pytest.approx(p[0], abs=1e-7)   # 1e-7: fp32 a and b carry slightly different masses
    assert P[0, 0] * P[1, 1] / (P[0, 1] * P[1, 0]) == pytest.approx(theta, rel=1e-12)


# ------------------------------------------------------------------ P8 independent convex solve

def newton_dual(C, a, b, eps, iters=200):
    """Maximise D(f,g) = <f,a> + <g,b> - eps sum exp((f_i+g_l-C_il)/eps) with g_{n-1} = 0 by a
    damped Newton method.  Written independently of the oracle (numpy only)."""
    n = C.shape[0]
    z = np.zeros(2 * n - 1)

    def parts(z):
        f, g = z[:n], np.append(z[n:], 0.0)
        P = np.exp((f[:, None] + g[None, :] - C) / eps)
        return f, g, P

    def D(z):
        f, g, P = parts(z)
        return f @ a + g @ b - eps * P.sum()

    for _ in range(iters):
        f, g, P = parts(z)
        grad = np.concatenate([a - P.sum(1), (b - P.sum(0))[:-1]])
        if np.abs(grad).max() < 1e-15:
            break
        H = np.zeros((2 * n - 1, 2 * n - 1))
        H[:n, :n] = np.diag(P.sum(1))
        H[n:, n:] = np.diag(P.sum(0)[:-1])
        H[:n, n:] = P[:, :-1]
        H[n:, :n] = P[:, :-1].T
        step = np.linalg.solve(H / eps, grad)
        t, d0 = 1.0, D(z)
        while D(z + t * step) < d0 and t > 1e-12:
            t *= 0.5
        z = z + t * step
    f, g, P = parts(z)
    return f, g, P


@pytest.mark.parametrize("n,eps,seed", [(3, 0.5, 0), (5, 0.3, 1), (8, 0.2, 2), (8, 1.0, 3)])
def test_against_newton_on_the_dual(n, eps, seed):
    C32 = random_cost(n, 500 + seed)
    a, b = dirichlet_pair(n, 600 + seed)
    a64 = a.astype(np.float64)
    b64 = b.astype(np.float64) * (a64.sum() / b.astype(np.float64).sum())   # exact equal mass in fp64
    b = b64.astype(np.float32)
    b64 = b.astype(np.float64)
    gap = abs(a64.sum() - b64.sum())
    C = C32.astype(np.float64)
    f, g, P = newton_dual(C, a64, b64 * (a64.sum() / b64.sum()), eps)
    u, v = oracle.sinkhorn_scaling(C32, C_, eps, a, b, 6000)
    Po = oracle.plan(C32, C_, eps, SC, u, v)
    np.testing.assert_allclose(Po, P, rtol=0, atol=1e-9 + 2 * gap)
    assert oracle.objectives(C32, C_, eps, SC, u, v, C32)["cost"] == pytest.approx((P * C).sum(), abs=1e-9 + 2 * gap)
    fl, gl = oracle.sinkhorn_log(C32, eps, a, b, 6000)
    np.testing.assert_allclose(oracle.plan(C32, C_, eps, LG, fl, gl), P, rtol=0, atol=1e-9 + 2 * gap)
    # duals agree up to the gauge (f + t, g - t)
    # (1e-7: the fp32 a and b carry masses that differ by ~1e-8, which moves the duals by that much)
    shift = (fl - f).mean()
    np.testing.assert_allclose(fl - shift, f, atol=1e-7)
    np.testing.assert_allclose(gl + shift, g, atol=1e-7)


# ------------------------------------------------------------------ error norms and log-domain marginals

def test_marginal_error_norms_on_hand_made_differences():
    """Section 5.3's err_a is a 2-norm; the acceptance bound uses the 1-norm.  Differences chosen as Pythagorean
    triples on a dyadic grid fix both exactly: rows (3, -4, 0)/1024 -> 7/1024 and 5/1024, columns
    (5, 0, -12)/1024 -> 17/1024 and 13/1024.  A dropped root, a swapped row/column slot or a swapped norm fails."""
    a = np.array([0.25, 0.5, 0.25], dtype=np.float32)
    b = np.array([0.5, 0.125, 0.375], dtype=np.float32)
    row = a.astype(np.float64) + np.array([3.0, -4.0, 0.0]) / 1024
    col = b.astype(np.float64) + np.array([5.0, 0.0, -12.0]) / 1024
    e = oracle.marginal_error_norms(row, col, a, b)
    assert e["row_l1"] == 7 / 1024 and e["row_l2"] == 5 / 1024
    assert e["col_l1"] == 17 / 1024 and e["col_l2"] == 13 / 1024


@pytest.mark.parametrize("domain", [SC, LG])
def test_marginal_errors_against_plan_sums_and_norm_inequalities(domain):
    """On a real (unconverged) state: the errors equal numpy's norms of the dense plan's row and column sums
    minus a, b, and satisfy ||d||_2 <= ||d||_1 <= sqrt(n) ||d||_2."""
    n, eps = 23, 0.2
    C = random_cost(n, 91)
    a, b = dirichlet_pair(n, 92)
    if domain == SC:
        x, y = oracle.sinkhorn_scaling(C, C_, eps, a, b, 2)
        rng = np.random.default_rng(93)
        x, y = x * (1 + 0.2 * (rng.random(n) - 0.5)), y * (1 + 0.1 * (rng.random(n) - 0.3))      # off both marginals
    else:
        x, y = oracle.sinkhorn_log(C, eps, a, b, 2)
        rng = np.random.default_rng(94)
        x, y = x + 0.04 * (rng.random(n) - 0.5), y - 0.02 * (rng.random(n) - 0.3)
    P = oracle.plan(C, C_, eps, domain, x, y)
    e = oracle.marginal_errors(C, C_, eps, domain, x, y, a, b)
    dr, dc = P.sum(1) - a.astype(np.float64), P.sum(0) - b.astype(np.float64)
    assert e["row_l1"] == pytest.approx(np.abs(dr).sum(), rel=1e-11)
    assert e["row_l2"] == pytest.approx(np.linalg.norm(dr), rel=1e-11)
    assert e["col_l1"] == pytest.approx(np.abs(dc).sum(), rel=1e-11)
    assert e["col_l2"] == pytest.approx(np.linalg.norm(dc), rel=1e-11)
    assert e["row_l1"] > 1e-3 and e["col_l1"] > 1e-3 and abs(e["row_l1"] - e["col_l1"]) > 1e-6
    for k in ("row", "col"):
        assert e[k + "_l2"] <= e[k + "_l1"] <= np.sqrt(n) * e[k + "_l2"]


def test_log_domain_marginals_rank1_closed_form_both_sides():
    """Additive cost C_il = x_i + y_l (x != y): at f = g = 0 the plan is exp(-x_i/eps) exp(-y_l/eps), so
    row_i = exp(-x_i/eps) sum_l exp(-y_l/eps) and col_l = exp(-y_l/eps) sum_i exp(-x_i/eps); after one log row
    half-step from g = 0 the row marginal is a, and after the column half-step the column marginal is b."""
    n, eps = 29, 0.13
    C, x, y = dyadic_additive(n, 77)
    a, b = dirichlet_pair(n, 78)
    z = np.zeros(n)
    row, col = oracle.marginals(C, C_, eps, LG, z, z)
    np.testing.assert_allclose(row, np.exp(-x / eps) * np.exp(-y / eps).sum(), rtol=1e-13)
    np.testing.assert_allclose(col, np.exp(-y / eps) * np.exp(-x / eps).sum(), rtol=1e-13)
    f = oracle.log_row_pass(C, eps, a, z)
    row, col = oracle.marginals(C, C_, eps, LG, f, z)
    np.testing.assert_allclose(row, a.astype(np.float64), rtol=1e-13)
    assert np.abs(col - b).max() > 1e-4                       # the other side is not yet matched
    g = oracle.log_col_pass(C, eps, b, f)
    row, col = oracle.marginals(C, C_, eps, LG, f, g)
    np.testing.assert_allclose(col, b.astype(np.float64), rtol=1e-13)


# ------------------------------------------------------------------ implicit kernel from points

def test_cost_from_points_hand_placed_integer_distances():
    """3-4-5 and 6-8-10 triangles: every squared distance is an integer fixed by hand; X != Y catches a
    transposed result, the scale factor is applied once."""
    X = np.array([[0, 0], [3, 4], [1, 1]], dtype=np.float32)
    Y = np.array([[0, 0], [6, 8], [1, 2]], dtype=np.float32)
    ref = np.array([[0, 100, 5], [25, 25, 8], [2, 74, 1]], dtype=np.float64)
    assert np.array_equal(oracle.cost_from_points(X, Y), ref)
    assert np.array_equal(oracle.cost_from_points(X, Y, 0.25), ref / 4)
    assert np.array_equal(oracle.cost_from_points(Y, X), ref.T)


def test_cost_from_points_symmetry_translation_and_generator():
    rng = np.random.default_rng(5)
    n, d = 40, 7
    X = (rng.integers(-512, 512, (n, d)) / 256.0).astype(np.float32)          # dyadic grid: shifts stay exact
    Y = (rng.integers(-512, 512, (n, d)) / 256.0).astype(np.float32)
    C1 = oracle.cost_from_points(X, X)
    assert np.array_equal(C1, C1.T) and np.all(np.diag(C1) == 0) and np.all(C1[~np.eye(n, dtype=bool)] > 0)
    shift = (rng.integers(-64, 64, d) / 16.0).astype(np.float32)
    assert np.array_equal(oracle.cost_from_points(X + shift, Y + shift), oracle.cost_from_points(X, Y))
    # the workload generator forms the same cost by the expanded square in fp64 and rounds it to fp32
    w = workloads.make(2, n=300, fp32_points=True, want_cost=True)
    C = oracle.cost_from_points(w.X, w.Y, w.cost_scale)
    assert np.max(np.abs(C - w.C.astype(np.float64))) <= 2.0 ** -24 * C.max() * 1.01
    assert C.max() == pytest.approx(1.0, rel=1e-12)                            # config 2 divides by the largest entry


def test_sinkhorn_points_equals_stored_cost_iteration():
    """On integer grid points every C_il is an integer, exact in fp32: the implicit iteration must reproduce the
    stored-cost iteration (pinned above by closed forms and the Newton solve) to rounding, two clouds, and
    its marginal errors those of the stored-cost state."""
    rng = np.random.default_rng(9)
    n, d, eps, scale = 31, 3, 6.0, 0.5
    X = rng.integers(0, 5, (n, d)).astype(np.float32)
    Y = rng.integers(0, 5, (n, d)).astype(np.float32)
    C = oracle.cost_from_points(X, Y, scale)
    C32 = C.astype(np.float32)
    assert np.array_equal(C32.astype(np.float64), C)
    a, b = dirichlet_pair(n, 10)
    for iters in (1, 7):
        u, v = oracle.sinkhorn_points(X, Y, scale, eps, a, b, iters)
        ur, vr = oracle.sinkhorn_scaling(C32, C_, eps, a, b, iters)
        np.testing.assert_allclose(u, ur, rtol=1e-13)
        np.testing.assert_allclose(v, vr, rtol=1e-13)
    e = oracle.marginal_errors_points(X, Y, scale, eps, u, v * 1.01, a, b)
    er = oracle.marginal_errors(C32, C_, eps, SC, ur, vr * 1.01, a, b)
    for k in e:
        assert e[k] == pytest.approx(er[k], rel=1e-11)
    assert e["row_l1"] > 1e-3


# ------------------------------------------------------------------ library-routine special case

def test_lse_against_scipy():
    n, eps = 50, 0.03
    C = random_cost(n, 17, scale=2.0)
    rng = np.random.default_rng(18)
    g = rng.standard_normal(n) * 0.1
    f = rng.standard_normal(n) * 0.1
    C64 = C.astype(np.float64)
    np.testing.assert_allclose(oracle.lse_rows(C, eps, g), logsumexp((g[None, :] - C64) / eps, axis=1), rtol=1e-13)
    np.testing.assert_allclose(oracle.lse_cols(C, eps, f), logsumexp((f[:, None] - C64) / eps, axis=0), rtol=1e-13)


def test_padded_leading_dimension():
    n = 19
    big = random_cost(32, 3)
    view = big[:n, :n]                      # ld = 32 > n
    dense = np.ascontiguousarray(view)
    a, b = dirichlet_pair(n, 4)
    u1, v1 = oracle.sinkhorn_scaling(view, C_, 0.2, a, b, 5)
    u2, v2 = oracle.sinkhorn_scaling(dense, C_, 0.2, a, b, 5)
    assert np.array_equal(u1, u2) and np.array_equal(v1, v2)


# ------------------------------------------------------------------ the paper's printed toy example

def read_golden(name):
    path = os.path.join(os.path.dirname(__file__), "golden", name)
    out, key = {}, None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if line.startswith("["):
            key = line.strip("[]")
            out[key] = []
        else:
            out[key].append([float(t) for t in line.split()])
    return {k: np.array(v) for k, v in out.items()}


def test_toy_portfolio_printed_values():
    gold = read_golden("toy_portfolio.txt")
    a = gold["x_shifted"][0] / gold["x_shifted"][0].sum()
    b = gold["xprime_shifted"][0] / gold["xprime_shifted"][0].sum()
    P = gold["P"]
    # what the printed plan does satisfy: its column sums are the stated b (to printed digits)
    np.testing.assert_allclose(P.sum(0), b, atol=2e-3)
    # what it does not: the row sums are not the stated a -- the example is inconsistent
    assert np.abs(P.sum(1) - a).max() > 0.05
    # the oracle on the printed C with the stated a, b and eps reaches the stated marginals
    C = gold["C"].astype(np.float32)
    u, v = oracle.sinkhorn_scaling(C, C_, 0.01, a.astype(np.float32), b.astype(np.float32), 5000)
    row, col = oracle.marginals(C, C_, 0.01, SC, u, v)
    np.testing.assert_allclose(col, b, atol=1e-7)
    np.testing.assert_allclose(row, a, atol=1e-6)
