"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU, no CUDA library).

Each test is chosen so that a plausible mistake in oracle/qn_oracle.c (a dropped term, a wrong
sign, a transposed V, a missing centring, sigma vs sigma^2) makes it fail.  Nothing here retypes
the oracle's own formula: the expected values come from closed forms, numpy's LAPACK routines,
explicitly built n x n matrices, or invariants of the construction in Section 2 of the paper.
"""
import numpy as np
import pytest

import oracle
import workloads as W


def _rand_problem(rng, n, m, cond=100.0, noise=0.0, spread=1.0):
    """theta[m][n], g[m][n] (fp32 storage) of a quadratic with SPD A (returned in fp64) and b."""
    Q, _ = np.linalg.qr(rng.standard_normal((n, n)))
    ev = np.geomspace(1.0, cond, n)
    A = (Q * ev) @ Q.T
    b = rng.standard_normal(n)
    theta = (rng.standard_normal(n)[None, :] + spread * rng.standard_normal((m, n))).astype(np.float32)
    g = theta.astype(np.float64) @ A.T - b[None, :] + noise * rng.standard_normal((m, n))
    return theta, g, A, b


def _as_f32_exact(x):
    """Round to fp32 so that the stored bits are what every side reads."""
    return np.ascontiguousarray(x, dtype=np.float32)


# ---------------------------------------------------------------- P1: SGD special case
@pytest.mark.parametrize("case", ["lambda_gt_1", "identical_g", "m1"])
def test_p1_j0_is_plain_sgd(case):
    """Section 2, sentence after Eq. (4): with j = 0 the update is standard SGD, thetabar - tau gbar."""
    rng = np.random.default_rng(1)
    n, m, tau, lam = 37, 5, 0.3, 0.01
    theta = _as_f32_exact(rng.standard_normal((m, n)))
    g = _as_f32_exact(rng.standard_normal((m, n)))
    if case == "lambda_gt_1":
        lam = 1.5
    elif case == "identical_g":
        g[:] = g[0]
    else:
        theta, g = theta[:1].copy(), g[:1].copy()
    r = oracle.update(theta, g, tau, lam)
    assert r.j == 0
    expect = theta.astype(np.float64).mean(0) - tau * g.astype(np.float64).mean(0)
    np.testing.assert_allclose(r.theta_new, expect, rtol=1e-15, atol=1e-15)


# ---------------------------------------------------------------- P2: Newton recovery
@pytest.mark.parametrize("n,m", [(2, 4), (3, 5), (4, 9), (6, 8), (6, 16)])
def test_p2_newton_step_on_quadratic(n, m):
    """Eq. (1)-(2): noise-free g_k = A theta_k - b gives G = A Theta; with m - 1 >= n and Theta of
    rank n the retained u_k span R^n, Hinv = A^-1, and tau = 1 lands on the minimiser A^-1 b."""
    rng = np.random.default_rng(100 + 10 * n + m)
    Q, _ = np.linalg.qr(rng.standard_normal((n, n)))
    A = (Q * np.geomspace(1.0, 50.0, n)) @ Q.T
    b = rng.standard_normal(n)
    theta = _as_f32_exact(rng.standard_normal(n)[None, :] + rng.standard_normal((m, n)))
    # gradients must be exact functions of the stored theta and storable in fp32 without loss of the
    # secant property: use fp64 math then store g in float32 only if exactly representable -- instead
    # keep A and b on a dyadic grid so that g is exact in fp32.
    A = np.round(A * 64) / 64
    A = (A + A.T) / 2
    b = np.round(b * 64) / 64
    theta = np.round(theta * 64) / 64
    g64 = theta.astype(np.float64) @ A.T - b[None, :]
    g = g64.astype(np.float32)
    assert np.array_equal(g.astype(np.float64), g64), "test construction must be exact in fp32"
    theta = theta.astype(np.float32)
    r = oracle.update(theta, g, 1.0, 1e-6)
    assert r.j == n
    newton = np.linalg.solve(A, b)  # Gaussian elimination, independent of the oracle
    assert np.linalg.norm(r.theta_new - newton) <= 1e-10 * np.linalg.norm(newton)


# ---------------------------------------------------------------- P3: orthonormal u_k
def test_p3_left_vectors_orthonormal():
    """Section 2: u_k are columns of the unitary U_G."""
    rng = np.random.default_rng(3)
    theta, g, _, _ = _rand_problem(rng, 40, 7, noise=0.05)
    g = _as_f32_exact(g)
    U, Y, sigma, j = oracle.left_vectors(theta, g, 1e-3)
    assert j == 6
    assert np.max(np.abs(U.T @ U - np.eye(j))) <= 1e-10


# ---------------------------------------------------------------- P4: agreement with a library SVD
@pytest.mark.parametrize("n,m", [(5, 3), (12, 6), (50, 8), (9, 12)])
def test_p4_svd_of_G(n, m):
    """Section 2: sigma_k and v_k are the singular values / right vectors of G, u_k the left ones.
    numpy's LAPACK SVD of the explicitly centred G is the independent reference."""
    rng = np.random.default_rng(40 + n + m)
    theta = _as_f32_exact(rng.standard_normal((m, n)))
    g = _as_f32_exact(rng.standard_normal((m, n)) * np.geomspace(1, 0.01, n)[None, :])
    G = (g.astype(np.float64) - g.astype(np.float64).mean(0)).T  # n x m, column k = Worker k
    Us, ss, Vts = np.linalg.svd(G, full_matrices=False)
    r = oracle.update(theta, g, 1.0, 1e-4)
    rank = min(m - 1, n)
    np.testing.assert_allclose(r.sigma[:rank], ss[:rank], rtol=0, atol=1e-10 * ss[0])
    assert np.all(r.sigma[rank:] <= 1e-6 * ss[0])
    # G v_k = sigma_k u_k with the oracle's own V and U (sign-free check), and v_k matches LAPACK's up to sign
    U, Y, sigma, j = oracle.left_vectors(theta, g, 1e-4)
    assert j == r.j
    for k in range(j):
        np.testing.assert_allclose(G @ r.V[:, k], sigma[k] * U[:, k], rtol=0, atol=1e-9 * ss[0])
        assert abs(abs(r.V[:, k] @ Vts[k]) - 1.0) <= 1e-8
        Theta = (theta.astype(np.float64) - theta.astype(np.float64).mean(0)).T
        np.testing.assert_allclose(Y[:, k], Theta @ r.V[:, k], rtol=0, atol=1e-12 * np.abs(Theta).max() * m)


def test_p4_eig_matches_lapack():
    """The Jacobi eigen-solver on a random symmetric matrix vs numpy.linalg.eigh."""
    rng = np.random.default_rng(44)
    for m in (1, 2, 3, 8, 17, 64):
        B = rng.standard_normal((m, m))
        C = B @ B.T
        mu, V = oracle.eig(C)
        ref = np.linalg.eigvalsh(C)[::-1]
        np.testing.assert_allclose(mu, ref, rtol=0, atol=1e-12 * abs(ref[0]))
        np.testing.assert_allclose(V @ np.diag(mu) @ V.T, C, rtol=0, atol=1e-12 * abs(ref[0]))
        np.testing.assert_allclose(V.T @ V, np.eye(m), rtol=0, atol=1e-13)
        assert np.all(np.diff(mu) <= 0)


# ---------------------------------------------------------------- P5: secant property and complement
def test_p5_secant_and_complement():
    """Eq. (3): Hinv maps sigma_k u_k to y_k (from H^-1 U Sigma = Theta V) for k <= j and is the identity
    on the orthogonal complement of span{u_1..u_j}."""
    rng = np.random.default_rng(5)
    n, m = 30, 6
    theta, g, _, _ = _rand_problem(rng, n, m, noise=0.1)
    g = _as_f32_exact(g)
    lam = 1e-3
    U, Y, sigma, j = oracle.left_vectors(theta, g, lam)
    assert j == m - 1
    for k in range(j):
        out, jj = oracle.apply_hinv(theta, g, lam, sigma[k] * U[:, k])
        assert jj == j
        np.testing.assert_allclose(out, Y[:, k], rtol=0, atol=1e-9 * np.linalg.norm(Y[:, k]))
    z = rng.standard_normal(n)
    z -= U @ (U.T @ z)
    out, _ = oracle.apply_hinv(theta, g, lam, z)
    np.testing.assert_allclose(out, z, rtol=0, atol=1e-12 * np.linalg.norm(z))


def test_p5_secant_equation_on_worker_differences():
    """Eq. (1): for the noise-free quadratic, Hinv (g_k - g_l) = theta_k - theta_l when all modes are kept."""
    rng = np.random.default_rng(55)
    n, m = 5, 9
    A = np.diag(np.array([1.0, 2.0, 4.0, 0.5, 8.0]))
    b = np.round(rng.standard_normal(n) * 16) / 16
    theta = (np.round(rng.standard_normal((m, n)) * 32) / 32).astype(np.float32)
    g = (theta.astype(np.float64) @ A - b).astype(np.float32)
    for (k, l) in [(0, 1), (3, 7), (8, 2)]:
        z = g[k].astype(np.float64) - g[l].astype(np.float64)
        out, j = oracle.apply_hinv(theta, g, 1e-6, z)
        assert j == n
        np.testing.assert_allclose(out, theta[k].astype(np.float64) - theta[l], rtol=0, atol=1e-10)


# ---------------------------------------------------------------- P6: m = 2 closed form
def test_p6_two_workers_closed_form():
    """m = 2: v_1 = (1,-1)/sqrt 2, sigma_1 = |g_1 - g_2|/sqrt 2, u = (g_1-g_2)/|g_1-g_2| and
    Hinv z = z - (z.u) u + (z.u) (theta_1 - theta_2)/|g_1 - g_2|."""
    rng = np.random.default_rng(6)
    n = 23
    theta = _as_f32_exact(rng.standard_normal((2, n)))
    g = _as_f32_exact(rng.standard_normal((2, n)))
    t64, g64 = theta.astype(np.float64), g.astype(np.float64)
    dg, dth = g64[0] - g64[1], t64[0] - t64[1]
    u = dg / np.linalg.norm(dg)
    z = rng.standard_normal(n)
    expect = z - (z @ u) * u + (z @ u) * dth / np.linalg.norm(dg)
    out, j = oracle.apply_hinv(theta, g, 0.5, z)
    assert j == 1
    np.testing.assert_allclose(out, expect, rtol=0, atol=1e-13 * np.linalg.norm(expect))
    tau = 0.7
    gbar = g64.mean(0)
    r = oracle.update(theta, g, tau, 0.5)
    expect_new = t64.mean(0) - tau * (gbar - (gbar @ u) * u + (gbar @ u) * dth / np.linalg.norm(dg))
    np.testing.assert_allclose(r.theta_new, expect_new, rtol=0, atol=1e-13 * np.linalg.norm(expect_new))
    np.testing.assert_allclose(r.sigma[0], np.linalg.norm(dg) / np.sqrt(2), rtol=1e-13)


# ---------------------------------------------------------------- P7: null vector of the centred Gram
def test_p7_null_vector_and_cap():
    """G 1 = 0 by construction of the centred columns, so sigma_m is round-off, v_m is parallel to 1 and j <= m-1."""
    rng = np.random.default_rng(7)
    n, m = 500, 8
    theta = _as_f32_exact(rng.standard_normal((m, n)))
    g = _as_f32_exact(5.0 + 0.1 * rng.standard_normal((m, n)))
    C = oracle.gram(g)
    np.testing.assert_allclose(C @ np.ones(m), 0, atol=1e-12 * np.abs(C).max())
    r = oracle.update(theta, g, 1.0, 1e-9)  # lambda so small that only the cap stops j
    assert r.j == m - 1
    assert r.sigma[-1] <= 1e-7 * r.sigma[0]
    vm = r.V[:, -1]
    assert abs(abs(vm @ np.ones(m)) / np.sqrt(m) - 1.0) <= 1e-8
    # centred Gram equals the explicit one built with numpy
    G = g.astype(np.float64) - g.astype(np.float64).mean(0)
    np.testing.assert_allclose(C, G @ G.T, rtol=0, atol=1e-12 * np.abs(C).max())


# ---------------------------------------------------------------- P8: collapsed form
def test_p8_collapse_identity():
    """theta_new = thetabar - tau (gbar - G d + Theta d) with d = V_j diag(sigma^-2) V_j^T G^T gbar, built here
    with numpy from the LAPACK SVD (not from the oracle's V), equals the oracle's literal Eq. (4)."""
    rng = np.random.default_rng(8)
    n, m, tau, lam = 64, 7, 0.4, 0.05
    theta, g, _, _ = _rand_problem(rng, n, m, noise=0.02)
    g = _as_f32_exact(g * np.geomspace(1, 0.05, n)[None, :])
    t64, g64 = theta.astype(np.float64), g.astype(np.float64)
    gbar, tbar = g64.mean(0), t64.mean(0)
    G, Th = (g64 - gbar).T, (t64 - tbar).T
    _, ss, Vt = np.linalg.svd(G, full_matrices=False)
    j = int(np.sum(ss >= lam * ss[0]))
    j = min(j, m - 1)
    Vj = Vt[:j].T
    d = Vj @ ((Vj.T @ (G.T @ gbar)) / ss[:j] ** 2)
    expect = tbar - tau * (gbar - G @ d + Th @ d)
    r = oracle.update(theta, g, tau, lam)
    assert r.j == j
    np.testing.assert_allclose(r.theta_new, expect, rtol=0, atol=1e-11 * np.linalg.norm(expect))


def test_p8_rank_cap():
    """A cap on j keeps the largest of the modes that the lambda rule retains: cap 0 is the SGD step, a cap at or
    above the rule's j changes nothing, and a cap in between equals the collapsed form built with numpy from
    LAPACK's SVD truncated at the cap."""
    rng = np.random.default_rng(18)
    n, m, tau, lam = 48, 8, 0.3, 0.02
    theta, g, _, _ = _rand_problem(rng, n, m, noise=0.02)
    g = _as_f32_exact(g * np.geomspace(1, 0.1, n)[None, :])
    t64, g64 = theta.astype(np.float64), g.astype(np.float64)
    gbar, tbar = g64.mean(0), t64.mean(0)
    G, Th = (g64 - gbar).T, (t64 - tbar).T
    _, ss, Vt = np.linalg.svd(G, full_matrices=False)
    free = oracle.update(theta, g, tau, lam)
    assert free.j >= 4
    r0 = oracle.update(theta, g, tau, lam, j_cap=0)
    assert r0.j == 0
    np.testing.assert_allclose(r0.theta_new, tbar - tau * gbar, rtol=0, atol=1e-14 * np.linalg.norm(tbar))
    for cap in (free.j, free.j + 1, m):
        r = oracle.update(theta, g, tau, lam, j_cap=cap)
        assert r.j == free.j and np.array_equal(r.theta_new, free.theta_new)
    for cap in (1, 3):
        Vj = Vt[:cap].T
        d = Vj @ ((Vj.T @ (G.T @ gbar)) / ss[:cap] ** 2)
        expect = tbar - tau * (gbar - G @ d + Th @ d)
        r = oracle.update(theta, g, tau, lam, j_cap=cap)
        assert r.j == cap
        np.testing.assert_allclose(r.theta_new, expect, rtol=0, atol=1e-11 * np.linalg.norm(expect))
        np.testing.assert_array_equal(r.sigma, free.sigma)  # sigma is reported in full whatever the cap
        assert np.linalg.norm(r.theta_new - free.theta_new) > 1e-6 * np.linalg.norm(free.theta_new)


def test_p8_learning_rate_cap():
    """tau is bounded by 1 / max_k sigma_k / ||Theta v_k||.  For noise-free gradients of a quadratic, G = A Theta
    and sigma_k u_k = A y_k, so the estimate is a quotient ||A y|| / ||y||: it lies between the extreme singular
    values of A, equals a for A = a I, and matches the same quantity built with numpy from LAPACK's SVD."""
    rng = np.random.default_rng(28)
    n, m, lam = 5, 9, 1e-6
    for kind in ("scaled identity", "spd"):
        if kind == "scaled identity":
            A = 4.0 * np.eye(n)
        else:
            Q, _ = np.linalg.qr(rng.standard_normal((n, n)))
            A = (Q * np.array([0.5, 1.0, 2.0, 3.0, 8.0])) @ Q.T
            A = np.round(A * 1024) / 1024
            A = (A + A.T) / 2
        b = np.round(rng.standard_normal(n) * 64) / 64
        theta = (np.round(rng.standard_normal((m, n)) * 64) / 64).astype(np.float32)
        g = (theta.astype(np.float64) @ A.T - b).astype(np.float32)
        assert np.array_equal(g.astype(np.float64), theta.astype(np.float64) @ A.T - b)  # exactly representable
        t64, g64 = theta.astype(np.float64), g.astype(np.float64)
        G, Th = (g64 - g64.mean(0)).T, (t64 - t64.mean(0)).T
        _, ss, Vt = np.linalg.svd(G, full_matrices=False)
        r_free = oracle.update(theta, g, 10.0, lam)
        jj = r_free.j
        est = max(ss[k] / np.linalg.norm(Th @ Vt[k]) for k in range(jj))
        sv = np.linalg.svd(A, compute_uv=False)
        assert sv[-1] * (1 - 1e-9) <= est <= sv[0] * (1 + 1e-9)
        if kind == "scaled identity":
            assert abs(est - 4.0) <= 1e-10
        r = oracle.update(theta, g, 10.0, lam, tau_cap=True)   # 10 is far above 1 / est: capped
        assert abs(r.tau_eff - 1.0 / est) <= 1e-9 / est
        expect = t64.mean(0) + (r.tau_eff / 10.0) * (r_free.theta_new - t64.mean(0))  # the step scales with tau
        np.testing.assert_allclose(r.theta_new, expect, rtol=0, atol=1e-10 * np.linalg.norm(expect))
        small = 0.01 / est
        r = oracle.update(theta, g, small, lam, tau_cap=True)  # below the bound: untouched
        assert r.tau_eff == small
        assert np.array_equal(r.theta_new, oracle.update(theta, g, small, lam).theta_new)


# ---------------------------------------------------------------- P9: symmetries
def test_p9_symmetries():
    rng = np.random.default_rng(9)
    n, m, tau, lam = 33, 6, 0.25, 0.01
    theta = (np.round(rng.standard_normal((m, n)) * 256) / 256).astype(np.float32)
    g = (np.round(rng.standard_normal((m, n)) * 256) / 256).astype(np.float32)
    base = oracle.update(theta, g, tau, lam)
    # Worker permutation leaves theta_new, sigma and j unchanged
    perm = rng.permutation(m)
    p = oracle.update(np.ascontiguousarray(theta[perm]), np.ascontiguousarray(g[perm]), tau, lam)
    assert p.j == base.j
    # sigma_m is the square root of round-off (G 1 = 0): compare the m-1 genuine values tightly
    np.testing.assert_allclose(p.sigma[:-1], base.sigma[:-1], rtol=0, atol=1e-12 * base.sigma[0])
    assert p.sigma[-1] <= 1e-7 * base.sigma[0] and base.sigma[-1] <= 1e-7 * base.sigma[0]
    np.testing.assert_allclose(p.theta_new, base.theta_new, rtol=0, atol=1e-11)
    # translating every theta_k by t translates theta_new by t (dyadic t: exact in fp32)
    t = (np.round(rng.standard_normal(n) * 4) / 4).astype(np.float32)
    s = oracle.update(theta + t[None, :], g, tau, lam)
    np.testing.assert_allclose(s.theta_new, base.theta_new + t, rtol=0, atol=1e-11)
    # scaling every g_k by c scales sigma by c, keeps j, scales the z-perp part and leaves the y part alone
    c = 4.0
    sc = oracle.update(theta, g * np.float32(c), tau, lam)
    assert sc.j == base.j
    np.testing.assert_allclose(sc.sigma[:-1], c * base.sigma[:-1], rtol=1e-12, atol=1e-12 * base.sigma[0])
    U, Y, sigma, j = oracle.left_vectors(theta, g, lam)
    g64 = g.astype(np.float64)
    gbar = g64.mean(0)
    alpha = U.T @ gbar
    zperp = gbar - U @ alpha
    ypart = Y @ (alpha / sigma[:j])
    tbar = theta.astype(np.float64).mean(0)
    np.testing.assert_allclose(base.theta_new, tbar - tau * (zperp + ypart), rtol=0, atol=1e-11)
    np.testing.assert_allclose(sc.theta_new, tbar - tau * (c * zperp + ypart), rtol=0, atol=1e-10)


# ---------------------------------------------------------------- P10: brute-force n x n operator
@pytest.mark.parametrize("n,m,lam", [(4, 3, 0.01), (6, 5, 0.2), (8, 6, 0.05), (8, 12, 1e-3)])
def test_p10_bruteforce_operator(n, m, lam):
    """Build Hinv as an explicit n x n matrix from Eq. (3): P U^T on span{u_k, k<=j} with p_k = y_k/sigma_k,
    identity on the complement, using LAPACK's SVD of G; compare the operator applied to unit vectors and
    the resulting update of Eq. (2)."""
    rng = np.random.default_rng(1000 + n * 13 + m)
    theta = _as_f32_exact(rng.standard_normal((m, n)))
    g = _as_f32_exact(rng.standard_normal((m, n)) * np.geomspace(1, 0.03, n)[None, :])
    t64, g64 = theta.astype(np.float64), g.astype(np.float64)
    gbar, tbar = g64.mean(0), t64.mean(0)
    G, Th = (g64 - gbar).T, (t64 - tbar).T
    Us, ss, Vt = np.linalg.svd(G, full_matrices=True)
    rank = min(m - 1, n)
    j = min(int(np.sum(ss[:rank] >= lam * ss[0])), m - 1)
    Uj = Us[:, :j]
    Pj = (Th @ Vt[:j].T) / ss[:j]
    H = Pj @ Uj.T + (np.eye(n) - Uj @ Uj.T)
    for e in range(n):
        z = np.zeros(n)
        z[e] = 1.0
        out, jj = oracle.apply_hinv(theta, g, lam, z)
        assert jj == j
        np.testing.assert_allclose(out, H[:, e], rtol=0, atol=1e-9 * np.abs(H).max())
    tau = 0.9
    r = oracle.update(theta, g, tau, lam)
    np.testing.assert_allclose(r.theta_new, tbar - tau * H @ gbar, rtol=0, atol=1e-9 * np.abs(H).max() * np.abs(gbar).max() * n)


# ---------------------------------------------------------------- cut-off rule
def test_cutoff_rule():
    """sigma_j >= lambda sigma_1 > sigma_{j+1} (Section 2, after Eq. (3)), with the m-1 cap and sigma_1 = 0."""
    mu = np.array([100.0, 25.0, 1.0, 1e-4, -1e-20])
    sigma, j = oracle.cutoff(mu, 0.1)
    np.testing.assert_allclose(sigma, [10, 5, 1, 1e-2, 0.0])
    assert j == 3
    assert oracle.cutoff(mu, 0.11)[1] == 2
    assert oracle.cutoff(mu, 1e-9)[1] == 4
    assert oracle.cutoff(np.zeros(4), 0.5)[1] == 0
    assert oracle.cutoff(mu, 1.0)[1] == 1
    assert oracle.cutoff(mu, 1.0001)[1] == 0
    assert oracle.cutoff(np.array([4.0, 4.0, 4.0]), 0.5)[1] == 2  # cap at m - 1


# ---------------------------------------------------------------- storage handling
def test_bf16_promotion_and_rounding():
    """bf16 bits are promoted exactly; fp64 -> bf16 rounding is nearest-even (checked against torch)."""
    import torch

    rng = np.random.default_rng(11)
    x = np.concatenate([rng.standard_normal(4000) * np.exp(rng.uniform(-60, 60, 4000)),
                        [0.0, -0.0, 1.0, 1.00390625, 1.001953125, 1.005859375, 3.3895313892515355e38, 1e-40, 9.1e-41,
                         4.6e-41, 4.5917748078809e-41]])
    # torch converts fp64 -> bf16 through fp32 (two roundings); feed values that are already fp32 so that
    # its result is the single nearest-even rounding the oracle performs
    x = x.astype(np.float32).astype(np.float64)
    got = oracle.round_storage(x, np.zeros(1, dtype=np.uint16))
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, ref)
    back = oracle.storage_to_f64(got)
    assert np.array_equal(back, torch.from_numpy(x).to(torch.bfloat16).double().numpy())
    # the C side reads bf16 bits the same way
    theta = rng.standard_normal((3, 16))
    tb = oracle.round_storage(theta, np.zeros(1, dtype=np.uint16))
    gb = oracle.round_storage(rng.standard_normal((3, 16)), np.zeros(1, dtype=np.uint16))
    r16 = oracle.update(tb, gb, 0.5, 0.01)
    r32 = oracle.update(oracle.storage_to_f64(tb).astype(np.float32), oracle.storage_to_f64(gb).astype(np.float32), 0.5, 0.01)
    assert r16.j == r32.j
    np.testing.assert_array_equal(r16.theta_new, r32.theta_new)


def test_sampled_outputs_and_threads():
    """Sampled pass 3 equals the full one at those columns; thread count does not change the result beyond round-off."""
    cfg = W.CONFIGS[0]
    theta, g = W.generate(cfg)
    tb, gb = W.to_bits(theta), W.to_bits(g)
    full = oracle.update(tb, gb, cfg.tau, cfg.lam, nthreads=1)
    idx = np.array([0, 1, 77, 4095, 2048], dtype=np.int64)
    samp = oracle.update(tb, gb, cfg.tau, cfg.lam, sample_idx=idx, nthreads=3)
    assert samp.j == full.j
    np.testing.assert_allclose(samp.theta_new, full.theta_new[idx], rtol=1e-12, atol=1e-12)


def test_quadratic_convergence_direction():
    """On the diagonal quadratic of config 0 the step moves thetabar towards A^-1 b inside span{y_k} and acts
    as plain gradient descent outside: J(theta_new) < J(thetabar - tau gbar) is not guaranteed, but the
    update must equal SGD's in every direction orthogonal to the u_k (Eq. (3), second branch)."""
    cfg = W.CONFIGS[0].with_shape(n=256)
    theta, g = W.generate(cfg)
    tb, gb = W.to_bits(theta), W.to_bits(g)
    r = oracle.update(tb, gb, cfg.tau, cfg.lam)
    U, Y, sigma, j = oracle.left_vectors(tb, gb, cfg.lam)
    t64, g64 = tb.astype(np.float64), gb.astype(np.float64)
    sgd = t64.mean(0) - cfg.tau * g64.mean(0)
    diff = r.theta_new - sgd
    # diff lies in span{u_k} + span{y_k}: its component orthogonal to both vanishes
    B, _ = np.linalg.qr(np.concatenate([U, Y], axis=1))
    resid = diff - B @ (B.T @ diff)
    assert np.linalg.norm(resid) <= 1e-9 * np.linalg.norm(diff)


def test_stored_small_cases_still_hold(oracle_mod):
    """Regression anchor: the oracle's results on formula-given inputs, as written by tests/golden/make_golden.py.
    (Not a pin: the values came from the oracle.  It makes a change of the oracle's arithmetic visible.)"""
    import importlib.util
    import json
    import os

    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "make_golden.py"))
    mg = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mg)
    with open(os.path.join(here, "oracle_small_cases.json")) as f:
        cases = json.load(f)["cases"]
    assert [(c["m"], c["n"], c["tau"], c["lam"]) for c in cases] == mg.CASES
    for c in cases:
        theta, g = mg.inputs(c["m"], c["n"])
        r = oracle_mod.update(theta, g, c["tau"], c["lam"])
        assert r.j == c["j"]
        sigma = np.array([float.fromhex(x) for x in c["sigma"]])
        want = np.array([float.fromhex(x) for x in c["theta_new"]])
        assert np.max(np.abs(r.sigma - sigma)) <= 1e-12 * sigma[0]
        assert np.max(np.abs(r.theta_new - want)) <= 1e-10 * np.max(np.abs(want))
