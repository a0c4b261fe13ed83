"""Pins for oracle/sde.py.  None of these retype the oracle's formulas: they use the closed
form of the Gaussian transport, a library ODE solver, library Gaussian densities, the
textbook Gaussian score, the marginal-preservation property the paper claims, and the
covariance it states for the branch noises."""
import math

import numpy as np
import pytest
from scipy import integrate, stats

from oracle import philox, sde, tree

S0 = 0.5


def _grid(T):
    return 1.0 - np.arange(T + 1) / T


def _vel(mu, t_grid):
    return lambda z, i, p: sde.linear_velocity(z.astype(np.float64), float(t_grid[i]), mu, S0)


def test_velocity_transports_gaussians_library_ode():
    """The flow of dz/dt = v(z,t) from t=1 to t=0 must be the monotone map between the two
    Gaussians N(0,1) and N(mu, s0^2): z_1 -> mu + s0 z_1."""
    mu = np.array([0.7, -1.3, 0.0])
    z1 = np.array([1.1, -0.4, 2.5])
    sol = integrate.solve_ivp(lambda t, z: sde.linear_velocity(z, t, mu, S0), (1.0, 0.0), z1,
                              rtol=1e-11, atol=1e-13)
    assert np.allclose(sol.y[:, -1], mu + S0 * z1, atol=1e-8)


def test_score_is_the_textbook_gaussian_score():
    mu = np.array([0.3, -2.0])
    z = np.array([0.9, 0.1])
    for t in (1.0, 0.6, 0.05):
        v = sde.linear_velocity(z, t, mu, S0)
        c_t = (1 - t) ** 2 * S0 ** 2 + t ** 2
        assert np.allclose(sde.score_from_velocity(z, v, t), -(z - (1 - t) * mu) / c_t, rtol=1e-12)


def test_ode_limit_sigma_zero():
    """sigma = 0: the discrete rollout converges (first order in 1/T) to mu + s0 z_0."""
    mu = np.array([0.5, -1.0, 2.0, 0.0])
    errs = []
    for T in (64, 128, 256):
        g = _grid(T)
        topo = tree.build_topology(T, 2, ())
        lat, logp = sde.rollout(topo, 4, g, 0.0, math.inf, seed=3, velocity_fn=_vel(mu, g))
        z0 = lat[0].astype(np.float64)
        errs.append(np.abs(lat[-1] - (mu + S0 * z0)).max())
        assert np.all(logp == 0.0)
    assert errs[2] < 5e-3
    assert 1.6 < errs[0] / errs[1] < 2.4 and 1.6 < errs[1] / errs[2] < 2.4


def _propagate(T, sigma):
    """Leaf law of one element given the root, obtained by pushing basis states through the
    oracle's own step functions: returns (P, V) with leaf ~ N(mu + P (z0 - 0), V) for mu = 0."""
    g = _grid(T)
    P, V = 1.0, 0.0
    for i in range(T):
        t, h = g[i], g[i] - g[i + 1]
        f = lambda z: sde.em_mean(np.array([z]), sde.linear_velocity(np.array([z]), t, np.array([0.0]), S0), t, h, sigma)[0]
        a = f(1.0) - f(0.0)
        assert abs(f(0.0)) < 1e-15
        P *= a
        V = a * a * V + sde.noise_scale(sigma, h) ** 2
    return P, V


@pytest.mark.parametrize("sigma", [0.3, 0.5, 1.0])
def test_marginal_preservation_in_the_limit(sigma):
    """Over a random root z_0 ~ N(0,1) the leaf variance P^2 + V must tend to s0^2 whatever
    sigma is ("keeping the marginal distribution unchanged"; boundary-distribution theorem)."""
    gaps = []
    for T in (256, 1024, 4096):
        P, V = _propagate(T, sigma)
        gaps.append(abs(P * P + V - S0 ** 2))
    assert gaps[2] < 3e-4 * max(1.0, sigma ** 2 * 4)
    assert gaps[0] > gaps[1] > gaps[2]
    # and the drift really depends on sigma: the deterministic part shrinks as noise grows
    assert _propagate(256, 1.0)[0] < _propagate(256, 0.3)[0] < _propagate(256, 0.0)[0]


def test_monte_carlo_leaf_law_tree_equals_sequential():
    """Empirical leaf mean and variance given the root match the propagated (P, V), for a
    branching tree and for a split-free rollout alike (leaf marginal preservation lemma)."""
    T, sigma, n = 8, 0.3, 2048
    g = _grid(T)
    mu = np.zeros(n)
    P, V = _propagate(T, sigma)
    for splits, s in (((), math.inf), ((0, 3), math.inf), ((0, 3), 1.0), ((1, 2, 5), 4.0)):
        topo = tree.build_topology(T, 2, splits)
        lat, _ = sde.rollout(topo, n, g, sigma, s, seed=11, velocity_fn=_vel(mu, g))
        z0 = lat[0].astype(np.float64)
        for leaf in topo.leaf_ids():
            resid = lat[leaf] - P * z0
            assert abs(resid.mean()) < 4.5 * math.sqrt(V / n)
            assert abs(resid.var() - V) < 4.5 * V * math.sqrt(2 / n)
        # with mu != 0 the mean path (1 - t) mu is followed exactly
    mu2 = np.full(n, 1.5)
    topo = tree.build_topology(T, 2, (0, 3))
    lat, _ = sde.rollout(topo, n, g, sigma, math.inf, seed=11, velocity_fn=_vel(mu2, g))
    resid = lat[-1] - (1.5 + P * lat[0].astype(np.float64))
    assert abs(resid.mean()) < 4.5 * math.sqrt(V / n)


def test_branch_noise_covariance():
    """Var(xi_b) = 1 and Cov(xi_b, xi_b') = 1/(1+s^2) (appendix, Branch Noise Construction)."""
    n = 1 << 20
    xi0 = philox.node_noise(5, 10, 2, philox.TAG_SHARED, n)
    e1 = philox.node_noise(5, 21, 2, philox.TAG_INNOV, n)
    e2 = philox.node_noise(5, 22, 2, philox.TAG_INNOV, n)
    for s in (1.0, 2.0, 4.0, 8.0):
        a, b = sde.branch_noise(xi0, e1, s), sde.branch_noise(xi0, e2, s)
        assert abs(a.var() - 1) < 5 * math.sqrt(2 / n) and abs(b.var() - 1) < 5 * math.sqrt(2 / n)
        assert abs(np.mean(a * b) - 1 / (1 + s * s)) < 5 / math.sqrt(n)
    assert sde.branch_noise(xi0, e1, math.inf) is e1
    assert np.allclose(sde.branch_noise(xi0, e1, 0.0), xi0)


def test_split_children_share_mean_and_use_eq2():
    """Children of one parent differ only through their noises, and with finite s their
    noises have the stated correlation; parents are stored once."""
    T, n, sigma, s = 3, 1 << 16, 0.3, 2.0
    g = _grid(T)
    topo = tree.build_topology(T, 2, (1,))
    mu = np.zeros(n)
    lat, logp, means = sde.rollout(topo, n, g, sigma, s, seed=2, velocity_fn=_vel(mu, g), return_means=True)
    c0, c1 = topo.children(1)
    assert np.array_equal(means[c0], means[c1])
    gi = sde.noise_scale(sigma, g[1] - g[2])
    x0, x1 = (lat[c0] - means[c0]) / gi, (lat[c1] - means[c1]) / gi
    assert abs(np.mean(x0 * x1) - 1 / (1 + s * s)) < 6 / math.sqrt(n)
    # a non-split step draws exactly the child's INNOV stream
    only = topo.children(0)[0]
    eta = philox.node_noise(2, only, 0, philox.TAG_INNOV, n)
    g0 = sde.noise_scale(sigma, g[0] - g[1])
    assert np.allclose((lat[only] - means[only]) / g0, eta, atol=2e-5)


def test_logp_is_the_library_gaussian_log_density():
    rng = np.random.default_rng(1)
    mean = rng.standard_normal(257)
    g = 0.075
    z = (mean + g * rng.standard_normal(257)).astype(np.float32)
    ref = stats.norm.logpdf(z.astype(np.float64), loc=mean, scale=g)
    assert math.isclose(sde.transition_logp(z, mean, g), ref.mean(), rel_tol=1e-12)
    assert math.isclose(sde.transition_logp(z[:1], mean[:1], g), ref[0], rel_tol=1e-12)
    # joint density of the D-dimensional isotropic Gaussian = D * per-element mean
    joint = stats.multivariate_normal.logpdf(z.astype(np.float64), mean=mean, cov=g * g)
    assert math.isclose(257 * sde.transition_logp(z, mean, g), joint, rel_tol=1e-10)


def test_rollout_logp_expected_value_and_recompute():
    T, n, sigma = 4, 1 << 15, 0.3
    g = _grid(T)
    mu = np.random.default_rng(0).standard_normal(n)
    topo = tree.build_topology(T, 2, (0, 2))
    vel = _vel(mu, g)
    lat, logp = sde.rollout(topo, n, g, sigma, math.inf, seed=42, velocity_fn=vel, tree_id=3, nodes_cap=20)
    for c in range(1, topo.nodes):
        i = int(topo.depth[c]) - 1
        gi = sigma * math.sqrt(g[i] - g[i + 1])
        expect = -0.5 - math.log(gi) - 0.5 * math.log(2 * math.pi)
        assert abs(logp[c] - expect) < 5 * math.sqrt(0.5 / n)     # Var(xi^2/2) = 1/2
        p = int(topo.parent[c])
        again = sde.edge_logp(lat[p], lat[c], vel(lat[p], i, p), g[i], g[i] - g[i + 1], sigma)
        assert again == logp[c]
    # node ids enter the stream: another tree id gives another root
    lat2, _ = sde.rollout(topo, 64, g, sigma, math.inf, seed=42, velocity_fn=lambda z, i, p: vel(np.pad(z, (0, n - 64)), i, p)[:64],
                          tree_id=4, nodes_cap=20)
    assert not np.array_equal(lat2[0], lat[0][:64])
    assert np.array_equal(lat[0], philox.node_noise(42, 60, 0, philox.TAG_ROOT, n).astype(np.float32))


def test_element_slices_agree_with_whole_rows():
    T, n = 4, 512
    g = _grid(T)
    mu = np.random.default_rng(5).standard_normal(n)
    topo = tree.build_topology(T, 2, (0, 2))
    full, _ = sde.rollout(topo, n, g, 0.3, 2.0, seed=1, velocity_fn=_vel(mu, g))
    part, _ = sde.rollout(topo, 64, g, 0.3, 2.0, seed=1, velocity_fn=_vel(mu[128:192], g), elem_start=128)
    assert np.array_equal(part, full[:, 128:192])


def test_hybrid_ode_sde_schedule():
    """ODE steps are deterministic (child = mean, log-prob 0), SDE steps unchanged, and a hybrid schedule still
    carries N(0,1) onto N(mu, s0^2) in the limit (every step, ODE or SDE, preserves the marginals)."""
    T, n = 6, 4096
    g = _grid(T)
    mu = np.zeros(n)
    topo = tree.build_topology(T, 2, (0, 3))
    sde_steps = [0, 3, 4]
    lat, logp, means = sde.rollout(topo, n, g, 0.3, math.inf, seed=9, velocity_fn=_vel(mu, g), return_means=True, sde_steps=sde_steps)
    full, logp_full = sde.rollout(topo, n, g, 0.3, math.inf, seed=9, velocity_fn=_vel(mu, g))
    for c in range(1, topo.nodes):
        i = int(topo.depth[c]) - 1
        if i in sde_steps:
            assert logp[c] != 0.0 and not np.array_equal(lat[c], means[c].astype(np.float32))
        else:
            assert logp[c] == 0.0 and np.array_equal(lat[c], means[c].astype(np.float32))
    # the first step is SDE in both runs and draws the same noise
    assert np.array_equal(lat[1], full[1]) and logp[1] == logp_full[1]
    # all-ODE equals the sigma = 0 rollout
    a, _ = sde.rollout(tree.build_topology(T, 2, ()), 64, g, 0.3, math.inf, seed=9, velocity_fn=_vel(mu[:64], g), sde_steps=[])
    b, _ = sde.rollout(tree.build_topology(T, 2, ()), 64, g, 0.0, math.inf, seed=9, velocity_fn=_vel(mu[:64], g))
    assert np.array_equal(a, b)
    # marginal preservation with every other step stochastic
    gaps = []
    for TT in (256, 2048):
        gg = _grid(TT)
        P, V = 1.0, 0.0
        for i in range(TT):
            t, h = gg[i], gg[i] - gg[i + 1]
            sig = 0.5 if i % 2 == 0 else 0.0
            f = lambda z: sde.em_mean(np.array([z]), sde.linear_velocity(np.array([z]), t, np.array([0.0]), S0), t, h, sig)[0]
            a_ = f(1.0) - f(0.0)
            P *= a_
            V = a_ * a_ * V + sde.noise_scale(sig, h) ** 2
        gaps.append(abs(P * P + V - S0 ** 2))
    assert gaps[1] < gaps[0] and gaps[1] < 5e-4
    with pytest.raises(AssertionError):
        sde.rollout(topo, 8, g, 0.3, math.inf, seed=9, velocity_fn=_vel(mu[:8], g), sde_steps=[3])   # split step 0 must be SDE
