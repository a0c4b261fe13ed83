"""Euler-Maruyama flow-SDE rollout over a tree (oracle, test infrastructure).

What the paper fixes
--------------------
* grid t_0 > t_1 > ... > t_T, h_i = t_i - t_{i+1}; one step is
  z_{i+1} = mu_theta(z_i, t_i) + g_i * eta_i,  g_i = g(t_i) * sqrt(h_i)
  (appendix "Branch Noise Construction");
* at a split step the K children share the mean and take the noises
  xi_b = (xi_0 + s * eta_b) / sqrt(1 + s^2), xi_0 shared, eta_b per branch,
  fresh at each split (Eq. 2);
* one root noise z_0 ~ N(0, I) per prompt ("Branch sampling"; "Init same noise").

Readings (the paper leaves mu_theta, f, g, epsilon of Eq. 1 uninstantiated)
--------------------------------------------------------------------------
* rectified-flow path z_t = (1 - t) x_0 + t * eps with velocity v = dz/dt, whose
  score is  grad log p_t(z) = -(z + (1 - t) v) / t;
* constant diffusion g(t) = sigma (the "Eta" hyper-parameter);
* reverse-time drift that keeps the marginals of the probability-flow ODE:
  mu_theta(z, t_i) = z - h_i v + (sigma^2 h_i / 2) * score
  (the drift-plus-score structure of Eq. 1);
* transition log-prob of the Gaussian step, normalised per element:
  log pi = -(1/D) sum_e (z'_e - mu_e)^2 / (2 g_i^2) - ln g_i - 0.5 ln(2 pi);
  multiply by D (and add nothing) for the joint log-density;
* s = +inf means xi_b = eta_b (independent children); a non-split step draws its
  single noise from the INNOV stream of the child.

Latents are stored as float32 (the state format of the latent pool); all
arithmetic between two stored states is float64.
"""
from __future__ import annotations

import math
from typing import Callable, Optional

import numpy as np

from . import philox
from .tree import Topology


def linear_velocity(z: np.ndarray, t: float, mu: np.ndarray, s0: float) -> np.ndarray:
    """Exact velocity field of the path z_t = (1-t) x_0 + t eps with x_0 ~ N(mu, s0^2 I), eps ~ N(0, I):
    the marginal is N((1-t) mu, c_t I), c_t = (1-t)^2 s0^2 + t^2, and
    v(z, t) = -mu + k_t (z - (1-t) mu),  k_t = (t - (1-t) s0^2) / c_t."""
    c_t = (1.0 - t) ** 2 * s0 ** 2 + t ** 2
    k_t = (t - (1.0 - t) * s0 ** 2) / c_t
    return -mu + k_t * (z - (1.0 - t) * mu)


def score_from_velocity(z: np.ndarray, v: np.ndarray, t: float) -> np.ndarray:
    """grad log p_t(z) = -E[eps | z] / t with E[eps | z] = z + (1 - t) v."""
    return -(z + (1.0 - t) * v) / t


def em_mean(z: np.ndarray, v: np.ndarray, t: float, h: float, sigma: float) -> np.ndarray:
    """mu_theta(z_i, t_i): one reverse-time Euler step of drift -v + (sigma^2/2) * score."""
    return z - h * v + 0.5 * sigma ** 2 * h * score_from_velocity(z, v, t)


def noise_scale(sigma: float, h: float) -> float:
    """g_i = g(t_i) sqrt(h_i) with g(t) = sigma."""
    return sigma * math.sqrt(h)


def branch_noise(xi0: np.ndarray, eta: np.ndarray, s: float) -> np.ndarray:
    """xi_b = (xi_0 + s eta_b) / sqrt(1 + s^2)  (Eq. 2); s = inf gives eta_b."""
    if math.isinf(s):
        return eta
    return (xi0 + s * eta) / math.sqrt(1.0 + s * s)


def transition_logp(z_child: np.ndarray, mean: np.ndarray, g: float) -> float:
    """Per-element mean of the Gaussian log-density of z_child under N(mean, g^2 I)."""
    if g == 0.0:
        return 0.0   # deterministic step: no density; the library writes 0
    d = np.asarray(z_child, dtype=np.float64) - mean
    return float(-np.mean(d * d) / (2.0 * g * g) - math.log(g) - 0.5 * math.log(2.0 * math.pi))


def root_latent(seed: int, root_id: int, n: int, elem_start: int = 0) -> np.ndarray:
    """z_0 ~ N(0, I) from the ROOT stream, rounded to the float32 state format."""
    return _noise(seed, root_id, 0, philox.TAG_ROOT, n, elem_start).astype(np.float32)


def _noise(seed, node_id, step, tag, n, elem_start):
    return philox.node_noise(seed, node_id, step, tag, n, elem_start)


VelocityFn = Callable[[np.ndarray, int, int], np.ndarray]
"""velocity_fn(z_parent float32 [n], step i, local parent index) -> v [n] (float64 or float32)."""


def rollout(topo: Topology, n_elem: int, t_grid, sigma: float, s: float, seed: int,
            velocity_fn: VelocityFn, tree_id: int = 0, nodes_cap: Optional[int] = None,
            elem_start: int = 0, return_means: bool = False, sde_steps=None):
    """Grow one tree (Algorithm 1, "Build rollout tree"): the root from the ROOT stream,
    then for i = 0..T-1 every node of depth i is advanced once, to K children at a split
    step and to one child otherwise.

    n_elem elements starting at element index elem_start of each latent row are
    computed (the whole row by default); log-probs are only meaningful for whole rows.
    Global node id (the Philox counter word) = tree_id * nodes_cap + local index.

    sde_steps: the hybrid ODE-SDE schedule of the ablation "Hybrid ODE-SDE" (all branching steps
    stay SDE, a window picks further SDE steps, the remaining updates are ODE steps): an iterable
    of the steps that are stochastic; None = all.  An ODE step uses sigma = 0 (drift -v, no noise,
    log-prob 0); a split step must be an SDE step.

    Returns (latents float32 [nodes][n_elem], logp float64 [nodes]) and, on request,
    the float64 means of every non-root node.
    """
    t = np.asarray(t_grid, dtype=np.float64)
    assert t.shape == (topo.T + 1,) and np.all(np.diff(t) < 0) and t[-2] > 0
    cap = topo.nodes if nodes_cap is None else nodes_cap
    base = tree_id * cap
    lat = np.zeros((topo.nodes, n_elem), dtype=np.float32)
    logp = np.zeros(topo.nodes, dtype=np.float64)
    means = np.zeros((topo.nodes, n_elem), dtype=np.float64) if return_means else None
    lat[0] = root_latent(seed, base, n_elem, elem_start)
    sde = None if sde_steps is None else set(int(x) for x in sde_steps)
    sigma_all = sigma
    for i in range(topo.T):
        h = float(t[i] - t[i + 1])
        sigma = sigma_all if (sde is None or i in sde) else 0.0
        is_split = i in topo.splits
        assert not (is_split and sigma == 0.0 and sigma_all != 0.0), "a split step must be an SDE step"
        g = noise_scale(sigma, h)
        for p in topo.level(i):
            z = lat[p].astype(np.float64)
            v = np.asarray(velocity_fn(lat[p], i, p), dtype=np.float64)
            mean = em_mean(z, v, float(t[i]), h, sigma)
            kids = topo.children(p)
            xi0 = None
            if is_split and not math.isinf(s) and g != 0.0:
                xi0 = _noise(seed, base + p, i, philox.TAG_SHARED, n_elem, elem_start)
            for c in kids:
                if g != 0.0:
                    eta = _noise(seed, base + c, i, philox.TAG_INNOV, n_elem, elem_start)
                    xi = branch_noise(xi0, eta, s) if is_split else eta
                    child = mean + g * xi
                else:
                    child = mean
                lat[c] = child.astype(np.float32)
                logp[c] = transition_logp(lat[c], mean, g)
                if return_means:
                    means[c] = mean
    if return_means:
        return lat, logp, means
    return lat, logp


def edge_logp(z_parent: np.ndarray, z_child: np.ndarray, v: np.ndarray, t: float, h: float, sigma: float) -> float:
    """log pi(z_child | z_parent) of one edge under a given velocity: the numerator or
    denominator of the ratio rho_e in Eq. 5, and the summand of s_l in Eq. 3."""
    mean = em_mean(np.asarray(z_parent, np.float64), np.asarray(v, np.float64), t, h, sigma)
    return transition_logp(z_child, mean, noise_scale(sigma, h))
