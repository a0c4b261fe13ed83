"""Leaf-reward stand-ins (oracle, test infrastructure).

The paper scores leaves with learned reward models (Algorithm 1, "Evaluate
rewards for leaves"); those are outside this library.  The workloads use two
closed-form stand-ins computed from the leaf latent, in float64:

    neg_mse(z, target) = -mean_e (z_e - target_e)^2
    cosine(z, target)  = <z, target> / (|z| |target|)
"""
from __future__ import annotations

import numpy as np


def neg_mse(z_leaf: np.ndarray, target: np.ndarray) -> float:
    d = np.asarray(z_leaf, dtype=np.float64) - np.asarray(target, dtype=np.float64)
    return float(-np.mean(d * d))


def cosine(z_leaf: np.ndarray, target: np.ndarray) -> float:
    a = np.asarray(z_leaf, dtype=np.float64)
    b = np.asarray(target, dtype=np.float64)
    return float(np.dot(a, b) / (np.sqrt(np.dot(a, a)) * np.sqrt(np.dot(b, b))))
