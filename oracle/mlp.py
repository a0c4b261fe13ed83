"""Per-token MLP velocity stand-in for the denoiser (oracle, test infrastructure).

The paper's mu_theta is a large network (FLUX.1-Dev, Wan2.1); the workloads here
replace it by a seeded per-token MLP  channels -> hidden -> channels  with GELU,
bf16 operands and wide accumulation.  The precision of that stand-in is fixed
by the workload definition, so the oracle emulates it step by step:

    zb = bf16(z)                      round-to-nearest-even
    h  = zb @ W1                      exact products, float64 accumulation
    a  = bf16(GELU(h))                GELU(x) = x/2 (1 + erf(x / sqrt 2))
    v  = float32(a @ W2)              float64 accumulation, float32 output

No bias and no time input (the workload gives none).
"""
from __future__ import annotations

import numpy as np
from scipy.special import erf


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round float32 to the nearest bf16 (ties to even); returns the value as float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    u = (u + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).reshape(np.shape(x))


def gelu_erf(x: np.ndarray) -> np.ndarray:
    return 0.5 * x * (1.0 + erf(x / np.sqrt(2.0)))


def mlp_velocity(z_tokens: np.ndarray, W1: np.ndarray, W2: np.ndarray, chunk: int = 8192) -> np.ndarray:
    """z_tokens float32 [n_tokens][channels]; W1 [channels][hidden], W2 [hidden][channels]
    (values bf16-representable).  Returns float32 [n_tokens][channels]."""
    z_tokens = np.asarray(z_tokens, dtype=np.float32)
    W1d = np.asarray(W1, dtype=np.float64)
    W2d = np.asarray(W2, dtype=np.float64)
    out = np.empty((z_tokens.shape[0], W2d.shape[1]), dtype=np.float32)
    for a in range(0, z_tokens.shape[0], chunk):
        zb = bf16_round(z_tokens[a:a + chunk]).astype(np.float64)
        h = zb @ W1d
        act = bf16_round(gelu_erf(h).astype(np.float32)).astype(np.float64)
        out[a:a + chunk] = (act @ W2d).astype(np.float32)
    return out
