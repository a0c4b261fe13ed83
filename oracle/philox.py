"""Counter-based Gaussian noise for the oracle (test infrastructure).

The paper only says the noises are N(0, I) draws (Eq. 2; appendix "Branch
Noise Construction": fresh (xi_0, {eta_b}) at every split step, no cross-time
sharing).  To make every draw reproducible the library *defines* the stream:

* generator: Philox4x32-10 exactly as published by Salmon, Moraes, Dror and
  Shaw, "Parallel random numbers: as easy as 1, 2, 3" (SC'11);
* key     = (seed low word, seed high word);
* counter = (element // 4, global node id, step index, stream tag);
* the four output words give the four elements 4*(element//4) + 0..3;
* uniform: u = ((x >> 9) + 0.5) * 2**-23, a 24-bit number strictly inside (0,1)
  that float32 holds exactly;
* normal: Box-Muller on word pairs (0,1) and (2,3):
  r = sqrt(-2 ln u_a), (r cos 2 pi u_b, r sin 2 pi u_b).

Everything here is float64; nothing is rounded.
"""
from __future__ import annotations

import numpy as np

PHILOX_M0 = 0xD2511F53
PHILOX_M1 = 0xCD9E8D57
PHILOX_W0 = 0x9E3779B9
PHILOX_W1 = 0xBB67AE85
MASK32 = 0xFFFFFFFF

TAG_ROOT = 0     # root latent z_0, keyed by the root's node id, step 0
TAG_SHARED = 1   # xi_0 of Eq. 2, keyed by the PARENT's node id
TAG_INNOV = 2    # eta_b of Eq. 2 and the noise of every non-split step, keyed by the CHILD's node id


def philox4x32_10(counter: np.ndarray, key) -> np.ndarray:
    """Philox4x32 with 10 rounds.  counter: (..., 4) integers < 2**32; key: 2 integers.
    Returns uint32 (..., 4).  One round maps (c0,c1,c2,c3) to
    (hi(M1*c2) ^ c1 ^ k0, lo(M1*c2), hi(M0*c0) ^ c3 ^ k1, lo(M0*c0)); the key is
    advanced by the Weyl constants between rounds."""
    c = np.asarray(counter).astype(np.uint64) & MASK32
    c0, c1, c2, c3 = (c[..., i].copy() for i in range(4))
    k0 = np.uint64(int(key[0]) & MASK32)
    k1 = np.uint64(int(key[1]) & MASK32)
    for rnd in range(10):
        if rnd > 0:
            k0 = np.uint64((int(k0) + PHILOX_W0) & MASK32)
            k1 = np.uint64((int(k1) + PHILOX_W1) & MASK32)
        p0 = np.uint64(PHILOX_M0) * c0   # < 2**64, no overflow
        p1 = np.uint64(PHILOX_M1) * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & np.uint64(MASK32)
        hi1, lo1 = p1 >> np.uint64(32), p1 & np.uint64(MASK32)
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def uniform_open(words: np.ndarray) -> np.ndarray:
    """Map uint32 words to float64 uniforms ((x >> 9) + 0.5) / 2**23 in (0, 1)."""
    return ((np.asarray(words, dtype=np.uint32) >> np.uint32(9)).astype(np.float64) + 0.5) * 2.0 ** -23


def box_muller(words: np.ndarray) -> np.ndarray:
    """(..., 4) uint32 -> (..., 4) float64 standard normals."""
    u = uniform_open(words)
    out = np.empty(u.shape, dtype=np.float64)
    for a, b in ((0, 1), (2, 3)):
        r = np.sqrt(-2.0 * np.log(u[..., a]))
        th = 2.0 * np.pi * u[..., b]
        out[..., a] = r * np.cos(th)
        out[..., b] = r * np.sin(th)
    return out


def seed_key(seed: int):
    return (seed & MASK32, (seed >> 32) & MASK32)


def noise_words(seed: int, node_id: int, step: int, tag: int, n_elements: int, elem_start: int = 0) -> np.ndarray:
    """The raw integer stream of one (node, step, tag) for elements
    [elem_start, elem_start + n_elements): uint32 (ceil(n/4), 4).  elem_start % 4 == 0."""
    assert elem_start % 4 == 0
    nblk = (n_elements + 3) // 4
    ctr = np.empty((nblk, 4), dtype=np.uint64)
    ctr[:, 0] = np.arange(nblk, dtype=np.uint64) + np.uint64(elem_start // 4)
    ctr[:, 1] = node_id
    ctr[:, 2] = step
    ctr[:, 3] = tag
    return philox4x32_10(ctr, seed_key(seed))


def node_noise(seed: int, node_id: int, step: int, tag: int, n_elements: int, elem_start: int = 0) -> np.ndarray:
    """float64 N(0,1) draws of one (node, step, tag) for elements [elem_start, elem_start + n_elements)."""
    return box_muller(noise_words(seed, node_id, step, tag, n_elements, elem_start)).reshape(-1)[:n_elements]
