"""CPU oracle of the expert similarity that the clustering step consumes (Sec. 3.1, Eq. 2-4).  TEST INFRASTRUCTURE ONLY.

    Eq. 2   S_param(i, j) = <w_i, w_j> / (|w_i| |w_j|),  w_i = expert i's weight matrix, flattened
    Eq. 3   S_task(i, j)  = <mu_i, mu_j> / (|mu_i| |mu_j|),  mu_i = expert i's activation centroid (Eq. 5 maintains it)
    Eq. 4   S = alpha S_param + (1 - alpha) S_task,  0 <= alpha <= 1

in numpy fp64, each formula written out as it stands.  Reading (the paper does not say): a vector of norm zero has
similarity 0 to every other vector and 1 to itself.

Pins (tests/test_similarity_oracle.py): hand-worked vectors at known angles (60 degrees, orthogonal, opposite, a
scaled copy); scikit-learn's cosine_similarity on random inputs; symmetry, unit diagonal, |S| <= 1 and a positive
semi-definite S_param; Eq. 4 at alpha = 0, 1 and its linearity in alpha.
"""
from __future__ import annotations

import numpy as np


def cosine_matrix(V: np.ndarray) -> np.ndarray:
    """V [E][n] -> [E][E] of <v_i, v_j> / (|v_i| |v_j|) (Eq. 2 / Eq. 3)."""
    V = np.asarray(V, dtype=np.float64).reshape(V.shape[0], -1)
    E = V.shape[0]
    out = np.zeros((E, E))
    norm = np.sqrt((V * V).sum(axis=1))
    for i in range(E):
        for j in range(E):
            if norm[i] > 0 and norm[j] > 0:
                out[i, j] = float(V[i] @ V[j]) / (norm[i] * norm[j])
            else:
                out[i, j] = 1.0 if i == j else 0.0
    return out


def fused_similarity(W: np.ndarray, mu: np.ndarray, alpha: float) -> dict:
    """W [E][...] expert weights, mu [E][d] centroids -> dict(S_param, S_task, S) (Eq. 2-4)."""
    assert 0.0 <= alpha <= 1.0
    S_param = cosine_matrix(W)
    S_task = cosine_matrix(mu)
    return dict(S_param=S_param, S_task=S_task, S=alpha * S_param + (1.0 - alpha) * S_task)
