"""CPU oracle for the offline EoRA solve, Algorithm 1 steps 1-6 (test infrastructure only).

Plain numpy, float64, the steps in the paper's order and notation (Section 3, Algorithm 1), library
eigendecomposition and SVD as the steps' primitives, nothing blocked or fused.  Only the test-suite, the
smoke check and the CPU baseline leg of the benchmark may import it; it shares no code with the CUDA path.

Paper orientation throughout this file:  W, W^ in R^{d x k} (d outputs, k inputs),  X~ in R^{k x n} (n
calibration columns),  B' in R^{d x r},  A in R^{r x k};  the compensated layer is  W^ X + B' A X.
The inference library stores A_lib = A^T [k][r] and B_lib = B'^T [r][d].

    1.  dW = W - W^
    2.  X~ X~^T = Q L Q^T                      (symmetric eigendecomposition)
    3.  Q' = Q sqrt(L)
    4.  dW' = dW Q'
    5.  dW' ~ U' S' V'^T, top r                (singular value decomposition);  B' = U' S',  A' = V'^T
    6.  A = A' Q'^{-1} = A' sqrt(L)^{-1} Q^T

Reading where the paper is silent: X~ X~^T of fewer calibration columns than k (or of correlated
activations) has eigenvalues that are zero up to rounding, and step 6 divides by their square roots.  The
eigenvalues are therefore clamped from below at `floor` times the largest one before step 3 (default
1e-12, in float64 far above rounding noise and far below anything that carries signal).  A direction whose
eigenvalue was clamped contributes (almost) nothing to dW', so it is never among the top r unless r exceeds
the numerical rank, and the product B' A is insensitive to the floor (pinned in the tests).
"""
from __future__ import annotations

import numpy as np


def gram(x_tilde: np.ndarray) -> np.ndarray:
    """X~ X~^T  (k x k)."""
    x = np.asarray(x_tilde, dtype=np.float64)
    return x @ x.T


def solve(w: np.ndarray, w_hat: np.ndarray, x_tilde: np.ndarray, r: int, floor: float = 1e-12) -> dict:
    """Algorithm 1, steps 1-6.  Returns B' (d x r), A (r x k), the eigenvalues L (ascending, after the
    clamp), the top-r singular values S' of dW', and all singular values of dW' (for the loss identity)."""
    w = np.asarray(w, dtype=np.float64)
    w_hat = np.asarray(w_hat, dtype=np.float64)
    d, k = w.shape
    assert w_hat.shape == (d, k) and x_tilde.shape[0] == k and 0 < r <= min(d, k)
    # 1
    dw = w - w_hat
    # 2
    lam, q = np.linalg.eigh(gram(x_tilde))
    lam = np.maximum(lam, floor * lam.max())
    # 3
    sqrt_lam = np.sqrt(lam)
    q_prime = q * sqrt_lam[None, :]
    # 4
    dw_prime = dw @ q_prime
    # 5
    u, s, vt = np.linalg.svd(dw_prime, full_matrices=False)
    b_prime = u[:, :r] * s[None, :r]
    a_prime = vt[:r, :]
    # 6
    q_prime_inv = (q / sqrt_lam[None, :]).T          # sqrt(L)^{-1} Q^T
    a = a_prime @ q_prime_inv
    return {"B": b_prime, "A": a, "lam": lam, "sigma": s[:r].copy(), "sigma_all": s, "dW": dw}


def layer_loss(dw: np.ndarray, b_prime: np.ndarray, a: np.ndarray, x_tilde: np.ndarray) -> float:
    """|| dW X~ - B' A X~ ||_F : the layer-wise compression loss that is left after compensation."""
    x = np.asarray(x_tilde, dtype=np.float64)
    return float(np.linalg.norm((np.asarray(dw, np.float64) - np.asarray(b_prime, np.float64) @ np.asarray(a, np.float64)) @ x))


def plain_svd(dw: np.ndarray, r: int) -> tuple[np.ndarray, np.ndarray]:
    """The baseline the paper compares with: rank-r SVD of dW itself, B = U S, A = V^T."""
    u, s, vt = np.linalg.svd(np.asarray(dw, dtype=np.float64), full_matrices=False)
    return u[:, :r] * s[None, :r], vt[:r, :]


def to_library_layout(b_prime: np.ndarray, a: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """(A_lib [k][r], B_lib [r][d]) of the inference path, Y = X W^T... + (X A_lib) B_lib."""
    return np.ascontiguousarray(a.T), np.ascontiguousarray(b_prime.T)
