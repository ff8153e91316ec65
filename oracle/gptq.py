"""CPU oracle of the weight quantizer the paper's experiments use: GPTQ with act-order (Sec. 4 "Quantization
Details": "GPTQ ... with act-order", per-channel symmetric 4-bit weights; Sec. 3.1 Remark 2 discusses its error bound
under expansion).  Test infrastructure only: plain numpy in fp64, in the order the GPTQ algorithm is published,
no blocking and no lazy batching.

The method works on the rows of the already expanded and rotated weight matrix W (one row per output channel,
K' columns) and on the Hessian H = X_hat^T X_hat of the layer's expanded, rotated calibration activations (K' x K').

Steps:
  1. damping: H <- H + damp * mean(diag H) * I; a channel whose diagonal entry is 0 gets the entry 1 and its weights 0;
  2. act-order: the channels are visited in descending order of diag(H) (stable for equal entries);
  3. U = upper Cholesky factor of H^-1 (H^-1 = U^T U), for the permuted H;
  4. every row keeps ONE scale for all its columns, s = max |w| / 7 of the unmodified row (1 for a zero row), rounded
     to fp32 as in the round-to-nearest path; the grid is the symmetric one, codes clamp to [-8, 7];
  5. columns j = 0, 1, ... in the visiting order: q_j = clamp(rne(w_j / s)); e_j = (w_j - s q_j) / U[j, j];
     every later column k > j receives w_k <- w_k - e_j U[j, k] (error feedback);
  6. the codes return to the original channel order.
The objective the method descends on is tr((W - Q) H (W - Q)^T) with Q = s * codes.
"""
from __future__ import annotations

import numpy as np


def act_order(H: np.ndarray) -> np.ndarray:
    """Visiting order: channel indices by descending diagonal of H, ties in ascending index."""
    return np.argsort(-np.diag(np.asarray(H, dtype=np.float64)), kind="stable")


def damped(H: np.ndarray, damp: float) -> tuple[np.ndarray, np.ndarray]:
    """(H with dead channels fixed and the damping added, mask of the dead channels)."""
    H = np.array(H, dtype=np.float64, copy=True)
    dead = np.diag(H) == 0.0
    H[dead, dead] = 1.0
    H[np.diag_indices_from(H)] += damp * np.mean(np.diag(H))
    return H, dead


def row_scales(W: np.ndarray) -> np.ndarray:
    """Per-row scale absmax / 7 (1 for a zero row), rounded to fp32 (the form in which it is stored)."""
    amax = np.max(np.abs(W), axis=1)
    s = np.where(amax > 0, amax / 7.0, 1.0)
    return s.astype(np.float32)


def gptq_quantize(W: np.ndarray, H: np.ndarray, damp: float = 0.01, order: bool = True):
    """codes int8 [N, K'] (original channel order), scales float32 [N]."""
    W = np.array(W, dtype=np.float64, copy=True)
    N, n = W.shape
    assert H.shape == (n, n)
    Hd, dead = damped(H, damp)
    W[:, dead] = 0.0
    s32 = row_scales(W)
    s = s32.astype(np.float64)
    perm = act_order(Hd) if order else np.arange(n)
    Wp = W[:, perm]
    Hp = Hd[np.ix_(perm, perm)]
    U = np.linalg.cholesky(np.linalg.inv(Hp)).T  # upper triangular, H^-1 = U^T U
    Q = np.zeros((N, n), dtype=np.int8)
    for j in range(n):
        q = np.clip(np.rint(Wp[:, j] / s), -8, 7)
        Q[:, j] = q.astype(np.int8)
        e = (Wp[:, j] - s * q) / U[j, j]
        Wp[:, j + 1:] -= np.outer(e, U[j, j + 1:])
    codes = np.empty_like(Q)
    codes[:, perm] = Q
    return codes, s32


def objective(W: np.ndarray, codes: np.ndarray, scales: np.ndarray, H: np.ndarray) -> float:
    """tr((W - Q) H (W - Q)^T), Q = scales[:, None] * codes, in fp64."""
    D = np.asarray(W, dtype=np.float64) - scales.astype(np.float64)[:, None] * codes.astype(np.float64)
    return float(np.einsum("ij,jk,ik->", D, np.asarray(H, dtype=np.float64), D))


def hessian(y: np.ndarray) -> np.ndarray:
    """H = Y^T Y of the (expanded, rotated) calibration activations Y [tokens, K'], fp64."""
    y = np.asarray(y, dtype=np.float64)
    return y.T @ y
