"""Distillation of the prefetch router from the frozen router (Sec. IV-C, Eq. (10)), on the CPU.

TEST INFRASTRUCTURE: the reference for ``apex_distill_router``.  Plain NumPy in fp64.

The prefetch router is a linear layer followed by a softmax, q_p = softmax(W_p h + b_p), fed with the hidden
state *before* attention; the teacher is the router's distribution q_r on the state *after* attention.  The loss is
the mean over the calibration tokens of KL(q_r || q_p) = sum_i q_r(i) log(q_r(i) / q_p(i)); its gradient with respect
to the student's logits is (q_p - q_r) / T.  Full-batch Adam (0.9 / 0.999 / 1e-8), fixed iteration count.
"""
from __future__ import annotations

import numpy as np


def softmax_rows(Z: np.ndarray) -> np.ndarray:
    Z = Z - Z.max(axis=1, keepdims=True)
    P = np.exp(Z)
    return P / P.sum(axis=1, keepdims=True)


def kl_loss(H: np.ndarray, Qr: np.ndarray, W: np.ndarray, b: np.ndarray) -> float:
    """Mean over tokens of KL(q_r || softmax(W h + b)); terms with q_r(i) = 0 contribute nothing."""
    Qp = softmax_rows(H.astype(np.float64) @ W.astype(np.float64).T + b.astype(np.float64))
    Qr = Qr.astype(np.float64)
    with np.errstate(divide="ignore", invalid="ignore"):
        t = np.where(Qr > 0, Qr * (np.log(Qr) - np.log(Qp)), 0.0)
    return float(t.sum(axis=1).mean())


def distill(H: np.ndarray, Qr: np.ndarray, W0: np.ndarray, b0: np.ndarray, iters: int = 200, lr: float = 0.01):
    """Returns (W [N][d], b [N]) in fp64 after `iters` Adam steps from (W0, b0)."""
    H = H.astype(np.float64)
    Qr = Qr.astype(np.float64)
    T = H.shape[0]
    W = W0.astype(np.float64).copy()
    b = b0.astype(np.float64).copy()
    mW = np.zeros_like(W); vW = np.zeros_like(W)
    mb = np.zeros_like(b); vb = np.zeros_like(b)
    for it in range(1, iters + 1):
        Qp = softmax_rows(H @ W.T + b)
        G = (Qp - Qr) / T                       # d loss / d logits
        gW = G.T @ H
        gb = G.sum(axis=0)
        c1, c2 = 1.0 - 0.9 ** it, 1.0 - 0.999 ** it
        mW = 0.9 * mW + 0.1 * gW; vW = 0.999 * vW + 0.001 * gW * gW
        mb = 0.9 * mb + 0.1 * gb; vb = 0.999 * vb + 0.001 * gb * gb
        W = W - lr * (mW / c1) / (np.sqrt(vW / c2) + 1e-8)
        b = b - lr * (mb / c1) / (np.sqrt(vb / c2) + 1e-8)
    return W, b
