"""ORACLE (test infrastructure, CPU only): per-minibatch loss and gradient of each model, in fp64.

``loss_and_grad(model, w, Xb, yb)`` returns ``(sum_q f(w; x_q, y_q), (1/m) sum_q grad f)`` for the
m rows of the minibatch: the stochastic gradient g(w, xi) of Section 2.2 (text under Eq. 2) of the
empirical risk of Eq. 1.  Parameters arrive as the fp32 values the server stores and every
operation below is carried out in fp64, so the result does not depend on summation order to the
accuracy the parity tests need.  Rows drawn twice count twice.

Models (the paper's analysis is for a generic differentiable f; these are the four used here):
  lsq       f = 1/2 (x.w - y)^2
  logistic  labels b in {0,1}, z = x.w, f = softplus(z) - b z, grad = (sigmoid(z) - b) x
  softmax   W in R^{C x d} (row-major in the parameter vector), f = -log softmax(W x)[label]
  mlp2      h = relu(W1^T x + b1), z = W2^T h + b2, f = -log softmax(z)[label]; parameter vector
            = [W1 (d x H, row-major), b1 (H), W2 (H x C, row-major), b2 (C)].  The two products
            with the d-sized dimension (x W1 and x^T delta1) take operands rounded to bfloat16
            (x, W1, delta1), as a bf16 tensor-core implementation does; everything else is
            unrounded.
"""
from __future__ import annotations

import numpy as np


def n_params(model: str, d: int, n_classes: int = 1, hidden: int = 0) -> int:
    if model in ("lsq", "logistic"):
        return d
    if model == "softmax":
        return n_classes * d
    if model == "mlp2":
        return d * hidden + hidden + hidden * n_classes + n_classes
    raise ValueError(model)


def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round to the nearest bfloat16 (ties to even), returned as fp64.

    The value is first rounded to fp32 (the precision the rounded tensor has on the device) and
    then its low 16 bits are rounded away."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) >> 16 << 16
    return u.astype(np.uint32).view(np.float32).astype(np.float64)


def _softmax_ce(Z: np.ndarray, label: np.ndarray):
    """Per-row loss -log softmax(Z)[label] and dLoss/dZ = softmax(Z) - onehot(label)."""
    zmax = Z.max(axis=1, keepdims=True)
    E = np.exp(Z - zmax)
    S = E.sum(axis=1, keepdims=True)
    lse = np.log(S[:, 0]) + zmax[:, 0]
    rows = np.arange(Z.shape[0])
    loss = lse - Z[rows, label]
    D = E / S
    D[rows, label] -= 1.0
    return loss, D


def loss_and_grad(model: str, w: np.ndarray, Xb: np.ndarray, yb: np.ndarray, n_classes: int = 1,
                  hidden: int = 0, bf16: bool = True):
    w = np.asarray(w, dtype=np.float64)
    Xb = np.asarray(Xb, dtype=np.float64)
    m, d = Xb.shape
    if model == "lsq":
        r = Xb @ w - np.asarray(yb, dtype=np.float64)
        return 0.5 * float(r @ r), (Xb.T @ r) / m
    if model == "logistic":
        b = np.asarray(yb, dtype=np.float64)
        z = Xb @ w
        softplus = np.maximum(z, 0.0) + np.log1p(np.exp(-np.abs(z)))
        ez = np.exp(-np.abs(z))
        sig = np.where(z >= 0, 1.0 / (1.0 + ez), ez / (1.0 + ez))
        return float(np.sum(softplus - b * z)), (Xb.T @ (sig - b)) / m
    lab = np.asarray(yb, dtype=np.int64)
    if model == "softmax":
        W = w.reshape(n_classes, d)
        loss, D = _softmax_ce(Xb @ W.T, lab)
        return float(loss.sum()), ((D.T @ Xb) / m).reshape(-1)
    if model == "mlp2":
        H, Cc = hidden, n_classes
        o1, o2, o3 = d * H, d * H + H, d * H + H + H * Cc
        W1, b1, W2, b2 = w[:o1].reshape(d, H), w[o1:o2], w[o2:o3].reshape(H, Cc), w[o3:]
        q = bf16_round if bf16 else (lambda a: np.asarray(a, dtype=np.float64))
        Xq = q(Xb)
        A1 = Xq @ q(W1) + b1
        Hh = np.maximum(A1, 0.0)
        loss, D2 = _softmax_ce(Hh @ W2 + b2, lab)
        D1 = (D2 @ W2.T) * (A1 > 0.0)
        g = np.concatenate([(Xq.T @ q(D1)).reshape(-1), D1.sum(axis=0),
                            (Hh.T @ D2).reshape(-1), D2.sum(axis=0)]) / m
        return float(loss.sum()), g
    raise ValueError(model)


def full_loss(model: str, w: np.ndarray, X: np.ndarray, y: np.ndarray, n_classes: int = 1, hidden: int = 0,
              bf16: bool = True, rows: int = 8192) -> float:
    """Empirical risk F(w) = (1/N) sum_n f(w, xi_n) over the whole data set (Eq. 1), fp64, in row
    blocks so that a large X needs no fp64 copy."""
    total = 0.0
    for a in range(0, X.shape[0], rows):
        total += loss_and_grad(model, w, X[a:a + rows], y[a:a + rows], n_classes, hidden, bf16)[0]
    return total / X.shape[0]
