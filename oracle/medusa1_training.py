"""CPU oracle of the Medusa-1 training objective (paper Sec. 2.2.1, Eq. 1).  TEST INFRASTRUCTURE, NOT THE PRODUCT.

Only tests may import this module.  Plain numpy in float64, one line per formula, matrix products through numpy's
matmul; no blocking, no fusion.  Pinned by tests/test_oracle_pins.py against torch's cross-entropy and autograd in
float64, central finite differences and closed forms (zero weights, saturated logits, lambda scaling, ignored labels).
"""
from __future__ import annotations

import numpy as np


def medusa1_loss_and_grads(h, W1, W2, labels, lam=None):
    """The Medusa-1 objective (Sec. 2.2.1, Eq. 1: frozen backbone, cross-entropy of every head against the token
    k + 1 positions ahead, weighted by lambda_k) and its gradient with respect to the heads' weights, in float64.

    h [N][d]: the backbone's last hidden states at N positions (constants: the backbone is frozen).
    W1 [K][d][d], W2 [K][V][d]: the heads of Sec. 2.1.1, p^(k) = softmax(W2_k (h + SiLU(W1_k h))).
    labels [K][N] int: labels[k][n] = the token head k + 1 should predict at position n, or -1 where the sequence has
    no such token (ignored).  lam [K]: lambda_k; default 0.8^k for k = 1..K (Sec. 2.2.1 weights the heads by
    powers of a constant and names 0.8).  Where the paper sums over the positions of one sequence, the reading here is the mean over the
    labelled positions of each head, so that the value does not depend on the batch size:
        L = sum_k lambda_k * mean_n( -log p_n^(k)(labels[k][n]) ).
    -> dict(loss_per_head [K], loss, grad_w1 [K][d][d], grad_w2 [K][V][d])
    """
    h = np.asarray(h, dtype=np.float64)
    W1 = np.asarray(W1, dtype=np.float64)
    W2 = np.asarray(W2, dtype=np.float64)
    y = np.asarray(labels, dtype=np.int64)
    K, V, d = W2.shape
    N = h.shape[0]
    lam = np.array([0.8 ** (k + 1) for k in range(K)]) if lam is None else np.asarray(lam, dtype=np.float64)
    loss_k = np.zeros(K)
    g1 = np.zeros_like(W1)
    g2 = np.zeros_like(W2)
    for k in range(K):
        a = h @ W1[k].T                      # [N][d]   W1_k h
        s = 1.0 / (1.0 + np.exp(-a))         # sigmoid
        h1 = h + a * s                       # residual + SiLU
        z = h1 @ W2[k].T                     # [N][V]   logits
        m = z.max(axis=1, keepdims=True)
        lse = m[:, 0] + np.log(np.exp(z - m).sum(axis=1))
        valid = y[k] >= 0
        nv = int(valid.sum())
        if nv == 0:
            continue
        rows = np.nonzero(valid)[0]
        loss_k[k] = float(np.mean(lse[rows] - z[rows, y[k][rows]]))
        dz = np.exp(z - lse[:, None])        # softmax
        dz[rows, y[k][rows]] -= 1.0
        dz[~valid] = 0.0
        dz *= lam[k] / nv
        g2[k] = dz.T @ h1
        dh1 = dz @ W2[k]
        da = dh1 * (s * (1.0 + a * (1.0 - s)))   # d SiLU(a) / da = s (1 + a (1 - s))
        g1[k] = da.T @ h
    return dict(loss_per_head=loss_k, loss=float((lam * loss_k).sum()), grad_w1=g1, grad_w2=g2)
