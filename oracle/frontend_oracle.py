"""Float64 CPU oracle of the layer front-end that produces the operator's w, beta and log f.

TEST INFRASTRUCTURE ONLY: the CUDA library never imports this module, and this
module never imports the CUDA package.

What it computes (paper Sec. 2.2, the footnote to the definition of H_t, and the
gate of Sec. 2.4):

* ``w_t``: the output ``z`` of a low-rank linear layer goes through a short
  convolution of filter size 3 and an L2 normalisation.  The linear layer is two
  plain matrix products, ``z = (x W1^T) W2^T`` (``lowrank_fwd`` / ``lowrank_bwd``
  at the end of this module); the front-end proper starts from ``z``.
* ``beta_t = 2 * sigmoid(beta_logit_t)`` with ``beta_logit_t = u^T x_t + b``.
* ``log f_t = log sigmoid(gate_logit_t)`` with ``gate_logit_t = u_f^T x_t + b_f``.

Readings where the paper gives no detail (they are this build's, stated in the
design notes): the convolution is causal and depthwise (one 3-tap filter per
channel, the sequence starts from zeros, no bias, no activation):
``y_t[c] = cw[c,0] z_{t-2}[c] + cw[c,1] z_{t-1}[c] + cw[c,2] z_t[c]``; the
normalisation is per head over its d channels, ``w = y / sqrt(sum y^2 + eps)``.

Layouts: ``z`` is ``[B, L, H*d]`` (head h owns channels ``h*d .. (h+1)*d``), the
logits are ``[B, L, H]``; outputs are in the operator's layouts ``[B, H, L, d]``
and ``[B, H, L]``.

The backward is the chain rule through these formulas written out term by term;
the tests pin it against central differences of ``frontend_fwd``.
"""
from __future__ import annotations

import numpy as np


def short_conv(z: np.ndarray, cw: np.ndarray) -> np.ndarray:
    """Causal depthwise 3-tap filter along the sequence: z [B, L, C], cw [C, 3] -> y [B, L, C]."""
    z = np.asarray(z, np.float64)
    cw = np.asarray(cw, np.float64)
    B, L, C = z.shape
    y = np.zeros_like(z)
    for t in range(L):
        for j in range(3):
            s = t - 2 + j
            if s >= 0:
                y[:, t, :] += cw[:, j] * z[:, s, :]
    return y


def frontend_fwd(z, cw, beta_logit, gate_logit, H: int, eps: float):
    """Returns (w [B,H,L,d], beta [B,H,L], log_f [B,H,L] or None)."""
    z = np.asarray(z, np.float64)
    B, L, C = z.shape
    d = C // H
    y = short_conv(z, cw).reshape(B, L, H, d)
    norm = np.sqrt((y * y).sum(-1, keepdims=True) + eps)
    w = (y / norm).transpose(0, 2, 1, 3).copy()
    bl = np.asarray(beta_logit, np.float64)
    beta = (2.0 / (1.0 + np.exp(-bl))).transpose(0, 2, 1).copy()
    log_f = None
    if gate_logit is not None:
        gl = np.asarray(gate_logit, np.float64)
        # log sigmoid(x) = -log(1 + exp(-x)), written so that neither branch overflows
        log_f = (np.minimum(gl, 0.0) - np.log1p(np.exp(-np.abs(gl)))).transpose(0, 2, 1).copy()
    return w, beta, log_f


def frontend_bwd(z, cw, beta_logit, gate_logit, dw, dbeta, dlog_f, H: int, eps: float):
    """Gradients of sum(w*dw) + sum(beta*dbeta) + sum(log_f*dlog_f) with respect to the inputs.

    dw [B,H,L,d], dbeta / dlog_f [B,H,L]  ->  dz [B,L,C], dcw [C,3], dbeta_logit [B,L,H], dgate_logit [B,L,H] or None.
    """
    z = np.asarray(z, np.float64)
    cw = np.asarray(cw, np.float64)
    B, L, C = z.shape
    d = C // H
    y = short_conv(z, cw).reshape(B, L, H, d)
    g = np.asarray(dw, np.float64).transpose(0, 2, 1, 3)            # [B, L, H, d]
    r = 1.0 / np.sqrt((y * y).sum(-1, keepdims=True) + eps)
    # w = y r, r = (y.y + eps)^(-1/2)  =>  dy = r g - r^3 y (y . g)
    dy = (r * g - (r ** 3) * y * (y * g).sum(-1, keepdims=True)).reshape(B, L, C)
    dz = np.zeros_like(z)
    dcw = np.zeros_like(cw)
    for t in range(L):
        for j in range(3):
            s = t - 2 + j                                            # y_t reads z_s through tap j
            if s >= 0:
                dz[:, s, :] += cw[:, j] * dy[:, t, :]
                dcw[:, j] += (dy[:, t, :] * z[:, s, :]).sum(0)
    bl = np.asarray(beta_logit, np.float64)
    sg = 1.0 / (1.0 + np.exp(-bl))
    dbl = np.asarray(dbeta, np.float64).transpose(0, 2, 1) * 2.0 * sg * (1.0 - sg)
    dgl = None
    if gate_logit is not None:
        gl = np.asarray(gate_logit, np.float64)
        dgl = np.asarray(dlog_f, np.float64).transpose(0, 2, 1) * (1.0 / (1.0 + np.exp(gl)))   # d log sigmoid = sigmoid(-x)
    return dz, dcw, dbl.copy(), None if dgl is None else dgl.copy()


def lowrank_fwd(x: np.ndarray, w1: np.ndarray, w2: np.ndarray):
    """The low-rank linear layer in front of the convolution (paper Sec. 2.2 footnote): x [M, D], W1 [r, D], W2 [C, r]
    (the layouts of a linear layer's weight) -> ``t = x W1^T`` [M, r] and ``z = t W2^T`` [M, C]."""
    x, w1, w2 = (np.asarray(a, np.float64) for a in (x, w1, w2))
    t = x @ w1.T
    return t @ w2.T, t


def lowrank_bwd(x: np.ndarray, w1: np.ndarray, w2: np.ndarray, dz: np.ndarray):
    """Gradients of ``sum(z * dz)``: ``dt = dz W2``, ``dW2 = dz^T t``, ``dx = dt W1``, ``dW1 = dt^T x``."""
    x, w1, w2, dz = (np.asarray(a, np.float64) for a in (x, w1, w2, dz))
    t = x @ w1.T
    dt = dz @ w2
    return dt @ w1, dt.T @ x, dz.T @ t
