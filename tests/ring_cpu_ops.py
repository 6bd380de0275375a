"""Float64 numpy restatement of the per-segment arithmetic of context-parallel PaTH (paper Sec. 3.5), for the CPU tests of
the ring schedule: the same four operations the GPU path offers (prepare / empty_message / step / finish), written from
the paper's description with explicit d x d transition matrices.  Test infrastructure only; it shares nothing with the CUDA
path.  One (batch, head) slice per call: tensors are [L, d] / [L].

    logit(i, j) = scale * k_j^T H_{j+1} ... H_i q_i + sum_{t=j+1..i} g_t,     H_t = I - beta_t w_t w_t^T
For a query i of segment r and a key j of an earlier segment c the chain of transitions splits into: the rest of segment c
after j (applied to the key: "keys advanced to the segment's end"), the whole segments in between (their products P), and
the start of segment r up to i (applied to the query: "queries pulled back to the segment's start").
"""
import numpy as np
import torch

from oracle import path_oracle


def _H(w, beta):
    return np.eye(len(w)) - beta * np.outer(w, w)


class CpuOps:
    def __init__(self, d, scale=1.0):
        self.d, self.scale = d, scale

    def prepare(self, seg):
        q, k, v, w, beta = (np.asarray(seg[n], dtype=np.float64) for n in ("q", "k", "v", "w", "beta"))
        g = np.asarray(seg["log_f"], dtype=np.float64) if seg.get("log_f") is not None else np.zeros(len(beta))
        L, d = q.shape
        o, lse = path_oracle.forward(q, k, v, w, beta, g, scale=self.scale)        # the segment's own causal attention
        x = np.empty_like(q)                                                       # x_i = H_0 H_1 ... H_i q_i (local indices)
        for i in range(L):
            u = q[i].copy()
            for t in range(i, -1, -1):
                u = _H(w[t], beta[t]) @ u
            x[i] = u
        kend = np.empty_like(k)                                                    # H_{L-1} ... H_{j+1} k_j
        for j in range(L):
            u = k[j].copy()
            for t in range(j + 1, L):
                u = _H(w[t], beta[t]) @ u
            kend[j] = u
        P = np.eye(d)                                                              # H_0 H_1 ... H_{L-1}
        for t in range(L):
            P = P @ _H(w[t], beta[t])
        G = np.cumsum(g)
        state = {"x": x, "gq": G.copy(), "o": o, "lse": lse}
        message = torch.from_numpy(np.concatenate([kend.ravel(), v.ravel(), P.ravel(), G - G[-1], [G[-1]]]))
        return state, message

    def empty_message(self, L):
        return torch.empty(2 * L * self.d + self.d * self.d + L + 1, dtype=torch.float64)

    def step(self, state, message, Lq, Lk):
        m, d = message.numpy(), self.d
        kend, v = m[:Lk * d].reshape(Lk, d), m[Lk * d:2 * Lk * d].reshape(Lk, d)
        P = m[2 * Lk * d:2 * Lk * d + d * d].reshape(d, d)
        gk, gtot = m[2 * Lk * d + d * d:2 * Lk * d + d * d + Lk], m[-1]
        s = self.scale * state["x"] @ kend.T + state["gq"][:, None] - gk[None, :]
        mx = s.max(1)
        e = np.exp(s - mx[:, None])
        lse_t = mx + np.log(e.sum(1))
        o_t = (e / e.sum(1, keepdims=True)) @ v
        top = np.maximum(state["lse"], lse_t)
        wa, wt = np.exp(state["lse"] - top), np.exp(lse_t - top)
        state["o"] = (state["o"] * wa[:, None] + o_t * wt[:, None]) / (wa + wt)[:, None]
        state["lse"] = top + np.log(wa + wt)
        state["x"] = state["x"] @ P.T                                              # column form: x <- P x
        state["gq"] = state["gq"] + gtot

    def finish(self, state, L):
        return state["o"], state["lse"]
