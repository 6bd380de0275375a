"""Float64 numpy restatement of the chunked algorithm the CUDA kernels implement.

Test-side only.  It exists to pin the *host-visible algebra* of the kernels --
signs, masks, transposes, dyadic indexing -- against the oracle before and
independently of any CUDA code.  It follows the paper's Sec. 3.3 (UT transform
per chunk, boundary-adjusted queries and keys, chunk products) and replaces the
paper's per-chunk query update by a dyadic meeting point, which is the same
product by associativity (the key-advance identity of Sec. 3.4):

for query chunk I and key chunk J < I let l = msb(I xor J) and e = (I >> l) << l.
Then   logits[I, J] = Qv[l][I] @ Kv[l][J]^T   where
    Qv[l][I] = Qleft_I  P_{I-1} ... P_e          (query pulled back to boundary e)
    Kv[l][J] = Kright_J P_{J+1}^T ... P_{e-1}^T  (key advanced to boundary e)
and both are built from products of aligned dyadic runs of chunk matrices,
Dy[l][b] = P_{(b+1) 2^l - 1} ... P_{b 2^l}.
"""
import numpy as np
import scipy.linalg


def _msb(x):
    return int(x).bit_length() - 1


def chunk_prep(Q, K, W, beta):
    """Per-chunk compact representation (paper Sec. 3.1 UT transform, Sec. 3.3 boundary-adjusted Q/K)."""
    B = Q.shape[0]
    Gm = W @ W.T
    A = np.eye(B) + np.tril(beta[:, None] * Gm, -1)
    Ainv = scipy.linalg.solve_triangular(A, np.eye(B), lower=True)
    T = Ainv * beta[None, :]
    U = T @ W
    P = np.eye(W.shape[1]) - W.T @ U
    Xq = np.tril(Q @ W.T)
    Xk = np.tril(W @ K.T, -1)
    Y = T @ Xk
    return dict(Gm=Gm, Ainv=Ainv, T=T, U=U, P=P, Xq=Xq, Xk=Xk, Y=Y,
                Ql=Q - Xq @ U, Kr=K - Y.T @ W)


def _pad(x, Lp):
    pad = [(0, Lp - x.shape[0])] + [(0, 0)] * (x.ndim - 1)
    return np.pad(x, pad)


def build_state(q, k, w, beta, B):
    """All forward intermediates of one slice, padded to a whole number of chunks (pad: w = 0, beta = 0)."""
    L, d = q.shape
    N = -(-L // B)
    Lp = N * B
    q, k, w, beta = (_pad(x, Lp) for x in (q, k, w, beta))
    ch = [chunk_prep(q[c * B:(c + 1) * B], k[c * B:(c + 1) * B], w[c * B:(c + 1) * B], beta[c * B:(c + 1) * B])
          for c in range(N)]
    nlev = max(1, _msb(max(N - 1, 1)) + 1)
    Dy = [dict() for _ in range(nlev)]
    for c in range(N):
        Dy[0][c] = ch[c]["P"]
    for l in range(nlev - 1):
        for b in range(N >> (l + 1)):
            Dy[l + 1][b] = Dy[l][2 * b + 1] @ Dy[l][2 * b]
    Qv = [dict() for _ in range(nlev)]
    Kv = [dict() for _ in range(nlev)]
    for I in range(1, N):
        prev = None
        for l in range(nlev):
            if not (I >> l) & 1:
                continue
            if prev is None:
                Qv[l][I] = ch[I]["Ql"]
            else:
                e2 = (I >> l) << l
                Qv[l][I] = Qv[prev][I] @ Dy[prev][e2 >> prev]
            prev = l
    for J in range(N - 1):
        prev = None
        for l in range(nlev):
            if (J >> l) & 1:
                continue
            if (((J >> l) + 1) << l) > N - 1:      # no query chunk meets this key at level l
                break
            if prev is None:
                Kv[l][J] = ch[J]["Kr"]
            else:
                E1 = ((J >> prev) + 1) << prev
                Kv[l][J] = Kv[prev][J] @ Dy[prev][E1 >> prev].T
            prev = l
    return dict(L=L, Lp=Lp, N=N, B=B, d=d, nlev=nlev, q=q, k=k, w=w, beta=beta, ch=ch, Dy=Dy, Qv=Qv, Kv=Kv)


def logits_blockwise(st, scale=1.0, G=None):
    N, B, Lp = st["N"], st["B"], st["Lp"]
    S = np.full((Lp, Lp), -np.inf)
    for I in range(N):
        c = st["ch"][I]
        qI, kI = st["q"][I * B:(I + 1) * B], st["k"][I * B:(I + 1) * B]
        D = qI @ kI.T - c["Xq"] @ c["Y"]
        S[I * B:(I + 1) * B, I * B:(I + 1) * B] = np.where(np.tril(np.ones((B, B), bool)), scale * D, -np.inf)
        for J in range(I):
            l = _msb(I ^ J)
            S[I * B:(I + 1) * B, J * B:(J + 1) * B] = scale * st["Qv"][l][I] @ st["Kv"][l][J].T
    if G is not None:
        Gp = _pad(G, Lp)
        S = S + Gp[:, None] - Gp[None, :]
    return S


def forward_blockwise(q, k, v, w, beta, g=None, scale=1.0, B=16):
    st = build_state(q, k, w, beta, B)
    L = st["L"]
    G = None if g is None else np.cumsum(g)
    S = logits_blockwise(st, scale, G)[:L, :L]
    lse = scipy.special.logsumexp(S, axis=1)
    P = np.exp(S - lse[:, None])
    return P @ v, lse, st, P


def backward_blockwise(q, k, v, w, beta, d_o, g=None, scale=1.0, B=16):
    """Gradients through the chunked formulation, in the order the CUDA backward takes."""
    o, lse, st, P = forward_blockwise(q, k, v, w, beta, g, scale, B)
    L, Lp, N, d, nlev = st["L"], st["Lp"], st["N"], st["d"], st["nlev"]
    delta = np.sum(d_o * o, axis=1)
    dP = d_o @ v.T
    dS = np.zeros((Lp, Lp))
    dS[:L, :L] = P * (dP - delta[:, None])
    dv = P.T @ d_o
    dG = -dS.sum(axis=0)[:L]                       # column sums; row sums vanish identically
    dS = scale * dS

    sl = lambda c: slice(c * B, (c + 1) * B)
    # attention-pair gradients w.r.t. the versions
    dQv = [dict() for _ in range(nlev)]
    dKv = [dict() for _ in range(nlev)]
    for I in range(N):
        for J in range(I):
            l = _msb(I ^ J)
            blk = dS[sl(I), sl(J)]
            dQv[l][I] = dQv[l].get(I, 0) + blk @ st["Kv"][l][J]
            dKv[l][J] = dKv[l].get(J, 0) + blk.T @ st["Qv"][l][I]
    # version chains, top level first
    dDy = [dict() for _ in range(nlev)]
    dQl = [np.zeros((B, d)) for _ in range(N)]
    dKr = [np.zeros((B, d)) for _ in range(N)]
    for I in range(1, N):
        bits = [l for l in range(nlev) if (I >> l) & 1]
        for a in range(len(bits) - 1, 0, -1):
            l2, l1 = bits[a], bits[a - 1]
            b = ((I >> l2) << l2) >> l1
            gup = dQv[l2].get(I, np.zeros((B, d)))
            dQv[l1][I] = dQv[l1].get(I, 0) + gup @ st["Dy"][l1][b].T
            dDy[l1][b] = dDy[l1].get(b, 0) + st["Qv"][l1][I].T @ gup
        dQl[I] = dQv[bits[0]].get(I, np.zeros((B, d)))
    for J in range(N - 1):
        bits = [l for l in range(nlev) if not (J >> l) & 1 and l in range(nlev) and J in st["Kv"][l]]
        for a in range(len(bits) - 1, 0, -1):
            l2, l1 = bits[a], bits[a - 1]
            b = (((J >> l1) + 1) << l1) >> l1
            gup = dKv[l2].get(J, np.zeros((B, d)))
            dKv[l1][J] = dKv[l1].get(J, 0) + gup @ st["Dy"][l1][b]
            dDy[l1][b] = dDy[l1].get(b, 0) + gup.T @ st["Kv"][l1][J]
        if bits:
            dKr[J] = dKv[bits[0]].get(J, np.zeros((B, d)))
    # dyadic products, top-down
    for l in range(nlev - 1, 0, -1):
        for b, dC in dDy[l].items():
            A_, B_ = st["Dy"][l - 1][2 * b + 1], st["Dy"][l - 1][2 * b]
            dDy[l - 1][2 * b + 1] = dDy[l - 1].get(2 * b + 1, 0) + dC @ B_.T
            dDy[l - 1][2 * b] = dDy[l - 1].get(2 * b, 0) + A_.T @ dC
    # chunk chain rule
    dq = np.zeros((Lp, d)); dk = np.zeros((Lp, d)); dw = np.zeros((Lp, d)); dbeta = np.zeros(Lp)
    tl = np.tril(np.ones((B, B)))
    tls = np.tril(np.ones((B, B)), -1)
    for c in range(N):
        ch = st["ch"][c]
        Q, K, W, bt = st["q"][sl(c)], st["k"][sl(c)], st["w"][sl(c)], st["beta"][sl(c)]
        dPc = dDy[0].get(c, np.zeros((d, d)))
        dSd = dS[sl(c), sl(c)] * tl
        U, Y, T, Xq, Xk, Ainv, Gm = (ch[n] for n in ("U", "Y", "T", "Xq", "Xk", "Ainv", "Gm"))
        dXq = tl * (-dQl[c] @ U.T - dSd @ Y.T)
        dU = -Xq.T @ dQl[c] - W @ dPc
        dY = -W @ dKr[c].T - Xq.T @ dSd
        dT = tl * (dY @ Xk.T + dU @ W.T)
        dXk = tls * (T.T @ dY)
        dA = tls * (-Ainv.T @ (dT * bt[None, :]) @ Ainv.T)
        dGm = bt[:, None] * dA
        dq[sl(c)] = dQl[c] + dSd @ K + dXq @ W
        dk[sl(c)] = dKr[c] + dSd.T @ Q + dXk.T @ W
        dw[sl(c)] = (-Y @ dKr[c] - U @ dPc.T + T.T @ dU + dXq.T @ Q + dXk @ K + (dGm + dGm.T) @ W)
        dbeta[sl(c)] = np.sum(Ainv * dT, axis=0) + np.sum(dA * Gm, axis=1)
    out = dict(dq=dq[:L], dk=dk[:L], dv=dv, dw=dw[:L], dbeta=dbeta[:L])
    if g is not None:
        out["dlog_f"] = np.cumsum(dG[::-1])[::-1]
    return out
