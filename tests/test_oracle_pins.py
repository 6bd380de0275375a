"""Pins of the float64 oracle against things other than itself (CPU only).

Each test checks the oracle against a fact fixed by the paper or by mathematics:
explicit matrix products, the paper's closed matrix form, the linear-RNN
unrolling, worked constructions from the appendix, special cases that reduce to
library routines, closed forms, finite differences, autograd of the closed
matrix form and exact gradient invariants.
"""
import math
import os

import numpy as np
import pytest
import scipy.linalg
import torch

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_problem(rng, L, d, S=None, unit_w=True, beta_lo=0.0, beta_hi=2.0, gate=False):
    shp = (L, d) if S is None else (S, L, d)
    q = rng.standard_normal(shp)
    k = rng.standard_normal(shp)
    v = rng.standard_normal(shp)
    w = rng.standard_normal(shp)
    if unit_w:
        w /= np.linalg.norm(w, axis=-1, keepdims=True)
    beta = rng.uniform(beta_lo, beta_hi, shp[:-1])
    g = np.log(1.0 / (1.0 + np.exp(-(rng.standard_normal(shp[:-1]) + 1.0)))) if gate else None
    return q, k, v, w, beta, g


def householder(w, beta):
    return np.eye(len(w)) - beta * np.outer(w, w)


def brute_logits(q, k, w, beta, g=None, scale=1.0):
    """k_j^T (H_{j+1} @ ... @ H_i) q_i with explicit d x d matrices (paper Sec. 2.1 definition)."""
    L, d = q.shape
    out = np.zeros((L, L))
    for i in range(L):
        for j in range(i + 1):
            M = np.eye(d)
            for s in range(j + 1, i + 1):
                M = M @ householder(w[s], beta[s])
            out[i, j] = scale * (k[j] @ M @ q[i])
            if g is not None:
                out[i, j] += g[j + 1:i + 1].sum()
    return out


def softmax_attend(S, v):
    """Causal softmax of a full logits matrix (lower triangle) and PV, via library routines."""
    L = S.shape[0]
    mask = np.tril(np.ones((L, L), dtype=bool))
    Sm = np.where(mask, S, -np.inf)
    lse = scipy.special.logsumexp(Sm, axis=1)
    P = np.exp(Sm - lse[:, None])
    return P @ v, lse


# ---------------------------------------------------------------- logits / product order

@pytest.mark.parametrize("gate", [False, True])
def test_logits_match_explicit_matrix_products(oracle, gate):
    rng = np.random.default_rng(1)
    q, k, v, w, beta, g = rand_problem(rng, L=13, d=5, unit_w=False, gate=gate)
    ref = brute_logits(q, k, w, beta, g, scale=0.7)
    got = oracle.logits(q, k, w, beta, g, scale=0.7)
    assert np.abs(got - ref).max() < 1e-12
    o, lse = oracle.forward(q, k, v, w, beta, g, scale=0.7)
    o_ref, lse_ref = softmax_attend(ref, v)
    assert np.abs(o - o_ref).max() < 1e-12 and np.abs(lse - lse_ref).max() < 1e-12


def test_logits_match_boxed_matrix_form(oracle):
    """Paper Sec. 3.2 boxed identity with the global inverse:
    A~ = lower(QK^T) - lower(QW^T) T^{-1} strictLower(WK^T),  T^{-1} = (I + strictLower(D W W^T))^{-1} D."""
    rng = np.random.default_rng(2)
    L, d = 48, 8
    q, k, v, w, beta, _ = rand_problem(rng, L, d)
    A = np.eye(L) + np.tril(np.diag(beta) @ w @ w.T, -1)
    Tinv = scipy.linalg.solve_triangular(A, np.diag(beta), lower=True)
    ref = np.tril(q @ k.T) - np.tril(q @ w.T) @ Tinv @ np.tril(w @ k.T, -1)
    got = oracle.logits(q, k, w, beta)
    assert np.abs(got - np.tril(ref)).max() < 1e-11


def test_linear_rnn_unrolling(oracle):
    """Paper Sec. 2.2: S_t = S_{t-1} H_t + v_t k_t^T, o_t = S_t q_t equals sum_j v_j a_tj (no softmax)."""
    rng = np.random.default_rng(3)
    L, d = 24, 6
    q, k, v, w, beta, _ = rand_problem(rng, L, d)
    a = oracle.logits(q, k, w, beta)
    S = np.zeros((d, d))
    for t in range(L):
        S = S @ householder(w[t], beta[t]) + np.outer(v[t], k[t])
        assert np.abs(S @ q[t] - a[t, :t + 1] @ v[:t + 1]).max() < 1e-11


def test_key_cache_recurrence(oracle):
    """Paper Sec. 3.4: keys updated in place, k_i <- H_t k_i for all i < t, give the logits as plain dot products."""
    rng = np.random.default_rng(4)
    L, d = 20, 7
    q, k, v, w, beta, _ = rand_problem(rng, L, d)
    a = oracle.logits(q, k, w, beta)
    cache = np.zeros((0, d))
    for t in range(L):
        H = householder(w[t], beta[t])
        cache = cache @ H.T  # every historical key <- H_t k
        cache = np.vstack([cache, k[t][None]])
        assert np.abs(cache @ q[t] - a[t, :t + 1]).max() < 1e-11


def test_key_cache_function_against_logits_products_and_special_cases(oracle):
    """The oracle's key cache (Sec. 3.4): its dot product with a query is that query's logit row; it equals the explicit
    matrix products H_{n-1} ... H_{j+1} k_j; beta = 0 leaves the keys alone; beta = 2 with unit w preserves their norms;
    a cache of n tokens extended by hand by one more transition equals the cache of n + 1 tokens."""
    rng = np.random.default_rng(41)
    L, d = 24, 6
    q, k, v, w, beta, _ = rand_problem(rng, L, d)
    a = oracle.logits(q, k, w, beta)
    for n in (1, 2, 9, L):
        kc = oracle.key_cache(k, w, beta, n)
        assert kc.shape == (n, d)
        assert np.abs(kc @ q[n - 1] - a[n - 1, :n]).max() < 1e-11          # logits of the last cached position
        for j in range(n):                                                 # explicit d x d products
            M = np.eye(d)
            for t in range(j + 1, n):
                M = householder(w[t], beta[t]) @ M
            assert np.abs(M @ k[j] - kc[j]).max() < 1e-11
    kc9, kc10 = oracle.key_cache(k, w, beta, 9), oracle.key_cache(k, w, beta, 10)
    step = np.vstack([kc9 @ householder(w[9], beta[9]).T, k[9][None]])
    assert np.abs(step - kc10).max() < 1e-12
    assert np.array_equal(oracle.key_cache(k, w, 0 * beta), k)
    wn = w / np.linalg.norm(w, axis=-1, keepdims=True)
    kc = oracle.key_cache(k, wn, 2.0 + 0 * beta)
    assert np.abs(np.linalg.norm(kc, axis=-1) - np.linalg.norm(k, axis=-1)).max() < 1e-12
    # batched call = per-slice calls
    kb = np.stack([k, 2 * k]); wb = np.stack([w, w[::-1]]); bb = np.stack([beta, beta[::-1]])
    kcb = oracle.key_cache(kb, wb, bb)
    assert np.array_equal(kcb[0], oracle.key_cache(k, w, beta)) and np.array_equal(kcb[1], oracle.key_cache(2 * k, w[::-1], beta[::-1]))


# ---------------------------------------------------------------- worked constructions

def _read_swaps():
    rows = []
    with open(os.path.join(GOLDEN, "thm_a1_swaps.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            sw, pi, tot = [x.strip() for x in line.split("|")]
            rows.append(([tuple(map(int, s.split("-"))) for s in sw.split()], int(tot)))
    return rows


@pytest.mark.parametrize("swaps,total", _read_swaps())
def test_theorem_a1_swap_tracking(oracle, swaps, total):
    n = len(swaps)
    L, d = n + 1, 6
    q = np.tile(n * np.array([1, 2, 3, 4, 5, 54.5]), (L, 1))
    k = np.zeros((L, d)); k[0] = [1, 2, 3, 4, 5, -1]
    v = np.zeros((L, d)); v[0, 0] = 1.0
    w = np.zeros((L, d))
    for t, (x, y) in enumerate(swaps, start=1):
        w[t, x - 1] = 1 / math.sqrt(2); w[t, y - 1] = -1 / math.sqrt(2)
    beta = np.full(L, 2.0)
    a = oracle.logits(q, k, w, beta)
    s0 = n * (total - 54.5)
    assert abs(a[n, 0] - s0) < 1e-9
    assert np.abs(a[n, 1:]).max() < 1e-12
    o, lse = oracle.forward(q, k, v, w, beta)
    expect = math.exp(s0) / (math.exp(s0) + n)
    assert abs(o[n, 0] - expect) < 1e-12 and np.abs(o[n, 1:]).max() == 0.0
    # identity permutation <=> s0 > n/2, otherwise s0 < -n/2 (rearrangement inequality)
    assert (s0 >= 0.5 * n - 1e-12) if total == 55 else (s0 <= -0.5 * n + 1e-12)


def test_theorem_a2_layer1_previous_token_pattern(oracle):
    """Appendix Theorem A.2, first layer: beta = 1, instruction tokens w = k = e_1, bit tokens w = e_2, k = 0,
    q = n e_1.  At a bit token i the only non-zero logit is j = i-1 and equals n."""
    n = 16
    L, d = 2 * n, 4
    q = np.zeros((L, d)); q[:, 0] = n
    k = np.zeros((L, d)); w = np.zeros((L, d))
    for t in range(L):
        if t % 2 == 0:
            k[t, 0] = 1.0; w[t, 0] = 1.0
        else:
            w[t, 1] = 1.0
    a = oracle.logits(q, k, w, np.ones(L))
    for i in range(1, L, 2):
        assert a[i, i - 1] == n
        row = a[i, :i + 1].copy(); row[i - 1] = 0.0
        assert np.abs(row).max() == 0.0


# ---------------------------------------------------------------- special cases / closed forms

def test_beta_zero_is_causal_softmax_attention(oracle):
    rng = np.random.default_rng(5)
    q, k, v, w, beta, _ = rand_problem(rng, L=40, d=16, S=3)
    o, lse = oracle.forward(q, k, v, w, np.zeros_like(beta), scale=0.25)
    for s in range(3):
        o_ref, lse_ref = softmax_attend(0.25 * q[s] @ k[s].T, v[s])
        assert np.abs(o[s] - o_ref).max() < 1e-12 and np.abs(lse[s] - lse_ref).max() < 1e-12


def test_beta_zero_with_gate_is_fox(oracle):
    """Paper's FoX equation: logit = k.q + sum_{s=j+1..i} log f_s."""
    rng = np.random.default_rng(6)
    L, d = 33, 8
    q, k, v, w, beta, g = rand_problem(rng, L, d, gate=True)
    G = np.cumsum(g)
    S = q @ k.T + G[:, None] - G[None, :]
    o_ref, lse_ref = softmax_attend(S, v)
    o, lse = oracle.forward(q, k, v, w, np.zeros(L), g)
    assert np.abs(o - o_ref).max() < 1e-12 and np.abs(lse - lse_ref).max() < 1e-12
    # constant gate = linear distance bias; zero gate = no gate
    c = 0.3
    a = oracle.logits(q, k, w, beta, np.full(L, -c))
    a0 = oracle.logits(q, k, w, beta)
    i, j = np.tril_indices(L)
    assert np.abs(a[i, j] - (a0[i, j] - c * (i - j))).max() < 1e-12
    assert np.abs(oracle.logits(q, k, w, beta, np.zeros(L)) - a0).max() == 0.0


def test_beta_two_unit_w_are_reflections(oracle):
    rng = np.random.default_rng(7)
    L, d = 30, 9
    q, k, v, w, beta, _ = rand_problem(rng, L, d)
    beta[:] = 2.0
    U = oracle.uchain(q, w, beta, L - 1)
    assert np.abs(np.linalg.norm(U, axis=1) - np.linalg.norm(q[L - 1])).max() < 1e-12
    # H^2 = I: repeating each w twice cancels
    w2 = np.repeat(w[: L // 2], 2, axis=0)
    U2 = oracle.uchain(q, w2, beta, L - 1)
    assert np.abs(U2[1::2] - q[L - 1]).max() < 1e-12


def test_constant_w_closed_form(oracle):
    """All w_t = w (unit): H's commute and prod H = I - (1 - prod(1-beta_s)) w w^T."""
    rng = np.random.default_rng(8)
    L, d = 25, 6
    q, k, v, w, beta, _ = rand_problem(rng, L, d)
    w[:] = w[0]
    a = oracle.logits(q, k, w, beta)
    for i in range(L):
        for j in range(i + 1):
            c = 1.0 - np.prod(1.0 - beta[j + 1:i + 1])
            assert abs(a[i, j] - (k[j] @ q[i] - c * (k[j] @ w[0]) * (w[0] @ q[i]))) < 1e-11


def test_axis_aligned_w_closed_form(oracle):
    """w_t = e_{t mod d}: diagonal H's, coordinate c scaled by prod over s in (j, i], s = c mod d, of (1 - beta_s)."""
    rng = np.random.default_rng(9)
    L, d = 23, 4
    q, k, v, w, beta, _ = rand_problem(rng, L, d)
    w[:] = np.eye(d)[np.arange(L) % d]
    a = oracle.logits(q, k, w, beta)
    for i in range(L):
        for j in range(i + 1):
            f = np.ones(d)
            for s in range(j + 1, i + 1):
                f[s % d] *= 1.0 - beta[s]
            assert abs(a[i, j] - np.sum(k[j] * f * q[i])) < 1e-11


def test_softmax_and_pv_properties(oracle):
    rng = np.random.default_rng(10)
    L, d = 37, 8
    q, k, v, w, beta, g = rand_problem(rng, L, d, gate=True)
    o, _ = oracle.forward(q, k, np.tile(v[0], (L, 1)), w, beta, g)
    assert np.abs(o - v[0]).max() < 1e-12          # convex combination of identical values
    o1, _ = oracle.forward(q, k, v, w, beta, g)
    v2 = rng.standard_normal((L, d))
    o2, _ = oracle.forward(q, k, v2, w, beta, g)
    o12, _ = oracle.forward(q, k, 2 * v - 3 * v2, w, beta, g)
    assert np.abs(o12 - (2 * o1 - 3 * o2)).max() < 1e-11  # linear in V
    # adding a constant to the gate prefix changes nothing: shift g_0 (which never enters a logit)
    g2 = g.copy(); g2[0] += 5.0
    o3, lse3 = oracle.forward(q, k, v, w, beta, g2)
    assert np.abs(o3 - o1).max() < 1e-12


def test_row_sampled_forward_equals_full(oracle):
    rng = np.random.default_rng(11)
    q, k, v, w, beta, g = rand_problem(rng, L=50, d=8, S=2, gate=True)
    o, lse = oracle.forward(q, k, v, w, beta, g)
    rows = [0, 7, 31, 49]
    o_r, lse_r = oracle.forward(q, k, v, w, beta, g, rows=rows)
    assert np.array_equal(o_r, o[:, rows]) and np.array_equal(lse_r, lse[:, rows])


# ---------------------------------------------------------------- gradients

def _loss(oracle, q, k, v, w, beta, g, d_o, scale):
    o, _ = oracle.forward(q, k, v, w, beta, g, scale=scale)
    return float(np.sum(o * d_o))


@pytest.mark.parametrize("gate", [False, True])
def test_backward_matches_central_differences(oracle, gate):
    rng = np.random.default_rng(12)
    L, d, scale = 11, 4, 0.8
    q, k, v, w, beta, g = rand_problem(rng, L, d, unit_w=False, gate=gate)
    d_o = rng.standard_normal((L, d))
    grads = oracle.backward(q, k, v, w, beta, d_o, g, scale=scale)
    args = {"q": q, "k": k, "v": v, "w": w, "beta": beta}
    names = {"q": "dq", "k": "dk", "v": "dv", "w": "dw", "beta": "dbeta"}
    if gate:
        args["g"] = g; names["g"] = "dlog_f"
    eps = 1e-6
    for name, arr in args.items():
        num = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            old = arr[idx]
            arr[idx] = old + eps; lp = _loss(oracle, q, k, v, w, beta, g, d_o, scale)
            arr[idx] = old - eps; lm = _loss(oracle, q, k, v, w, beta, g, d_o, scale)
            arr[idx] = old
            num[idx] = (lp - lm) / (2 * eps)
        err = np.abs(num - grads[names[name]]).max()
        assert err < 2e-7 * max(1.0, np.abs(num).max()), (name, err)


@pytest.mark.parametrize("gate", [False, True])
def test_backward_with_an_lse_gradient_matches_central_differences(oracle, gate):
    """Loss sum(O dO) + sum(lse dlse): the lse term alone, against central differences of the forward's lse, and
    the sum rule (gradients add)."""
    rng = np.random.default_rng(15)
    L, d, scale = 9, 4, 0.7
    q, k, v, w, beta, g = rand_problem(rng, L, d, unit_w=False, gate=gate)
    d_o = rng.standard_normal((L, d))
    d_lse = rng.standard_normal(L)
    both = oracle.backward(q, k, v, w, beta, d_o, g, scale=scale, d_lse=d_lse)
    only_o = oracle.backward(q, k, v, w, beta, d_o, g, scale=scale)
    only_l = oracle.backward(q, k, v, w, beta, np.zeros_like(d_o), g, scale=scale, d_lse=d_lse)
    for n in both:
        assert np.abs(both[n] - (only_o[n] + only_l[n])).max() < 1e-12, n
    assert np.abs(only_l["dv"]).max() == 0.0                      # lse does not depend on v
    lse_loss = lambda: float(np.sum(oracle.forward(q, k, v, w, beta, g, scale=scale)[1] * d_lse))
    args = {"q": q, "k": k, "w": w, "beta": beta}
    names = {"q": "dq", "k": "dk", "w": "dw", "beta": "dbeta"}
    if gate:
        args["g"] = g; names["g"] = "dlog_f"
    eps = 1e-6
    for name, arr in args.items():
        num = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            old = arr[idx]
            arr[idx] = old + eps; lp = lse_loss()
            arr[idx] = old - eps; lm = lse_loss()
            arr[idx] = old
            num[idx] = (lp - lm) / (2 * eps)
        err = np.abs(num - only_l[names[name]]).max()
        assert err < 2e-7 * max(1.0, np.abs(num).max()), (name, err)


def _boxed_forward_torch(q, k, v, w, beta, g, scale):
    """The paper's closed matrix form (Sec. 3.2) in torch float64, differentiable by autograd."""
    L = q.shape[0]
    A = torch.eye(L, dtype=torch.float64) + torch.tril(torch.diag(beta) @ w @ w.T, -1)
    Tinv = torch.linalg.solve_triangular(A, torch.diag(beta), upper=False)
    S = scale * (torch.tril(q @ k.T) - torch.tril(q @ w.T) @ Tinv @ torch.tril(w @ k.T, -1))
    if g is not None:
        G = torch.cumsum(g, 0)
        S = S + G[:, None] - G[None, :]
    mask = torch.tril(torch.ones(L, L, dtype=torch.bool))
    P = torch.softmax(S.masked_fill(~mask, float("-inf")), dim=1)
    return P @ v


@pytest.mark.parametrize("gate", [False, True])
def test_backward_matches_autograd_of_boxed_form(oracle, gate):
    rng = np.random.default_rng(13)
    L, d, scale = 40, 8, 0.5
    q, k, v, w, beta, g = rand_problem(rng, L, d, gate=gate)
    d_o = rng.standard_normal((L, d))
    grads = oracle.backward(q, k, v, w, beta, d_o, g, scale=scale)
    ts = [torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (q, k, v, w, beta)]
    tg = torch.tensor(g, dtype=torch.float64, requires_grad=True) if gate else None
    o = _boxed_forward_torch(*ts, tg, scale)
    (o * torch.tensor(d_o)).sum().backward()
    for t, name in zip(ts, ["dq", "dk", "dv", "dw", "dbeta"]):
        ref = t.grad.numpy()
        assert np.abs(grads[name] - ref).max() < 1e-10 * max(1.0, np.abs(ref).max()), name
    if gate:
        assert np.abs(grads["dlog_f"] - tg.grad.numpy()).max() < 1e-10


def test_gradient_invariants(oracle):
    """H_t is invariant under w -> c w, beta -> beta / c^2  =>  w_t . dw_t = 2 beta_t dbeta_t;
    the logit is bilinear in (q, k) and softmax is shift-free  =>  sum q.dq = sum k.dk per slice;
    H_0 and g_0 enter no logit  =>  their gradients vanish;  dO = 0  =>  all gradients vanish."""
    rng = np.random.default_rng(14)
    S, L, d = 2, 64, 16
    q, k, v, w, beta, g = rand_problem(rng, L, d, S=S, unit_w=False, gate=True)
    w *= 0.5
    d_o = rng.standard_normal((S, L, d))
    gr = oracle.backward(q, k, v, w, beta, d_o, g, scale=0.3)
    assert np.abs(np.sum(w * gr["dw"], -1) - 2 * beta * gr["dbeta"]).max() < 1e-12
    assert np.abs(np.sum(q * gr["dq"], (-1, -2)) - np.sum(k * gr["dk"], (-1, -2))).max() < 1e-11
    assert np.abs(gr["dw"][:, 0]).max() == 0.0 and np.abs(gr["dbeta"][:, 0]).max() == 0.0
    assert np.abs(gr["dlog_f"][:, 0]).max() < 1e-13
    z = oracle.backward(q, k, v, w, beta, np.zeros_like(d_o), g, scale=0.3)
    assert all(np.abs(x).max() == 0.0 for x in z.values())
