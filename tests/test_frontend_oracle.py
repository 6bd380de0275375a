"""Pins of the front-end oracle (w from the short convolution and L2 normalisation, beta, log f: paper Sec. 2.2
footnote and the gate of Sec. 2.4) against things it does not compute itself: a library convolution, closed forms,
invariants and central differences of its own forward for the hand-written backward."""
import numpy as np
import pytest

from oracle import frontend_oracle as fo


def _inputs(seed, B=2, L=9, H=2, d=4, gate=True):
    rng = np.random.default_rng(seed)
    z = rng.standard_normal((B, L, H * d))
    cw = rng.standard_normal((H * d, 3))
    bl = rng.standard_normal((B, L, H))
    gl = rng.standard_normal((B, L, H)) + 2.0 if gate else None
    return z, cw, bl, gl


def test_short_conv_is_the_library_convolution_truncated_to_the_sequence():
    z, cw, _, _ = _inputs(0, B=1, L=11)
    y = fo.short_conv(z, cw)
    for c in range(z.shape[2]):
        # np.convolve flips its second argument: tap j multiplies z_{t-2+j}, so the kernel in convolve order is cw[c, ::-1]
        ref = np.convolve(z[0, :, c], cw[c, ::-1])[: z.shape[1]]
        np.testing.assert_allclose(y[0, :, c], ref, rtol=0, atol=1e-13)


def test_impulse_response_and_causality():
    B, L, C = 1, 8, 3
    cw = np.array([[1.0, 2.0, 3.0], [-1.0, 0.5, 0.25], [0.0, 0.0, 1.0]])
    z = np.zeros((B, L, C))
    z[0, 3, :] = 1.0
    y = fo.short_conv(z, cw)
    assert np.all(y[0, :3] == 0.0)                       # nothing before the impulse
    np.testing.assert_array_equal(y[0, 3], cw[:, 2])     # the current position sees the last tap
    np.testing.assert_array_equal(y[0, 4], cw[:, 1])
    np.testing.assert_array_equal(y[0, 5], cw[:, 0])
    assert np.all(y[0, 6:] == 0.0)                       # the filter has three taps
    # the first two positions use zeros for the missing history
    z2 = np.arange(1.0, L + 1)[None, :, None] * np.ones((1, 1, C))
    y2 = fo.short_conv(z2, cw)
    np.testing.assert_allclose(y2[0, 0], cw[:, 2] * 1.0)
    np.testing.assert_allclose(y2[0, 1], cw[:, 1] * 1.0 + cw[:, 2] * 2.0)


def test_w_rows_have_unit_norm_per_head_and_identity_filter_is_plain_normalisation():
    z, cw, bl, gl = _inputs(1, B=2, L=7, H=3, d=5)
    w, beta, log_f = fo.frontend_fwd(z, cw, bl, gl, H=3, eps=0.0)
    np.testing.assert_allclose((w * w).sum(-1), 1.0, rtol=0, atol=1e-13)
    ident = np.zeros_like(cw)
    ident[:, 2] = 1.0
    w_id, _, _ = fo.frontend_fwd(z, ident, bl, gl, H=3, eps=0.0)
    zz = z.reshape(2, 7, 3, 5)
    ref = (zz / np.linalg.norm(zz, axis=-1, keepdims=True)).transpose(0, 2, 1, 3)
    np.testing.assert_allclose(w_id, ref, rtol=0, atol=1e-14)
    # a positive eps only shrinks: |w|^2 = s / (s + eps)
    w_e, _, _ = fo.frontend_fwd(z, ident, bl, gl, H=3, eps=0.5)
    s = (zz * zz).sum(-1).transpose(0, 2, 1)
    np.testing.assert_allclose((w_e * w_e).sum(-1), s / (s + 0.5), rtol=1e-13)


def test_w_is_causal_in_z_and_heads_do_not_mix():
    z, cw, bl, gl = _inputs(2, B=1, L=10, H=2, d=4)
    w0, _, _ = fo.frontend_fwd(z, cw, bl, gl, H=2, eps=1e-6)
    z1 = z.copy()
    z1[0, 6, :4] += 1.0                                  # head 0, position 6
    w1, _, _ = fo.frontend_fwd(z1, cw, bl, gl, H=2, eps=1e-6)
    np.testing.assert_array_equal(w0[0, :, :6], w1[0, :, :6])      # earlier positions unchanged
    np.testing.assert_array_equal(w0[0, 1], w1[0, 1])              # the other head unchanged everywhere
    assert np.all(np.abs(w0[0, 0, 6:9] - w1[0, 0, 6:9]).max(-1) > 0)   # three positions see it
    np.testing.assert_array_equal(w0[0, 0, 9:], w1[0, 0, 9:])


def test_beta_and_gate_closed_forms_and_layout():
    B, L, H = 2, 3, 2
    bl = np.zeros((B, L, H))
    gl = np.zeros((B, L, H))
    bl[1, 2, 0] = np.log(3.0)            # sigmoid = 3/4
    gl[0, 1, 1] = -np.log(3.0)           # sigmoid = 1/4
    bl[0, 0, 1] = 800.0                  # saturates without overflow
    gl[1, 0, 0] = -800.0
    z = np.ones((B, L, H * 2))
    cw = np.ones((H * 2, 3))
    with np.errstate(over="ignore"):
        _, beta, log_f = fo.frontend_fwd(z, cw, bl, gl, H=H, eps=0.0)
    assert beta.shape == (B, H, L) and log_f.shape == (B, H, L)
    assert beta[0, 0, 1] == 1.0 and np.isclose(log_f[0, 0, 0], -np.log(2.0), rtol=1e-15)
    assert np.isclose(beta[1, 0, 2], 1.5, rtol=1e-15)               # [b, h, t] <- logits [b, t, h]
    assert np.isclose(log_f[0, 1, 1], np.log(0.25), rtol=1e-15)
    assert beta[0, 1, 0] == 2.0 and log_f[1, 0, 0] == -800.0
    assert np.all(beta >= 0) and np.all(beta <= 2) and np.all(log_f <= 0)
    # no gate given, none returned
    assert fo.frontend_fwd(z, cw, bl, None, H=H, eps=0.0)[2] is None


def _objective(z, cw, bl, gl, dw, dbeta, dlf, H, eps):
    w, beta, lf = fo.frontend_fwd(z, cw, bl, gl, H, eps)
    val = (w * dw).sum() + (beta * dbeta).sum()
    if gl is not None:
        val += (lf * dlf).sum()
    return val


@pytest.mark.parametrize("gate,eps", [(True, 1e-3), (False, 0.0)])
def test_backward_matches_central_differences_of_the_forward(gate, eps):
    B, L, H, d = 2, 7, 2, 3
    z, cw, bl, gl = _inputs(3, B, L, H, d, gate)
    rng = np.random.default_rng(30)
    dw = rng.standard_normal((B, H, L, d))
    dbeta = rng.standard_normal((B, H, L))
    dlf = rng.standard_normal((B, H, L)) if gate else None
    dz, dcw, dbl, dgl = fo.frontend_bwd(z, cw, bl, gl, dw, dbeta, dlf, H, eps)
    assert (dgl is None) == (not gate)
    h = 1e-6

    def numeric(arr):
        out = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            keep = arr[i]
            arr[i] = keep + h
            fp = _objective(z, cw, bl, gl, dw, dbeta, dlf, H, eps)
            arr[i] = keep - h
            fm = _objective(z, cw, bl, gl, dw, dbeta, dlf, H, eps)
            arr[i] = keep
            out[i] = (fp - fm) / (2 * h)
        return out

    np.testing.assert_allclose(dz, numeric(z), rtol=2e-6, atol=2e-8)
    np.testing.assert_allclose(dcw, numeric(cw), rtol=2e-6, atol=2e-8)
    np.testing.assert_allclose(dbl, numeric(bl), rtol=2e-6, atol=2e-8)
    if gate:
        np.testing.assert_allclose(dgl, numeric(gl), rtol=2e-6, atol=2e-8)


def test_backward_invariants_of_the_normalisation():
    # with eps = 0, w does not change when z (or the filter) is scaled, so the gradient is orthogonal to both (Euler)
    B, L, H, d = 1, 8, 2, 4
    z, cw, bl, gl = _inputs(4, B, L, H, d, False)
    rng = np.random.default_rng(40)
    dw = rng.standard_normal((B, H, L, d))
    dz, dcw, _, _ = fo.frontend_bwd(z, cw, bl, None, dw, np.zeros((B, H, L)), None, H, 0.0)
    for h_ in range(H):
        sl = slice(h_ * d, (h_ + 1) * d)
        assert abs((dz[..., sl] * z[..., sl]).sum()) < 1e-12 * np.abs(dz).max() * z.size
        assert abs((dcw[sl] * cw[sl]).sum()) < 1e-12 * np.abs(dcw).max() * cw.size
    # a gradient along w itself is annihilated: dz = 0 for dw = w
    w, _, _ = fo.frontend_fwd(z, cw, bl, None, H, 0.0)
    dz2, dcw2, _, _ = fo.frontend_bwd(z, cw, bl, None, w, np.zeros((B, H, L)), None, H, 0.0)
    assert np.abs(dz2).max() < 1e-13 and np.abs(dcw2).max() < 1e-13


def test_lowrank_layer_is_two_library_linear_layers_and_its_backward_is_their_autograd():
    """z = Linear_2(Linear_1(x)) without biases, against torch's own linear layers and their autograd in float64."""
    import torch
    rng = np.random.default_rng(21)
    M, D, r, C = 7, 10, 3, 8
    x, w1, w2, dz = rng.standard_normal((M, D)), rng.standard_normal((r, D)), rng.standard_normal((C, r)), rng.standard_normal((M, C))
    z, t = fo.lowrank_fwd(x, w1, w2)
    tx, t1, t2 = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (x, w1, w2))
    tz = torch.nn.functional.linear(torch.nn.functional.linear(tx, t1), t2)
    assert np.abs(z - tz.detach().numpy()).max() < 1e-12
    assert np.abs(t - (x @ w1.T)).max() < 1e-12
    (tz * torch.tensor(dz)).sum().backward()
    dx, dw1, dw2 = fo.lowrank_bwd(x, w1, w2, dz)
    for got, ref in ((dx, tx.grad), (dw1, t1.grad), (dw2, t2.grad)):
        assert np.abs(got - ref.numpy()).max() < 1e-12
    # rank: z has at most r independent columns
    assert np.linalg.matrix_rank(z) <= r
