"""The chunked / dyadic formulation (numpy restatement of what the kernels do) against the oracle, CPU only."""
import numpy as np
import pytest

from blockwise_ref import backward_blockwise, forward_blockwise
from test_oracle_pins import rand_problem


@pytest.mark.parametrize("L,B,gate", [(64, 16, False), (112, 16, True), (77, 8, True), (40, 64, False), (8, 8, False)])
def test_forward_blockwise_equals_oracle(oracle, L, B, gate):
    rng = np.random.default_rng(L + B)
    q, k, v, w, beta, g = rand_problem(rng, L, 12, gate=gate)
    o, lse, _, _ = forward_blockwise(q, k, v, w, beta, g, scale=0.6, B=B)
    o_ref, lse_ref = oracle.forward(q, k, v, w, beta, g, scale=0.6)
    assert np.abs(o - o_ref).max() < 1e-11 and np.abs(lse - lse_ref).max() < 1e-11


@pytest.mark.parametrize("L,B,gate", [(64, 16, False), (112, 16, True), (77, 8, True), (40, 64, True)])
def test_backward_blockwise_equals_oracle(oracle, L, B, gate):
    rng = np.random.default_rng(100 + L + B)
    q, k, v, w, beta, g = rand_problem(rng, L, 12, gate=gate)
    d_o = rng.standard_normal((L, 12))
    got = backward_blockwise(q, k, v, w, beta, d_o, g, scale=0.6, B=B)
    ref = oracle.backward(q, k, v, w, beta, d_o, g, scale=0.6)
    for name, r in ref.items():
        assert np.abs(got[name] - r).max() < 1e-10 * max(1.0, np.abs(r).max()), name
