"""Parity of the layer front-end kernels (paper Sec. 2.2 footnote: short convolution and L2 normalisation for w,
beta = 2 sigmoid; gate of Sec. 2.4) with the float64 oracle, through the C ABI.

The kernels compute in float32 from bf16 / float32 inputs that the oracle receives exactly, so the differences are the
rounding of the bf16 outputs (half an ulp, 2^-9 relative) plus float32 noise:
  w, dz        : |got - ref| <= 2^-8 max|ref| elementwise and rel-Fro <= 3e-3 (bf16 outputs);
  beta, log f, logit gradients : 1e-5 relative to the largest entry (float32 outputs, expf / log1pf);
  dconv_w      : 1e-4 relative to the largest entry (float32 sums of B*L products, added by atomics in any order).
"""
import numpy as np
import pytest
import torch

from oracle import frontend_oracle as fo
from paper_2505_16381_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2505_16381_b200 import binding as b
    b.load()
    assert torch.cuda.is_available()
    return b


def f64(t):
    return synth.to_f64(t)


def rel_fro(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


def close_bf16(got, ref):
    return np.abs(got - ref).max() <= 2.0 ** -8 * np.abs(ref).max() and rel_fro(got, ref) <= 3e-3


def close_f32(got, ref, tol=1e-5):
    return np.abs(got - ref).max() <= tol * max(np.abs(ref).max(), 1e-30)


SHAPES = [
    (1, 2, 256, 64, False),
    (2, 3, 1000, 128, True),     # ragged: 1000 = 7 CTAs of 128 positions + 104, and 62 warps + a half-filled one
    (1, 1, 1, 64, True),         # a single position: only the last tap sees data
    (1, 2, 2, 128, False),
    (3, 1, 17, 64, False),       # one row into a second warp
    (1, 4, 129, 128, True),      # one row into a second CTA
    (2, 2, 4096, 64, True),
]


@pytest.mark.parametrize("B,H,L,d,gate", SHAPES)
def test_frontend_forward_matches_oracle(binding, B, H, L, d, gate):
    inp = synth.make_frontend_inputs(B, H, L, d, gate, seed=900 + L + d)
    dev = {n: (t.cuda() if torch.is_tensor(t) else t) for n, t in inp.items()}
    eps = 1e-6
    w, beta, log_f = binding.path_attn_frontend_fwd(dev["z"], dev["conv_w"], dev["beta_logit"], dev["gate_logit"], H=H, eps=eps)
    torch.cuda.synchronize()
    assert binding.last_launch_count() == 1
    rw, rb, rf = fo.frontend_fwd(f64(inp["z"]), f64(inp["conv_w"]), f64(inp["beta_logit"]), f64(inp["gate_logit"]), H, eps)
    assert w.shape == (B, H, L, d) and w.dtype == torch.bfloat16
    assert close_bf16(f64(w), rw)
    assert close_f32(f64(beta), rb)
    assert (log_f is None) == (not gate)
    if gate:
        assert close_f32(f64(log_f), rf)


@pytest.mark.parametrize("B,H,L,d,gate", SHAPES)
def test_frontend_backward_matches_oracle(binding, B, H, L, d, gate):
    inp = synth.make_frontend_inputs(B, H, L, d, gate, seed=950 + L + d)
    dev = {n: (t.cuda() if torch.is_tensor(t) else t) for n, t in inp.items()}
    eps = 1e-6
    dz, dcw, dbl, dgl = binding.path_attn_frontend_bwd(dev["z"], dev["conv_w"], dev["beta_logit"], dev["dw"], dev["dbeta"],
                                                       dev["gate_logit"], dev["dlog_f"], H=H, eps=eps)
    torch.cuda.synchronize()
    assert binding.last_launch_count() == 1
    rz, rcw, rbl, rgl = fo.frontend_bwd(f64(inp["z"]), f64(inp["conv_w"]), f64(inp["beta_logit"]), f64(inp["gate_logit"]),
                                        f64(inp["dw"]), f64(inp["dbeta"]), f64(inp["dlog_f"]), H, eps)
    assert dz.shape == inp["z"].shape and dz.dtype == torch.bfloat16
    assert close_bf16(f64(dz), rz)
    assert close_f32(f64(dcw), rcw, 1e-4)
    assert close_f32(f64(dbl), rbl)
    assert (dgl is None) == (not gate)
    if gate:
        assert close_f32(f64(dgl), rgl)


def test_frontend_edge_values(binding):
    """Zero rows (0/sqrt(eps) = 0, no NaN), saturated logits, eps = 0 with non-zero rows."""
    B, H, L, d = 1, 2, 40, 64
    inp = synth.make_frontend_inputs(B, H, L, d, True, seed=77)
    inp["z"][:, :5] = 0                                   # y = 0 at t < 5
    inp["beta_logit"][0, 0, 0] = 200.0
    inp["beta_logit"][0, 1, 0] = -200.0
    inp["gate_logit"][0, 2, 1] = -200.0
    inp["gate_logit"][0, 3, 1] = 200.0
    dev = {n: (t.cuda() if torch.is_tensor(t) else t) for n, t in inp.items()}
    w, beta, log_f = binding.path_attn_frontend_fwd(dev["z"], dev["conv_w"], dev["beta_logit"], dev["gate_logit"], H=H, eps=1e-6)
    assert torch.isfinite(w.float()).all() and torch.all(w[:, :, :5] == 0)
    assert beta[0, 0, 0].item() == 2.0 and beta[0, 0, 1].item() == 0.0     # [b, h, t] <- logits [b, t, h]
    assert log_f[0, 1, 2].item() == -200.0 and log_f[0, 1, 3].item() == 0.0
    dz, dcw, dbl, dgl = binding.path_attn_frontend_bwd(dev["z"], dev["conv_w"], dev["beta_logit"], dev["dw"], dev["dbeta"],
                                                       dev["gate_logit"], dev["dlog_f"], H=H, eps=1e-6)
    for t in (dz.float(), dcw, dbl, dgl):
        assert torch.isfinite(t).all()
    with np.errstate(over="ignore"):
        rz, rcw, rbl, rgl = fo.frontend_bwd(f64(inp["z"]), f64(inp["conv_w"]), f64(inp["beta_logit"]), f64(inp["gate_logit"]),
                                            f64(inp["dw"]), f64(inp["dbeta"]), f64(inp["dlog_f"]), H, 1e-6)
    # rows with y = 0 have r = 1/sqrt(eps) = 1000: dz there is large and the bf16 bound scales with it
    assert close_bf16(f64(dz), rz) and close_f32(f64(dcw), rcw, 1e-4) and close_f32(f64(dbl), rbl) and close_f32(f64(dgl), rgl)
    # eps = 0 on rows that are not zero
    w0, _, _ = binding.path_attn_frontend_fwd(dev["z"][:, 5:].contiguous(), dev["conv_w"], dev["beta_logit"][:, 5:].contiguous(),
                                              None, H=H, eps=0.0)
    n = w0.float().norm(dim=-1)
    assert torch.all((n - 1).abs() <= 2.0 ** -8)


def test_frontend_feeds_the_operator(binding, oracle):
    """End to end on a small case: front-end -> operator forward and backward -> front-end backward, against the two
    oracles composed the same way (the operator's bounds apply to what passes through it)."""
    B, H, L, d = 1, 2, 300, 64
    inp = synth.make_frontend_inputs(B, H, L, d, True, seed=5)
    att = synth.make_inputs(B, H, L, d, "bf16", gate=True, seed=6)
    dev = {n: (t.cuda() if torch.is_tensor(t) else t) for n, t in inp.items()}
    q, k, v, d_o = (att[n].cuda() for n in ("q", "k", "v", "d_o"))
    eps = 1e-6
    w, beta, log_f = binding.path_attn_frontend_fwd(dev["z"], dev["conv_w"], dev["beta_logit"], dev["gate_logit"], H=H, eps=eps)
    ws = binding.alloc_workspace(q, True, True)
    o, lse = binding.path_attn_fwd(q, k, v, w, beta, log_f, workspace=ws)
    g = binding.path_attn_bwd(q, k, v, w, beta, o, lse, d_o, log_f, workspace=ws)
    dz, dcw, dbl, dgl = binding.path_attn_frontend_bwd(dev["z"], dev["conv_w"], dev["beta_logit"], g["dw"], g["dbeta"],
                                                       dev["gate_logit"], g["dlog_f"], H=H, eps=eps)
    assert binding.device_status(ws) == 0
    # oracle chain in float64, fed the same bf16 w the operator saw (so the operator's own rounding is not double counted)
    rw, rb, rf = fo.frontend_fwd(f64(inp["z"]), f64(inp["conv_w"]), f64(inp["beta_logit"]), f64(inp["gate_logit"]), H, eps)
    assert close_bf16(f64(w), rw)
    go = oracle.backward(f64(att["q"]), f64(att["k"]), f64(att["v"]), f64(w), f64(beta), f64(att["d_o"]), log_f=f64(log_f))
    rz, rcw, rbl, rgl = fo.frontend_bwd(f64(inp["z"]), f64(inp["conv_w"]), f64(inp["beta_logit"]), f64(inp["gate_logit"]),
                                        go["dw"].reshape(B, H, L, d), go["dbeta"].reshape(B, H, L), go["dlog_f"].reshape(B, H, L),
                                        H, eps)
    assert rel_fro(f64(dz), rz) <= 1e-2 and rel_fro(f64(dcw), rcw) <= 1e-2
    assert rel_fro(f64(dbl), rbl) <= 1e-2 and rel_fro(f64(dgl), rgl) <= 1e-2


@pytest.mark.parametrize("B,L,D,r,C", [
    (2, 300, 256, 64, 128),        # ragged row count, one output tile per product
    (1, 1, 64, 64, 64),            # a single row, the smallest sizes
    (3, 517, 1024, 128, 512),      # several tiles and stages in every direction
    (2, 1024, 2048, 64, 2048),     # the headline layer: H = 16 heads of d = 128, hidden size 2048
])
def test_lowrank_layer_matches_oracle(binding, B, L, D, r, C):
    """Forward and backward of the low-rank linear layer (paper Sec. 2.2 footnote) against float64 matrix products."""
    g = torch.Generator().manual_seed(77 + L + D)
    x = torch.randn(B, L, D, generator=g).bfloat16()
    w1 = (torch.randn(r, D, generator=g) / D ** 0.5).bfloat16()
    w2 = (torch.randn(C, r, generator=g) / r ** 0.5).bfloat16()
    dz = torch.randn(B, L, C, generator=g).bfloat16()
    z, t = binding.path_attn_lowrank_fwd(x.cuda(), w1.cuda(), w2.cuda())
    z_ref, t_ref = fo.lowrank_fwd(f64(x).reshape(-1, D), f64(w1), f64(w2))
    assert rel_fro(f64(t).reshape(-1, r), t_ref) <= 3e-3 and rel_fro(f64(z).reshape(-1, C), z_ref) <= 5e-3
    assert close_bf16(f64(z).reshape(-1, C), z_ref)
    dx, dw1, dw2 = binding.path_attn_lowrank_bwd(x.cuda(), w1.cuda(), w2.cuda(), t, dz.cuda())
    rx, r1, r2 = fo.lowrank_bwd(f64(x).reshape(-1, D), f64(w1), f64(w2), f64(dz).reshape(-1, C))
    assert rel_fro(f64(dx).reshape(-1, D), rx) <= 5e-3
    assert rel_fro(f64(dw1), r1) <= 5e-3 and rel_fro(f64(dw2), r2) <= 5e-3      # (t and dt enter rounded to bf16)
    dx2, dw1b, dw2b = binding.path_attn_lowrank_bwd(x.cuda(), w1.cuda(), w2.cuda(), t, dz.cuda())
    assert torch.equal(dx, dx2)
    for a, b_ in ((dw1, dw1b), (dw2, dw2b)):                      # float32 atomics: equal to rounding, not bitwise
        assert (a - b_).abs().max().item() <= 1e-5 * a.abs().max().item()


def test_lowrank_layer_argument_errors(binding):
    x = torch.zeros(4, 96, dtype=torch.bfloat16, device="cuda")                   # D not a multiple of 64
    with pytest.raises(binding.PathAttnError) as e:
        binding.path_attn_lowrank_fwd(x, torch.zeros(64, 96, dtype=torch.bfloat16, device="cuda"),
                                      torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == -2
