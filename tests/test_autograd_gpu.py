"""The torch.autograd wrappers are argument marshalling over the binding: their gradients must be the ones the C-ABI
backward returns, and the chain front-end -> operator must match the two oracles composed (paper Sec. 2.2, 2.4)."""
import numpy as np
import pytest
import torch

from oracle import frontend_oracle as fo
from paper_2505_16381_b200 import synth

pytestmark = pytest.mark.gpu


def rel_fro(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


@pytest.mark.parametrize("gate", [False, True])
def test_path_attention_autograd_matches_oracle(oracle, gate):
    from paper_2505_16381_b200.autograd import path_attention
    B, H, L, d = 1, 2, 384, 64
    inp = synth.make_inputs(B, H, L, d, "bf16", gate=gate, seed=8100 + gate)
    leaves = {n: inp[n].cuda().requires_grad_(True) for n in ("q", "k", "v", "w", "beta")}
    log_f = inp["log_f"].cuda().requires_grad_(True) if gate else None
    o = path_attention(leaves["q"], leaves["k"], leaves["v"], leaves["w"], leaves["beta"], log_f)
    o.backward(inp["d_o"].cuda())
    f64 = synth.to_f64
    ref_o, _ = oracle.forward(f64(inp["q"]), f64(inp["k"]), f64(inp["v"]), f64(inp["w"]), f64(inp["beta"]), f64(inp["log_f"]))
    ref = oracle.backward(f64(inp["q"]), f64(inp["k"]), f64(inp["v"]), f64(inp["w"]), f64(inp["beta"]), f64(inp["d_o"]),
                          f64(inp["log_f"]))
    assert rel_fro(f64(o).reshape(ref_o.shape), ref_o) <= 1e-2
    for n, g in (("dq", leaves["q"].grad), ("dk", leaves["k"].grad), ("dv", leaves["v"].grad), ("dw", leaves["w"].grad),
                 ("dbeta", leaves["beta"].grad)):
        assert rel_fro(f64(g).reshape(ref[n].shape), ref[n]) <= 1e-2, n
    if gate:
        assert rel_fro(f64(log_f.grad).reshape(ref["dlog_f"].shape), ref["dlog_f"]) <= 1e-2


@pytest.mark.parametrize("retain", [False, True])
def test_path_attention_autograd_takes_transposed_views(oracle, retain):
    """The usual layer layout: q, k, v, w arrive as [B, L, H, d].transpose(1, 2) and beta, log_f as [B, L, H].transpose(1, 2):
    none of them contiguous, all of them requiring grad."""
    from paper_2505_16381_b200.autograd import path_attention
    B, H, L, d = 1, 2, 200, 64
    inp = synth.make_inputs(B, H, L, d, "bf16", gate=True, seed=8150)
    base = {n: inp[n].transpose(1, 2).contiguous().cuda().requires_grad_(True) for n in ("q", "k", "v", "w", "beta", "log_f")}
    view = {n: t.transpose(1, 2) for n, t in base.items()}
    assert not view["q"].is_contiguous() and not view["beta"].is_contiguous()
    o = path_attention(view["q"], view["k"], view["v"], view["w"], view["beta"], view["log_f"], retain_state=retain)
    o.backward(inp["d_o"].cuda())
    f64 = synth.to_f64
    ref = oracle.backward(f64(inp["q"]), f64(inp["k"]), f64(inp["v"]), f64(inp["w"]), f64(inp["beta"]), f64(inp["d_o"]),
                          f64(inp["log_f"]))
    for n, r in (("q", "dq"), ("k", "dk"), ("v", "dv"), ("w", "dw"), ("beta", "dbeta"), ("log_f", "dlog_f")):
        got = f64(base[n].grad.transpose(1, 2)).reshape(ref[r].shape)
        assert rel_fro(got, ref[r]) <= 1e-2, r


def test_frontend_then_operator_autograd_chain(oracle):
    from paper_2505_16381_b200.autograd import path_attention, path_frontend
    B, H, L, d = 1, 2, 300, 64
    fi = synth.make_frontend_inputs(B, H, L, d, True, seed=8200)
    att = synth.make_inputs(B, H, L, d, "bf16", gate=True, seed=8201)
    z = fi["z"].cuda().requires_grad_(True)
    cw = fi["conv_w"].cuda().requires_grad_(True)
    bl = fi["beta_logit"].cuda().requires_grad_(True)
    gl = fi["gate_logit"].cuda().requires_grad_(True)
    q, k, v = (att[n].cuda() for n in ("q", "k", "v"))
    w, beta, log_f = path_frontend(z, cw, bl, gl, H=H, eps=1e-6)
    o = path_attention(q, k, v, w, beta, log_f)
    o.backward(att["d_o"].cuda())
    f64 = synth.to_f64
    go = oracle.backward(f64(att["q"]), f64(att["k"]), f64(att["v"]), f64(w), f64(beta), f64(att["d_o"]), log_f=f64(log_f))
    rz, rcw, rbl, rgl = fo.frontend_bwd(f64(fi["z"]), f64(fi["conv_w"]), f64(fi["beta_logit"]), f64(fi["gate_logit"]),
                                        go["dw"].reshape(B, H, L, d), go["dbeta"].reshape(B, H, L),
                                        go["dlog_f"].reshape(B, H, L), H, 1e-6)
    assert rel_fro(f64(z.grad), rz) <= 1e-2 and rel_fro(f64(cw.grad), rcw) <= 1e-2
    assert rel_fro(f64(bl.grad), rbl) <= 1e-2 and rel_fro(f64(gl.grad), rgl) <= 1e-2


def test_wrappers_refuse_cpu_tensors():
    from paper_2505_16381_b200.autograd import path_attention
    inp = synth.make_inputs(1, 1, 128, 64, "bf16", seed=1)
    with pytest.raises(Exception):
        path_attention(inp["q"], inp["k"], inp["v"], inp["w"], inp["beta"])
