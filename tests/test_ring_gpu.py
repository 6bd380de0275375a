"""Context-parallel PaTH (paper Sec. 3.5): the segment-level C-ABI calls, driven as 2 to 8 virtual ranks on one device in
ring order, against the float64 oracle's forward over the whole sequence."""
import numpy as np
import pytest
import torch

from paper_2505_16381_b200 import synth

pytestmark = pytest.mark.gpu


def split(inp, cuts):
    segs, lo = [], 0
    for hi in cuts:
        seg = {n: inp[n][:, :, lo:hi].contiguous().cuda() for n in ("q", "k", "v", "w", "beta")}
        if inp["log_f"] is not None:
            seg["log_f"] = inp["log_f"][:, :, lo:hi].contiguous().cuda()
        segs.append(seg)
        lo = hi
    return segs


@pytest.mark.parametrize("B,H,L,d,gate,cuts,scale", [
    (1, 2, 1024, 128, False, [512, 1024], 1.0),                       # 2 ranks
    (1, 2, 1024, 64, True, [256, 512, 768, 1024], 1.0),               # 4 ranks, PaTH-FoX
    (2, 1, 2048, 128, True, [256 * i for i in range(1, 9)], 0.5),     # 8 ranks
    (1, 3, 1000, 64, True, [300, 500, 1000], 1.0),                    # unequal, ragged segments
    (1, 2, 700, 128, False, [1, 130, 700], -0.25),                    # a one-token segment, negative scale
])
def test_virtual_ring_matches_the_oracle(oracle, B, H, L, d, gate, cuts, scale):
    from paper_2505_16381_b200 import ring
    inp = synth.make_inputs(B, H, L, d, "bf16", gate=gate, seed=9100 + L + d, sharp=(L == 1000))
    ops = ring.GpuOps(B, H, d, scale=scale, has_gate=gate)
    outs = ring.virtual_ring_forward(ops, split(inp, cuts))
    o = torch.cat([x[0] for x in outs], dim=2)
    lse = torch.cat([x[1] for x in outs], dim=2)
    f = synth.to_f64
    o_ref, lse_ref = oracle.forward(f(inp["q"]), f(inp["k"]), f(inp["v"]), f(inp["w"]), f(inp["beta"]),
                                    None if inp["log_f"] is None else f(inp["log_f"]), scale=scale)
    got = f(o)
    assert np.isfinite(got).all()
    assert np.linalg.norm(got - o_ref) <= 1e-2 * np.linalg.norm(o_ref)
    assert np.abs(got - o_ref).max() <= 2e-2 * max(1.0, np.abs(o_ref).max())
    assert np.abs(f(lse) - lse_ref).max() <= 2e-3 * max(1.0, np.abs(lse_ref).max())


def test_one_segment_is_the_ordinary_forward(oracle):
    from paper_2505_16381_b200 import binding, ring
    inp = synth.make_inputs(1, 2, 640, 128, "bf16", gate=True, seed=9200)
    seg = split(inp, [640])[0]
    (o, lse), = ring.virtual_ring_forward(ring.GpuOps(1, 2, 128, has_gate=True), [seg])
    o2, lse2 = binding.path_attn_fwd(seg["q"], seg["k"], seg["v"], seg["w"], seg["beta"], seg["log_f"])
    assert torch.equal(o, o2) and torch.allclose(lse, lse2, rtol=0, atol=1e-6)
