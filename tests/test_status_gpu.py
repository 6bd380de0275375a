"""The device status word: a bounded wait that runs out is reported as PATH_ERR_TIMEOUT, and the workspace is usable
again afterwards.  The wait that runs out is the library's own self-test (a barrier nothing arrives on, with a limit of a
millisecond): nothing faults, traps or hangs."""
import numpy as np
import pytest
import torch

from paper_2505_16381_b200 import synth

pytestmark = pytest.mark.gpu


def test_an_expired_wait_is_reported_and_the_workspace_recovers(oracle):
    from paper_2505_16381_b200 import binding as b
    inp = synth.make_inputs(1, 2, 300, 64, "bf16", seed=77)
    dev = {k: (v.cuda() if torch.is_tensor(v) else v) for k, v in inp.items()}
    ws = b.alloc_workspace(dev["q"], False, True)
    args = (dev["q"], dev["k"], dev["v"], dev["w"], dev["beta"])
    o0, lse0 = b.path_attn_fwd(*args, workspace=ws)
    assert b.device_status(ws) == 0
    t0 = torch.cuda.Event(enable_timing=True)
    t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    b.selftest_timeout(ws, limit_us=1000)
    t1.record()
    with pytest.raises(b.PathAttnError) as e:
        b.device_status(ws)
    assert e.value.status == -8 and "0x7f1" in str(e.value)
    assert 0.3 <= t0.elapsed_time(t1) <= 50.0           # the wait gave up after about its limit (1 ms), not at once, not never
    # the context and the workspace are intact: the next calls are clean and right
    o1, lse1 = b.path_attn_fwd(*args, workspace=ws)
    assert b.device_status(ws) == 0
    assert torch.equal(o0, o1) and torch.equal(lse0, lse1)
    g = b.path_attn_bwd(*args, o1, lse1, dev["d_o"], workspace=ws, reuse=True)
    assert b.device_status(ws) == 0
    f = synth.to_f64
    x = [f(inp[n]).reshape(-1, *inp[n].shape[2:]) for n in ("q", "k", "v", "w", "beta", "d_o")]
    ref = oracle.backward(x[0], x[1], x[2], x[3], x[4], x[5], None)
    for n, r in ref.items():
        got = g[n].float().cpu().double().numpy().reshape(r.shape)
        assert np.linalg.norm(got - r) <= 1e-2 * np.linalg.norm(r), n


def test_selftest_argument_errors():
    from paper_2505_16381_b200 import binding as b
    ws = torch.empty(1024, dtype=torch.uint8, device="cuda")
    for bad in (0, 200000):
        with pytest.raises(b.PathAttnError) as e:
            b.selftest_timeout(ws, limit_us=bad)
        assert e.value.status == -2
