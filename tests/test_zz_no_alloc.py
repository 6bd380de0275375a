"""path_attn_fwd_static: the forward entry point for callers that may not allocate device memory.

Such callers (code running under CUDA-graph stream capture, plug-ins of a runtime that owns the whole device pool,
loops that cannot afford cudaMalloc's implicit synchronisation) pass only inputs and outputs; the scratch memory is a
fixed buffer inside the library.  The GPU test drives the entry point through the C ABI twice in a row, with different
problems so that the second call meets the first call's leftovers in the shared buffer, and checks each result against
the ordinary path_attn_fwd on the same inputs and against the float64 oracle.  This file sorts last on purpose: a run that stops at the first failure
has then already run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2505_16381_b200 import synth


def test_static_entry_point_rejects_oversized_problems_on_the_host():
    from paper_2505_16381_b200 import binding, build
    build.build()
    lib = binding.load()
    P = 0x4000
    big = dict(B=4, H=16, L=4096, d=128)
    assert binding.workspace_bytes(**big) > binding.STATIC_SCRATCH_BYTES
    rc = lib.path_attn_fwd_static(P, P, P, P, P, None, P, P, big["B"], big["H"], big["L"], big["d"], 1.0, 0, None, None)
    assert rc == -9
    assert "static buffer" in lib.path_attn_strerror(rc).decode()
    assert lib.path_attn_fwd_static(P, P, P, P, P, None, P, P, 1, 1, 128, 96, 1.0, 0, None, None) == -2
    assert lib.path_attn_fwd_static(P, P, P, P, P, None, P, P, 1, 1, 128, 64, 1.0, 9, None, None) == -3


@pytest.mark.gpu
def test_static_entry_point_matches_workspace_entry_point_twice_in_a_row(oracle):
    from paper_2505_16381_b200 import binding
    binding.load()
    problems = [dict(B=1, H=2, L=640, d=128, gate=True, seed=41), dict(B=2, H=2, L=300, d=64, gate=False, seed=42)]
    for prob in problems:
        assert binding.workspace_bytes(prob["B"], prob["H"], prob["L"], prob["d"], has_gate=prob["gate"]) \
            <= binding.STATIC_SCRATCH_BYTES
        inp = synth.make_inputs(prob["B"], prob["H"], prob["L"], prob["d"], "bf16", gate=prob["gate"], seed=prob["seed"])
        dev = {k: (v.cuda() if torch.is_tensor(v) else v) for k, v in inp.items()}
        args = (dev["q"], dev["k"], dev["v"], dev["w"], dev["beta"], dev["log_f"])
        o_ref, lse_ref = binding.path_attn_fwd(*args, scale=1.0)
        # outputs are the caller's: allocate them up front, the call itself allocates nothing
        o = torch.full_like(dev["q"], float("nan"))
        lse = torch.full_like(dev["beta"], float("nan"))
        allocations = lambda: torch.cuda.memory_stats()["allocation.all.allocated"]   # count of torch allocator requests
        binding.path_attn_fwd_static(*args, scale=1.0, out=(o, lse))   # (the first call on a device looks the buffer up)
        torch.cuda.synchronize()
        o.fill_(float("nan")); lse.fill_(float("nan"))
        torch.cuda.synchronize()
        before, free_before = allocations(), torch.cuda.mem_get_info()[0]     # free bytes as the driver counts them
        _, _, scratch = binding.path_attn_fwd_static(*args, scale=1.0, out=(o, lse))
        torch.cuda.synchronize()
        # neither torch's allocator nor the driver (a cudaMalloc inside the library would show here) handed out memory
        assert allocations() == before and torch.cuda.mem_get_info()[0] == free_before
        # same kernels, same order: the tolerances of the parity tests hold with room to spare
        assert torch.isfinite(o).all() and torch.isfinite(lse).all()
        err = (o.float() - o_ref.float()).abs().max().item()
        rel = ((o.float() - o_ref.float()).norm() / o_ref.float().norm()).item()
        assert err <= 2e-2 and rel <= 1e-2, (prob, err, rel)
        assert (lse - lse_ref).abs().max().item() <= 2e-3
        # and directly against the oracle, with the parity tests' bounds
        f = synth.to_f64
        o64, lse64 = oracle.forward(f(inp["q"]), f(inp["k"]), f(inp["v"]), f(inp["w"]), f(inp["beta"]),
                                    None if inp["log_f"] is None else f(inp["log_f"]), scale=1.0)
        got = f(o)
        assert np.linalg.norm(got - o64) <= 1e-2 * np.linalg.norm(o64)
        assert np.abs(got - o64).max() <= 2e-2 * max(1.0, np.abs(o64).max())
        assert np.abs(f(lse) - lse64).max() <= 2e-3 * max(1.0, np.abs(lse64).max())
        # the scratch address handed back is a device pointer usable with the status query
        detail = ctypes.c_uint(123)
        st = torch.cuda.current_stream().cuda_stream
        rc = binding.load().path_attn_device_status(ctypes.c_void_p(scratch), ctypes.c_void_p(st), ctypes.byref(detail))
        assert rc == 0 and detail.value == 0
