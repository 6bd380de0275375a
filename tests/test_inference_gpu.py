"""Parity of the inference entry points (paper Sec. 3.4) with the float64 oracle, through the C ABI.

* the key cache after a prefill against the oracle's key-cache recurrence;
* decoding steps against rows of the oracle's full forward (a decoded token's output is that row of causal attention over
  the whole sequence) and, after the last step, the updated cache against the oracle's cache of the longer prefix.

Tolerances: the prefill cache is built from bf16 tensor-core tiles (keys rounded once to bf16 after the chunk transform,
chunk products carried as bf16 pairs), so it is held to the training path's bounds (rel-Fro 1e-2, max-abs 2e-2); the
decoding step itself is float32 arithmetic on the cache, so starting from an exact cache its outputs are held to 2^-8
(o is stored in bf16) and the cache to 1e-5.
"""
import numpy as np
import pytest
import torch

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


@pytest.mark.parametrize("B,H,L,d,gate", [
    (1, 2, 512, 64, False),
    (2, 1, 700, 128, True),      # ragged length
    (1, 3, 100, 128, False),     # a single chunk
    (1, 1, 2304, 64, True),      # 18 chunks
    (1, 2, 4224, 128, True),     # 33 chunks: the walk is cut into 4 ranges (9, 9, 9, 6 chunks) + suffix products
    (2, 1, 8300, 64, False),     # 65 chunks, ragged: 8 ranges of 9 chunks, the last one of 2
])
def test_prefill_cache_matches_oracle(binding, oracle, B, H, L, d, gate):
    inp = synth.make_inputs(B, H, L, d, "bf16", gate=gate, seed=50 + L)
    dev = {n: (t.cuda() if torch.is_tensor(t) else t) for n, t in inp.items()}
    cap = L + 5
    cache = binding.alloc_cache(B, H, cap, d, gate)
    cache["kc"].fill_(7.0)
    ws = binding.path_attn_prefill_cache(dev["k"], dev["v"], dev["w"], dev["beta"], cache, dev["log_f"])
    assert binding.device_status(ws) == 0
    ref = oracle.key_cache(f64(inp["k"]), f64(inp["w"]), f64(inp["beta"]))
    got = cache["kc"][:, :, :L].cpu().double().numpy()
    assert rel_fro(got, ref) <= 1e-2 and np.abs(got - ref).max() <= 2e-2 * max(1.0, np.abs(ref).max())
    assert torch.all(cache["kc"][:, :, L:] == 7.0)                       # rows past the prompt are left alone
    assert torch.equal(cache["vc"][:, :, :L], dev["v"])
    if gate:
        G = np.cumsum(f64(inp["log_f"]), axis=-1)
        assert np.abs(cache["gc"][:, :, :L].cpu().double().numpy() - G).max() <= 1e-4 * max(1.0, np.abs(G).max())


@pytest.mark.parametrize("B,H,L0,T,d,gate,scale", [
    (1, 2, 0, 40, 64, False, 1.0),        # decoding from an empty cache
    (2, 2, 300, 33, 128, True, 1.0),      # crosses a 256-position block of the split
    (1, 1, 1000, 8, 64, True, 0.5),
])
def test_decode_steps_match_oracle_rows(binding, oracle, B, H, L0, T, d, gate, scale):
    L = L0 + T
    inp = synth.make_inputs(B, H, L, d, "bf16", gate=gate, seed=70 + L)
    q, k, v, w, beta, lf = (f64(inp[n]) for n in ("q", "k", "v", "w", "beta", "log_f"))
    dev = {n: (t.cuda() if torch.is_tensor(t) else t) for n, t in inp.items()}
    cache = binding.alloc_cache(B, H, L, d, gate)
    # start from the oracle's exact cache of the first L0 tokens, so that only the decoding arithmetic is under test
    if L0:
        cache["kc"][:, :, :L0] = torch.from_numpy(oracle.key_cache(k, w, beta, L0)).float().cuda()
        cache["vc"][:, :, :L0] = dev["v"][:, :, :L0]
        if gate:
            cache["gc"][:, :, :L0] = torch.from_numpy(np.cumsum(lf, axis=-1)[..., :L0]).float().cuda()
    ws = binding.decode_workspace(B, H, L, d)
    o_ref, lse_ref = oracle.forward(q, k, v, w, beta, lf, scale=scale, rows=list(range(L0, L)))
    for i, t in enumerate(range(L0, L)):
        tok = lambda n: dev[n][:, :, t].contiguous()
        o_t, lse_t = binding.path_attn_decode_step(tok("q"), tok("k"), tok("v"), tok("w"), dev["beta"][:, :, t].contiguous(),
                                                   cache, t, dev["log_f"][:, :, t].contiguous() if gate else None,
                                                   scale=scale, workspace=ws)
        got = o_t.float().cpu().double().numpy()
        ref = o_ref[..., i, :]
        assert np.abs(got - ref).max() <= 2 ** -8 * max(1.0, np.abs(ref).max()), ("o", t)
        assert np.abs(lse_t.cpu().double().numpy() - lse_ref[..., i]).max() <= 1e-4 * max(1.0, np.abs(lse_ref).max()), ("lse", t)
    kc_ref = oracle.key_cache(k, w, beta, L)
    got = cache["kc"].cpu().double().numpy()
    assert np.abs(got - kc_ref).max() <= 1e-5 * max(1.0, np.abs(kc_ref).max())
    assert torch.equal(cache["vc"], dev["v"])


def test_prefill_then_decode_end_to_end(binding, oracle):
    """Prompt through path_attn_prefill_cache, then decoding steps: outputs within the training path's bounds."""
    B, H, L0, T, d = 1, 2, 640, 6, 128
    L = L0 + T
    inp = synth.make_inputs(B, H, L, d, "bf16", gate=True, seed=99)
    q, k, v, w, beta, lf = (f64(inp[n]) for n in ("q", "k", "v", "w", "beta", "log_f"))
    dev = {n: (t.cuda() if torch.is_tensor(t) else t) for n, t in inp.items()}
    cache = binding.alloc_cache(B, H, L, d, True)
    pre = lambda n: dev[n][:, :, :L0].contiguous()
    binding.path_attn_prefill_cache(pre("k"), pre("v"), pre("w"), pre("beta"), cache, pre("log_f"))
    o_ref, _ = oracle.forward(q, k, v, w, beta, lf, rows=list(range(L0, L)))
    for i, t in enumerate(range(L0, L)):
        tok = lambda n: dev[n][:, :, t].contiguous()
        o_t, _ = binding.path_attn_decode_step(tok("q"), tok("k"), tok("v"), tok("w"), tok("beta"), cache, t, tok("log_f"))
        got = o_t.float().cpu().double().numpy()
        ref = o_ref[..., i, :]
        assert rel_fro(got, ref) <= 1e-2 and np.abs(got - ref).max() <= 2e-2 * max(1.0, np.abs(ref).max())


def test_inference_argument_checks(binding):
    cache = binding.alloc_cache(1, 1, 16, 64, False)
    x = torch.zeros(1, 1, 64, dtype=torch.bfloat16, device="cuda")
    b = torch.ones(1, 1, dtype=torch.float32, device="cuda")
    with pytest.raises(binding.PathAttnError) as e:
        binding.path_attn_decode_step(x, x, x, x, b, cache, 16)          # t == capacity
    assert e.value.status == -2
    with pytest.raises(binding.PathAttnError) as e:
        binding.path_attn_decode_step(x, x, x, x, b, cache, 0, log_f_t=b)   # gate given without a gate cache
    assert e.value.status == -1
    k = torch.zeros(1, 1, 32, 64, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.PathAttnError) as e:
        binding.path_attn_prefill_cache(k, k, k, torch.ones(1, 1, 32, device="cuda"), cache)   # prompt longer than the cache
    assert e.value.status == -2
