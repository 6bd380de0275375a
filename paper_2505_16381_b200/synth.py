"""Seeded synthetic inputs shaped like the paper's language-model workloads.

This module holds no arithmetic of the method itself: it only draws random
tensors, normalises w, squashes beta and the gate, and rounds to the I/O dtype.
Both the CPU oracle's tests and the CUDA path's tests / benchmark feed on it, so
that the two are always compared on identical values.

Recipe (fixed draw order q, k, v, w_raw, z_beta, z_f, dO from one CPU
generator): q, k ~ N(0,1) (divided by sqrt(d) when ``qk_scaled``), v ~ N(0,1),
w = w_raw / ||w_raw||_2, beta = 2*sigmoid(z_beta), log f = logsigmoid(z_f + 3),
dO ~ N(0,1).  q, k, v, w, dO are rounded to the I/O dtype; beta and log f stay
float32.
"""
from __future__ import annotations

import torch

BASE_SEED = 250516381

# name -> (B, H, L, d, dtype, qk_scaled, gate, backward)
CONFIGS = {
    "C1": dict(B=1, H=2, L=256, d=64, dtype="fp32", qk_scaled=False, gate=False, backward=False, index=0),
    "C2": dict(B=8, H=16, L=2048, d=64, dtype="bf16", qk_scaled=True, gate=False, backward=True, index=1),
    "C3": dict(B=4, H=16, L=4096, d=128, dtype="bf16", qk_scaled=True, gate=False, backward=True, index=2),
    "C4": dict(B=2, H=16, L=8192, d=128, dtype="bf16", qk_scaled=True, gate=True, backward=True, index=3),
    "C5": dict(B=1, H=32, L=32768, d=128, dtype="bf16", qk_scaled=True, gate=False, backward=False, index=4),
}

_DTYPES = {"bf16": torch.bfloat16, "fp32": torch.float32}


def make_inputs(B, H, L, d, dtype="bf16", qk_scaled=True, gate=False, seed=BASE_SEED, sharp=False,
                **_unused):
    """Returns a dict of CPU tensors: q, k, v, w, d_o ``[B,H,L,d]`` in ``dtype``; beta ``[B,H,L]``
    float32; log_f ``[B,H,L]`` float32 or None; scale (always 1.0: the 1/sqrt(d) of the
    workloads is folded into q and k).

    ``sharp=True`` keeps q at unit variance and scales only k, which gives unit-variance
    logits instead of the near-uniform attention of the default recipe.
    """
    gen = torch.Generator(device="cpu")
    gen.manual_seed(int(seed))
    td = _DTYPES[dtype]

    def draw(*shape):
        return torch.randn(*shape, generator=gen, dtype=torch.float32)

    q = draw(B, H, L, d)
    k = draw(B, H, L, d)
    v = draw(B, H, L, d)
    w_raw = draw(B, H, L, d)
    z_beta = draw(B, H, L)
    z_f = draw(B, H, L)
    d_o = draw(B, H, L, d)
    if sharp:
        k = k / d ** 0.5
    elif qk_scaled:
        q = q / d ** 0.5
        k = k / d ** 0.5
    w = w_raw / w_raw.norm(dim=-1, keepdim=True)
    beta = 2.0 * torch.sigmoid(z_beta)
    log_f = torch.nn.functional.logsigmoid(z_f + 3.0) if gate else None
    return {
        "q": q.to(td).contiguous(), "k": k.to(td).contiguous(), "v": v.to(td).contiguous(),
        "w": w.to(td).contiguous(), "d_o": d_o.to(td).contiguous(),
        "beta": beta.contiguous(), "log_f": None if log_f is None else log_f.contiguous(),
        "scale": 1.0,
    }


def make_frontend_inputs(B, H, L, d, gate=False, seed=BASE_SEED):
    """Random inputs of the layer front-end (CPU tensors): z ``[B,L,H*d]`` bf16 ~ N(0,1), conv_w ``[H*d,3]`` float32
    ~ N(0,1/3), beta_logit ``[B,L,H]`` ~ N(0,1), gate_logit ~ N(3,1) or None, and upstream gradients dw ``[B,H,L,d]``
    bf16, dbeta, dlog_f ``[B,H,L]`` float32 ~ N(0,1).  Draw order as listed."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(int(seed))

    def draw(*shape):
        return torch.randn(*shape, generator=gen, dtype=torch.float32)

    z = draw(B, L, H * d)
    conv_w = draw(H * d, 3) / 3 ** 0.5
    beta_logit = draw(B, L, H)
    gate_logit = draw(B, L, H) + 3.0
    dw = draw(B, H, L, d)
    dbeta = draw(B, H, L)
    dlog_f = draw(B, H, L)
    return {
        "z": z.to(torch.bfloat16).contiguous(), "conv_w": conv_w.contiguous(), "beta_logit": beta_logit.contiguous(),
        "gate_logit": gate_logit.contiguous() if gate else None, "dw": dw.to(torch.bfloat16).contiguous(),
        "dbeta": dbeta.contiguous(), "dlog_f": dlog_f.contiguous() if gate else None,
    }


def make_config(name: str):
    """Inputs of one of the named workloads (seed = BASE_SEED + its index)."""
    c = CONFIGS[name]
    return make_inputs(c["B"], c["H"], c["L"], c["d"], dtype=c["dtype"], qk_scaled=c["qk_scaled"],
                       gate=c["gate"], seed=BASE_SEED + c["index"])


def to_f64(t):
    """Exact upcast of a (possibly bf16) CPU tensor to a float64 numpy array."""
    return None if t is None else t.detach().cpu().to(torch.float64).numpy()
