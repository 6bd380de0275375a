"""``torch.autograd`` entry points over the binding: the operator and the layer front-end as differentiable functions.

Argument marshalling only: every forward and backward below is one call of :mod:`binding` (the C-ABI library).  There is
no other implementation behind them: without the built library, or on a non-CUDA tensor, they raise.

    o = path_attention(q, k, v, w, beta, log_f=None, scale=1.0)            # [B,H,L,d] bf16; beta / log_f [B,H,L] float32
    w, beta, log_f = path_frontend(z, conv_w, beta_logit, gate_logit, H)   # z [B,L,H*d] bf16, logits [B,L,H] float32
"""
from __future__ import annotations

import torch

from . import binding


class _PathAttention(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, w, beta, log_f, scale, retain_state):
        # (requires_grad of the copies .contiguous() makes is always False here: ask autograd itself)
        need_grad = any(ctx.needs_input_grad[:6])
        q, k, v, w = (t.contiguous() for t in (q, k, v, w))
        beta = beta.contiguous()
        log_f = None if log_f is None else log_f.contiguous()
        # Default: a forward-sized workspace that is released right away; the backward recomputes the chunk preparation.
        # retain_state keeps a backward-sized workspace (about ten times the size of q, k, v, w together) alive from
        # forward to backward so that the backward can skip that recomputation.
        keep = bool(retain_state) and need_grad
        ws = binding.alloc_workspace(q, log_f is not None, keep)
        o, lse = binding.path_attn_fwd(q, k, v, w, beta, log_f, scale=scale, workspace=ws)
        ctx.save_for_backward(q, k, v, w, beta, log_f, o, lse)
        ctx.scale, ctx.ws = scale, (ws if keep else None)
        ctx.mark_non_differentiable(lse)
        return o, lse

    @staticmethod
    def backward(ctx, d_o, _d_lse):
        q, k, v, w, beta, log_f, o, lse = ctx.saved_tensors
        g = binding.path_attn_bwd(q, k, v, w, beta, o, lse, d_o.contiguous(), log_f, scale=ctx.scale, workspace=ctx.ws,
                                  reuse=ctx.ws is not None)
        ctx.ws = None
        return g["dq"], g["dk"], g["dv"], g["dw"], g["dbeta"], g.get("dlog_f"), None, None


def path_attention(q, k, v, w, beta, log_f=None, scale: float = 1.0, return_lse: bool = False, retain_state: bool = False):
    """PaTH attention (paper Sec. 2.2; PaTH-FoX when ``log_f`` is given), differentiable in q, k, v, w, beta, log_f.

    ``retain_state=True`` trades memory for time: the forward's chunk preparation stays in a backward-sized workspace
    until the backward has used it (see ``path_attn_bwd_reuse``)."""
    o, lse = _PathAttention.apply(q, k, v, w, beta, log_f, float(scale), bool(retain_state))
    return (o, lse) if return_lse else o


class _PathFrontend(torch.autograd.Function):
    @staticmethod
    def forward(ctx, z, conv_w, beta_logit, gate_logit, H, eps):
        z, conv_w, beta_logit = z.contiguous(), conv_w.contiguous(), beta_logit.contiguous()
        gate_logit = None if gate_logit is None else gate_logit.contiguous()
        w, beta, log_f = binding.path_attn_frontend_fwd(z, conv_w, beta_logit, gate_logit, H=H, eps=eps)
        ctx.save_for_backward(z, conv_w, beta_logit, gate_logit)
        ctx.H, ctx.eps = H, eps
        return w, beta, log_f

    @staticmethod
    def backward(ctx, dw, dbeta, dlog_f):
        z, conv_w, beta_logit, gate_logit = ctx.saved_tensors
        if gate_logit is not None and dlog_f is None:
            dlog_f = torch.zeros(dbeta.shape, dtype=torch.float32, device=z.device)
        dz, dcw, dbl, dgl = binding.path_attn_frontend_bwd(z, conv_w, beta_logit, dw.contiguous(), dbeta.contiguous(),
                                                           gate_logit, None if gate_logit is None else dlog_f.contiguous(),
                                                           H=ctx.H, eps=ctx.eps)
        return dz, dcw, dbl, dgl, None, None


def path_frontend(z, conv_w, beta_logit, gate_logit=None, H: int = 1, eps: float = 1e-6):
    """Layer front-end (paper Sec. 2.2 footnote, Sec. 2.4 gate): ``(w, beta, log_f)`` in the operator's layouts,
    differentiable in z, conv_w and the logits.  ``log_f`` is None when ``gate_logit`` is."""
    return _PathFrontend.apply(z, conv_w, beta_logit, gate_logit, int(H), float(eps))
