"""Ring schedule of context-parallel PaTH attention (paper Sec. 3.5, "Compatibility with context-parallelism").

The sequence is cut into contiguous segments, rank r holding segment r.  Every rank prepares its segment (its own causal
attention, its queries pulled back to the segment's start, and the message ``(transformed keys, values, segment
product)`` for the holders of later queries); then the messages travel around the ring, one hop per step, and a rank
attends the message of segment ``r - t`` at step ``t`` if that segment is an earlier one, nearest first, updating its
query state after each.  A received message always lands in a buffer of the receiving rank's own memory before any
kernel reads it.

The per-segment arithmetic is behind an ``ops`` object (``prepare``, ``empty_message``, ``step``, ``finish``):
:class:`GpuOps` marshals to the C-ABI calls ``path_attn_cp_*`` (there is no other implementation in this package; the
schedule itself is plain ``torch.distributed`` point-to-point traffic and runs on any backend).
"""
from __future__ import annotations

import torch


class GpuOps:
    """``path_attn_cp_prepare / step / finish`` on the current CUDA device for slices ``[B, H, ., d]``."""

    def __init__(self, B, H, d, scale=1.0, has_gate=False, device="cuda"):
        from . import binding
        self.b, self.B, self.H, self.d, self.scale, self.gate, self.device = binding, B, H, d, scale, has_gate, device

    def prepare(self, seg):
        """``seg``: dict with q, k, v, w ``[B,H,L,d]`` bf16, beta and optional log_f ``[B,H,L]`` float32."""
        state, message, self.ws = self.b.path_attn_cp_prepare(seg["q"], seg["k"], seg["v"], seg["w"], seg["beta"],
                                                              seg.get("log_f"), scale=self.scale)
        return state, message

    def empty_message(self, L):
        n = int(self.b.load().path_attn_cp_message_bytes(self.B, self.H, int(L), self.d))
        return torch.empty(n, dtype=torch.uint8, device=self.device)

    def step(self, state, message, Lq, Lk):
        self.b.path_attn_cp_step(state, message, self.B, self.H, int(Lq), int(Lk), self.d, scale=self.scale, workspace=self.ws)

    def finish(self, state, L):
        return self.b.path_attn_cp_finish(state, self.B, self.H, int(L), self.d)


def virtual_ring_forward(ops, segments):
    """All ranks of the ring played one after the other by ONE process (no communication): returns the list of
    ``finish`` results, one per segment.  ``segments[r]`` is rank r's input dict; ``segments[r]["q"].shape[-2]`` its length."""
    lengths = [int(s["q"].shape[-2]) for s in segments]
    prepared = [ops.prepare(s) for s in segments]
    out = []
    for r, (state, _) in enumerate(prepared):
        for t in range(1, r + 1):                      # nearest earlier segment first
            ops.step(state, prepared[r - t][1], lengths[r], lengths[r - t])
        out.append(ops.finish(state, lengths[r]))
    return out


def ring_forward(ops, seg, group=None):
    """One rank of the ring: ``seg`` is this rank's segment.  Returns this segment's ``finish`` result.

    ``world - 1`` hops; in hop ``t`` every rank passes the message it holds to rank + 1 and receives the one of segment
    ``rank - t`` from rank - 1, which it attends if ``rank - t >= 0`` (causality: later segments' messages are forwarded
    but never read)."""
    import torch.distributed as dist
    rank, world = dist.get_rank(group), dist.get_world_size(group)
    L = int(seg["q"].shape[-2])
    state, message = ops.prepare(seg)
    lengths = [torch.zeros(1, dtype=torch.int64, device=message.device) for _ in range(world)]
    dist.all_gather(lengths, torch.tensor([L], dtype=torch.int64, device=message.device), group=group)
    lengths = [int(x.item()) for x in lengths]
    held = message
    nxt, prv = (rank + 1) % world, (rank - 1) % world
    for t in range(1, world):
        owner = (rank - t) % world
        incoming = ops.empty_message(lengths[owner])
        reqs = dist.batch_isend_irecv([dist.P2POp(dist.isend, held, nxt, group), dist.P2POp(dist.irecv, incoming, prv, group)])
        for r in reqs:
            r.wait()
        held = incoming
        if rank - t >= 0:
            ops.step(state, held, L, lengths[owner])
    return ops.finish(state, L)
