"""Python binding of the C-ABI library: argument marshalling only.

Every step of the path runs in the CUDA kernels behind ``include/path_attn.h``;
torch is used here for device memory and the current stream.  There is no CPU
fallback: if the shared library has not been built or the tensors are not on a
CUDA device, the calls raise.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_LIB_PATH = Path(__file__).resolve().parent / "libpath_attn.so"
_lib = None

PATH_BF16, PATH_FP32 = 0, 1
PATH_OK = 0
EXPORTS = ["path_attn_workspace_bytes", "path_attn_fwd", "path_attn_bwd", "path_attn_bwd_reuse", "path_attn_fwd_static",
           "path_attn_device_status", "path_attn_selftest_timeout",
           "path_attn_prefill_cache", "path_attn_decode_workspace_bytes", "path_attn_decode_step",
           "path_attn_frontend_fwd", "path_attn_frontend_bwd", "path_attn_skipped_chunk_pairs",
           "path_attn_lowrank_workspace_bytes", "path_attn_lowrank_fwd", "path_attn_lowrank_bwd",
           "path_attn_cp_state_bytes", "path_attn_cp_message_bytes", "path_attn_cp_workspace_bytes",
           "path_attn_cp_prepare", "path_attn_cp_step", "path_attn_cp_finish",
           "path_attn_strerror", "path_attn_last_cuda_error", "path_attn_last_launch_count",
           "path_attn_profile_enable", "path_attn_profile_read", "path_attn_profile_stage_name"]


class PathAttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        lib = load()
        msg = lib.path_attn_strerror(status).decode()
        extra = f" (cudaError {lib.path_attn_last_cuda_error()})" if status == -7 else ""
        super().__init__(f"{where}: {msg}{extra} [status {status}]")
        self.status = status


def load():
    """Loads ``libpath_attn.so`` (built by ``paper_2505_16381_b200.build``); raises if it is missing."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise FileNotFoundError(
                f"{_LIB_PATH} not found: build it with `python -m paper_2505_16381_b200.build` (there is no fallback)")
        lib = ctypes.CDLL(str(_LIB_PATH))
        P, I, F, Z = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        lib.path_attn_workspace_bytes.restype = Z
        lib.path_attn_workspace_bytes.argtypes = [I, I, I, I, I, I, I]
        lib.path_attn_fwd.restype = I
        lib.path_attn_fwd.argtypes = [P, P, P, P, P, P, P, P, I, I, I, I, F, I, P, Z, P]
        lib.path_attn_fwd_static.restype = I
        lib.path_attn_fwd_static.argtypes = [P, P, P, P, P, P, P, P, I, I, I, I, F, I, P, ctypes.POINTER(P)]
        lib.path_attn_bwd.restype = I
        lib.path_attn_bwd.argtypes = [P] * 15 + [I, I, I, I, F, I, P, Z, P]
        lib.path_attn_bwd_reuse.restype = I
        lib.path_attn_bwd_reuse.argtypes = [P] * 15 + [I, I, I, I, F, I, P, Z, P]
        lib.path_attn_selftest_timeout.restype = I
        lib.path_attn_selftest_timeout.argtypes = [P, ctypes.c_uint, P]
        lib.path_attn_prefill_cache.restype = I
        lib.path_attn_prefill_cache.argtypes = [P] * 8 + [I, I, I, I, I, I, P, Z, P]
        lib.path_attn_decode_workspace_bytes.restype = Z
        lib.path_attn_decode_workspace_bytes.argtypes = [I, I, I, I]
        lib.path_attn_decode_step.restype = I
        lib.path_attn_decode_step.argtypes = [P] * 9 + [I, I, P, P, I, I, I, F, I, P, Z, P]
        lib.path_attn_frontend_fwd.restype = I
        lib.path_attn_frontend_fwd.argtypes = [P] * 7 + [I, I, I, I, F, P]
        lib.path_attn_frontend_bwd.restype = I
        lib.path_attn_frontend_bwd.argtypes = [P] * 11 + [I, I, I, I, F, P]
        for fn in (lib.path_attn_cp_state_bytes, lib.path_attn_cp_message_bytes):
            fn.restype, fn.argtypes = Z, [I, I, I, I]
        lib.path_attn_cp_workspace_bytes.restype = Z
        lib.path_attn_cp_workspace_bytes.argtypes = [I, I, I, I, I]
        lib.path_attn_cp_prepare.restype = I
        lib.path_attn_cp_prepare.argtypes = [P] * 8 + [I, I, I, I, F, I, P, Z, P]
        lib.path_attn_cp_step.restype = I
        lib.path_attn_cp_step.argtypes = [P, P, I, I, I, I, I, F, P, Z, P]
        lib.path_attn_cp_finish.restype = I
        lib.path_attn_cp_finish.argtypes = [P, P, P, I, I, I, I, P]
        LL = ctypes.c_longlong
        lib.path_attn_lowrank_workspace_bytes.restype = Z
        lib.path_attn_lowrank_workspace_bytes.argtypes = [LL, I, I, I]
        lib.path_attn_lowrank_fwd.restype = I
        lib.path_attn_lowrank_fwd.argtypes = [P] * 5 + [LL, I, I, I, P, Z, P]
        lib.path_attn_lowrank_bwd.restype = I
        lib.path_attn_lowrank_bwd.argtypes = [P] * 8 + [LL, I, I, I, P, Z, P]
        lib.path_attn_skipped_chunk_pairs.restype = I
        lib.path_attn_skipped_chunk_pairs.argtypes = [P, P, ctypes.POINTER(ctypes.c_ulonglong), ctypes.POINTER(ctypes.c_ulonglong)]
        lib.path_attn_device_status.restype = I
        lib.path_attn_device_status.argtypes = [P, P, ctypes.POINTER(ctypes.c_uint)]
        lib.path_attn_strerror.restype = ctypes.c_char_p
        lib.path_attn_strerror.argtypes = [I]
        lib.path_attn_last_cuda_error.restype = I
        lib.path_attn_last_launch_count.restype = I
        lib.path_attn_profile_enable.restype = I
        lib.path_attn_profile_enable.argtypes = [I]
        lib.path_attn_profile_read.restype = I
        lib.path_attn_profile_read.argtypes = [ctypes.POINTER(ctypes.c_float), I]
        lib.path_attn_profile_stage_name.restype = ctypes.c_char_p
        lib.path_attn_profile_stage_name.argtypes = [I]
        _lib = lib
    return _lib


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return PATH_BF16
    if t.dtype == torch.float32:
        return PATH_FP32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _check(q, *others):
    if not q.is_cuda:
        raise RuntimeError("path_attn: tensors must live on a CUDA device (there is no CPU path)")
    for t in others:
        if t is not None and (t.device != q.device or not t.is_contiguous()):
            raise RuntimeError("path_attn: all tensors must be contiguous and on the same device")
    if q.dim() != 4 or not q.is_contiguous():
        raise RuntimeError("path_attn: q must be a contiguous [B, H, L, d] tensor")


def workspace_bytes(B, H, L, d, dtype=PATH_BF16, has_gate=False, for_backward=False) -> int:
    return int(load().path_attn_workspace_bytes(B, H, L, d, dtype, int(has_gate), int(for_backward)))


def alloc_workspace(q, has_gate=False, for_backward=False) -> torch.Tensor:
    B, H, L, d = q.shape
    n = workspace_bytes(B, H, L, d, _dt(q), has_gate, for_backward)
    if n == 0:
        raise PathAttnError(-2, "path_attn_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=q.device)


def path_attn_fwd(q, k, v, w, beta, log_f=None, scale=1.0, workspace=None, out=None):
    """Forward.  Returns ``(o, lse)``; asynchronous on the current stream."""
    _check(q, k, v, w, beta, log_f)
    lib = load()
    B, H, L, d = q.shape
    if workspace is None:
        workspace = alloc_workspace(q, log_f is not None, False)
    o = torch.empty_like(q) if out is None else out[0]
    lse = torch.empty(B, H, L, dtype=torch.float32, device=q.device) if out is None else out[1]
    st = torch.cuda.current_stream(q.device).cuda_stream
    with torch.cuda.device(q.device):
        rc = lib.path_attn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(w), _ptr(beta), _ptr(log_f), _ptr(o), _ptr(lse),
                               B, H, L, d, float(scale), _dt(q), _ptr(workspace), workspace.numel(),
                               ctypes.c_void_p(st))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_fwd")
    return o, lse


STATIC_SCRATCH_BYTES = 16 << 20


def path_attn_fwd_static(q, k, v, w, beta, log_f=None, scale=1.0, out=None):
    """Forward through the entry point that takes no workspace: its scratch is a fixed buffer inside the library,
    so nothing is allocated by the call itself (the output tensors are the caller's; pass ``out=(o, lse)`` to
    reuse preallocated ones).  Only problems needing at most ``STATIC_SCRATCH_BYTES`` of scratch are accepted.
    Returns ``(o, lse, scratch_address)``."""
    _check(q, k, v, w, beta, log_f)
    lib = load()
    B, H, L, d = q.shape
    o = torch.empty_like(q) if out is None else out[0]
    lse = torch.empty(B, H, L, dtype=torch.float32, device=q.device) if out is None else out[1]
    st = torch.cuda.current_stream(q.device).cuda_stream
    addr = ctypes.c_void_p(0)
    with torch.cuda.device(q.device):
        rc = lib.path_attn_fwd_static(_ptr(q), _ptr(k), _ptr(v), _ptr(w), _ptr(beta), _ptr(log_f), _ptr(o), _ptr(lse),
                                      B, H, L, d, float(scale), _dt(q), ctypes.c_void_p(st), ctypes.byref(addr))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_fwd_static")
    return o, lse, addr.value


def path_attn_bwd(q, k, v, w, beta, o, lse, d_o, log_f=None, scale=1.0, workspace=None, out=None, reuse=False):
    """Backward.  Returns a dict dq, dk, dv, dw, dbeta (and dlog_f when gated).

    ``reuse=True`` calls ``path_attn_bwd_reuse``: the chunk preparation is taken from ``workspace``, where the forward of
    this very problem must have left it (backward-sized workspace, nothing written in between); a mismatch shows up as
    status -10 from :func:`device_status`."""
    _check(q, k, v, w, beta, log_f, o, lse, d_o)
    lib = load()
    B, H, L, d = q.shape
    if reuse and workspace is None:
        raise ValueError("reuse=True needs the workspace the forward ran on")
    if workspace is None:
        workspace = alloc_workspace(q, log_f is not None, True)
    if out is None:
        out = {n: torch.empty_like(q) for n in ("dq", "dk", "dv", "dw")}
        out["dbeta"] = torch.empty_like(beta)
        if log_f is not None:
            out["dlog_f"] = torch.empty_like(log_f)
    st = torch.cuda.current_stream(q.device).cuda_stream
    fn = lib.path_attn_bwd_reuse if reuse else lib.path_attn_bwd
    with torch.cuda.device(q.device):
        rc = fn(_ptr(q), _ptr(k), _ptr(v), _ptr(w), _ptr(beta), _ptr(log_f), _ptr(o), _ptr(lse),
                _ptr(d_o), _ptr(out["dq"]), _ptr(out["dk"]), _ptr(out["dv"]), _ptr(out["dw"]),
                _ptr(out["dbeta"]), _ptr(out.get("dlog_f")), B, H, L, d, float(scale), _dt(q),
                _ptr(workspace), workspace.numel(), ctypes.c_void_p(st))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_bwd")
    return out


def device_status(workspace) -> int:
    """Synchronises the current stream and returns the device status word of the last call on ``workspace``
    (0 = clean).  Raises on a timed-out device wait."""
    lib = load()
    detail = ctypes.c_uint(0)
    st = torch.cuda.current_stream(workspace.device).cuda_stream
    with torch.cuda.device(workspace.device):
        rc = lib.path_attn_device_status(_ptr(workspace), ctypes.c_void_p(st), ctypes.byref(detail))
    if rc != PATH_OK:
        raise PathAttnError(rc, f"path_attn_device_status (word 0x{detail.value:x})")
    return int(detail.value)


def selftest_timeout(workspace, limit_us=1000) -> None:
    """Launches the library's wait self-test on ``workspace``: a bounded wait that runs out after ``limit_us``
    microseconds and reports itself through the status word (read it with :func:`device_status`)."""
    lib = load()
    st = torch.cuda.current_stream(workspace.device).cuda_stream
    with torch.cuda.device(workspace.device):
        rc = lib.path_attn_selftest_timeout(_ptr(workspace), int(limit_us), ctypes.c_void_p(st))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_selftest_timeout")


def skipped_chunk_pairs(workspace):
    """(kept, all) chunk pairs of the last gated forward on ``workspace`` (block skipping; synchronises the stream)."""
    lib = load()
    kept, total = ctypes.c_ulonglong(0), ctypes.c_ulonglong(0)
    st = torch.cuda.current_stream(workspace.device).cuda_stream
    with torch.cuda.device(workspace.device):
        rc = lib.path_attn_skipped_chunk_pairs(_ptr(workspace), ctypes.c_void_p(st), ctypes.byref(kept), ctypes.byref(total))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_skipped_chunk_pairs")
    return kept.value, total.value


def last_launch_count() -> int:
    return int(load().path_attn_last_launch_count())


def profile_enable(on: bool = True) -> None:
    """Turns the library's per-stage CUDA-event timing on or off for the calling thread."""
    load().path_attn_profile_enable(int(on))


def profile_read() -> dict:
    """Milliseconds per stage of the most recent fwd / bwd call (stages that did not run are omitted)."""
    lib = load()
    buf = (ctypes.c_float * 16)()
    n = lib.path_attn_profile_read(buf, 16)
    if n < 0:
        raise PathAttnError(n, "path_attn_profile_read")
    return {lib.path_attn_profile_stage_name(i).decode(): float(buf[i]) for i in range(n) if buf[i] >= 0}


# ----------------------------------------------------------------------------------------- inference (key cache)

def alloc_cache(B, H, cap, d, gate=False, device="cuda"):
    """Empty caches for ``cap`` tokens: ``kc`` float32 and ``vc`` bf16 ``[B,H,cap,d]``, ``gc`` float32 ``[B,H,cap]`` or None."""
    return {"kc": torch.zeros(B, H, cap, d, dtype=torch.float32, device=device),
            "vc": torch.zeros(B, H, cap, d, dtype=torch.bfloat16, device=device),
            "gc": torch.zeros(B, H, cap, dtype=torch.float32, device=device) if gate else None}


def path_attn_prefill_cache(k, v, w, beta, cache, log_f=None, workspace=None):
    """Fills positions ``0..L-1`` of ``cache`` from a prompt: ``kc_j = H_{L-1} ... H_{j+1} k_j``, ``vc = v``, gate prefix."""
    _check(k, k, v, w, beta, log_f)
    lib = load()
    B, H, L, d = k.shape
    cap = cache["kc"].shape[2]
    if workspace is None:
        workspace = alloc_workspace(k, log_f is not None, False)
    st = torch.cuda.current_stream(k.device).cuda_stream
    with torch.cuda.device(k.device):
        rc = lib.path_attn_prefill_cache(_ptr(k), _ptr(v), _ptr(w), _ptr(beta), _ptr(log_f), _ptr(cache["kc"]),
                                         _ptr(cache["vc"]), _ptr(cache["gc"]), B, H, L, d, cap, _dt(k), _ptr(workspace),
                                         workspace.numel(), ctypes.c_void_p(st))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_prefill_cache")
    return workspace


def decode_workspace(B, H, cap, d, device="cuda"):
    n = int(load().path_attn_decode_workspace_bytes(B, H, cap, d))
    if n == 0:
        raise PathAttnError(-2, "path_attn_decode_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def path_attn_decode_step(q_t, k_t, v_t, w_t, beta_t, cache, t, log_f_t=None, scale=1.0, workspace=None, out=None):
    """One decoding step at position ``t`` (= number of cached tokens): updates ``cache`` in place, returns ``(o_t, lse_t)``.
    ``q_t, k_t, v_t, w_t``: ``[B,H,d]`` bf16; ``beta_t, log_f_t``: ``[B,H]`` float32."""
    for x in (q_t, k_t, v_t, w_t, beta_t):
        if not (x.is_cuda and x.is_contiguous()):
            raise ValueError("decode inputs must be contiguous CUDA tensors")
    lib = load()
    B, H, d = q_t.shape
    cap = cache["kc"].shape[2]
    if workspace is None:
        workspace = decode_workspace(B, H, cap, d, q_t.device)
    o = torch.empty_like(q_t) if out is None else out[0]
    lse = torch.empty(B, H, dtype=torch.float32, device=q_t.device) if out is None else out[1]
    st = torch.cuda.current_stream(q_t.device).cuda_stream
    with torch.cuda.device(q_t.device):
        rc = lib.path_attn_decode_step(_ptr(q_t), _ptr(k_t), _ptr(v_t), _ptr(w_t), _ptr(beta_t), _ptr(log_f_t),
                                       _ptr(cache["kc"]), _ptr(cache["vc"]), _ptr(cache["gc"]), int(t), cap, _ptr(o),
                                       _ptr(lse), B, H, d, float(scale), _dt(q_t), _ptr(workspace), workspace.numel(),
                                       ctypes.c_void_p(st))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_decode_step")
    return o, lse


# ----------------------------------------------------------------------------------------- layer front-end

def _frontend_check(z, conv_w, beta_logit, gate_logit, H):
    B, L, C = z.shape
    if C % H:
        raise ValueError("z's channel count must be a multiple of H")
    d = C // H
    if z.dtype != torch.bfloat16:
        raise ValueError("z must be bf16")
    if conv_w.shape != (C, 3) or conv_w.dtype != torch.float32:
        raise ValueError("conv_w must be float32 [H*d, 3]")
    for x in (beta_logit, gate_logit):
        if x is not None and (x.shape != (B, L, H) or x.dtype != torch.float32):
            raise ValueError("logits must be float32 [B, L, H]")
    for x in (z, conv_w, beta_logit, gate_logit):
        if x is not None and not (x.is_cuda and x.is_contiguous()):
            raise ValueError("front-end inputs must be contiguous CUDA tensors")
    return B, L, d


def path_attn_frontend_fwd(z, conv_w, beta_logit, gate_logit=None, H=1, eps=1e-6):
    """``z`` ``[B,L,H*d]`` bf16, ``conv_w`` ``[H*d,3]``, logits ``[B,L,H]`` float32 -> ``(w [B,H,L,d] bf16, beta, log_f [B,H,L])``."""
    B, L, d = _frontend_check(z, conv_w, beta_logit, gate_logit, H)
    lib = load()
    w = torch.empty(B, H, L, d, dtype=torch.bfloat16, device=z.device)
    beta = torch.empty(B, H, L, dtype=torch.float32, device=z.device)
    log_f = torch.empty_like(beta) if gate_logit is not None else None
    st = torch.cuda.current_stream(z.device).cuda_stream
    with torch.cuda.device(z.device):
        rc = lib.path_attn_frontend_fwd(_ptr(z), _ptr(conv_w), _ptr(beta_logit), _ptr(gate_logit), _ptr(w), _ptr(beta),
                                        _ptr(log_f), B, H, L, d, float(eps), ctypes.c_void_p(st))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_frontend_fwd")
    return w, beta, log_f


def path_attn_frontend_bwd(z, conv_w, beta_logit, dw, dbeta, gate_logit=None, dlog_f=None, H=1, eps=1e-6):
    """Backward of :func:`path_attn_frontend_fwd`: returns ``(dz, dconv_w, dbeta_logit, dgate_logit or None)``."""
    B, L, d = _frontend_check(z, conv_w, beta_logit, gate_logit, H)
    if dw.shape != (B, H, L, d) or dw.dtype != torch.bfloat16 or dbeta.shape != (B, H, L) or dbeta.dtype != torch.float32:
        raise ValueError("dw must be bf16 [B,H,L,d] and dbeta float32 [B,H,L]")
    if (gate_logit is None) != (dlog_f is None):
        raise ValueError("gate_logit and dlog_f go together")
    for x in (dw, dbeta, dlog_f):
        if x is not None and not (x.is_cuda and x.is_contiguous()):
            raise ValueError("front-end gradients must be contiguous CUDA tensors")
    lib = load()
    dz = torch.empty_like(z)
    dcw = torch.empty_like(conv_w)
    dbl = torch.empty_like(beta_logit)
    dgl = torch.empty_like(gate_logit) if gate_logit is not None else None
    st = torch.cuda.current_stream(z.device).cuda_stream
    with torch.cuda.device(z.device):
        rc = lib.path_attn_frontend_bwd(_ptr(z), _ptr(conv_w), _ptr(beta_logit), _ptr(gate_logit), _ptr(dw), _ptr(dbeta),
                                        _ptr(dlog_f), _ptr(dz), _ptr(dcw), _ptr(dbl), _ptr(dgl), B, H, L, d, float(eps),
                                        ctypes.c_void_p(st))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_frontend_bwd")
    return dz, dcw, dbl, dgl


def _lowrank_check(x, w1, w2):
    for t in (x, w1, w2):
        if not (t.is_cuda and t.is_contiguous() and t.dtype == torch.bfloat16):
            raise ValueError("low-rank layer operands must be contiguous bf16 CUDA tensors")
    M, D = x.reshape(-1, x.shape[-1]).shape
    r, C = w1.shape[0], w2.shape[0]
    if w1.shape != (r, D) or w2.shape != (C, r):
        raise ValueError("w1 must be [r, D] and w2 [C, r]")
    return M, D, r, C


def path_attn_lowrank_fwd(x, w1, w2):
    """``x [..., D]``, ``w1 [r, D]``, ``w2 [C, r]`` bf16 -> ``(z [..., C], t [..., r])``: ``t = x w1^T``, ``z = t w2^T``."""
    M, D, r, C = _lowrank_check(x, w1, w2)
    lib = load()
    t = torch.empty(*x.shape[:-1], r, dtype=torch.bfloat16, device=x.device)
    z = torch.empty(*x.shape[:-1], C, dtype=torch.bfloat16, device=x.device)
    ws = torch.empty(256, dtype=torch.uint8, device=x.device)
    st = torch.cuda.current_stream(x.device).cuda_stream
    with torch.cuda.device(x.device):
        rc = lib.path_attn_lowrank_fwd(_ptr(x), _ptr(w1), _ptr(w2), _ptr(t), _ptr(z), M, D, r, C, _ptr(ws), ws.numel(),
                                       ctypes.c_void_p(st))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_lowrank_fwd")
    return z, t


def path_attn_lowrank_bwd(x, w1, w2, t, dz, workspace=None):
    """Backward of :func:`path_attn_lowrank_fwd`: ``(dx bf16, dw1 float32 [r, D], dw2 float32 [C, r])``."""
    M, D, r, C = _lowrank_check(x, w1, w2)
    lib = load()
    if workspace is None:
        workspace = torch.empty(int(lib.path_attn_lowrank_workspace_bytes(M, D, r, C)), dtype=torch.uint8, device=x.device)
    dx = torch.empty_like(x)
    dw1 = torch.empty(r, D, dtype=torch.float32, device=x.device)
    dw2 = torch.empty(C, r, dtype=torch.float32, device=x.device)
    st = torch.cuda.current_stream(x.device).cuda_stream
    with torch.cuda.device(x.device):
        rc = lib.path_attn_lowrank_bwd(_ptr(x), _ptr(w1), _ptr(w2), _ptr(t), _ptr(dz.contiguous()), _ptr(dx), _ptr(dw1), _ptr(dw2),
                                       M, D, r, C, _ptr(workspace), workspace.numel(), ctypes.c_void_p(st))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_lowrank_bwd")
    return dx, dw1, dw2


# ----------------------------------------------------------------------------------------- context-parallel path

def _u8(n, device):
    return torch.empty(n, dtype=torch.uint8, device=device)


def cp_alloc(B, H, L, d, has_gate=False, device="cuda"):
    """(state, message, workspace) buffers for a segment of L positions (paper Sec. 3.5)."""
    lib = load()
    sizes = (lib.path_attn_cp_state_bytes(B, H, L, d), lib.path_attn_cp_message_bytes(B, H, L, d),
             lib.path_attn_cp_workspace_bytes(B, H, L, d, int(has_gate)))
    if 0 in sizes:
        raise PathAttnError(-2, "path_attn_cp_*_bytes")
    return tuple(_u8(int(n), device) for n in sizes)


def path_attn_cp_prepare(q, k, v, w, beta, log_f=None, scale=1.0, state=None, message=None, workspace=None):
    """This device's segment: fills ``state`` (resident queries + running result) and ``message`` (what later segments'
    holders need from this one).  Returns ``(state, message, workspace)``."""
    _check(q, k, v, w, beta, log_f)
    lib = load()
    B, H, L, d = q.shape
    if state is None or message is None or workspace is None:
        s_, m_, w_ = cp_alloc(B, H, L, d, log_f is not None, q.device)
        state = s_ if state is None else state
        message = m_ if message is None else message
        workspace = w_ if workspace is None else workspace
    st = torch.cuda.current_stream(q.device).cuda_stream
    with torch.cuda.device(q.device):
        rc = lib.path_attn_cp_prepare(_ptr(q), _ptr(k), _ptr(v), _ptr(w), _ptr(beta), _ptr(log_f), _ptr(state), _ptr(message),
                                      B, H, L, d, float(scale), _dt(q), _ptr(workspace), workspace.numel(), ctypes.c_void_p(st))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_cp_prepare")
    return state, message, workspace


def path_attn_cp_step(state, message, B, H, Lq, Lk, d, scale=1.0, workspace=None):
    """The resident queries (``state``, Lq positions) attend an earlier segment's ``message`` (Lk positions) and move on."""
    lib = load()
    if workspace is None:
        workspace = _u8(int(lib.path_attn_cp_workspace_bytes(B, H, Lq, d, 0)), state.device)
    st = torch.cuda.current_stream(state.device).cuda_stream
    with torch.cuda.device(state.device):
        rc = lib.path_attn_cp_step(_ptr(state), _ptr(message), B, H, Lq, Lk, d, float(scale), _ptr(workspace),
                                   workspace.numel(), ctypes.c_void_p(st))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_cp_step")
    return workspace


def path_attn_cp_finish(state, B, H, L, d):
    """``(o [B,H,L,d] bf16, lse [B,H,L] float32)`` of the segment from its state."""
    lib = load()
    o = torch.empty(B, H, L, d, dtype=torch.bfloat16, device=state.device)
    lse = torch.empty(B, H, L, dtype=torch.float32, device=state.device)
    st = torch.cuda.current_stream(state.device).cuda_stream
    with torch.cuda.device(state.device):
        rc = lib.path_attn_cp_finish(_ptr(state), _ptr(o), _ptr(lse), B, H, L, d, ctypes.c_void_p(st))
    if rc != PATH_OK:
        raise PathAttnError(rc, "path_attn_cp_finish")
    return o, lse
