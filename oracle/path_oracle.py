"""ctypes front-end of the float64 CPU oracle (``path_oracle.c``).

TEST INFRASTRUCTURE ONLY: the CUDA library never imports this module, and this
module never imports the CUDA package.  It compiles ``path_oracle.c`` with gcc
(OpenMP) into ``oracle/_build/`` on first use.

All functions take and return float64 numpy arrays shaped ``[..., L, d]``
(q, k, v, w, o and gradients) and ``[..., L]`` (beta, log-gate, lse); leading
dimensions are flattened into independent slices.  Inputs of lower precision
are upcast exactly, so feeding bf16-rounded values gives the exact-arithmetic
answer for those rounded inputs.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "path_oracle.c"
_LIB = _HERE / "_build" / "libpath_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle's C source; returns the shared-library path."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        _LIB.parent.mkdir(exist_ok=True)
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", str(tmp), str(_SRC), "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(str(build()))
        P = ctypes.c_void_p
        I = ctypes.c_int
        D = ctypes.c_double
        lib.path_oracle_num_threads.restype = I
        lib.path_oracle_fwd_rows.argtypes = [P, P, P, P, P, P, I, I, I, D, P, I, P, P]
        lib.path_oracle_fwd.argtypes = [P, P, P, P, P, P, I, I, I, D, P, P]
        lib.path_oracle_logits.argtypes = [P, P, P, P, P, I, I, D, P]
        lib.path_oracle_uchain.argtypes = [P, P, P, I, I, I, P]
        lib.path_oracle_key_cache.argtypes = [P, P, P, I, I, I, I, P]
        lib.path_oracle_bwd.argtypes = [P, P, P, P, P, P, P, I, I, I, D, P, P, P, P, P, P]
        lib.path_oracle_bwd_lse.restype = ctypes.c_int
        lib.path_oracle_bwd_lse.argtypes = [P, P, P, P, P, P, P, P, I, I, I, D, P, P, P, P, P, P]
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the oracle's OpenMP loops will use."""
    return int(_load().path_oracle_num_threads())


def _f64(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _flatten(q, k, v, w, beta, log_f):
    q, k, v, w, beta = map(_f64, (q, k, v, w, beta))
    L, d = q.shape[-2:]
    S = int(np.prod(q.shape[:-2], dtype=np.int64)) if q.ndim > 2 else 1
    for t in (k, v, w):
        assert t.shape == q.shape
    assert beta.shape == q.shape[:-1]
    g = None if log_f is None else _f64(log_f)
    if g is not None:
        assert g.shape == beta.shape
    return q, k, v, w, beta, g, S, L, d


def forward(q, k, v, w, beta, log_f=None, scale: float = 1.0, rows=None):
    """O and LSE (natural log, scale and gate included).

    ``rows``: optional 1-D list of query positions; then only those rows are
    computed (same rows for every slice) and the outputs are ``[..., len(rows), d]``
    and ``[..., len(rows)]``.
    """
    q, k, v, w, beta, g, S, L, d = _flatten(q, k, v, w, beta, log_f)
    lead = q.shape[:-2]
    if rows is None:
        n, rp = L, None
    else:
        rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int32))
        assert rows.ndim == 1 and rows.min() >= 0 and rows.max() < L
        n, rp = len(rows), _ptr(rows)
    o = np.empty(lead + (n, d))
    lse = np.empty(lead + (n,))
    rc = _load().path_oracle_fwd_rows(_ptr(q), _ptr(k), _ptr(v), _ptr(w), _ptr(beta), _ptr(g),
                                      S, L, d, float(scale), rp, n, _ptr(o), _ptr(lse))
    if rc != 0:
        raise MemoryError("path_oracle_fwd_rows failed")
    return o, lse


def logits(q, k, w, beta, log_f=None, scale: float = 1.0):
    """[L, L] logits of ONE slice (q, k, w are [L, d]); entries with j > i are 0."""
    q, k, w, beta = map(_f64, (q, k, w, beta))
    assert q.ndim == 2
    L, d = q.shape
    g = None if log_f is None else _f64(log_f)
    out = np.empty((L, L))
    rc = _load().path_oracle_logits(_ptr(q), _ptr(k), _ptr(w), _ptr(beta), _ptr(g), L, d, float(scale), _ptr(out))
    if rc != 0:
        raise MemoryError("path_oracle_logits failed")
    return out


def uchain(q, w, beta, i: int):
    """Carried vectors of query row ``i`` of ONE slice: ``U[j] = H_{j+1} ... H_i q_i``, j = 0..i."""
    q, w, beta = map(_f64, (q, w, beta))
    L, d = q.shape
    U = np.empty((i + 1, d))
    rc = _load().path_oracle_uchain(_ptr(q), _ptr(w), _ptr(beta), L, d, int(i), _ptr(U))
    if rc != 0:
        raise MemoryError("path_oracle_uchain failed")
    return U


def key_cache(k, w, beta, n=None):
    """Decoding key cache after the first ``n`` tokens (default: all): ``kc[..., j, :] = H_{n-1} ... H_{j+1} k_j``,
    built by the recurrence itself (every earlier key gets ``k <- H_t k`` when token t arrives).  ``[..., n, d]``."""
    k, w, beta = map(_f64, (k, w, beta))
    L, d = k.shape[-2:]
    S = int(np.prod(k.shape[:-2], dtype=np.int64)) if k.ndim > 2 else 1
    assert w.shape == k.shape and beta.shape == k.shape[:-1]
    n = L if n is None else int(n)
    assert 0 <= n <= L
    kc = np.empty(k.shape[:-2] + (n, d))
    rc = _load().path_oracle_key_cache(_ptr(k), _ptr(w), _ptr(beta), S, L, d, n, _ptr(kc))
    if rc != 0:
        raise MemoryError("path_oracle_key_cache failed")
    return kc


def backward(q, k, v, w, beta, d_o, log_f=None, scale: float = 1.0, d_lse=None):
    """Gradients of sum(O * d_o) (+ sum(lse * d_lse) when ``d_lse`` is given): dict with dq, dk, dv, dw, dbeta and
    (if gated) dlog_f."""
    q, k, v, w, beta, g, S, L, d = _flatten(q, k, v, w, beta, log_f)
    d_o = _f64(d_o)
    assert d_o.shape == q.shape
    d_lse = None if d_lse is None else _f64(d_lse)
    assert d_lse is None or d_lse.shape == beta.shape
    dq, dk, dv, dw = (np.empty_like(q) for _ in range(4))
    dbeta = np.empty_like(beta)
    dg = None if g is None else np.empty_like(beta)
    rc = _load().path_oracle_bwd_lse(_ptr(q), _ptr(k), _ptr(v), _ptr(w), _ptr(beta), _ptr(g), _ptr(d_o), _ptr(d_lse),
                                     S, L, d, float(scale), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dw),
                                     _ptr(dbeta), _ptr(dg))
    if rc != 0:
        raise MemoryError("path_oracle_bwd failed")
    out = {"dq": dq, "dk": dk, "dv": dv, "dw": dw, "dbeta": dbeta}
    if dg is not None:
        out["dlog_f"] = dg
    return out
