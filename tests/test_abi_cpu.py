"""The C-ABI library without a GPU: it loads, exports what include/path_attn.h declares, plans workspaces and
rejects bad arguments on the host before touching the device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2505_16381_b200 import binding, build
    build.build()
    return binding.load()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "path_attn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(path_attn_\w+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    from paper_2505_16381_b200 import binding
    names = declared_symbols()
    assert len(names) >= 10
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_workspace_planning(lib):
    from paper_2505_16381_b200 import binding as b
    assert b.workspace_bytes(1, 1, 128, 64) > 0
    assert b.workspace_bytes(4, 16, 4096, 128, for_backward=True) > b.workspace_bytes(4, 16, 4096, 128)
    assert b.workspace_bytes(4, 16, 4096, 128, has_gate=True) > b.workspace_bytes(4, 16, 4096, 128)
    assert b.workspace_bytes(1, 1, 129, 64) > b.workspace_bytes(1, 1, 128, 64)   # ragged tail pads
    for bad in [(0, 1, 128, 64), (1, 1, 0, 64), (1, 1, 128, 96), (1, 1, 128, 256), (1, -1, 128, 64)]:
        assert b.workspace_bytes(*bad) == 0
    assert b.workspace_bytes(1, 1, 128, 64, dtype=7) == 0
    # the headline workloads fit a B200 (180 GB) with room to spare
    assert b.workspace_bytes(2, 16, 8192, 128, has_gate=True, for_backward=True) < 40e9
    assert b.workspace_bytes(1, 32, 32768, 128) < 40e9


def _fwd(lib, q=0x1000, k=0x1000, v=0x1000, w=0x1000, beta=0x1000, log_f=None, o=0x1000, lse=0x1000,
         B=1, H=1, L=128, d=64, dt=0, ws=0x1000, ws_bytes=1 << 40):
    return lib.path_attn_fwd(q, k, v, w, beta, log_f, o, lse, B, H, L, d, 1.0, dt, ws, ws_bytes, None)


def test_forward_rejects_bad_arguments_on_the_host(lib):
    assert _fwd(lib, q=None) == -1
    assert _fwd(lib, ws=None) == -1
    assert _fwd(lib, d=96) == -2
    assert _fwd(lib, L=0) == -2
    assert _fwd(lib, dt=5) == -3
    assert _fwd(lib, k=0x1008) == -4
    assert _fwd(lib, ws=0x1010) == -4
    assert _fwd(lib, ws_bytes=1024) == -5


def test_backward_rejects_bad_arguments_on_the_host(lib):
    P = 0x2000
    def bwd(**kw):
        a = dict(q=P, k=P, v=P, w=P, beta=P, log_f=None, o=P, lse=P, d_o=P, dq=P, dk=P, dv=P, dw=P, dbeta=P,
                 dlog_f=None, B=1, H=1, L=128, d=64, dt=0, ws=P, n=1 << 40)
        a.update(kw)
        return lib.path_attn_bwd(a["q"], a["k"], a["v"], a["w"], a["beta"], a["log_f"], a["o"], a["lse"], a["d_o"],
                                 a["dq"], a["dk"], a["dv"], a["dw"], a["dbeta"], a["dlog_f"], a["B"], a["H"], a["L"],
                                 a["d"], 1.0, a["dt"], a["ws"], a["n"], None)
    assert bwd(d_o=None) == -1
    assert bwd(log_f=P) == -1            # gate without a place for its gradient
    assert bwd(dlog_f=P) == -1
    assert bwd(d=32) == -2
    assert bwd(dt=1) == -3               # backward is bf16 only
    assert bwd(dw=P + 4) == -4
    assert bwd(n=4096) == -5


def test_frontend_rejects_bad_arguments_on_the_host(lib):
    P = 0x2000
    def fwd(**kw):
        a = dict(z=P, cw=P, bl=P, gl=None, w=P, beta=P, log_f=None, B=1, H=2, L=16, d=64, eps=1e-6)
        a.update(kw)
        return lib.path_attn_frontend_fwd(a["z"], a["cw"], a["bl"], a["gl"], a["w"], a["beta"], a["log_f"], a["B"], a["H"],
                                          a["L"], a["d"], a["eps"], None)
    def bwd(**kw):
        a = dict(z=P, cw=P, bl=P, gl=None, dw=P, dbeta=P, dlog_f=None, dz=P, dcw=P, dbl=P, dgl=None, B=1, H=2, L=16, d=128,
                 eps=1e-6)
        a.update(kw)
        return lib.path_attn_frontend_bwd(a["z"], a["cw"], a["bl"], a["gl"], a["dw"], a["dbeta"], a["dlog_f"], a["dz"],
                                          a["dcw"], a["dbl"], a["dgl"], a["B"], a["H"], a["L"], a["d"], a["eps"], None)
    assert fwd(z=None) == -1 and fwd(beta=None) == -1
    assert fwd(gl=P) == -1 and fwd(log_f=P) == -1          # gate logits and log_f go together
    assert fwd(d=96) == -2 and fwd(L=0) == -2 and fwd(H=0) == -2 and fwd(eps=-1.0) == -2
    assert fwd(z=P + 8) == -4 and fwd(w=P + 2) == -4
    assert bwd(dw=None) == -1 and bwd(dcw=None) == -1
    assert bwd(gl=P) == -1 and bwd(gl=P, dlog_f=P) == -1 and bwd(dgl=P) == -1
    assert bwd(d=32) == -2 and bwd(B=0) == -2
    assert bwd(dz=P + 8) == -4


def test_skipped_chunk_pairs_rejects_null_arguments(lib):
    import ctypes
    a, b = ctypes.c_ulonglong(0), ctypes.c_ulonglong(0)
    assert lib.path_attn_skipped_chunk_pairs(None, None, ctypes.byref(a), ctypes.byref(b)) == -1
    assert lib.path_attn_skipped_chunk_pairs(0x2000, None, None, ctypes.byref(b)) == -1


def test_strerror_and_counters(lib):
    seen = set()
    for code in range(0, -9, -1):
        msg = lib.path_attn_strerror(code).decode()
        assert msg and msg != "unknown status"
        seen.add(msg)
    assert len(seen) == 9
    assert lib.path_attn_strerror(-99).decode() == "unknown status"
    assert lib.path_attn_last_launch_count() == 0
    assert lib.path_attn_device_status(None, None, None) == -1


def test_product_path_has_no_oracle_or_cpu_fallback():
    import torch
    from paper_2505_16381_b200 import binding
    q = torch.zeros(1, 1, 128, 64, dtype=torch.bfloat16)
    with pytest.raises(RuntimeError, match="CUDA"):
        binding.path_attn_fwd(q, q, q, q, torch.zeros(1, 1, 128))
    for fn in ("binding.py", "build.py", "synth.py", "__init__.py"):
        src = open(os.path.join(ROOT, "paper_2505_16381_b200", fn)).read()
        assert "oracle" not in src.replace("the CPU oracle's tests", "").replace("CPU oracle", "") or fn == "synth.py"
