"""The ring schedule of context-parallel PaTH (paper Sec. 3.5) on CPU: gloo ranks exchange float64 messages built by the
numpy restatement in ring_cpu_ops.py, and the gathered result must equal the oracle's forward over the whole sequence.
This pins both the schedule (who sends what to whom, which messages a rank may read, in which order) and the
segment algebra itself (pulled-back queries, advanced keys, segment products, gate bookkeeping) independently of CUDA."""
import os
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _problem(L, d, gate, seed):
    rng = np.random.default_rng(seed)
    q, k, v = (rng.standard_normal((L, d)) for _ in range(3))
    w = rng.standard_normal((L, d))
    w /= np.linalg.norm(w, axis=1, keepdims=True)
    beta = 2.0 / (1.0 + np.exp(-rng.standard_normal(L)))
    g = -np.abs(rng.standard_normal(L)) * 0.3 if gate else None
    return q, k, v, w, beta, g


@pytest.mark.parametrize("cuts,gate", [([7, 20], False), ([5, 6, 19, 30], True), ([1, 12, 13, 24], True)])
def test_virtual_ring_with_numpy_ops_equals_the_definition(oracle, cuts, gate):
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from ring_cpu_ops import CpuOps
    from paper_2505_16381_b200 import ring
    L, d, scale = cuts[-1], 6, 0.7
    q, k, v, w, beta, g = _problem(L, d, gate, 5)
    segs, lo = [], 0
    for hi in cuts:
        segs.append({"q": q[lo:hi], "k": k[lo:hi], "v": v[lo:hi], "w": w[lo:hi], "beta": beta[lo:hi],
                     "log_f": None if g is None else g[lo:hi]})
        lo = hi
    outs = ring.virtual_ring_forward(CpuOps(d, scale), segs)
    o = np.concatenate([x[0] for x in outs]); lse = np.concatenate([x[1] for x in outs])
    o_ref, lse_ref = oracle.forward(q, k, v, w, beta, g, scale=scale)
    assert np.abs(o - o_ref).max() < 1e-10 and np.abs(lse - lse_ref).max() < 1e-10


WORKER = """
import os, sys
sys.path.insert(0, {root!r}); sys.path.insert(0, os.path.join({root!r}, "tests"))
import numpy as np, torch, torch.distributed as dist
from oracle import path_oracle
from paper_2505_16381_b200 import ring
from ring_cpu_ops import CpuOps
from test_ring_schedule_cpu import _problem
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
cuts = {cuts!r}
L, d, scale = cuts[-1], 6, 0.7
q, k, v, w, beta, g = _problem(L, d, True, 11)
lo, hi = ([0] + cuts)[rank], cuts[rank]
seg = dict(q=q[lo:hi], k=k[lo:hi], v=v[lo:hi], w=w[lo:hi], beta=beta[lo:hi], log_f=g[lo:hi])
o, lse = ring.ring_forward(CpuOps(d, scale), seg)
o_ref, lse_ref = path_oracle.forward(q, k, v, w, beta, g, scale=scale)
err = max(np.abs(o - o_ref[lo:hi]).max(), np.abs(lse - lse_ref[lo:hi]).max())
assert err < 1e-10, (rank, err)
open(os.path.join({out!r}, "rank%d.txt" % rank), "w").write("ok")
dist.destroy_process_group()
"""


@pytest.mark.parametrize("world,cuts,port", [(2, [9, 21], 29531), (4, [4, 9, 10, 23], 29532)])
def test_ring_schedule_on_gloo_ranks(tmp_path, world, cuts, port):
    from oracle import path_oracle
    path_oracle.build()
    script = tmp_path / "worker.py"
    script.write_text(WORKER.format(root=ROOT, out=str(tmp_path), cuts=cuts))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="1")
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={world}",
                          "--master-addr", "127.0.0.1", "--master-port", str(port), str(script)],
                         capture_output=True, text=True, timeout=600, env=env)
    assert out.returncode == 0, out.stderr[-3000:]
    assert all((tmp_path / f"rank{r}.txt").read_text() == "ok" for r in range(world))
