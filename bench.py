#!/usr/bin/env python
"""Benchmark of the PaTH attention hot path (forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload C3]

One step = one pass of the whole hot path over one batch of seeded synthetic input:
path_attn_fwd followed by path_attn_bwd on the headline workload (B=4, H=16, L=4096,
d=128, bf16).  Rank 0 prints ONE JSON line.  With N > 1 (launched by torchrun) every
rank runs its own batch of the same shape (the (batch, head) slices are independent:
no data-path collective), times are reduced with max over ranks, and `value` is the
aggregate of all ranks ("weak" scaling).

FLOP models (both reported; neither counts masked-out work):
  M1  attention-equivalent: forward 2*B*H*L*(L+1)*d, backward 2.5x forward.  `value` uses M1.
  M2  M1 + the Householder work the method executes at chunk size 128 (chunk preparation,
      run products, version chains, diagonal corrections and their chain rules), each
      contraction counted once (no split-precision or recomputation multipliers).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2505_16381_b200 import synth  # noqa: E402

CHUNK = 128
METRIC = "PaTH attn fwd+bwd TFLOP/s (attention-equivalent FLOPs) at L=4096, d=128"


def metric_name(cfg):
    """The headline metric's name; the other workloads (--workload) carry their own length and head size in it."""
    return METRIC.replace("L=4096, d=128", f"L={cfg['L']}, d={cfg['d']}")
UNIT = "TFLOP/s"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the kernel named by `roofline.kernel`,
# from the ncu capture summarised under profiles/ (None until one exists for that kernel).
# DRAM bytes per launch PER (batch, head) SLICE at the C3 shape (L=4096, d=128), from the ncu captures at batch 1
# (16 slices) summarised under profiles/; slices are independent, so a launch over S slices moves S times this.
NCU_TRAFFIC_BYTES_PER_SLICE = {
    "chunk_prep": 12.71e6,         # backward instance (the step's forward runs on the shared workspace)
    "levels_fwd": 2.13e6 + 6.35e6,   # dyadic_fused (one launch for three levels) + version_fwd
    "fa_fwd": 11.18e6,
    "fa_bwd_dkv": 15.24e6,
    "fa_bwd_dq": 8.62e6,
    "bwd_levels": 12.64e6,         # level_bwd (4 launches)
    "bwd_chunk_chain": 18.29e6,
}

# DRAM bytes per launch of frontend_bwd_kernel PER BATCH ROW at H=32, L=4096, d=64 with the gate, from the ncu capture at
# batch 16 summarised under profiles/ (573.76 MB read + 255.33 MB written); batch rows are independent.
NCU_FRONTEND_BWD_TRAFFIC_PER_BATCH_ROW = (573.76e6 + 255.33e6) / 16


# ----------------------------------------------------------------------------------------- FLOP models
def flops_m1(B, H, L, d):
    fwd = 2.0 * B * H * L * (L + 1) * d
    return fwd, 2.5 * fwd


def _version_steps(N):
    """(query-side, key-side) number of (chunk, level) version-chain products of one slice."""
    nlev = (N - 1).bit_length() if N > 1 else 0
    nq = nk = 0
    for l2 in range(1, nlev):
        for c in range(N):
            low = c & ((1 << l2) - 1)
            if (c >> l2) & 1 and low:
                nq += 1
            lowz = ~c & ((1 << l2) - 1)
            if not (c >> l2) & 1 and lowz and (((c >> l2) + 1) << l2) <= N - 1:
                nk += 1
    return nq, nk, nlev


def flops_m2(B, H, L, d):
    S = B * H
    N = -(-L // CHUNK)
    Bc = CHUNK
    f1, b1 = flops_m1(B, H, L, d)
    prep = S * N * (12 * Bc * Bc * d + 2 * Bc * d * d + 2.67 * Bc ** 3)
    nq, nk, nlev = _version_steps(N)
    dy = sum(S * (N >> l) * 2 * d ** 3 for l in range(1, max(nlev - 1, 0)))
    ver = S * (nq + nk) * 2 * Bc * d * d
    diag = S * N * 2 * Bc ** 3
    fwd = f1 + prep + dy + ver + diag
    chain = S * N * (14 * 2 * Bc * Bc * d + 6 * 2 * Bc ** 3 + 2 * 2 * Bc * d * d)
    bwd = b1 + (prep + dy + ver) + 2 * diag + 2 * ver + 2 * dy + chain
    return fwd, bwd


def mma_flops(n, ksteps):
    """One tcgen05 product group: `ksteps` instructions of shape 128 x n x 16."""
    return 2.0 * 128 * n * 16 * ksteps


def chunk_kernel_flops(d):
    """Executed tensor-core FLOPs per 128-token chunk of the two per-chunk kernels (every issued product, the low parts
    of the bf16 pairs included), read off their product lists."""
    kd = d // 16
    prep = (3 * mma_flops(128, kd) + 2 * mma_flops(d, 8) + 3 * mma_flops(128, 8) + 3 * mma_flops(d, 8) +
            2 * mma_flops(d, 8) + 2 * mma_flops(d, 8))
    chain = (mma_flops(128, kd) + mma_flops(128, 8) + mma_flops(d, 8) + mma_flops(d, kd) +                       # phase 0
             mma_flops(128, kd) + mma_flops(128, 8) + mma_flops(d, 8) + mma_flops(d, kd) + mma_flops(128, kd) +  # phase 1
             mma_flops(128, 8) + mma_flops(128, kd) +                                                            # phase 2
             2 * mma_flops(128, 8) + 2 * mma_flops(d, 8) +                                                       # phase 3
             6 * mma_flops(128, 8) +                                                                             # phase 4
             10 * mma_flops(d, 8))                                                                               # phase 5
    return prep, chain


def level_bytes(S, N, d):
    """Algorithmic bytes of the level kernels (run products and version chains), forward and backward: every tile a
    launch has to read or write once, counted from the step lists (t = 128 x d bf16 tile, m = d x d bf16 matrix)."""
    t, m = CHUNK * d * 2, d * d * 2
    nq, nk, nlev = _version_steps(N)
    chains_q = sum(1 for c in range(N) if bin(c).count("1") >= 2)
    chains_k = nk and sum(1 for c in range(N) if any(
        not (c >> l2) & 1 and (~c & ((1 << l2) - 1)) and (((c >> l2) + 1) << l2) <= N - 1 for l2 in range(1, nlev)))
    runs = lambda l: N >> l
    # run products: a launch builds up to three levels; it reads the hi + lo pairs of its input level once and writes
    # every product's pair (the levels in between stay in shared memory)
    dy = 0
    l = 0
    while l + 1 <= nlev - 2:
        fuse = min(3, nlev - 2 - l)
        dy += 2 * runs(l + 1) * 2 * m + sum(runs(l + j) for j in range(1, fuse + 1)) * 2 * m
        l += fuse
    fwd = S * (dy + (nq + nk) * (2 * m + t) + (chains_q + chains_k) * t)
    top = max(nlev - 2, 0)
    run_cnt = sum(runs(l) for l in range(0, top + 1))
    parents = sum(runs(l) for l in range(0, top))
    bwd = S * ((nq + nk) * 4 * t + run_cnt * 2 * m + parents * 2 * m)
    return fwd, bwd


# ----------------------------------------------------------------------------------------- helpers
def shard_info():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def max_over_ranks(x: float, world: int, device=None) -> float:
    """Maximum of a per-rank scalar over all ranks (identity for one rank)."""
    if world == 1:
        return float(x)
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"burst": p["bf16_tflops"], "sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "hbm": p["hbm_gbs"], "source": "measured"}
    return {"burst": 1590.0, "sustained": 1400.0, "hbm": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons of one GPU with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) >= 6:
                self.samples.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        sm = sorted(int(s[0]) for s in self.samples if s[0].isdigit())
        mx = [int(s[1]) for s in self.samples if s[1].isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(s[2 + i].lower().startswith("active") for s in self.samples)]
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        ids = [x for x in vis.split(",") if x.strip() != ""]
        if local < len(ids) and ids[local].strip().isdigit():
            return int(ids[local])
    return local


# ----------------------------------------------------------------------------------------- reference arm
def oracle_sample(cfg, inp, n_slices=1):
    """Forward + backward of the float64 oracle on the first `n_slices` (batch, head) slices.  Returns seconds."""
    from oracle import path_oracle as po
    f = synth.to_f64
    sl = lambda t: None if t is None else f(t.reshape(-1, *t.shape[2:])[:n_slices])
    q, k, v, w, beta, d_o, g = (sl(inp[n]) for n in ("q", "k", "v", "w", "beta", "d_o", "log_f"))
    t0 = time.perf_counter()
    po.forward(q, k, v, w, beta, g, scale=inp["scale"])
    po.backward(q, k, v, w, beta, d_o, g, scale=inp["scale"])
    return time.perf_counter() - t0, po.num_threads()


def run_reference(args, cfg):
    rank, world, _ = shard_info()
    if rank != 0:
        return
    inp = synth.make_config(args.workload)
    f1, b1 = flops_m1(1, 1, cfg["L"], cfg["d"])  # one slice per step
    for _ in range(args.warmup):
        oracle_sample(cfg, inp)
    secs = []
    cores = 1
    for _ in range(args.steps):
        s, cores = oracle_sample(cfg, inp)
        secs.append(s)
    ms = 1e3 * sum(secs) / len(secs)
    val = (f1 + b1) / (ms * 1e-3) / 1e12
    sample = f"1 of {cfg['B'] * cfg['H']} (batch, head) slices of {args.workload} per step, forward + backward, float64"
    line = {
        "impl": "reference", "metric": metric_name(cfg), "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.workload}: B={cfg['B']} H={cfg['H']} L={cfg['L']} d={cfg['d']} fwd+bwd",
                   "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------- our arm
def run_ours(args, cfg):
    from paper_2505_16381_b200 import binding
    rank, world, local = shard_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the hot path has no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    binding.load()

    B, H, L, d = cfg["B"], cfg["H"], cfg["L"], cfg["d"]
    inp = synth.make_inputs(B, H, L, d, dtype=cfg["dtype"], qk_scaled=cfg["qk_scaled"], gate=cfg["gate"],
                            seed=synth.BASE_SEED + cfg["index"] + 1000 * rank)
    names = ["q", "k", "v", "w", "beta", "d_o"] + (["log_f"] if cfg["gate"] else [])
    host = {n: inp[n].pin_memory() for n in names}
    devt = {n: host[n].to(dev, non_blocking=True) for n in names}
    devt.setdefault("log_f", None)
    scale = inp["scale"]
    ws = binding.alloc_workspace(devt["q"], cfg["gate"], True)
    o = torch.empty_like(devt["q"])
    lse = torch.empty(B, H, L, dtype=torch.float32, device=dev)
    gout = {n: torch.empty_like(devt["q"]) for n in ("dq", "dk", "dv", "dw")}
    gout["dbeta"] = torch.empty_like(devt["beta"])
    if cfg["gate"]:
        gout["dlog_f"] = torch.empty_like(devt["beta"])
    launches = [0]

    def step(t):
        binding.path_attn_fwd(t["q"], t["k"], t["v"], t["w"], t["beta"], t["log_f"], scale=scale, workspace=ws,
                              out=(o, lse))
        n = binding.last_launch_count()
        binding.path_attn_bwd(t["q"], t["k"], t["v"], t["w"], t["beta"], o, lse, t["d_o"], t["log_f"], scale=scale,
                              workspace=ws, out=gout, reuse=True)
        launches[0] = n + binding.last_launch_count()

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing, with per-stage events
    for _ in range(args.warmup):
        step(devt)
    binding.device_status(ws)
    binding.profile_enable(True)
    sampler = ClockSampler(physical_gpu_index(local))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed_pass():
        """EXACTLY args.steps steps between two events, no host synchronisation inside; ms per step and the stage times
        of the pass's last step (the stage events are re-recorded by every step)."""
        barrier()
        e0.record()
        for _ in range(args.steps):
            step(devt)
        e1.record()
        barrier()
        return e0.elapsed_time(e1) / args.steps, dict(binding.profile_read())

    # A pass of K steps lasts only tens of milliseconds: the same pass is repeated back to back until the GPU has been
    # under this load for more than a second (so that the clock sampler sees the clocks the number was measured at),
    # and the MEDIAN pass is reported.
    barrier()
    if rank == 0:
        sampler.start()
    passes = [timed_pass()]
    n_pass = args.passes if args.passes > 0 else int(min(40, max(3, -(-1200.0 // (passes[0][0] * args.steps)))))
    n_pass += 1 - n_pass % 2
    while len(passes) < n_pass:
        passes.append(timed_pass())
    clocks = sampler.stop() if rank == 0 else None
    passes.sort(key=lambda x: x[0])
    ms, stage_ms = passes[len(passes) // 2]
    ms_best = passes[0][0]
    binding.device_status(ws)
    ms = max_over_ranks(ms, world, dev)

    # ---- the metric's other half and the price of not holding the workspace: forward alone on a forward-sized
    # workspace, and a step whose backward recomputes the chunk preparation (nothing kept between the two calls)
    ws_fwd = binding.alloc_workspace(devt["q"], cfg["gate"], False)

    def fwd_only(t):
        binding.path_attn_fwd(t["q"], t["k"], t["v"], t["w"], t["beta"], t["log_f"], scale=scale, workspace=ws_fwd, out=(o, lse))

    def step_no_reuse(t):
        fwd_only(t)
        binding.path_attn_bwd(t["q"], t["k"], t["v"], t["w"], t["beta"], o, lse, t["d_o"], t["log_f"], scale=scale,
                              workspace=ws, out=gout)

    def time_fn(fn):
        for _ in range(3):
            fn(devt)
        res = []
        for _ in range(5):
            barrier()
            e0.record()
            for _ in range(args.steps):
                fn(devt)
            e1.record()
            barrier()
            res.append(e0.elapsed_time(e1) / args.steps)
        return max_over_ranks(sorted(res)[len(res) // 2], world, dev)

    fwd_ms = no_reuse_ms = float("nan")
    fwd_stage_ms = {}
    if not args.only_step:
        fwd_ms = time_fn(fwd_only)
        fwd_stage_ms = {k_: v_ for k_, v_ in binding.profile_read().items() if k_ in ("chunk_prep", "levels_fwd", "fa_fwd")}
        no_reuse_ms = time_fn(step_no_reuse)
    binding.profile_enable(False)
    binding.device_status(ws_fwd)
    del ws_fwd

    # ---- end to end: host buffers in, host buffers out, every step
    hout = {n: torch.empty(t.shape, dtype=t.dtype).pin_memory() for n, t in gout.items()}
    h2d = sum(host[n].numel() * host[n].element_size() for n in names)
    d2h = sum(t.numel() * t.element_size() for t in hout.values())

    # Three streams (copy-in, compute, copy-out) and two sets of device buffers: every step still copies its inputs
    # from pinned host memory and its results back inside the timed region, but the copies of neighbouring steps
    # overlap the kernels, as an input pipeline would.
    cur = torch.cuda.current_stream(dev)
    s_in, s_cmp, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    din = [{n: torch.empty_like(devt[n]) for n in names} for _ in range(2)]
    for t in din:
        t.setdefault("log_f", None)
    gouts = [gout, {n: torch.empty_like(v_) for n, v_ in gout.items()}]
    ev = lambda: torch.cuda.Event()
    in_ready, in_free, out_ready, out_free = ([ev(), ev()] for _ in range(4))

    def e2e_run(nsteps):
        for st in (s_in, s_cmp, s_out):
            st.wait_stream(cur)
        for i in range(nsteps):
            b = i & 1
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(in_free[b])
                for n in names:
                    din[b][n].copy_(host[n], non_blocking=True)
                in_ready[b].record(s_in)
            with torch.cuda.stream(s_cmp):
                s_cmp.wait_event(in_ready[b])
                if i >= 2:
                    s_cmp.wait_event(out_free[b])
                t = din[b]
                binding.path_attn_fwd(t["q"], t["k"], t["v"], t["w"], t["beta"], t["log_f"], scale=scale, workspace=ws,
                                      out=(o, lse))
                binding.path_attn_bwd(t["q"], t["k"], t["v"], t["w"], t["beta"], o, lse, t["d_o"], t["log_f"],
                                      scale=scale, workspace=ws, out=gouts[b], reuse=True)
                in_free[b].record(s_cmp)
                out_ready[b].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(out_ready[b])
                for n in hout:
                    hout[n].copy_(gouts[b][n], non_blocking=True)
                out_free[b].record(s_out)
        for st in (s_in, s_cmp, s_out):
            cur.wait_stream(st)

    ms_e2e = float("nan")
    if not args.only_step:
        e2e_run(min(args.warmup, 3))
        barrier()
        e0.record()
        e2e_run(args.steps)
        e1.record()
        barrier()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1) / args.steps, world, dev)

    # ---- report
    f1, b1 = flops_m1(B, H, L, d)
    f2, b2 = flops_m2(B, H, L, d)
    peaks = load_peaks()
    tf = lambda fl, t_ms: fl / (t_ms * 1e-3) / 1e12
    value = world * tf(f1 + b1, ms)
    # Work models of the stages.  Attention sweeps: executed FLOPs (tensor-bound).  Per-chunk kernels: BOTH their
    # algorithmic bytes and their executed tensor-core FLOPs (they turn out to be bound by the latter).  Level
    # kernels: algorithmic bytes.
    S, N = B * H, -(-L // CHUNK)
    nch = S * N
    diag = nch * 2 * CHUNK ** 3
    prep_fl, chain_fl = chunk_kernel_flops(d)
    stage_flops = {"fa_fwd": f1 + diag, "fa_bwd_dkv": 2.0 * f1 + diag, "fa_bwd_dq": 1.5 * f1,
                   "chunk_prep": nch * prep_fl, "bwd_chunk_prep": nch * prep_fl, "bwd_chunk_chain": nch * chain_fl}
    if cfg["gate"]:   # the sweeps execute the kept chunk pairs only: their rooflines count those
        kept_, total_ = binding.skipped_chunk_pairs(ws)
        pair_fl = 4.0 * CHUNK * CHUNK * d          # one S product + one P V product of a full 128 x 128 pair
        stage_flops.update({"fa_fwd": kept_ * pair_fl, "fa_bwd_dkv": 2.0 * kept_ * pair_fl,
                            "fa_bwd_dq": 1.5 * max(kept_ - nch, 0) * pair_fl})
    t_d, t_b = CHUNK * d * 2, CHUNK * CHUNK * 2                 # bytes of a [128 x d] / [128 x 128] bf16 tile
    prep_bytes = nch * (3 * t_d + 2 * t_d + 2 * t_b + 2 * d * d * 2)
    lev_f, lev_b = level_bytes(S, N, d)
    # (the step's forward runs on the backward-sized workspace: its chunk preparation also stores T~ and (I+N)^-1 as
    # hi + lo, Xk [128 x 128] and U [128 x d]; the chain rule reads w, q, k, U, seven [128 x 128] tiles, (s dSd)^T, bf16
    # dQl / dKr / dP and writes dq, dk, dw)
    stage_bytes = {"chunk_prep": prep_bytes + nch * (5 * t_b + t_d), "bwd_chunk_prep": prep_bytes + nch * (5 * t_b + t_d),
                   "bwd_chunk_chain": nch * (4 * t_d + 7 * t_b + t_b + 2 * t_d + d * d * 2 + 3 * t_d),
                   "levels_fwd": lev_f, "bwd_levels": lev_b, "bwd_levels_fwd": lev_f}
    if cfg["gate"]:   # version chains are built only up to the levels the kept pairs use: no closed-form byte count
        for k_ in ("levels_fwd", "bwd_levels", "bwd_levels_fwd"):
            stage_bytes.pop(k_)

    def ncu_traffic(kernel):
        per_slice = NCU_TRAFFIC_BYTES_PER_SLICE.get(kernel)
        return per_slice * B * H if (per_slice is not None and (L, d) == (4096, 128)) else None

    # every stage against the roofline that binds it: the larger of its two fractions (a kernel cannot be further from
    # its bound than from the nearer of the two ceilings); fractions are of the MEASURED peaks, tensor = burst figure
    stage_roof = {}
    for k_, t_ms in stage_ms.items():
        fr_t = tf(stage_flops[k_], t_ms) / peaks["burst"] if k_ in stage_flops else None
        fr_h = stage_bytes[k_] / (t_ms * 1e-3) / 1e9 / peaks["hbm"] if k_ in stage_bytes else None
        if fr_t is None and fr_h is None:
            continue
        bound = "tensor" if (fr_h is None or (fr_t is not None and fr_t >= fr_h)) else "hbm"
        stage_roof[k_] = {"bound": bound, "frac": fr_t if bound == "tensor" else fr_h, "ms": t_ms,
                          "tflops": tf(stage_flops[k_], t_ms) if k_ in stage_flops else None,
                          "gbs": stage_bytes[k_] / (t_ms * 1e-3) / 1e9 if k_ in stage_bytes else None}
    furthest = min(stage_roof, key=lambda k_: stage_roof[k_]["frac"]) if stage_roof else None
    top = max(stage_roof, key=lambda k_: stage_roof[k_]["ms"]) if stage_roof else None
    roof = None
    if top is not None:
        r = stage_roof[top]
        if r["bound"] == "tensor":
            roof = {"kernel": top, "bound": "tensor", "achieved": r["tflops"], "peak": peaks["burst"], "unit": "TFLOP/s",
                    "frac": r["tflops"] / peaks["burst"], "traffic": ncu_traffic(top),
                    "peak_source": f"{peaks['source']} cuBLAS bf16, burst (the timed passes run at full clock; see clocks)",
                    "peak_sustained": peaks["sustained"], "frac_of_sustained": r["tflops"] / peaks["sustained"],
                    "ms_per_launch": r["ms"], "flops_per_launch": stage_flops[top]}
        else:
            roof = {"kernel": top, "bound": "hbm", "achieved": r["gbs"], "peak": peaks["hbm"], "unit": "GB/s",
                    "frac": r["gbs"] / peaks["hbm"], "traffic": ncu_traffic(top),
                    "peak_source": f"{peaks['source']} copy bandwidth", "ms_per_launch": r["ms"],
                    "bytes_per_launch": stage_bytes[top]}
    skipping = None
    if cfg["gate"]:   # gated workloads: the sweeps leave out chunk pairs the gate has made negligible; the FLOP models do not
        kept, total = binding.skipped_chunk_pairs(ws)
        skipping = {"kept_chunk_pairs": kept, "all_chunk_pairs": total,
                    "note": "TFLOP/s are attention-equivalent FLOPs of the full causal problem per second, skipped pairs included"}
    executed = sum(stage_flops[k_] for k_ in stage_ms if k_ in stage_flops)
    line = {
        "metric": metric_name(cfg), "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": f"{args.workload}: B={B} H={H} L={L} d={d} bf16 fwd+bwd per GPU", "global_batch": B * world,
                   "seq_len": L, "parallelism": f"{world} independent replicas (no collective)",
                   "l2_policy": "inputs + workspace exceed L2 (no flush needed)", "chunk": CHUNK,
                   "state": "forward on the backward-sized workspace, path_attn_bwd_reuse (see detail.step_ms_no_reuse)",
                   "timing": f"median of {len(passes)} back-to-back passes of {args.steps} steps", "block_skipping": skipping},
        "clocks": clocks,
        "e2e": {"value": world * tf(f1 + b1, ms_e2e), "unit": UNIT, "ms_per_step": ms_e2e, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h},
        "gpu_launches": launches[0] * args.steps,
        "roofline": roof,
        "detail": {
            "tflops_m2": world * tf(f2 + b2, ms),
            "frac_of_burst_peak_m1": tf(f1 + b1, ms) / peaks["burst"], "frac_of_burst_peak_m2": tf(f2 + b2, ms) / peaks["burst"],
            "frac_of_nominal_m1": tf(f1 + b1, ms) / 2250.0,
            "ms_per_step_best_pass": ms_best,
            "fwd_ms": fwd_ms, "fwd_tflops_m1": world * tf(f1, fwd_ms), "fwd_frac_of_burst_peak_m1": tf(f1, fwd_ms) / peaks["burst"],
            "fwd_frac_of_burst_peak_m2": tf(f2, fwd_ms) / peaks["burst"], "fwd_stage_ms": fwd_stage_ms,
            "bwd_ms": ms - sum(stage_ms.get(k_, 0.0) for k_ in ("chunk_prep", "levels_fwd", "fa_fwd")),
            "step_ms_no_reuse": no_reuse_ms, "tflops_m1_no_reuse": world * tf(f1 + b1, no_reuse_ms),
            "workspace_bytes": {"forward": binding.workspace_bytes(B, H, L, d, has_gate=cfg["gate"], for_backward=False),
                                "backward": ws.numel()},
            "executed_tensor_tflops": tf(executed, ms), "executed_frac_of_burst_peak": tf(executed, ms) / peaks["burst"],
            "stage_ms": stage_ms,
            "stage_roofline": stage_roof, "furthest_below_roofline": furthest,
            "launches_per_step": launches[0], "peaks": peaks,
        },
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        secs1, cores = oracle_sample(cfg, inp)                       # sizes the sample: aim at ~15 s of CPU work
        n = int(min(B * H, max(1, round(15.0 / max(secs1, 1e-3)))))
        secs, cores = oracle_sample(cfg, inp, n)
        s1, sb1 = flops_m1(1, 1, L, d)
        line["cpu_baseline"] = {"value": n * (s1 + sb1) / secs / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"{n} of {B * H} (batch, head) slices of {args.workload}, forward + backward, "
                                          f"float64, {secs:.1f} s"}
    else:
        line["cpu_baseline"] = None
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_decode(args):
    """Inference arm (paper Sec. 3.4), 1 GPU: prefill of the key cache for the C5 prompt shape, then `--steps` decoding
    steps on top of it.  One JSON line: decoding throughput and the step's algorithmic cache bytes against the measured
    copy bandwidth (the step is one read-modify-write pass over the float32 key cache plus a read of the bf16 values)."""
    from paper_2505_16381_b200 import binding
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    c = synth.CONFIGS["C5"]
    B, H, L, d = (args.batch or c["B"]), c["H"], c["L"], c["d"]
    g = torch.Generator(device=dev); g.manual_seed(synth.BASE_SEED)
    rn = lambda *sh: torch.randn(*sh, device=dev, generator=g)
    k = (rn(B, H, L, d) / d ** 0.5).bfloat16(); v = rn(B, H, L, d).bfloat16()
    w = rn(B, H, L, d); w = (w / w.norm(dim=-1, keepdim=True)).bfloat16(); beta = 2 * torch.sigmoid(rn(B, H, L))
    n_tok = args.warmup + args.steps
    cache = binding.alloc_cache(B, H, L + n_tok, d, False, dev)
    ws = binding.alloc_workspace(k, False, False)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    for _ in range(3):
        binding.path_attn_prefill_cache(k, v, w, beta, cache, workspace=ws)
    torch.cuda.synchronize()
    prefill_ms = []
    for _ in range(5):       # (one call moves 1.4 GB: more than L2, no flush needed)
        p0, p1 = ev(), ev()
        p0.record()
        binding.path_attn_prefill_cache(k, v, w, beta, cache, workspace=ws)
        p1.record()
        torch.cuda.synchronize()
        prefill_ms.append(p0.elapsed_time(p1))
    prefill_ms = sorted(prefill_ms)[2]
    assert binding.device_status(ws) == 0
    tok = [(rn(B, H, d) / d ** 0.5).bfloat16() for _ in range(2)] + [rn(B, H, d).bfloat16()]
    wt = rn(B, H, d); wt = (wt / wt.norm(dim=-1, keepdim=True)).bfloat16(); bt = 2 * torch.sigmoid(rn(B, H))
    dws = binding.decode_workspace(B, H, L + n_tok, d, dev)
    out = (torch.empty(B, H, d, dtype=torch.bfloat16, device=dev), torch.empty(B, H, dtype=torch.float32, device=dev))
    for i in range(args.warmup):
        binding.path_attn_decode_step(tok[0], tok[1], tok[2], wt, bt, cache, L + i, workspace=dws, out=out)
    sampler = ClockSampler(physical_gpu_index(0))
    torch.cuda.synchronize()
    sampler.start()
    e0, e1 = ev(), ev()
    e0.record()
    for i in range(args.steps):      # the cache (5.4 GB at the default shape) exceeds L2: no flush needed
        binding.path_attn_decode_step(tok[0], tok[1], tok[2], wt, bt, cache, L + args.warmup + i, workspace=dws, out=out)
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / args.steps
    peaks = load_peaks()
    T = L + args.warmup + (args.steps - 1) / 2.0            # mean number of cached tokens over the timed steps
    byt = B * H * T * (2 * 4 * d + 2 * d)
    gbs = byt / (ms * 1e-3) / 1e9
    line = {"metric": "PaTH decode steps/s per sequence at 32k cached tokens (B*H = %d heads)" % (B * H), "value": 1e3 / ms,
            "unit": "steps/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"decode: B={B} H={H} cached tokens={L} d={d}, float32 key cache, bf16 values",
                       "l2_policy": "cache exceeds L2 (no flush needed)"},
            "clocks": clocks, "gpu_launches": 2 * args.steps,
            "roofline": {"kernel": "decode_update_kernel", "bound": "hbm", "achieved": gbs, "peak": peaks["hbm"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm"], "traffic": None, "peak_source": f"{peaks['source']} copy bandwidth",
                         "bytes_per_launch": byt},
            "detail": {"prefill_cache_ms": prefill_ms, "prefill_tokens": B * L}}
    print(json.dumps(line), flush=True)


def run_frontend(args):
    """Layer front-end arm (paper Sec. 2.2 footnote, Sec. 2.4 gate), 1 GPU: one step = forward (z, logits -> w, beta, log f)
    plus backward (dw, dbeta, dlog f -> dz, dconv_w, dlogits) at the paper's benchmark shape B=32, H=32, L=4096, d=64
    with the gate.  One JSON line; the roofline entry is the backward kernel (the longer of the two): algorithmic bytes
    per (b, h, t) row = 2d (z) + 2d (dw) + 2d (dz) + 24 (six float32 scalars) against the measured copy bandwidth."""
    from paper_2505_16381_b200 import binding
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    B, H, L, d, gate = (args.batch or 32), 32, 4096, 64, True
    inp = synth.make_frontend_inputs(B, H, L, d, gate, seed=synth.BASE_SEED)
    x = {n: (t.to(dev) if torch.is_tensor(t) else t) for n, t in inp.items()}
    fwd = lambda: binding.path_attn_frontend_fwd(x["z"], x["conv_w"], x["beta_logit"], x["gate_logit"], H=H)
    bwd = lambda: binding.path_attn_frontend_bwd(x["z"], x["conv_w"], x["beta_logit"], x["dw"], x["dbeta"], x["gate_logit"],
                                                 x["dlog_f"], H=H)
    for _ in range(args.warmup):
        fwd(); bwd()
    ev = lambda: torch.cuda.Event(enable_timing=True)
    marks = [(ev(), ev(), ev()) for _ in range(args.steps)]
    sampler = ClockSampler(physical_gpu_index(0))
    torch.cuda.synchronize()
    sampler.start()
    for a, b, c in marks:      # the tensors of one step (2.9 GB at the default shape) exceed L2: no flush needed
        a.record(); fwd(); b.record(); bwd(); c.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = marks[0][0].elapsed_time(marks[-1][2]) / args.steps
    ms_f = sum(a.elapsed_time(b) for a, b, _ in marks) / args.steps
    ms_b = sum(b.elapsed_time(c) for _, b, c in marks) / args.steps
    rows = B * H * L
    byt_f, byt_b = rows * (4 * d + 16), rows * (6 * d + 24)
    peaks = load_peaks()
    gbs = byt_b / (ms_b * 1e-3) / 1e9
    line = {"metric": "PaTH layer front-end positions/s (forward + backward, all heads)", "value": B * L / (ms * 1e-3),
            "unit": "positions/s", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": f"front-end: B={B} H={H} L={L} d={d} gate={gate}, bf16 z / w / dw / dz, float32 scalars",
                       "l2_policy": "tensors exceed L2 (no flush needed)"},
            "clocks": clocks, "gpu_launches": 2 * args.steps,
            "roofline": {"kernel": "frontend_bwd_kernel", "bound": "hbm", "achieved": gbs, "peak": peaks["hbm"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm"], "traffic": NCU_FRONTEND_BWD_TRAFFIC_PER_BATCH_ROW * B,
                         "peak_source": f"{peaks['source']} copy bandwidth", "bytes_per_launch": byt_b},
            "detail": {"fwd_ms": ms_f, "bwd_ms": ms_b, "fwd_GBps": byt_f / (ms_f * 1e-3) / 1e9, "fwd_bytes_per_launch": byt_f}}
    # the low-rank linear layer in front (hidden size D = H*d, rank 64): z = (x W1^T) W2^T and its backward
    Dm, rk, C = H * d, 64, H * d
    gl = torch.Generator(device=dev); gl.manual_seed(synth.BASE_SEED + 1)
    xl = torch.randn(B, L, Dm, device=dev, generator=gl).bfloat16()
    w1 = (torch.randn(rk, Dm, device=dev, generator=gl) / Dm ** 0.5).bfloat16()
    w2 = (torch.randn(C, rk, device=dev, generator=gl) / rk ** 0.5).bfloat16()
    zl, tl = binding.path_attn_lowrank_fwd(xl, w1, w2)
    lws = torch.empty(int(binding.load().path_attn_lowrank_workspace_bytes(B * L, Dm, rk, C)), dtype=torch.uint8, device=dev)
    for _ in range(3):
        binding.path_attn_lowrank_fwd(xl, w1, w2); binding.path_attn_lowrank_bwd(xl, w1, w2, tl, x["z"], workspace=lws)
    la, lb, lc = ev(), ev(), ev()
    torch.cuda.synchronize()
    la.record()
    for _ in range(args.steps):
        binding.path_attn_lowrank_fwd(xl, w1, w2)
    lb.record()
    for _ in range(args.steps):
        binding.path_attn_lowrank_bwd(xl, w1, w2, tl, x["z"], workspace=lws)
    lc.record()
    torch.cuda.synchronize()
    lr_f, lr_b = la.elapsed_time(lb) / args.steps, lb.elapsed_time(lc) / args.steps
    Mr = B * L
    lr_bytes_f = Mr * (Dm + 2 * rk + C) * 2                       # x in; t out and in again; z out
    lr_bytes_b = Mr * (2 * C + 2 * rk + rk + 2 * Dm) * 2          # dz twice, dt out and in twice, t, x, dx
    line["detail"].update({"lowrank_fwd_ms": lr_f, "lowrank_bwd_ms": lr_b, "lowrank_fwd_GBps": lr_bytes_f / (lr_f * 1e-3) / 1e9,
                           "lowrank_bwd_GBps": lr_bytes_b / (lr_b * 1e-3) / 1e9,
                           "lowrank_shape": f"M={Mr} D={Dm} r={rk} C={C}"})
    if not args.no_cpu_baseline:
        from oracle import frontend_oracle as fo
        import time
        Ls = 256                                             # one batch row, the first 256 positions, all heads
        f64 = lambda t: None if t is None else synth.to_f64(t[:1, :Ls] if t.shape[1] == L else t[:1, :, :Ls])
        t0 = time.perf_counter()
        fo.frontend_fwd(f64(inp["z"]), synth.to_f64(inp["conv_w"]), f64(inp["beta_logit"]), f64(inp["gate_logit"]), H, 1e-6)
        fo.frontend_bwd(f64(inp["z"]), synth.to_f64(inp["conv_w"]), f64(inp["beta_logit"]), f64(inp["gate_logit"]),
                        f64(inp["dw"]), f64(inp["dbeta"]), f64(inp["dlog_f"]), H, 1e-6)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": Ls / dt, "unit": "positions/s", "cores": 1, "kind": "oracle",
                                "sample": f"B=1, first {Ls} positions, all {H} heads, forward + backward"}
    print(json.dumps(line), flush=True)


def run_ring(args):
    """Context-parallel arm (paper Sec. 3.5), 1 GPU: the headline sequence cut into `--segments` equal segments, all ranks of
    the ring played one after the other on this device (prepare for every segment, then every step of every rank:
    D (D - 1) / 2 segment-against-segment sweeps).  One JSON line: forward TFLOP/s (attention-equivalent FLOPs of the
    whole causal problem) of the virtual ring next to the monolithic forward.  Nothing is sent anywhere: this times the
    per-device arithmetic, not a ring."""
    from paper_2505_16381_b200 import binding, ring
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    c = synth.CONFIGS[args.workload]
    B, H, L, d, D = (args.batch or c["B"]), c["H"], c["L"], c["d"], args.segments
    inp = synth.make_inputs(B, H, L, d, dtype="bf16", qk_scaled=c["qk_scaled"], gate=c["gate"], seed=synth.BASE_SEED + c["index"])
    names = ["q", "k", "v", "w", "beta"] + (["log_f"] if c["gate"] else [])
    full = {n: inp[n].to(dev) for n in names}
    cuts = [L * (i + 1) // D for i in range(D)]
    segs, lo = [], 0
    for hi in cuts:
        segs.append({n: full[n][:, :, lo:hi].contiguous() for n in names})
        lo = hi
    ops = ring.GpuOps(B, H, d, scale=inp["scale"], has_gate=c["gate"], device=dev)
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def timed(fn):
        for _ in range(args.warmup):
            fn()
        res = []
        for _ in range(args.steps):
            a, b_ = ev(), ev()
            torch.cuda.synchronize()
            a.record(); fn(); b_.record()
            torch.cuda.synchronize()
            res.append(a.elapsed_time(b_))
        return sorted(res)[len(res) // 2]

    sampler = ClockSampler(physical_gpu_index(0))
    sampler.start()
    ms_ring = timed(lambda: ring.virtual_ring_forward(ops, segs))
    ws = binding.alloc_workspace(full["q"], c["gate"], False)
    ms_mono = timed(lambda: binding.path_attn_fwd(full["q"], full["k"], full["v"], full["w"], full["beta"], full.get("log_f"),
                                                  scale=inp["scale"], workspace=ws))
    clocks = sampler.stop()
    f1, _ = flops_m1(B, H, L, d)
    peaks = load_peaks()
    line = {"metric": f"PaTH attn forward TFLOP/s (attention-equivalent FLOPs), {D} virtual context-parallel ranks on one GPU, L={L}, d={d}",
            "value": f1 / (ms_ring * 1e-3) / 1e12, "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_ring, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": f"{args.workload} forward: B={B} H={H} L={L} d={d}, {D} segments of {L // D} positions, "
                                   f"prepare x{D} + {D * (D - 1) // 2} steps + finish x{D}, no communication",
                       "l2_policy": "inputs + workspaces exceed L2 (no flush needed)"},
            "clocks": clocks, "gpu_launches": None,
            "roofline": {"kernel": "whole virtual ring (sweeps + preparations)", "bound": "tensor", "achieved": f1 / (ms_ring * 1e-3) / 1e12,
                         "peak": peaks["burst"], "unit": "TFLOP/s", "frac": f1 / (ms_ring * 1e-3) / 1e12 / peaks["burst"], "traffic": None,
                         "peak_source": f"{peaks['source']} cuBLAS bf16, burst"},
            "detail": {"monolithic_forward_ms": ms_mono, "monolithic_forward_tflops": f1 / (ms_mono * 1e-3) / 1e12,
                       "ring_over_monolithic": ms_ring / ms_mono}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="C3", choices=[n for n, c in synth.CONFIGS.items() if c["backward"]])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch size (profiling captures)")
    ap.add_argument("--only-step", action="store_true",
                    help="time the fwd+bwd step only: no forward-only / no-reuse / end-to-end arms (profiling captures)")
    ap.add_argument("--passes", type=int, default=0,
                    help="number of timed passes of --steps steps (default: as many as keep the GPU busy for > 1 s; profiling captures pass 1)")
    ap.add_argument("--path", choices=["train", "decode", "frontend", "ring"], default="train",
                    help="train: the fwd+bwd step (the headline); decode: the inference arm; frontend: the layer front-end "
                         "kernels; ring: the context-parallel calls as virtual ranks (all 1 GPU, not part of the headline)")
    ap.add_argument("--segments", type=int, default=4, help="--path ring: number of virtual ranks")
    args = ap.parse_args()
    if args.path == "decode":
        args.warmup = max(args.warmup, 3)
        return run_decode(args)
    if args.path == "frontend":
        args.warmup = max(args.warmup, 3)
        return run_frontend(args)
    if args.path == "ring":
        args.warmup = max(args.warmup, 3)
        return run_ring(args)
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = dict(synth.CONFIGS[args.workload])
    if args.batch > 0:
        cfg["B"] = args.batch
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
