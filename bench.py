#!/usr/bin/env python
"""Benchmark of the KATA chunked forward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one ``kata_fwd_chunked`` call (rows a0-a6 of the hot path: normalise, feature
products, state update, inter-chunk read, intra-chunk scores and apply, gate/normalise epilogue)
on the long-context workload B=1, H=16, T=131072, d_k=d_v=64, C=64, bf16, q,k,v iid N(0,1) from
seed 3.  The metric is tokens/s (B*T per step).  With N > 1 every rank runs its own copy of the
workload (heads and batches are independent, no collective in the data path): weak scaling.

The JSON line also carries: ``roofline`` for the dominant kernel, ``e2e`` (the same call through
``kata_fwd_host`` with pinned host buffers, copies inside the timed region), ``cpu_baseline`` (the
fp64 oracle timed on a bounded sample on the host cores), ``clocks`` sampled during the timed
region, and ``extra`` with separately timed figures for the quadratic form and the scan forms.

``--impl reference`` times the oracle itself (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "kata_chunked_fwd_tokens_per_s_T131072_d64"
UNIT = "tokens/s"
WORKLOAD = dict(B=1, H=16, T=131072, d_k=64, d_v=64, C=64)

# Algorithmic work per (b,h,t) of the chunked form with the packed symmetric feature
# n = d(d+1)/2 = 2080: state update 2*n*d_v + inter-chunk read 2*n*d_v + intra-chunk
# (C+1)/2 * 2*(d + d_v) + normaliser via the d x d Gram 3*d^2.
def chunked_flops_per_head_token(d=64, dv=64, C=64):
    n = d * (d + 1) // 2
    return 4 * n * dv + (C + 1) * (d + dv) + 3 * d * d


def quadratic_flops(B, H, T, d=64, dv=64):
    return B * H * (T * (T + 1) // 2) * (2 * d + 2 * dv)


def load_traffic(T: int):
    """DRAM bytes per launch of the dominant kernel, scaled linearly in T from the ncu capture recorded beside its
    summary under profiles/ (null if the record is missing)."""
    path = os.path.join(ROOT, "profiles", "tc_split_kernel_c4_T32768_traffic.json")
    if not os.path.exists(path):
        return None, "kata::tc_split_kernel (tcgen05 feature-split chunked forward)"
    with open(path) as f:
        rec = json.load(f)
    scale = T / rec["T"]
    return scale * (rec["dram_bytes_read"] + rec["dram_bytes_write"]), rec["kernel"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons in the background."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0]))
                smax.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(names, r[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(smax) if smax else None,
                    samples=len(sm), reasons=sorted(reasons))


# The bounded sample of the workload the oracle is timed on, in the `cpu_baseline` leg and in `--impl reference` alike.
ORACLE_SAMPLE = dict(heads=1, tokens=65536)
ORACLE_SAMPLE_TEXT = ("fp64 numpy oracle, Algorithm-1 chunked form (direct d^2 feature), {heads} of the 16 heads x {tokens} "
                      "of the 131072 tokens of the workload per step; tokens/s extrapolated to H=16 heads (linear in T "
                      "and H)").format(**ORACLE_SAMPLE)


def time_oracle_sample(heads: int = 1, tokens: int = 8192):
    """The fp64 oracle's chunked form on `heads` heads x `tokens` tokens of the benchmark workload."""
    import numpy as np
    from oracle import kata_oracle as ko
    from paper_2607_17419_b200 import inputs
    w = inputs.gaussian_workload("cpu_sample", "bf16", 1, heads, tokens, 64, 64, 64, 3)
    t0 = time.perf_counter()
    for h in range(heads):
        o = ko.kata_chunked(w.q_ref[0, h], w.k_ref[0, h], w.v_ref[0, h], 64, "psd_direct")
    dt = time.perf_counter() - t0
    assert np.all(np.isfinite(o))
    # whole-job tokens/s: a token counts once its H heads are done
    per_head_token = dt / (heads * tokens)
    return 1.0 / (per_head_token * WORKLOAD["H"]), dt


def host_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy  # noqa: F401  (loads BLAS so that host_threads sees it)
    for _ in range(args.warmup):
        time_oracle_sample(1, 2048)
    times, vals = [], []
    for _ in range(args.steps):
        v, dt = time_oracle_sample(**ORACLE_SAMPLE)
        times.append(dt)
        vals.append(v)
    value = statistics.mean(vals)
    ms = 1e3 * statistics.mean(times)
    sample = ORACLE_SAMPLE_TEXT
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic",
                config=dict(workload="c4 long-context chunked forward B=1 H=16 T=131072 d_k=d_v=64 C=64 bf16 inputs; each "
                                     "step is the bounded sample: " + ORACLE_SAMPLE_TEXT, **WORKLOAD),
                cpu_baseline=dict(value=value, unit=UNIT, cores=host_threads(), kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    from paper_2607_17419_b200 import binding as kb
    from paper_2607_17419_b200 import build as kbuild
    from paper_2607_17419_b200 import inputs, sharding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        kbuild.build()
    if world > 1:
        dist.barrier()
    kb.lib()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    W = WORKLOAD
    w = inputs.gaussian_workload("c4_long_bf16", "bf16", W["B"], W["H"], W["T"], W["d_k"], W["d_v"], W["C"], 3)

    def tt(a):
        return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    hq, hk, hv = (tt(a).pin_memory() for a in (w.q_dev, w.k_dev, w.v_dev))
    ho = torch.empty_like(hv).pin_memory()
    q, k, v = hq.to(dev), hk.to(dev), hv.to(dev)
    out = torch.empty_like(v)
    stream = torch.cuda.current_stream(dev)
    inter = kb.KATA_SCAN if args.mode == "scan" else kb.KATA_SEQUENTIAL

    def step():
        kb.kata_fwd_chunked(q, k, v, out, inter_chunk=inter)

    for _ in range(max(args.warmup, 3)):
        step()
    launches_per_step = kb.kata_last_launch_count()
    impl = "tensor" if kb.kata_last_impl() == kb.KATA_IMPL_TENSOR else "simt"
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    ms_total = e0.elapsed_time(e1)
    # the same step, each one timed by its own pair of events (median and best of at least 20)
    n_single = max(20, args.steps)
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_single)]
    for a, b in pairs:
        a.record(stream)
        step()
        b.record(stream)
    barrier()
    single = sorted(a.elapsed_time(b) for a, b in pairs)
    clocks = sampler.stop() if rank == 0 else None

    # ---- end to end: pinned host buffers through kata_fwd_host, copies inside the timed region ----
    ws = kb.Workspace()
    for _ in range(2):
        kb.kata_fwd_host(kb.KATA_FN_CHUNKED, hq, hk, hv, ho, inter_chunk=inter, workspace=ws)
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_steps = max(2, min(args.steps, 5))
    f0.record(stream)
    for _ in range(e2e_steps):
        kb.kata_fwd_host(kb.KATA_FN_CHUNKED, hq, hk, hv, ho, inter_chunk=inter, workspace=ws)
        stream.synchronize()          # the caller reads the result of each step
    f1.record(stream)
    barrier()
    e2e_ms_total = f0.elapsed_time(f1)
    # the host route works in pieces that hand the state over and runs them on the streaming kernel, the device call
    # on the feature-split kernel: the same function, rounded at different places
    diff = (ho.to(dev).float() - out.float()).abs().amax(dim=-1)
    assert bool((diff <= 3e-2 * out.float().abs().amax(dim=-1).clamp_min(1e-3)).all()), "host route and device call disagree"

    ms_total, e2e_ms_total = sharding.max_over_ranks([ms_total, e2e_ms_total], device=dev)

    if rank == 0:
        peaks = load_peaks()
        tokens = W["B"] * W["T"]
        ms_step = ms_total / args.steps
        value = sharding.whole_job_rate(tokens, world, ms_step)
        e2e_value = sharding.whole_job_rate(tokens, world, e2e_ms_total / e2e_steps)
        flops = chunked_flops_per_head_token() * W["B"] * W["H"] * W["T"]
        achieved = flops / (ms_step * 1e-3) / 1e12
        if impl == "tensor":
            sustained = ms_total > 1000.0
            peak = peaks["bf16_sustained"] if sustained else peaks["bf16_burst"]
            traffic, kernel_name = load_traffic(W["T"])
            roof = dict(bound="tensor", achieved=achieved, peak=peak, unit="TFLOP/s", frac=achieved / peak,
                        traffic=traffic, kernel=kernel_name,
                        note=f"algorithmic flops (packed feature n=2080) / CUDA-event time; peak = "
                             f"{'sustained' if sustained else 'burst'} bf16 cuBLAS of {peaks['source']}")
        else:
            alu_peak = 148 * 128 * 2 * 1.965e9 / 1e12      # SMs x fp32 lanes x FMA x max clock
            roof = dict(bound="alu", achieved=achieved, peak=alu_peak, unit="TFLOP/s", frac=achieved / alu_peak,
                        traffic=None, kernel="chunk_simt_kernel (fp32 FMA path)",
                        note="algorithmic flops / CUDA-event time; peak = 148 SMs x 128 fp32 lanes x 2 x 1.965 GHz")
        extra = measure_extra(kb, inputs, dev, stream, q, k, v, out, peaks) if args.extra else None
        cpu_runs = [time_oracle_sample(**ORACLE_SAMPLE) for _ in range(3)]
        cpu_val, cpu_dt = statistics.mean(r[0] for r in cpu_runs), sum(r[1] for r in cpu_runs)
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=max(args.warmup, 3),
                    ms_per_step=ms_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16",
                    data="synthetic",
                    config=dict(workload="c4 long-context chunked forward B=1 H=16 T=131072 d_k=d_v=64 C=64 bf16 "
                                         "(per GPU; q,k,v iid N(0,1), seed 3)",
                                inter_chunk=args.mode, impl=impl, l2="inputs (805 MB) larger than L2", **W),
                    e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=int(3 * q.numel() * 2),
                             d2h_bytes_per_step=int(out.numel() * 2), ms_per_step=e2e_ms_total / e2e_steps,
                             bound="host link",
                             host_link_gbs=(3 * q.numel() * 2 + out.numel() * 2) / (e2e_ms_total / e2e_steps * 1e-3) / 1e9),
                    step_ms=dict(median=statistics.median(single), best=single[0], n=len(single),
                                 note="each step between its own pair of CUDA events; ms_per_step is the K-step region / K"),
                    gpu_launches=int(launches_per_step * args.steps),
                    roofline=roof,
                    cpu_baseline=dict(value=cpu_val, unit=UNIT, cores=host_threads(), kind="oracle",
                                      sample=ORACLE_SAMPLE_TEXT + f"; mean of 3 such steps ({cpu_dt:.1f} s in all)"),
                    clocks=clocks, extra=extra)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_small(args):
    """Profiler case: the chunked forward on B=1, H=16, T=32768 (inputs 201 MB > L2, well under a GB)."""
    import numpy as np
    import torch
    from paper_2607_17419_b200 import binding as kb, build as kbuild, inputs
    kbuild.build()
    torch.cuda.set_device(0)
    w = inputs.gaussian_workload("c4_T32768", "bf16", 1, 16, 32768, 64, 64, 64, 3)
    q, k, v = (torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda() for a in (w.q_dev, w.k_dev, w.v_dev))
    out = torch.empty_like(v)
    inter = kb.KATA_SCAN if args.mode == "scan" else kb.KATA_SEQUENTIAL
    for _ in range(args.warmup):
        kb.kata_fwd_chunked(q, k, v, out, inter_chunk=inter)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.steps):
        kb.kata_fwd_chunked(q, k, v, out, inter_chunk=inter)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / args.steps
    print(json.dumps(dict(case="small", T=32768, ms_per_step=ms, tokens_per_s=32768 / (ms * 1e-3),
                          impl="tensor" if kb.kata_last_impl() == kb.KATA_IMPL_TENSOR else "simt")))


def run_decode(args):
    """Profiler case of the decode step: B=16, H=16, d=64, bf16 tokens, fp32 state (273 MB > L2); short line."""
    import torch
    from paper_2607_17419_b200 import binding as kb, build as kbuild
    kbuild.build()
    torch.cuda.set_device(0)
    Bd, Hd, d = 16, 16, 64
    g = torch.Generator(device="cpu").manual_seed(5)
    qd, kd, vd = (torch.randn(Bd, Hd, d, generator=g).to(torch.bfloat16).cuda() for _ in range(3))
    n_psi = kb.decode_n_psi(d)
    S = torch.zeros(Bd, Hd, n_psi, d, device="cuda")
    Z = torch.zeros(Bd, Hd, n_psi, device="cuda")
    od = torch.empty_like(vd)
    for _ in range(args.warmup):
        kb.kata_decode_step(qd, kd, vd, S, Z, od)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.steps):
        kb.kata_decode_step(qd, kd, vd, S, Z, od)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / args.steps
    nbytes = 2 * Bd * Hd * n_psi * (d + 1) * 4
    print(json.dumps(dict(case="decode", heads=Bd * Hd, ms_per_step=ms, state_bytes_per_step=nbytes,
                          gbs=nbytes / (ms * 1e-3) / 1e9)))


def order1_inputs(B, T, dev, seed=11):
    """Non-negative first-order features (|N(0,1)|-like: uniform here, the kernel's speed does not depend on the
    values), H = 16, d = 64, bf16: the shapes of the paper's scan benchmark."""
    import torch
    g = torch.Generator(device=dev).manual_seed(seed)
    return tuple(torch.rand(B, 16, T, 64, device=dev, generator=g).to(torch.bfloat16) for _ in range(3))


def run_order1(args):
    """Profiler case of the first-order tensor-core kernel: B=16, H=16, T=8192, C=128 (inputs 805 MB > L2, 256
    CTAs), one kernel per step in both forms (--mode scan: eight groups per head, every group walked twice); short line."""
    import torch
    from paper_2607_17419_b200 import binding as kb, build as kbuild
    kbuild.build()
    torch.cuda.set_device(0)
    B, T = 16, 8192
    q, k, v = order1_inputs(B, T, torch.device("cuda", 0))
    out = torch.empty_like(v)
    kw = dict(feature_order=1, C=128)
    if args.mode == "scan":
        kw.update(inter_chunk=kb.KATA_SCAN, scan_group=8)
    for _ in range(args.warmup):
        kb.kata_fwd_chunked(q, k, v, out, **kw)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.steps):
        kb.kata_fwd_chunked(q, k, v, out, **kw)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / args.steps
    nbytes = B * 16 * T * 512
    print(json.dumps(dict(case="order1", B=B, T=T, ms_per_step=ms, tokens_per_s=B * T / (ms * 1e-3),
                          algorithmic_bytes=nbytes, gbs=nbytes / (ms * 1e-3) / 1e9, launches=kb.kata_last_launch_count(),
                          impl="tensor" if kb.kata_last_impl() == kb.KATA_IMPL_TENSOR else "simt")))


def run_quadratic(args):
    """Profiler case of the quadratic forward: config 2 (B=4, H=16, T=4096, d=64, bf16; inputs 134 MB > L2); short line."""
    import numpy as np
    import torch
    from paper_2607_17419_b200 import binding as kb, build as kbuild, inputs
    kbuild.build()
    torch.cuda.set_device(0)
    w = inputs.config(2)
    q, k, v = (torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda() for a in (w.q_dev, w.k_dev, w.v_dev))
    out = torch.empty_like(v)
    for _ in range(args.warmup):
        kb.kata_fwd_quadratic(q, k, v, out)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.steps):
        kb.kata_fwd_quadratic(q, k, v, out)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / args.steps
    fl = quadratic_flops(w.B, w.H, w.T)
    print(json.dumps(dict(case="quadratic", ms_per_step=ms, tokens_per_s=w.B * w.T / (ms * 1e-3), tflops=fl / (ms * 1e-3) / 1e12,
                          launches=kb.kata_last_launch_count(),
                          impl="tensor" if kb.kata_last_impl() == kb.KATA_IMPL_TENSOR else "simt")))


def run_bwd(args):
    """Profiler case of the backward pass: config 2 (B=4, H=16, T=4096, d=64, bf16; inputs 134 MB > L2); short line."""
    import numpy as np
    import torch
    from paper_2607_17419_b200 import binding as kb, build as kbuild, inputs
    kbuild.build()
    torch.cuda.set_device(0)
    w = inputs.config(2)
    q, k, v = (torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda() for a in (w.q_dev, w.k_dev, w.v_dev))
    g = torch.randn(v.shape, device="cuda", generator=torch.Generator(device="cuda").manual_seed(7)).to(torch.bfloat16)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    for _ in range(args.warmup):
        kb.kata_bwd_quadratic(q, k, v, g, dq, dk, dv)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.steps):
        kb.kata_bwd_quadratic(q, k, v, g, dq, dk, dv)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / args.steps
    fl = quadratic_flops(w.B, w.H, w.T) / 256.0 * 640.0
    print(json.dumps(dict(case="bwd", ms_per_step=ms, tokens_per_s=w.B * w.T / (ms * 1e-3), tflops=fl / (ms * 1e-3) / 1e12,
                          launches=kb.kata_last_launch_count(),
                          impl="tensor" if kb.kata_last_impl() == kb.KATA_IMPL_TENSOR else "simt")))


def run_scan(args):
    """Profiler case of the scan form of the chunked forward: config 4 at T = 32768 (B=1, H=16, d=64, bf16), two
    groups of 128 tiles: a state-only pass over the first group, then both groups restarted; short line."""
    import numpy as np
    import torch
    from paper_2607_17419_b200 import binding as kb, build as kbuild, inputs
    kbuild.build()
    torch.cuda.set_device(0)
    w = inputs.config(4, 32768)
    q, k, v = (torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda() for a in (w.q_dev, w.k_dev, w.v_dev))
    out = torch.empty_like(v)
    for _ in range(args.warmup):
        kb.kata_fwd_chunked(q, k, v, out, inter_chunk=kb.KATA_SCAN)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.steps):
        kb.kata_fwd_chunked(q, k, v, out, inter_chunk=kb.KATA_SCAN)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / args.steps
    print(json.dumps(dict(case="scan", ms_per_step=ms, tokens_per_s=w.B * w.T / (ms * 1e-3),
                          launches=kb.kata_last_launch_count(),
                          impl="tensor" if kb.kata_last_impl() == kb.KATA_IMPL_TENSOR else "simt")))


def measure_extra(kb, inputs, dev, stream, q, k, v, out, peaks):
    """Separately timed secondary figures: scan forms on the same workload, quadratic form on config 2."""
    import numpy as np
    import torch

    def timed(fn, reps=5, warm=2):
        for _ in range(warm):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        for _ in range(reps):
            fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    res = {}
    T = q.shape[2]
    for name, fn in (("chunked_seq", lambda: kb.kata_fwd_chunked(q, k, v, out, inter_chunk=kb.KATA_SEQUENTIAL)),
                     ("chunked_scan", lambda: kb.kata_fwd_chunked(q, k, v, out, inter_chunk=kb.KATA_SCAN)),
                     ("chunk_state_scan", lambda: kb.kata_chunk_state_scan(q, k, v, out))):
        ms = timed(fn)
        res[name] = dict(ms=ms, tokens_per_s=T / (ms * 1e-3), launches=kb.kata_last_launch_count())
    B_, H_ = q.shape[0], q.shape[1]

    def plan(fn_code, mode, scan_group=0):
        ng, cpg, rounds = kb.kata_scan_plan(fn_code, B_, H_, T, 64, 64, 64,
                                            kb.make_opts(kb.KATA_BF16, inter_chunk=mode, scan_group=scan_group))
        return dict(n_groups=ng, chunks_per_group=cpg, scan_rounds=rounds)
    res["chunked_scan"].update(plan(kb.KATA_FN_CHUNKED, kb.KATA_SCAN))
    res["chunk_state_scan"].update(plan(kb.KATA_FN_CHUNK_STATE_SCAN, kb.KATA_SEQUENTIAL))
    # the scan forms with the chunk axis cut into 16 groups (four rounds of the state scan)
    sg = (T // 64) // 16
    for name, fn, code, mode in (
            ("chunked_scan_g16", lambda: kb.kata_fwd_chunked(q, k, v, out, inter_chunk=kb.KATA_SCAN, scan_group=sg),
             kb.KATA_FN_CHUNKED, kb.KATA_SCAN),
            ("chunk_state_scan_g16", lambda: kb.kata_chunk_state_scan(q, k, v, out, scan_group=sg),
             kb.KATA_FN_CHUNK_STATE_SCAN, kb.KATA_SEQUENTIAL)):
        ms = timed(fn)
        res[name] = dict(ms=ms, tokens_per_s=T / (ms * 1e-3), launches=kb.kata_last_launch_count(), **plan(code, mode, sg))
    # one batch element, four of the sixteen heads of the same workload: 32 CTAs on the sequential walk, where
    # the scan form (and inter_chunk = AUTO, which picks it here) fills the GPU with groups of tiles
    q4, k4, v4, o4 = (a[:, :4] for a in (q, k, v, out))
    q4, k4, v4, o4 = q4.contiguous(), k4.contiguous(), v4.contiguous(), o4.contiguous()
    for name, mode in (("seq", kb.KATA_SEQUENTIAL), ("scan", kb.KATA_SCAN), ("auto", kb.KATA_INTER_AUTO)):
        ms = timed(lambda: kb.kata_fwd_chunked(q4, k4, v4, o4, inter_chunk=mode))
        res[f"chunked_{name}_H4"] = dict(ms=ms, tokens_per_s=T / (ms * 1e-3), launches=kb.kata_last_launch_count())
    del q4, k4, v4, o4
    w2 = inputs.config(2)
    q2, k2, v2 = (torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).to(dev) for a in (w2.q_dev, w2.k_dev, w2.v_dev))
    o2 = torch.empty_like(v2)
    ms = timed(lambda: kb.kata_fwd_quadratic(q2, k2, v2, o2))
    fl = quadratic_flops(w2.B, w2.H, w2.T)
    res["quadratic_c2"] = dict(ms=ms, tokens_per_s=w2.B * w2.T / (ms * 1e-3), tflops=fl / (ms * 1e-3) / 1e12,
                               frac_of_bf16_burst=fl / (ms * 1e-3) / 1e12 / peaks["bf16_burst"],
                               impl="tensor" if kb.kata_last_impl() == kb.KATA_IMPL_TENSOR else "simt")
    # blockwise map (KATA-Mg): one-pass chunked form on the headline workload, quadratic form on config 2
    for g in (2, 4):
        ms = timed(lambda: kb.kata_fwd_chunked(q, k, v, out, feature_groups=g))
        res[f"chunked_seq_M{g}"] = dict(ms=ms, tokens_per_s=T / (ms * 1e-3), launches=kb.kata_last_launch_count(),
                                        ratio_to_M1=ms / res["chunked_seq"]["ms"],
                                        impl="tensor" if kb.kata_last_impl() == kb.KATA_IMPL_TENSOR else "simt")
        ms = timed(lambda: kb.kata_fwd_quadratic(q2, k2, v2, o2, feature_groups=g))
        res[f"quadratic_c2_M{g}"] = dict(ms=ms, tokens_per_s=w2.B * w2.T / (ms * 1e-3), tflops=fl / (ms * 1e-3) / 1e12,
                                         impl="tensor" if kb.kata_last_impl() == kb.KATA_IMPL_TENSOR else "simt")
    # the same forms on config 2 (64 heads x 4096 tokens), where the CTAs per head of a layout decide the number of
    # waves of the grid: the blockwise maps against the full lift, with the ratio
    ms1 = timed(lambda: kb.kata_fwd_chunked(q2, k2, v2, o2))
    res["chunked_seq_c2"] = dict(ms=ms1, tokens_per_s=w2.B * w2.T / (ms1 * 1e-3), launches=kb.kata_last_launch_count())
    for g in (2, 4):
        ms = timed(lambda: kb.kata_fwd_chunked(q2, k2, v2, o2, feature_groups=g))
        res[f"chunked_seq_c2_M{g}"] = dict(ms=ms, tokens_per_s=w2.B * w2.T / (ms * 1e-3), ratio_to_M1=ms / ms1,
                                           launches=kb.kata_last_launch_count())
    # backward of the quadratic form on config 2 (tensor-core kernels; recomputation, 5 matrix products of
    # 2 * 64 flops per causal pair = 640 algorithmic flops per pair)
    g2 = torch.randn(v2.shape, device=dev, generator=torch.Generator(device=dev).manual_seed(7)).to(torch.bfloat16)
    dq2, dk2, dv2 = torch.empty_like(q2), torch.empty_like(k2), torch.empty_like(v2)
    ms = timed(lambda: kb.kata_bwd_quadratic(q2, k2, v2, g2, dq2, dk2, dv2))
    flb = fl / 256.0 * 640.0
    res["bwd_quadratic_c2"] = dict(ms=ms, tokens_per_s=w2.B * w2.T / (ms * 1e-3), tflops=flb / (ms * 1e-3) / 1e12,
                                   frac_of_bf16_burst=flb / (ms * 1e-3) / 1e12 / peaks["bf16_burst"],
                                   launches=kb.kata_last_launch_count(),
                                   impl="tensor" if kb.kata_last_impl() == kb.KATA_IMPL_TENSOR else "simt")
    ms = timed(lambda: kb.kata_bwd_quadratic(q2, k2, v2, g2, dq2, dk2, dv2, feature_groups=2))
    res["bwd_quadratic_c2_M2"] = dict(ms=ms, tokens_per_s=w2.B * w2.T / (ms * 1e-3), tflops=flb / (ms * 1e-3) / 1e12,
                                      launches=kb.kata_last_launch_count(),
                                      impl="tensor" if kb.kata_last_impl() == kb.KATA_IMPL_TENSOR else "simt")
    # O(T) two-pass backward against the quadratic-form backward on one batch element of 16 heads (the first T tokens
    # of the headline workload): where the linear-state form takes over
    gfull = torch.randn(v.shape, device=dev, generator=torch.Generator(device=dev).manual_seed(9)).to(torch.bfloat16)
    cross = None
    for Tb in (4096, 16384, 65536, T):
        qb, kb_, vb, gb = (a[:, :, :Tb].contiguous() for a in (q, k, v, gfull))
        dqb, dkb, dvb = torch.empty_like(qb), torch.empty_like(kb_), torch.empty_like(vb)
        ms_c = timed(lambda: kb.kata_bwd_chunked(qb, kb_, vb, gb, dqb, dkb, dvb), reps=3, warm=1)
        lc = kb.kata_last_launch_count()
        ms_q = timed(lambda: kb.kata_bwd_quadratic(qb, kb_, vb, gb, dqb, dkb, dvb), reps=3, warm=1)
        res[f"bwd_chunked_H16_T{Tb}"] = dict(ms=ms_c, tokens_per_s=Tb / (ms_c * 1e-3), launches=lc, impl="simt",
                                             bwd_quadratic_ms=ms_q, speedup_over_quadratic=ms_q / ms_c)
        if cross is None and ms_c < ms_q:
            cross = Tb
        del qb, kb_, vb, gb, dqb, dkb, dvb
    res["bwd_chunked_crossover"] = dict(first_T_where_chunked_is_faster=cross, shapes="B=1 H=16 d=64 bf16, T in 4096, 16384, 65536, 131072")
    del gfull
    # first-order feature (rows of q, k as features; matched d x d state, C = 128): shapes of the paper's scan
    # benchmark; HBM-bound, 512 algorithmic bytes per token and head (q, k, v read, o written)
    for Bo, To in ((1, 8192), (1, 131072), (4, 32768), (16, 8192), (32, 32768)):
        qo, ko_, vo = order1_inputs(Bo, To, dev)
        oo = torch.empty_like(vo)
        nb = Bo * 16 * To * 512
        for name, fn in (("seq", lambda: kb.kata_fwd_chunked(qo, ko_, vo, oo, feature_order=1, C=128)),
                         ("scan", lambda: kb.kata_chunk_state_scan(qo, ko_, vo, oo, feature_order=1, C=128))):
            ms = timed(fn)
            res[f"order1_{name}_B{Bo}_T{To}"] = dict(ms=ms, tokens_per_s=Bo * To / (ms * 1e-3), gbs=nb / (ms * 1e-3) / 1e9,
                                                     frac_of_hbm=nb / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                                     launches=kb.kata_last_launch_count())
        del qo, ko_, vo, oo
    # decode step: B=16, H=16, d=64, bf16 tokens, fp32 state in the direct layout (285 MB of state > L2);
    # HBM-bound: the state is read and written once per token
    Bd, Hd, d = 16, 16, 64
    g = torch.Generator(device="cpu").manual_seed(5)
    qd, kd, vd = (torch.randn(Bd, Hd, d, generator=g).to(torch.bfloat16).to(dev) for _ in range(3))
    n_psi = kb.decode_n_psi(d)
    S = torch.zeros(Bd, Hd, n_psi, d, device=dev)
    Z = torch.zeros(Bd, Hd, n_psi, device=dev)
    od = torch.empty_like(vd)
    ms = timed(lambda: kb.kata_decode_step(qd, kd, vd, S, Z, od), reps=20, warm=3)
    nbytes = 2 * Bd * Hd * n_psi * (d + 1) * 4
    res["decode_step"] = dict(ms=ms, tokens_per_s=Bd / (ms * 1e-3), heads=Bd * Hd, state_bytes_per_step=nbytes,
                              gbs=nbytes / (ms * 1e-3) / 1e9, frac_of_hbm=nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                              launches=kb.kata_last_launch_count())
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--mode", default="sequential", choices=["sequential", "scan"])
    ap.add_argument("--no-extra", dest="extra", action="store_false")
    ap.add_argument("--case", default="full", choices=["full", "small", "decode", "order1", "bwd", "quadratic", "scan"],
                    help="small: the same kernel on T=32768 only; decode: the decode step only; order1: the "
                         "first-order tensor-core kernel on B=16, T=8192 (all for profiler captures; they print a "
                         "short line)")
    args = ap.parse_args()
    if args.case == "small":
        run_small(args)
    elif args.case == "decode":
        run_decode(args)
    elif args.case == "order1":
        run_order1(args)
    elif args.case == "bwd":
        run_bwd(args)
    elif args.case == "quadratic":
        run_quadratic(args)
    elif args.case == "scan":
        run_scan(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
