#!/usr/bin/env python
"""Benchmark of the STaMP-quantized linear layer on B200.

A step is one pass of the whole hot path -- sequence transform, per-token mixed-precision
quantization, int8 tensor-core GEMM, de-quantization, inverse transform, bias -- over one
synthetic activation batch, through the C ABI (stamp_linear_fused).  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl native|reference] [--workload NAME]

N > 1 (launched by torch.distributed.run) runs N independent replicas, one per GPU: the layer
has no cross-GPU exchange, so there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2510_26771_b200 import inputs as gen  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
NOMINAL_I8_OVER_BF16 = 2.0      # dense tensor peaks: 4.5 POPS int8 vs 2.25 PFLOPS bf16
NOMINAL_I8_TOPS = 4500.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
DEFAULT_WORKLOAD = "sweep_L32768_D8192"   # the largest single-GPU shape of the throughput sweep
SECONDARY_WORKLOAD = "llm_mlp_up"         # read as well (extra.secondary): the LLM layer of the named configurations

# DRAM bytes per launch of the dominant kernel from an ncu capture of the kernel as it stands (see profiles/);
# a workload is listed only while that capture is current.
NCU_TRAFFIC_BYTES = {
    # k_gemm_i8<256, 6, EPI_HAAR_BF16, pair>: dram__bytes_read.sum 736.34 MB + dram__bytes_write.sum 519.52 MB, one
    # launch, single-pass capture at full size (profiles/k_gemm_i8_pair_dram_sweep_L32768_D8192.txt)
    "sweep_L32768_D8192": 1255860000,
    # the same kernel on the small case: 54.27 MB + 16.40 MB
    "llm_mlp_up": 70661376,
}


def workloads():
    w = dict(gen.named_configs())
    for L in gen.SWEEP_L:
        for D in gen.SWEEP_D:
            c = gen.config_sweep(L, D)
            w[c.name] = c
    return w


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_burst": float(p["bf16_tflops"]),
                "bf16_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_burst": FALLBACK_BF16_TFLOPS, "bf16_sustained": 1400.0,
            "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the GPU is under load."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"], stdout=self.tmp,
                                         stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.tmp.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if sm:
            # samples under load = the upper half of the observed clocks (idle samples sit at the floor)
            out["sm_mhz"] = statistics.median(sorted(sm)[len(sm) // 2:])
            out["sm_max_mhz"] = max(smax)
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


def time_loop(fn, iters, warm=3):
    """Mean milliseconds per call of fn(i) over `iters` back-to-back calls (CUDA events on the current stream)."""
    import torch
    for i in range(warm):
        fn(i)
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(iters):
        fn(i)
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) / iters


def measure_i8_ceilings(st, local_rank):
    """The int8 tensor ceilings of THIS GPU, taken in this run:
    * the issue-only tcgen05.mma kind::i8 loop on tiles resident in shared memory (stamp_measure_i8_mma_issue):
      burst = best of 5 launches of about 4 ms, sustained = mean over about a second of back-to-back launches,
      with the SM clock sampled meanwhile;
    * torch._int_mm 8192^3 (the vendor library's int8 GEMM), burst and mean."""
    import torch
    out = {}
    nbatch = 1000
    ops = st.stamp_measure_i8_mma_issue(nbatch)   # warm-up, sets the function attribute
    torch.cuda.synchronize()
    best = min(time_loop(lambda i: st.stamp_measure_i8_mma_issue(nbatch), 1, warm=0) for _ in range(5))
    out["issue_only_burst_tops"] = ops / (best * 1e-3) / 1e12
    sampler = ClockSampler(local_rank)
    n = max(10, int(1000.0 / best))
    mean = time_loop(lambda i: st.stamp_measure_i8_mma_issue(nbatch), n, warm=0)
    clk = sampler.stop()
    out["issue_only_sustained_tops"] = ops / (mean * 1e-3) / 1e12
    out["issue_only_sustained_sm_mhz"] = clk["sm_mhz"]
    out["issue_only_reasons"] = clk["reasons"]
    out["issue_only_shape"] = "M128 x N256 x K32, cta_group::1, one CTA per SM, 64000 instructions per CTA and launch"
    try:
        a = torch.randint(-8, 8, (8192, 8192), dtype=torch.int8, device="cuda")
        b = torch.randint(-8, 8, (8192, 8192), dtype=torch.int8, device="cuda").t()
        torch._int_mm(a, b)
        torch.cuda.synchronize()
        t_best = min(time_loop(lambda i: torch._int_mm(a, b), 1, warm=0) for _ in range(10))
        t_mean = time_loop(lambda i: torch._int_mm(a, b), 20, warm=0)
        out["torch_int_mm_8192_burst_tops"] = 2.0 * 8192 ** 3 / (t_best * 1e-3) / 1e12
        out["torch_int_mm_8192_tops"] = 2.0 * 8192 ** 3 / (t_mean * 1e-3) / 1e12
        del a, b
    except Exception:
        out["torch_int_mm_8192_burst_tops"] = out["torch_int_mm_8192_tops"] = None
    if st.stamp_last_device_status() != 0:
        raise RuntimeError("device status word raised by the issue-only loop")
    return out


def max_over_ranks_ms(local_ms: float, device="cpu") -> float:
    """Timed-region duration of the whole job: the slowest rank's (all-reduce MAX; identity for one rank)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(local_ms)
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tops(ops_per_replica_step: float, world: int, ms_per_step: float) -> float:
    """Replicas only: every rank runs the same step on its own GPU, so the job did world x the work
    in the time of the slowest rank."""
    return world * ops_per_replica_step / (ms_per_step * 1e-3) / 1e12


def cpu_oracle_sample(cfg, seconds_target=15.0):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload: all tokens and
    features, a subset of output channels chosen so that the run takes roughly seconds_target."""
    from oracle import stamp_oracle as orc
    orc.build()
    X = gen.make_activation(cfg)
    def run(ncol):
        Wc = gen.make_weight(cfg, np.arange(ncol))
        t0 = time.perf_counter()
        orc.stamp_linear(X, Wc, None, transform=cfg.transform, block=cfg.block, levels=cfg.levels, k_hi=cfg.k_hi, grid_w=cfg.grid, asym=cfg.zero_point,
                         want=("Y",))
        return time.perf_counter() - t0
    # two probes separate the fixed cost (transform + quantizer) from the per-channel cost (GEMM, inverse)
    c1, c2 = min(cfg.N, 8), min(cfg.N, 64)
    t1, t2 = run(c1), run(c2)
    per_col = max((t2 - t1) / max(c2 - c1, 1), 1e-6)
    fixed = max(t1 - per_col * c1, 0.0)
    ncols = int(min(cfg.N, max(c2, (seconds_target - fixed) / per_col)))
    ncols = max(8, (ncols // 8) * 8)
    W = gen.make_weight(cfg, np.arange(ncols))
    t0 = time.perf_counter()
    orc.stamp_linear(X, W, None, transform=cfg.transform, block=cfg.block, levels=cfg.levels, k_hi=cfg.k_hi,
                     grid_w=cfg.grid, asym=cfg.zero_point, want=("Y",))
    dt = time.perf_counter() - t0
    tops = 2.0 * cfg.M * ncols * cfg.K / dt / 1e12
    return {"value": tops, "unit": "TOPS", "cores": orc.num_threads(), "kind": "oracle",
            "sample": f"all {cfg.M} tokens x {cfg.K} features, {ncols} of {cfg.N} output channels, "
                      f"{dt:.1f} s of oracle time"}, (X, W, ncols)


def run_reference(args, cfg):
    """--impl reference: the CPU oracle timed on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import stamp_oracle as orc
    base, (X, W, ncols) = cpu_oracle_sample(cfg, seconds_target=8.0)

    def step():
        orc.stamp_linear(X, W, None, transform=cfg.transform, block=cfg.block, levels=cfg.levels, k_hi=cfg.k_hi, grid_w=cfg.grid, asym=cfg.zero_point,
                         want=("Y",))
    for _ in range(min(args.warmup, 1)):
        step()
    steps = max(1, min(args.steps, 3))
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / steps
    tops = 2.0 * cfg.M * ncols * cfg.K / dt / 1e12
    line = {"impl": "reference", "metric": "stamp_linear_tops", "value": tops, "unit": "TOPS", "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": {"workload": cfg.name, "B": cfg.B, "L": cfg.L, "K": cfg.K, "N": cfg.N,
                       "sample_output_channels": ncols},
            "cpu_baseline": {"value": tops, "unit": "TOPS", "cores": base["cores"], "kind": "oracle",
                             "sample": f"all {cfg.M} tokens x {cfg.K} features, {ncols} of {cfg.N} output channels "
                                       "per step"},
            "e2e": {"value": tops, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def quick_reading(st, cfg, y_t, steps):
    """ms per step, layer TOPS and GEMM share of another workload through the same call (no side measurements)."""
    import torch
    c = st.make_config(cfg.transform, cfg.block, cfg.levels, cfg.k_hi, grid_w=cfg.grid, zero_point=cfg.zero_point)
    x_t = torch.bfloat16 if cfg.dtype == gen.BF16 else torch.float32
    X_host = torch.from_numpy(gen.make_activation(cfg)).to(x_t)
    W_dev = torch.from_numpy(gen.make_weight(cfg)).cuda().to(x_t)
    bias = torch.from_numpy(gen.make_bias(cfg)).cuda()
    wq, w_scale = st.stamp_quantize_weights(c, W_dev)
    w_op, w_fmt, _ = weight_operand(st, c, wq)
    n_x = max(2, -(-2 * L2_BYTES // (X_host.numel() * X_host.element_size())))
    n_w = max(2, -(-2 * L2_BYTES // (w_op.numel() * w_op.element_size())))
    Xs = [X_host.cuda() for _ in range(n_x)]
    Ws = [w_op.clone() for _ in range(n_w)]
    Y = torch.empty((cfg.B, cfg.L, cfg.N), dtype=y_t, device="cuda")
    ws = st.alloc_workspace(c, cfg.B, cfg.L, cfg.K, cfg.N)
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record()      # (an event has no handle to pass to the library before its first record)
    g1.record()

    def step(i):
        st.stamp_linear_fused(c, Xs[i % n_x], Ws[i % n_w], w_fmt, w_scale, bias, ws, out=Y, n_out=cfg.N)
    ms = time_loop(step, steps, warm=20)
    launches = st.stamp_last_launch_count()
    st.stamp_profile_gemm_events(g0, g1)
    gms = []
    for i in range(20):
        step(i)
        torch.cuda.synchronize()
        gms.append(g0.elapsed_time(g1))
    st.stamp_profile_gemm_events(None, None)
    ops = 2.0 * cfg.M * cfg.N * cfg.K
    gemm_ms = statistics.mean(gms)
    return {"workload": cfg.name, "steps": steps, "ms_per_step": ms, "tops": ops / (ms * 1e-3) / 1e12,
            "gemm_ms": gemm_ms, "gemm_tops": ops / (gemm_ms * 1e-3) / 1e12, "launches_per_step": launches,
            "device_status": st.stamp_last_device_status()}


def weight_operand(st, c, wq):
    """The weight operand the benchmark hands to the layer: prepared once, offline (weights are static)."""
    both = st.stamp_prepare_weights_both(c, wq)
    return both, st.W_INT8_AND_PACKED4, ("int4 codes prepared offline: one per int8 for the tensor cores, "
                                         "packed two per byte for the kernels that only stream them")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="native", choices=("native", "reference"))
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--out-dtype", default="bf16", choices=("bf16", "f32"))
    ap.add_argument("--levels", type=int, default=None,
                    help="override the workload's Haar level count (0 = full depth) and, with --k-hi, its 8-bit rows")
    ap.add_argument("--k-hi", type=int, default=None)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true", help="skip the second reading on the LLM layer")
    ap.add_argument("--quick", action="store_true",
                    help="timed region only (no side measurements, no CPU baseline): for profiler captures")
    ap.add_argument("--stage", default="fused", choices=("fused", "quantize", "inverse"),
                    help="with --quick: the call each step makes (the whole layer, or one of its passes alone)")
    args = ap.parse_args()
    cfg = workloads()[args.workload]
    if args.levels is not None:
        cfg = gen.scaled(cfg, levels=args.levels)
    if args.k_hi is not None:
        cfg = gen.scaled(cfg, k_hi=args.k_hi)

    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist
    from paper_2510_26771_b200 import binding as st

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    st.lib()  # fails loudly if the CUDA library is missing
    warmup = max(args.warmup, 3)
    steps = max(args.steps, 1)
    peaks = measured_peaks()

    # ---- inputs: generated on the host, resident in HBM before the timed region ----
    c = st.make_config(cfg.transform, cfg.block, cfg.levels, cfg.k_hi, grid_w=cfg.grid, zero_point=cfg.zero_point)
    B, L, K, N, M = cfg.B, cfg.L, cfg.K, cfg.N, cfg.M
    x_t = torch.bfloat16 if cfg.dtype == gen.BF16 else torch.float32
    y_t = torch.bfloat16 if args.out_dtype == "bf16" else torch.float32
    X_host = torch.from_numpy(gen.make_activation(cfg)).to(x_t).pin_memory()
    W_dev = torch.from_numpy(gen.make_weight(cfg)).cuda().to(x_t)
    bias = torch.from_numpy(gen.make_bias(cfg)).cuda()
    wq, w_scale = st.stamp_quantize_weights(c, W_dev)       # offline: weights are static
    w8, w_fmt, weights_note = weight_operand(st, c, wq)
    del W_dev
    x_bytes = X_host.numel() * X_host.element_size()
    y_bytes = M * N * (2 if y_t == torch.bfloat16 else 4)
    # rotate over enough distinct copies that consecutive steps never find their inputs in L2
    n_x = max(2, -(-2 * L2_BYTES // x_bytes))
    n_w = max(2, -(-2 * L2_BYTES // (w8.numel() * w8.element_size())))
    Xs = [X_host.cuda() for _ in range(n_x)]
    Ws = [w8.clone() for _ in range(n_w)]
    Y = torch.empty((B, L, N), dtype=y_t, device="cuda")
    ws = st.alloc_workspace(c, B, L, K, N)

    def step(i):
        st.stamp_linear_fused(c, Xs[i % n_x], Ws[i % n_w], w_fmt, w_scale, bias, ws, out=Y, n_out=cfg.N)

    if args.quick and args.stage == "quantize":
        def step(i):  # noqa: F811
            st.stamp_quantize(c, Xs[i % n_x], ws)
    elif args.quick and args.stage == "inverse":
        Yt_in = torch.randn((B, L, N), device="cuda")

        def step(i):  # noqa: F811
            st.stamp_inverse(c, Yt_in, bias, ws, out=Y)

    for i in range(warmup):
        step(i)
    launches_per_step = st.stamp_last_launch_count()
    torch.cuda.synchronize()
    if st.stamp_last_device_status() != 0:
        raise RuntimeError("device status word raised during warm-up")

    # ---- timed region: exactly `steps` steps, CUDA events, GEMM bracketed by its own events ----
    sampler = ClockSampler(local_rank) if rank == 0 else None
    # the GEMM of every `ev_stride`-th step is bracketed by its own events: up to 200 samples spread over the whole region
    ev_stride = max(1, -(-steps // 200))
    n_ev = -(-steps // ev_stride)
    g0 = [torch.cuda.Event(enable_timing=True) for _ in range(n_ev)]
    g1 = [torch.cuda.Event(enable_timing=True) for _ in range(n_ev)]
    for e in g0 + g1:
        e.record()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ev0.record()
    for i in range(steps):
        if i % ev_stride == 0:
            st.stamp_profile_gemm_events(g0[i // ev_stride], g1[i // ev_stride])
        elif i % ev_stride == 1:
            st.stamp_profile_gemm_events(None, None)
        step(i)
    ev1.record()
    st.stamp_profile_gemm_events(None, None)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    total_ms = ev0.elapsed_time(ev1)
    total_ms = max_over_ranks_ms(total_ms, device="cuda")
    ms_per_step = total_ms / steps
    gemm_ms = statistics.mean(a.elapsed_time(b) for a, b in zip(g0, g1)) if args.stage == "fused" or not args.quick else 0.0
    status = st.stamp_last_device_status()

    # keep the GPU under the same load a little longer if the timed region was too short to sample clocks
    clocks = None
    if sampler is not None:
        t_end = time.time() + (0.0 if args.quick else max(0.0, 1.0 - total_ms / 1e3))
        i = 0
        while time.time() < t_end:
            step(i)
            i += 1
            if i % 64 == 0:
                torch.cuda.synchronize()
        torch.cuda.synchronize()
        clocks = sampler.stop()

    ops = 2.0 * M * N * K
    value = whole_job_tops(ops, world, ms_per_step)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    if args.quick:
        gemm_tops = ops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else None
        print(json.dumps({"metric": "stamp_linear_tops", "value": value, "unit": "TOPS", "n_gpus": world,
                          "steps": steps, "warmup": warmup, "ms_per_step": ms_per_step, "quick": True,
                          "config": {"workload": cfg.name, "stage": args.stage},
                          "extra": {"gemm_ms": gemm_ms, "gemm_tops": gemm_tops},
                          "gpu_launches": launches_per_step * steps, "clocks": clocks}), flush=True)
        return

    # ---- the bandwidth-bound passes, timed alone on this same workload (L2 defeated by the same rotation) ----
    iters = max(10, min(steps, 200))
    nh = st.n_hi_rows(c, B, L)
    quant_bytes = x_bytes + nh * K + (M - nh) * K // 2 + 4 * M
    q_ms = time_loop(lambda i: st.stamp_quantize(c, Xs[i % n_x], ws), iters)
    n_yt = max(2, -(-2 * L2_BYTES // (M * N * 4)))
    Yts = [torch.randn((B, L, N), device="cuda") for _ in range(n_yt)]
    inv_bytes = M * N * 4 + y_bytes
    i_ms = time_loop(lambda i: st.stamp_inverse(c, Yts[i % n_yt], bias, ws, out=Y), iters)
    del Yts

    # ---- end to end: host buffers, copies inside the timed region, through the C ABI ----
    # Two calls are kept in flight, on two streams with a workspace and a pinned result buffer each, so that
    # one step's result copy (device to host) overlaps the next step's input copy (host to device): the link is
    # full duplex.  Every step still copies its X in and its Y out inside the timed region.
    ws_bytes_h = st.stamp_workspace_bytes_host(c, B, L, K, N, st._dtype_code(X_host), 1 if y_t == torch.bfloat16 else 0)
    del ws
    lanes = [(torch.cuda.Stream(), torch.empty(ws_bytes_h, dtype=torch.uint8, device="cuda"),
              torch.empty((B, L, N), dtype=y_t).pin_memory()) for _ in range(2)]
    e2e_steps = max(6, min(steps, 100, int(2000.0 / max(ms_per_step * 8, 1e-3))))

    def e2e_loop(iters):
        main = torch.cuda.current_stream()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(main)
        for lane in lanes:
            lane[0].wait_event(a)
        for i in range(iters):
            stream, ws_h, Y_host = lanes[i % 2]
            with torch.cuda.stream(stream):
                st.stamp_linear_fused_host(c, X_host, Ws[i % n_w], w_fmt, w_scale, bias, Y_host, ws_h, n_out=N)
        for lane in lanes:
            done = torch.cuda.Event()
            done.record(lane[0])
            main.wait_event(done)
        b.record(main)
        torch.cuda.synchronize()
        return a.elapsed_time(b) / iters

    e2e_loop(4)
    e2e_ms = e2e_loop(e2e_steps)
    e2e = {"value": world * ops / (e2e_ms * 1e-3) / 1e12, "unit": "TOPS", "h2d_bytes_per_step": x_bytes,
           "d2h_bytes_per_step": y_bytes, "ms_per_step": e2e_ms, "in_flight": 2, "steps": e2e_steps}
    del lanes, Xs, Ws, Y

    # ---- a second reading on the LLM layer of the named configurations (same code path, smaller shape) ----
    secondary = None
    if cfg.name != SECONDARY_WORKLOAD and not args.no_secondary:
        secondary = quick_reading(st, workloads()[SECONDARY_WORKLOAD], y_t, min(steps, 1000))

    # ---- int8 ceilings of this GPU, measured now ----
    ceil = measure_i8_ceilings(st, local_rank)

    # The GEMM's denominator.  A timed region shorter than about a second runs at boost clocks (burst regime);
    # a longer one settles under the power cap (sustained regime): the measured ceilings of the same regime apply.
    burst = total_ms < 1000.0
    regime = "burst" if burst else "sustained"
    bf16x2 = (peaks["bf16_burst"] if burst else peaks["bf16_sustained"]) * NOMINAL_I8_OVER_BF16
    candidates = {
        f"issue-only tcgen05.mma kind::i8 loop, {regime}": ceil["issue_only_burst_tops" if burst else "issue_only_sustained_tops"],
        f"torch._int_mm 8192^3, {regime}": ceil["torch_int_mm_8192_burst_tops" if burst else "torch_int_mm_8192_tops"],
        f"2 x {peaks['source']} bf16 {regime} ({peaks['bf16_burst' if burst else 'bf16_sustained']} TFLOP/s)": bf16x2,
    }
    peak_name, i8_peak = max(((k, v) for k, v in candidates.items() if v), key=lambda kv: kv[1])
    gemm_tops = ops / (gemm_ms * 1e-3) / 1e12
    roofline = {"bound": "tensor", "kernel": "k_gemm_i8", "achieved": gemm_tops, "peak": i8_peak, "unit": "TFLOP/s",
                "frac": gemm_tops / i8_peak, "frac_of_nominal": gemm_tops / NOMINAL_I8_TOPS,
                "traffic": NCU_TRAFFIC_BYTES.get(cfg.name),
                "note": f"int8 ops; timed region {total_ms:.0f} ms => {regime} regime; peak = the highest of the int8 "
                        f"ceilings measured in this run for that regime: {peak_name}; all candidates (TOPS): "
                        + ", ".join(f"{k} = {v:.0f}" for k, v in candidates.items() if v)
                        + f"; nominal dense int8 {NOMINAL_I8_TOPS:.0f}"}
    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        cpu_baseline, _ = cpu_oracle_sample(cfg)

    sm_mhz = clocks["sm_mhz"] if clocks else None
    line = {
        "metric": "stamp_linear_tops", "value": value, "unit": "TOPS", "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": cfg.name, "B": B, "L": L, "K": K, "N": N, "transform": int(cfg.transform),
                   "block": cfg.block, "levels": cfg.levels, "k_hi": cfg.k_hi, "x_dtype": str(x_t).split(".")[-1],
                   "y_dtype": str(y_t).split(".")[-1], "weights": weights_note,
                   "l2": f"inputs rotate over {n_x} activation and {n_w} weight copies (> 2x L2)",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * steps, "roofline": roofline,
        "cpu_baseline": cpu_baseline,
        "extra": {"gemm_ms": gemm_ms, "gemm_tops": gemm_tops, "timed_region_ms": total_ms,
                  "ms_per_step_x_sm_mhz": ms_per_step * sm_mhz if sm_mhz else None,
                  "layer_frac_of_i8_peak": value / world / i8_peak,
                  "layer_frac_of_nominal": value / world / NOMINAL_I8_TOPS,
                  "quant_ms": q_ms, "quant_gbs": quant_bytes / (q_ms * 1e-3) / 1e9, "quant_bytes": quant_bytes,
                  "quant_frac_hbm": quant_bytes / (q_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                  "inverse_ms": i_ms, "inverse_gbs": inv_bytes / (i_ms * 1e-3) / 1e9, "inverse_bytes": inv_bytes,
                  "inverse_frac_hbm": inv_bytes / (i_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                  "i8_ceilings": ceil, "secondary": secondary, "launches_per_step": launches_per_step,
                  "device_status": status, "peaks": peaks},
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
