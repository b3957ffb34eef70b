#!/usr/bin/env python
"""Benchmark of the RMM linear layer (forward + backward through the C ABI) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = rmm_forward + rmm_backward on one batch of synthetic, seeded input of the
named workload.  Prints ONE JSON line.  With N > 1 (launched under torchrun) every rank
runs an independent replica of the same layer (the path does not shard); the value is
the aggregate over ranks, timed on the device, maximum over ranks.

--impl reference times the CPU fp64 oracle (oracle/) on this machine's host cores, on a
bounded sample of the same workload.
"""
import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import rmm_inputs as R  # noqa: E402

METRIC = "RMM linear fwd+bwd TFLOP/s (bf16)"
UNIT = "TFLOP/s"
DEFAULT_WORKLOAD = "large_ffn_up_rho0.1"
# (workload, step) -> DRAM bytes of the kernels of that pass, from the ncu capture at 4096 tokens summarised in
# profiles/dram_bytes_per_kernel_n4096_din1024_dout4096_k1638.md: (bytes read per token row, bytes read once, bytes
# written).  Backward pass: the sketch kernel reads dY once (33.61 MB per 4096 tokens) and so does the dX kernel
# (33.59 MB; cold caches, the two kernels serialised by ncu: side by side the second reader is served by L2 as far
# as dY fits); W 8.39 MB, G + X_proj 16.81 MB once; written at full size: dX, G and dW (at 4096 tokens they stay in L2).
NCU_DRAM_BYTES = {("large_ffn_up_rho0.1", "bwd"): ((33.613312e6 + 33.59e6) / 4096, 8.39e6 + 16.81e6,
                                                  lambda w: (w.n_tokens * w.d_in + w.b_proj * w.d_out + w.d_in * w.d_out) * 2)}

STEP_ORDER = ("fwd", "bwd", "y", "sketch", "dx", "sdy", "dw", "db")
E2E_LANES = 3    # streams (each with its own staging buffers and thread) that take the end-to-end steps in turn


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index, period=0.001):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.power = [], set(), []
        self.stop_flag = threading.Event()
        self.max_mhz = None
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {"hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap,
                 "hw_power_brake": nv.nvmlClocksThrottleReasonHwPowerBrakeSlowdown}
        while not self.stop_flag.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for n, bit in names.items():
                    if mask & bit:
                        self.reasons.add(n)
            except Exception:
                pass
            time.sleep(self.period)

    def result(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w": float(np.median(self.power)) if self.power else None}


def physical_gpu_index(local_index):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


# ----------------------------------------------------------------------------- oracle legs
def oracle_sample_seconds(w, n_tokens):
    """One forward+backward of the oracle on the first n_tokens rows (same rho); returns (seconds, flops)."""
    from oracle import oracle as O
    ws = R.Workload(w.name, w.dtype, n_tokens, w.d_in, w.d_out, w.rho, w.dist, w.seed, w.x_std, w.w_std, w.dy_std)
    X, W, b, dY = R.make_inputs(w, n_tokens=n_tokens)
    X, W, dY = X.astype(np.float64), W.astype(np.float64), dY.astype(np.float64)
    store = O.STORE_BF16 if w.dtype == R.DTYPE_BF16 else O.STORE_F32
    t0 = time.perf_counter()
    S = O.generate_s(ws.seed, n_tokens, ws.b_proj, ws.dist, store)
    _, Xp = O.forward(X, W, None, S)
    O.backward(dY, W, Xp, S)
    dt = time.perf_counter() - t0
    return dt, ws.flops()["total"], ws.b_proj


def pick_sample_tokens(w, budget_s):
    """Token count whose oracle pass should take about budget_s, from a small calibration pass.
    The oracle's strided loops slow down as the sample grows, hence the factor 3 of caution."""
    n0 = min(w.n_tokens, 256)
    t, f, _ = oracle_sample_seconds(w, n0)
    rate = f / max(t, 1e-6) / 3.0
    n = n0
    while n * 2 <= w.n_tokens:
        ws = R.Workload(w.name, w.dtype, n * 2, w.d_in, w.d_out, w.rho, w.dist, w.seed)
        if ws.flops()["total"] / rate > budget_s:
            break
        n *= 2
    return n


def cpu_baseline(w, budget_s=20.0):
    from oracle import oracle as O
    n = pick_sample_tokens(w, budget_s)
    t, f, k = oracle_sample_seconds(w, n)
    return {"value": f / t / 1e12, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
            "sample": f"first {n} of {w.n_tokens} token rows, B_proj = {k} (same rho), one fwd+bwd in {t:.2f} s",
            "seconds": t}


def run_reference(args, w):
    """The reference arm: the oracle as it stands on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as O
    total_budget = args.reference_budget_s
    per_step = total_budget / max(1, args.steps + args.warmup)
    n = pick_sample_tokens(w, per_step)
    for _ in range(args.warmup):
        oracle_sample_seconds(w, n)
    ts, fl, k = [], 0, 0
    for _ in range(args.steps):
        t, fl, k = oracle_sample_seconds(w, n)
        ts.append(t)
    tot = float(np.sum(ts))
    value = fl * args.steps / tot / 1e12
    sample = f"first {n} of {w.n_tokens} token rows, B_proj = {k} (same rho) per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_variance_probe(args, w, P, Xd, dYd):
    """Times rmm_variance_probe (the variance diagnostics of Section 2.3 on the device) on the workload's X and dY."""
    import torch
    pws = torch.empty(P.rmm_variance_probe_workspace_bytes(w.n_tokens, w.d_in, w.d_out), dtype=torch.uint8, device="cuda")
    out = torch.empty(8, dtype=torch.float64, device="cuda")
    for _ in range(args.warmup):
        P.rmm_variance_probe(Xd, dYd, w.b_proj, w.dist, out=out, workspace=pws)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        P.rmm_variance_probe(Xd, dYd, w.b_proj, w.dist, out=out, workspace=pws)
    e1.record()
    torch.cuda.synchronize()
    assert P.rmm_last_device_status(pws) == P.RMM_OK
    print(json.dumps({"metric": "rmm_variance_probe time", "unit": "ms", "value": e0.elapsed_time(e1) / args.steps,
                      "config": workload_config(w), "values": dict(zip(P.VARIANCE_FIELDS, out.cpu().tolist()))}), flush=True)


def workload_config(w):
    touched = (2 * w.n_tokens * (w.d_in + w.d_out) * 2 + 3 * w.d_in * w.d_out + 2 * w.b_proj * (w.d_in + w.d_out)) * w.elem_bytes
    return {"workload": w.name, "n_tokens": w.n_tokens, "d_in": w.d_in, "d_out": w.d_out, "rho": w.rho,
            "b_proj": w.b_proj, "sketch": ("gaussian", "rademacher", "identity", "sors_hadamard", "sors_dct")[w.dist], "seed": w.seed,
            "l2": f"inputs larger than L2: about {touched / 1e6:.0f} MB of tensors touched per step, no flush"}


# ----------------------------------------------------------------------------- N > 1: independent replicas
def max_over_ranks(ms_local, device):
    """Job time = the slowest rank's device time (all ranks get it). One process: the value itself."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(flops_per_replica, world, ms_step):
    """Whole-job TFLOP/s: every rank runs one replica of the layer (weak scaling, no collective on the data path)."""
    return world * flops_per_replica / (ms_step * 1e-3) / 1e12


# ----------------------------------------------------------------------------- GPU arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(R.WORKLOADS))
    ap.add_argument("--shape", type=int, nargs=4, metavar=("N", "D_IN", "D_OUT", "B_PROJ"), default=None,
                    help="an ad-hoc bf16 layer instead of a named workload (small cases for profilers)")
    ap.add_argument("--dist", default="gaussian", choices=["gaussian", "rademacher", "sors", "dct"], help="sketch of --shape")
    ap.add_argument("--pass-mode", type=int, default=0, choices=[0, 1, 2],
                    help="0: the two kernels of a pass side by side (default), 1: one launch per pass, 2: one after the other")
    ap.add_argument("--cycle-trace", action="store_true",
                    help="with the cycle-accounting build of the library (RMM_LIBRARY=...): print the per-role cycle "
                         "counters of the last sketch / one-launch kernel to stderr (median and maximum over CTAs)")
    ap.add_argument("--forward-only", action="store_true", help="steps are forward passes only (for profilers)")
    ap.add_argument("--variance-probe", action="store_true",
                    help="time rmm_variance_probe on the workload's X and dY instead of the layer")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=30)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--reference-budget-s", type=float, default=300.0,
                    help="wall-clock budget of the whole --impl reference run (sizes its token sample)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.shape is not None:
        n, di, do, k = args.shape
        dist = {"gaussian": R.DIST_GAUSSIAN, "rademacher": R.DIST_RADEMACHER, "sors": R.DIST_SORS, "dct": R.DIST_DCT}[args.dist]
        w = R.Workload(f"shape_{n}_{di}_{do}_k{k}_{args.dist}", R.DTYPE_BF16, n, di, do, k / n, dist, 0, k_fixed=k)
    else:
        w = R.WORKLOADS[args.workload]

    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist

    import paper_2201_13195_b200 as P

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    P.rmm_set_pass_mode(args.pass_mode)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    # ---- inputs, resident in HBM before the timed region
    X, W, b, dY = R.make_inputs(w)
    td = torch.bfloat16 if w.dtype == R.DTYPE_BF16 else torch.float32
    Xd, Wd, dYd = [torch.from_numpy(a).cuda().to(td).contiguous() for a in (X, W, dY)]
    N, k = w.n_tokens, w.b_proj
    Y = torch.empty((N, w.d_out), dtype=td, device="cuda")
    Xp = torch.empty((k, w.d_in), dtype=td, device="cuda")
    dX = torch.empty((N, w.d_in), dtype=td, device="cuda")
    dW = torch.empty((w.d_out, w.d_in), dtype=td, device="cuda")
    db = torch.empty((w.d_out,), dtype=td, device="cuda")
    ws = P.alloc_workspace(N, w.d_in, w.d_out, k, w.dtype, dist=w.dist)
    stream = torch.cuda.current_stream()

    if args.variance_probe:
        run_variance_probe(args, w, P, Xd, dYd)
        return

    def step(i):
        seed = w.seed + i          # a fresh S every step (Algorithm 1)
        P.rmm_forward(Xd, Wd, None, seed, k, w.dist, Y=Y, X_proj=Xp, workspace=ws, stream=stream)
        if not args.forward_only:
            P.rmm_backward(dYd, Wd, Xp, seed, w.dist, dX=dX, dW=dW, db=db, workspace=ws, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    t_warm = time.perf_counter()
    for i in range(args.warmup):
        step(i)
    barrier()
    t_warm = (time.perf_counter() - t_warm) / max(args.warmup, 1)
    assert P.rmm_last_device_status(ws) == P.RMM_OK

    launches_before = P.rmm_layer_launch_count()
    # per-kernel events for the first 50 timed steps only: a pair of events per pass costs a 4096-token step 6 %
    P.rmm_profile_enable(min(args.steps, 50) * 6)
    # about fifty samples over the timed region, at least one per millisecond's worth of it for short runs: a sampler
    # thread that wakes every millisecond competes with the launching thread of a host-bound (4096-token) run
    period = min(0.05, max(0.001, t_warm * args.steps / 50))
    sampler = ClockSampler(physical_gpu_index(local_rank), period)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        step(args.warmup + i)
    e1.record(stream)
    barrier()
    sampler.stop_flag.set()
    sampler.join()
    gpu_launches = P.rmm_layer_launch_count() - launches_before     # the library's own count of its kernel launches
    ms_total = e0.elapsed_time(e1)
    assert P.rmm_last_device_status(ws) == P.RMM_OK
    records = P.rmm_profile_read(min(args.steps, 50) * 6)
    P.rmm_profile_enable(0)
    if args.cycle_trace and rank == 0:
        tr = P.rmm_debug_pass_trace()
        if tr is None:
            sys.stderr.write("no cycle counters: load the cycle-accounting build with RMM_LIBRARY=...\n")
        else:
            for name, v in tr.items():
                lead, peer = [x for x in v[0::2] if x], [x for x in v[1::2] if x]
                fmt = lambda a: f"median {int(np.median(a)):9d} max {max(a):9d}" if a else "-"
                sys.stderr.write(f"{name:22s} even CTAs {fmt(lead)}   odd CTAs {fmt(peer)}\n")

    ms_total = max_over_ranks(ms_total, torch.device("cuda", local_rank))
    ms_step = ms_total / args.steps
    fl = w.flops()
    value = job_value(fl["total"], world, ms_step)

    # ---- per-kernel durations and roofline of the dominant kernel
    per_kernel = {}
    for name in STEP_ORDER:
        v = [ms for n, ms in records if n == name]
        if v:
            per_kernel[name] = {"ms": float(np.mean(v)), "launches_timed": len(v)}
    peaks = load_peaks()
    flops_of = {"y": fl["y"], "sketch": fl["sketch"], "dx": fl["dx"], "sdy": fl["sdy"], "dw": fl["dw"],
                "fwd": fl["y"] + fl["sketch"], "bwd": fl["dx"] + fl["sdy"]}
    if "bwd" in per_kernel and "dw" not in per_kernel:
        flops_of["bwd"] += fl["dw"]          # dW ran inside the backward pass (beside dX, after the sketch)
    for name, d in per_kernel.items():
        if name in flops_of:
            d["tflops"] = flops_of[name] / (d["ms"] * 1e-3) / 1e12
    dom = max((n for n in per_kernel if n in flops_of), key=lambda n: per_kernel[n]["ms"])
    achieved = per_kernel[dom]["tflops"]
    # Denominator: the burst figure when the timed region is short and ran at full clock (a kernel timed alone),
    # the sustained one when the region is long or the power cap was active (a kernel inside a long step).
    clocks = sampler.result()
    capped = "sw_power_cap" in (clocks.get("reasons") or [])
    use_burst = ms_total < 1000.0 and not capped
    peak = peaks["bf16_tflops"] if use_burst else peaks["bf16_tflops_sustained"]
    roofline = {"bound": "tensor", "kernel": dom, "achieved": achieved, "peak": peak,
                "unit": "TFLOP/s", "frac": achieved / peak,
                "peak_kind": f"{'burst' if use_burst else 'sustained'} bf16 GEMM, of {peaks['source']}",
                "frac_of_burst": achieved / peaks["bf16_tflops"],
                "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                "traffic": None, "algorithmic_flops_per_launch": flops_of[dom],
                "kernel_note": {"fwd": "forward pass: dense kernel (Y) beside sketch kernel (X_proj) + its reduction",
                                "bwd": "backward pass: dense kernel (dX) beside sketch kernel (S^T dY, db) + reduction + dW kernel"
                                }.get(dom, dom)}
    # DRAM bytes of the dominant pass, from an ncu capture taken at 4096 tokens; the token-sized reads grow in
    # proportion to the tokens.
    ncu_traffic = NCU_DRAM_BYTES.get((w.name, dom))
    if ncu_traffic is not None and args.pass_mode == 0:
        roofline["traffic"] = ncu_traffic[0] * w.n_tokens + ncu_traffic[1] + ncu_traffic[2](w)
        roofline["algorithmic_bytes"] = (w.n_tokens * (w.d_out + w.d_in) + w.d_in * w.d_out * 2 + w.b_proj * (2 * w.d_out + w.d_in)) * 2
        roofline["traffic_note"] = ("dram read+write of the kernels of the backward pass (dX kernel, sketch kernel, dW kernel): "
                                    "ncu at 4096 tokens, cold cache per kernel, token-sized reads scaled by the token count, "
                                    "results counted once")

    # ---- end to end through the host-buffer entry points (pinned host memory)
    e2e = None
    if (rank == 0 or world > 1) and args.e2e_steps > 0:
        # E2E_LANES lanes (stream, device staging, workspace, host result buffers) take the steps in turn, so that
        # the host->device copies of one step overlap the device->host copies of the step before it (the two
        # copy directions are separate engines); every step still copies all its inputs in and all its results out.
        hX, hW, hdY = [torch.from_numpy(a).to(td).pin_memory() for a in (X, W, dY)]
        nb = max(P.rmm_host_staging_bytes(N, w.d_in, w.d_out, k, w.dtype, bw, o) for bw in (0, 1) for o in (0, 1))
        lanes = []
        for li in range(E2E_LANES):
            ln = {"stream": stream if li == 0 else torch.cuda.Stream(),
                  "hY": torch.empty_like(Y, device="cpu").pin_memory(), "hXp": torch.empty_like(Xp, device="cpu").pin_memory(),
                  "hd": [torch.empty_like(a, device="cpu").pin_memory() for a in (dX, dW, db)],
                  "dev_in": torch.empty(nb, dtype=torch.uint8, device="cuda"),
                  "dev_out": torch.empty(nb, dtype=torch.uint8, device="cuda"),
                  "ws": ws if li == 0 else P.alloc_workspace(N, w.d_in, w.d_out, k, w.dtype, dist=w.dist)}
            lanes.append(ln)

        def e2e_step(i):
            ln = lanes[i % E2E_LANES]
            seed = w.seed + 100000 + i
            P.rmm_forward_host(hX, hW, None, seed, k, w.dist, ln["hY"], ln["hXp"], ln["dev_in"], ln["dev_out"], ln["ws"],
                               stream=ln["stream"])
            P.rmm_backward_host(hdY, hW, ln["hXp"], seed, w.dist, *ln["hd"], ln["dev_in"], ln["dev_out"], ln["ws"],
                                stream=ln["stream"])

        for i in range(2 * E2E_LANES):
            e2e_step(i)
        torch.cuda.synchronize()
        barrier()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(lanes[0]["stream"])
        for ln in lanes[1:]:
            ln["stream"].wait_event(g0)               # no lane starts before the start mark
        # The host entry points return when their results are in host memory, so each lane runs in its own
        # thread (ctypes releases the interpreter lock during the call).
        def lane_worker(li):
            for i in range(li, args.e2e_steps, E2E_LANES):
                e2e_step(2 * E2E_LANES + i)

        workers = [threading.Thread(target=lane_worker, args=(li,)) for li in range(E2E_LANES)]
        for t in workers:
            t.start()
        for t in workers:
            t.join()
        for ln in lanes[1:]:                          # the end mark follows the last step of every lane
            done = torch.cuda.Event()
            done.record(ln["stream"])
            lanes[0]["stream"].wait_event(done)
        g1.record(lanes[0]["stream"])
        torch.cuda.synchronize()
        for ln in lanes:
            assert P.rmm_last_device_status(ln["ws"]) == P.RMM_OK
        dt = g0.elapsed_time(g1) * 1e-3
        tt = torch.tensor([dt], dtype=torch.float64, device="cuda")
        if world > 1:
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        dt = float(tt.item())
        eb = w.elem_bytes
        h2d = (N * w.d_in + w.d_out * w.d_in) * eb + (N * w.d_out + w.d_out * w.d_in + k * w.d_in) * eb
        d2h = (N * w.d_out + k * w.d_in) * eb + (N * w.d_in + w.d_out * w.d_in + w.d_out) * eb
        e2e = {"value": world * fl["total"] * args.e2e_steps / dt / 1e12, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": args.e2e_steps, "ms_per_step": 1e3 * dt / args.e2e_steps,
               "streams": E2E_LANES}

    if rank == 0:
        cpu = None if args.no_cpu_baseline or world > 1 else cpu_baseline(w)
        saved = w.saved_bytes()
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16" if w.dtype == R.DTYPE_BF16 else "f32", "data": "synthetic",
                "config": workload_config(w), "pass_mode": args.pass_mode, "clocks": clocks, "e2e": e2e,
                "gpu_launches": gpu_launches, "roofline": roofline, "cpu_baseline": cpu,
                "pct_of_tensor_peak": {"burst": 100 * value / world / peaks["bf16_tflops"],
                                       "sustained": 100 * value / world / peaks["bf16_tflops_sustained"],
                                       "of": peaks["source"]},
                "sm_cycles_per_step": (ms_step * 1e-3 * clocks["sm_mhz"] * 1e6) if clocks.get("sm_mhz") else None,
                "effective_tflops_exact_layer_flops": world * fl["exact_layer"] / (ms_step * 1e-3) / 1e12,
                "saved_activation_bytes": saved, "workspace_bytes": int(ws.numel()), "per_kernel": per_kernel,
                "replicas": "independent layers, no collective" if world > 1 else None}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
