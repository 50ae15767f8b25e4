#!/usr/bin/env python
"""Benchmark of the blocked adaptive randomized range finder on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg2]

One "step" is one complete run of the hot path (Algorithm 2: norm, sample, panel QR, WY
update, norms, stop rule, for every block until the tolerance is met) on one seeded synthetic
matrix.  The default workload is the 8192 x 8192 float64 configuration (polynomial spectrum,
b = 64, relative tolerance 1e-4, rank cap 1024).  The metric is the method's own arithmetic,
sum_i (6 m_i n b + 3 m_i b^2) over the executed blocks, per second.  With N > 1 every rank runs
an independent replica (the path has no exchange step): value = N runs' flops / slowest rank.
Rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel of the default
# workload, from the ncu capture summarised in profiles/kernels_cfg2_4096x4096_b64.md (captured on a
# 4096 x 4096 case and scaled to the bench's average launch by the elements processed).
NCU_TRAFFIC_BYTES = {("cfg2", "update"): 1.07e9, ("cfg2", "vtw"): 136.3e6 * 3.875,
                     # tcgen05 kernels, block step 0 (profiles/kernels_cfg4_4096x11008_fp32_b64_tcgen05.md); of the update's
                     # 180 MB of writes 59 MB were still in L2 when the launch ended
                     ("cfg4", "update"): 185.4e6 + 120.9e6, ("cfg4", "vtw"): 178.6e6 + 6.4e6}

NOMINAL_FP64_OVER_BF16 = 37.0 / 2250.0   # HGX B200 dense figures: FP64 tensor 37 TF, bf16 2250 TF


def method_flops(m: int, n: int, b: int, steps: int) -> float:
    return float(sum(6.0 * (m - i * b) * n * b + 3.0 * (m - i * b) * b * b for i in range(steps)))


def measured_peaks() -> dict:
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f)
    except Exception:
        return {}


class ClockSampler:
    """nvidia-smi clock / throttle samples while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx = float(f[1])
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def max_over_ranks(ms: float, world: int, device) -> float:
    """Slowest rank's time: every multi-GPU number is the maximum over ranks."""
    if world == 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tflops(flops_per_replica: float, world: int, ms_step: float) -> float:
    """Whole-job rate of `world` independent replicas that all took `ms_step` (the slowest rank's time)."""
    return world * flops_per_replica / (ms_step * 1e-3) / 1e12


def oracle_run(A, Om, w, blocks=None):
    from oracle import rrf_oracle as orc
    max_rank = w.max_rank if blocks is None else min(w.max_rank, blocks * w.b)
    t0 = time.perf_counter()
    r = orc.rrf(A, Om, w.b, w.tol, max_rank)
    dt = time.perf_counter() - t0
    return r, dt


def host_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def generate(w, device):
    """A on the device (or host when device is None) and Omega^T, both in the path's dtype."""
    import torch
    from paper_2608_28941_b200 import workloads as wl
    A, _ = wl.make_matrix(w, device=device)
    Om = wl.make_omega(w).astype(w.np_dtype)
    OmT = np.ascontiguousarray(Om.T)
    if device is not None:
        OmT = torch.from_numpy(OmT).to(device)
    return A, Om, OmT


def run_reference(args, w, rank, world):
    """The oracle, as it stands, timed on the host cores (rank 0 only)."""
    if rank != 0:
        return
    import torch
    dev = "cuda:0" if torch.cuda.is_available() else None
    A, Om, _ = generate(w, dev)
    A = A.cpu().numpy().astype(np.float64) if dev else A.astype(np.float64)
    Om = Om.astype(np.float64)
    # bound the sample: a full run if K+W of them fit in about three minutes, else a prefix of blocks
    _, t_full = oracle_run(A, Om, w, blocks=2)
    est_full = t_full / 2 * (w.max_rank // w.b) * 0.7
    blocks = None
    budget = 180.0 / max(1, args.steps + args.warmup)
    if est_full > budget:
        blocks = max(1, int(budget / (t_full / 2)))
    for _ in range(args.warmup):
        oracle_run(A, Om, w, blocks)
    times, steps_done, r = [], 0, None
    for _ in range(args.steps):
        r, dt = oracle_run(A, Om, w, blocks)
        times.append(dt)
        steps_done = r.steps
    sec = float(np.mean(times))
    tf = method_flops(w.m, w.n, w.b, steps_done) / sec / 1e12
    sample = "full workload" if blocks is None else f"first {steps_done} block steps of the workload"
    line = {"impl": "reference", "metric": "rangefinder_tflops", "value": tf, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
            "config": {"workload": w.name, "m": w.m, "n": w.n, "b": w.b, "tol": w.tol, "max_rank": w.max_rank,
                       "k": r.k, "block_steps": r.steps, "status": r.status, "sample": sample},
            "cpu_baseline": {"value": tf, "unit": "TFLOP/s", "cores": host_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": tf, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


class Problem:
    """One workload resident on the device: inputs, outputs and workspace of rrf_run."""

    def __init__(self, h, w, dev, sched, estimator=0, panel_ctas=0):
        import torch
        from paper_2608_28941_b200 import rrf
        self.h, self.w, self.dev, self.sched, self.estimator, self.panel_ctas = h, w, dev, sched, estimator, panel_ctas
        self.A, self.Om, self.OmT = generate(w, dev)
        self.tdt, self.esize = self.A.dtype, self.A.element_size()
        p = rrf.make_params(rrf.RRF_F64 if w.dtype == "f64" else rrf.RRF_F32, w.m, w.n, w.b, w.tol, w.max_rank)
        self.ws = torch.empty(rrf.rrf_workspace_bytes(p), dtype=torch.uint8, device=dev)
        self.V = torch.empty((w.m, w.max_rank), dtype=self.tdt, device=dev)
        self.T = torch.empty((w.b, w.max_rank), dtype=self.tdt, device=dev)
        self.B = torch.empty((w.max_rank, w.n), dtype=self.tdt, device=dev)

    def step(self, A=None, omegaT="resident", flags=0, out=None):
        from paper_2608_28941_b200 import rrf
        w = self.w
        om = self.OmT if isinstance(omegaT, str) else omegaT
        V, T, B = (self.V, self.T, self.B) if out is None else out
        return rrf.rrf_run(self.h, self.A if A is None else A, w.b, w.tol, w.max_rank, omegaT=om, V=V, T=T,
                           B=B, workspace=self.ws, flags=self.sched | flags, seed=w.seed, estimator=self.estimator, panel_ctas=self.panel_ctas)


def time_problem(pb, steps, warmup, world, barrier):
    """Timed region (the call as a user makes it) and, right after it, the per-kernel event profile."""
    import torch
    from paper_2608_28941_b200 import rrf
    h = pb.h
    rrf.rrf_set_profiling(h, False)
    res = None
    for _ in range(max(warmup, 1)):
        res = pb.step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        res = pb.step()
    e1.record()
    barrier()
    ms_step = max_over_ranks(e0.elapsed_time(e1), world, pb.dev) / steps
    # per-kernel events lengthen a step by several percent, so they are kept out of the timed region
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rrf.rrf_set_profiling(h, True)
    for _ in range(2):
        pb.step()
    prof = {}
    barrier()
    p0.record()
    for _ in range(steps):
        pb.step()
        for name, (ms, cnt) in rrf.rrf_get_profile(h).items():
            a = prof.setdefault(name, [0.0, 0])
            a[0] += ms
            a[1] += cnt
    p1.record()
    barrier()
    rrf.rrf_set_profiling(h, False)
    return res, ms_step, prof, p0.elapsed_time(p1) / steps


def roofline_of(pb, res, prof, steps, value_per_gpu, ms_step, ms_profiled, peaks, local):
    """Roofline of the dominant kernel from the event profile.  `frac` is against the whole device's peak."""
    import torch
    from paper_2608_28941_b200 import rrf
    w, h = pb.w, pb.h
    gemm = {"sample", "vtw", "update"}
    top = max((nm for nm in prof if nm not in ("skipped",)), key=lambda nm: prof[nm][0])
    ms, cnt = prof[top]
    mi = [w.m - i * w.b for i in range(res.steps)]
    kind = 0 if w.dtype == "f64" else 3
    peak = rrf.rrf_measure_peak(h, kind, 200.0)
    if w.dtype == "f32":
        peak /= 3.0                               # three TF32 products per fp32 product
    tc = w.dtype == "f32" and getattr(pb, "f32_engine", "mma") == "tcgen05"
    if top in gemm and tc:
        # Single precision on tcgen05: per 64 KB of W read and written the tensor core needs about half the time
        # HBM does, so HBM is the roof of these kernels.  Algorithmic bytes: the rows of W each launch must read
        # (update: and write back); V, Zt and OmegaT are smaller by n / b and stay in L2.
        hbm = peaks.get("hbm_gbs", 6650.0)
        per_row = {"update": 2.0, "vtw": 1.0, "sample": 1.0}[top] * w.n * pb.esize
        byts = steps * (w.m * per_row if top == "sample" else sum(r * per_row for r in mi))
        achieved = byts / (ms * 1e-3) / 1e9
        work = steps * sum((4.0 if top == "update" else 2.0) * r * w.n * w.b for r in mi)
        sms = torch.cuda.get_device_properties(local).multi_processor_count
        share = (sms - res.panel_ctas) / sms if (res.queues == 2 and top == "update") else 1.0
        tf32 = peaks.get("bf16_tflops", 1590.0) * 0.5 / 3.0
        rl = {"kernel": top, "bound": "hbm", "achieved": achieved, "peak": hbm, "unit": "GB/s",
              "frac": achieved / hbm, "traffic": NCU_TRAFFIC_BYTES.get((w.name, top)),
              "peak_source": "MEASURED_PEAKS.json (of measured)" if "hbm_gbs" in peaks else "of fallback",
              "avg_launch_ms": ms / max(cnt, 1), "launches": cnt, "sm_share": share,
              "tensor_tflops": work / (ms * 1e-3) / 1e12, "tensor_peak_3xtf32": tf32,
              "tensor_peak_source": "bf16 peak x nominal TF32/bf16 ratio / 3 products per fp32 product"}
        peak = tf32
    elif top in gemm:
        work = steps * sum(2.0 * r * w.n * w.b for r in mi)
        if top == "update":                       # the fused kernel also samples a later panel in most passes
            work += steps * sum(2.0 * (r - w.b) * w.n * w.b for r in mi[:res.fused_samples])   # rows below B_i
        if top == "sample":
            work = steps * 2.0 * w.m * w.n * w.b
        achieved = work / (ms * 1e-3) / 1e12
        recipe = peaks.get("bf16_tflops", 1590.0) * NOMINAL_FP64_OVER_BF16 if w.dtype == "f64" else None
        sms = torch.cuda.get_device_properties(local).multi_processor_count
        share = (sms - res.panel_ctas) / sms if (res.queues == 2 and top == "update") else 1.0
        rl = {"kernel": top, "bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
              "frac": achieved / peak, "traffic": NCU_TRAFFIC_BYTES.get((w.name, top)),
              "peak_source": ("FP64 mma.sync rate of the whole device, measured live by rrf_measure_peak" if w.dtype == "f64"
                              else "TF32 mma.sync rate / 3 of the whole device, measured live by rrf_measure_peak"),
              "peak_recipe": recipe, "frac_recipe": achieved / recipe if recipe else None,
              "peak_recipe_source": ("MEASURED_PEAKS.json bf16 x nominal FP64/bf16 ratio (of measured)"
                                     if "bf16_tflops" in peaks else "fallback bf16 x nominal ratio (of fallback)"),
              "avg_launch_ms": ms / max(cnt, 1), "launches": cnt,
              # under the look-ahead schedule the kernel is launched on the SMs the panel kernel leaves it
              "sm_share": share, "frac_of_own_sms": achieved / (peak * share)}
    else:
        hbm = peaks.get("hbm_gbs", 6650.0)
        byts = steps * sum(2.0 * r * w.b * pb.esize for r in mi)
        achieved = byts / (ms * 1e-3) / 1e9
        rl = {"kernel": top, "bound": "hbm", "achieved": achieved, "peak": hbm, "unit": "GB/s",
              "frac": achieved / hbm, "traffic": NCU_TRAFFIC_BYTES.get((w.name, top)),
              "peak_source": "MEASURED_PEAKS.json (of measured)" if "hbm_gbs" in peaks else "of fallback",
              "avg_launch_ms": ms / max(cnt, 1), "launches": cnt}
    rl["whole_step_frac"] = value_per_gpu / peak
    rl["phases_ms_per_step"] = {nm: prof[nm][0] / steps for nm in prof}
    rl["profiled_over"] = ("%d steps right after the timed region, with an event before every kernel "
                           "(%.3f ms per step with the events, %.3f without)" % (steps, ms_profiled, ms_step))
    return rl

def e2e_of(pb, res, steps, world, barrier, flops):
    """The same metric through the C ABI from pinned host memory: every step copies A in and B, V, T out.
    Omega is drawn on the device by the library (seed), so it does not travel."""
    import torch
    from paper_2608_28941_b200 import rrf
    w, dev = pb.w, pb.dev
    A_h = pb.A.cpu().pin_memory()
    B_h = torch.empty((w.max_rank, w.n), dtype=pb.tdt).pin_memory()
    V_h = torch.empty((w.m, w.max_rank), dtype=pb.tdt).pin_memory()
    T_h = torch.empty((w.b, w.max_rank), dtype=pb.tdt).pin_memory()
    # Two device input buffers and two sets of output buffers: the input of step s+1 travels on a copy stream and
    # the results of step s-1 go back on another one while step s computes, as a caller that streams problems
    # through the library would do (the link carries both directions at once).
    A_d = [torch.empty_like(pb.A), torch.empty_like(pb.A)]
    outs = [(pb.V, pb.T, pb.B), (torch.empty_like(pb.V), torch.empty_like(pb.T), torch.empty_like(pb.B))]
    arrived = [torch.cuda.Event(), torch.cuda.Event()]
    returned = [torch.cuda.Event(), torch.cuda.Event()]
    copy_stream = torch.cuda.Stream()
    back_stream = torch.cuda.Stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    # the pinned host-to-device rate on its own, to tell the link from the loop
    barrier()
    e0.record()
    for _ in range(3):
        A_d[0].copy_(A_h, non_blocking=True)
    e1.record()
    barrier()
    h2d_gbs = 3 * A_h.numel() * pb.esize / (e0.elapsed_time(e1) * 1e-3) / 1e9

    def send(slot):
        with torch.cuda.stream(copy_stream):
            A_d[slot].copy_(A_h, non_blocking=True)
            arrived[slot].record(copy_stream)

    def loop(nsteps):
        copy_stream.wait_stream(torch.cuda.current_stream())
        send(0)
        r = None
        for s in range(nsteps):
            slot = s & 1
            if s + 1 < nsteps:
                send(1 - slot)                 # the previous user of that slot has finished: rrf_run synchronises
            torch.cuda.current_stream().wait_event(arrived[slot])
            if s >= 2:
                torch.cuda.current_stream().wait_event(returned[slot])   # this set's results of step s-2 are on the host
            V_d, T_d, B_d = outs[slot]
            r = pb.step(A=A_d[slot], omegaT=None, flags=rrf.RRF_FLAG_NO_GRAPH, out=outs[slot])   # the inputs alternate: nothing to replay
            # rrf_run has synchronised: the results are complete.  B's rows are contiguous; V and T go back whole (a
            # strided copy of their first k columns runs at 2 GB/s, the whole buffers at the link's rate)
            with torch.cuda.stream(back_stream):
                B_h[:r.k].copy_(B_d[:r.k], non_blocking=True)
                V_h.copy_(V_d, non_blocking=True)
                T_h.copy_(T_d, non_blocking=True)
                returned[slot].record(back_stream)
        torch.cuda.current_stream().wait_stream(back_stream)     # the timed region ends when the last results are back
        torch.cuda.current_stream().synchronize()
        return r

    loop(2)
    barrier()
    n_e2e = max(2, min(steps, 12))
    e0.record()
    r = loop(n_e2e)
    e1.record()
    barrier()
    ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / n_e2e
    fl = method_flops(w.m, w.n, w.b, r.steps)
    return {"value": job_tflops(fl, world, ms), "unit": "TFLOP/s", "ms_per_step": ms,
            "h2d_bytes_per_step": int(A_h.numel() * pb.esize),
            "d2h_bytes_per_step": int((r.k * w.n + w.m * w.max_rank + w.b * w.max_rank) * pb.esize),
            "k": r.k, "omega": "drawn on the device from the seed (rrf_fill_omega), not copied",
            "pinned_h2d_gbs_alone": h2d_gbs,
            "pipelined": "the input of step s+1 is copied in on a second stream and the results of step s-1 out on a "
                         "third while step s computes; %d steps timed, first copy in and last copy out not overlapped" % n_e2e}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--m", type=int, default=0, help="override the workload's rows (profiling captures)")
    ap.add_argument("--n", type=int, default=0, help="override the workload's columns")
    ap.add_argument("--max-rank", type=int, default=0, help="override the workload's rank cap")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="skip the short runs of the other four configurations")
    ap.add_argument("--schedule", default="auto", choices=["auto", "one", "two"],
                    help="one queue (sequential), two queues (look-ahead), or the library's own rule")
    ap.add_argument("--panel", default="column", choices=["column", "blocked", "tree"],
                    help="panel kernel: column by column (default), blocked in micro-panels of eight, or the tree kernel (b <= 64)")
    ap.add_argument("--variant", default="in-place", choices=["in-place", "no-update"],
                    help="no-update: A is left unchanged and B is not formed (one pass over A per block instead of "
                         "three); stops on the sampled Frobenius estimate.  Flops are counted as the in-place schedule's")
    ap.add_argument("--estimator", type=int, default=0, choices=[0, 1, 2, 3])
    ap.add_argument("--f32-engine", default="tcgen05", choices=["mma", "tcgen05"],
                    help="tensor-core path of the single-precision V^T W product")
    ap.add_argument("--tc-chunk", type=int, default=2,
                    help="tcgen05: 64-row tiles summed in tensor memory between round-to-nearest adds (0: all)")
    ap.add_argument("--panel-ctas", type=int, default=0, help="look-ahead schedule: SMs given to the panel chain (0: library's rule)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    from paper_2608_28941_b200 import workloads as wl
    w = wl.CONFIGS[args.workload]
    custom = bool(args.m or args.n or args.max_rank)
    if custom:
        w = w.scaled(args.m or w.m, args.n or w.n, max_rank=args.max_rank or w.max_rank)

    if args.impl == "reference":
        run_reference(args, w, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2608_28941_b200 import build as _build, rrf

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()
    h = rrf.rrf_create(local)
    rrf.rrf_set_single_engine(h, 1 if args.f32_engine == "tcgen05" else 0, args.tc_chunk)
    sched = {"auto": 0, "one": rrf.RRF_FLAG_ONE_QUEUE, "two": rrf.RRF_FLAG_TWO_QUEUES}[args.schedule]
    if args.panel == "tree":
        sched |= rrf.RRF_FLAG_PANEL_TREE
    if args.panel == "blocked":
        sched |= rrf.RRF_FLAG_PANEL_BLOCKED

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    estimator = args.estimator
    if args.variant == "no-update":
        sched = rrf.RRF_FLAG_NO_UPDATE
        estimator = estimator if estimator >= 2 else 2
        args.no_e2e = True
        args.no_per_config = True
    peaks = measured_peaks()
    pb = Problem(h, w, dev, sched, estimator, args.panel_ctas)
    pb.f32_engine = args.f32_engine
    sampler = ClockSampler(local)
    pb.step()
    barrier()
    sampler.start()
    res, ms_step, prof, ms_profiled = time_problem(pb, args.steps, args.warmup, world, barrier)
    clocks = sampler.stop()
    flops = method_flops(w.m, w.n, w.b, res.steps)
    value = job_tflops(flops, world, ms_step)
    launches = args.steps * res.kernel_launches      # counted by the library: every kernel it put on the device

    e2e = None if args.no_e2e else e2e_of(pb, res, args.steps, world, barrier, flops)
    roofline = roofline_of(pb, res, prof, args.steps, value / world, ms_step, ms_profiled, peaks, local) if rank == 0 else None

    # ---- CPU baseline: the oracle on the host cores (rank 0, single-GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        A64 = pb.A.cpu().numpy().astype(np.float64)
        Om64 = pb.Om.astype(np.float64)
        _, t2 = oracle_run(A64, Om64, w, blocks=2)
        est = t2 / 2 * (w.max_rank // w.b)
        blocks = None if est < 40 else max(1, int(25.0 / (t2 / 2)))
        r, dt = oracle_run(A64, Om64, w, blocks)
        cpu = {"value": method_flops(w.m, w.n, w.b, r.steps) / dt / 1e12, "unit": "TFLOP/s", "cores": host_threads(),
               "kind": "oracle", "seconds": dt, "k": r.k,
               "sample": "full workload, one run" if blocks is None else f"first {r.steps} block steps, one run"}
        del A64, Om64

    # ---- the other configurations, briefly: time, rate, fraction of the peak, dominant kernel
    per_config = None
    if rank == 0 and world == 1 and not custom and not args.no_per_config:
        del pb
        torch.cuda.empty_cache()
        per_config = []
        for name in ("cfg1", "cfg2", "cfg3", "cfg4", "cfg5"):
            if name == w.name:
                continue
            wc = wl.CONFIGS[name]
            n_steps = 3 if name == "cfg5" else 10
            pc = Problem(h, wc, dev, sched)
            pc.f32_engine = args.f32_engine
            r, ms, pr, msp = time_problem(pc, n_steps, 3, 1, barrier)
            v = job_tflops(method_flops(wc.m, wc.n, wc.b, r.steps), 1, ms)
            rl = roofline_of(pc, r, pr, n_steps, v, ms, msp, peaks, local)
            per_config.append({"workload": name, "dtype": wc.dtype, "m": wc.m, "n": wc.n, "b": wc.b, "tol": wc.tol,
                               "max_rank": wc.max_rank, "k": r.k, "block_steps": r.steps, "status": r.status,
                               "queues": r.queues, "panel_ctas": r.panel_ctas, "steps_timed": n_steps,
                               "ms_per_step": ms, "tflops": v, "peak_tflops": rl["peak"] if rl["bound"] == "tensor" else None,
                               "whole_step_frac": rl["whole_step_frac"], "dominant_kernel": rl["kernel"],
                               "dominant_bound": rl["bound"], "dominant_frac": rl["frac"],
                               "phases_ms_per_step": rl["phases_ms_per_step"]})
            del pc
            torch.cuda.empty_cache()

    if rank == 0:
        esize = 8 if w.dtype == "f64" else 4
        line = {"metric": "rangefinder_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
                "config": {"workload": w.name, "m": w.m, "n": w.n, "b": w.b, "tol": w.tol, "max_rank": w.max_rank,
                           "k": res.k, "block_steps": res.steps, "status": res.status,
                           "l2": "inputs larger than L2 (A is %.0f MB)" % (w.m * w.n * esize / 1e6),
                           "queues": res.queues, "panel_ctas": res.panel_ctas, "panel_kernel": args.panel,
                           "variant": args.variant, "estimator": estimator,
                           "passes_over_A_per_block": 1 if args.variant == "no-update" else 3,
                           "fused_samples": res.fused_samples, "extra_samples": res.extra_samples,
                           "parallelism": "replicas only" if world > 1 else "single GPU"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
                "roofline": roofline, "cpu_baseline": cpu, "per_config": per_config}
        print(json.dumps(line))
    rrf.rrf_destroy(h)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
