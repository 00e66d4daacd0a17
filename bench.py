#!/usr/bin/env python
"""Benchmark of the SF hot path: `python bench.py --gpus N --steps K --warmup W [--impl reference]`.

A step is one pass of the whole path (factor computation -> SF buffer -> rank-K apply, i.e. one
`sfb_step`) over one synthetic minibatch of the named workload.  Prints ONE JSON line (rank 0).

* `value`: SF-step samples/s with inputs resident in HBM, device-timed (CUDA events), max over ranks.
* `e2e`: the same metric with the step's inputs copied from pinned host memory and a result read
  back to the host inside the timed region, all through the C ABI.
* `roofline`: the dominant kernel (the rank-K apply) against the measured peak for its bound.
* `cpu_baseline`: the fp64 oracle, as it stands, on a bounded sample on the host cores.
* `--impl reference`: times the oracle (the only reference implementation there is) instead.

With N > 1 (torchrun) every rank runs an independent replica of the workload ("replicas only": the
path has no exchange step on one node because the P workers are simulated inside one SF buffer).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "SF-step samples/s"
UNIT = "samples/s"
SMEM_TBS = 148 * 128 * 1.965e9 / 1e12           # shared-memory load path of the whole chip
L2_TBS = 24.5                                   # L2 read rate at which ncu reports lts__throughput = 100 % (17.9 TB/s at 73 %)
DATASHEET_BF16_TFLOPS = 2250.0
FP32_FMA_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12     # 148 SMs x 128 lanes x 2 flop x max SM clock
ORACLE_IMPL = "fp64 numpy oracle (contractions on the host BLAS), as it stands"
# A timed region shorter than this finishes before the power controller settles: the burst peak is its denominator;
# a longer one runs under the power cap and is compared with the sustained peak.
BURST_REGION_S = 1.0


def tensor_peak(peaks, path, region_s):
    """(peak TFLOP/s, label) for a tensor-core kernel timed inside a region of `region_s` seconds."""
    # tf32 nominal rate is half of bf16; the compensated path spends, per algorithmic product, one tf32 product and
    # one bf16 product of twice the reduction length (as long as a tf32 one): two tf32 products' worth
    scale = {"bf16": 1.0, "tf32": 0.5, "tf32x3": 0.5 / 2.0}[path]
    kind = "burst" if region_s < BURST_REGION_S else "sustained"
    base = peaks["bf16"] if kind == "burst" else peaks["bf16_sustained"]
    label = (f"{peaks['source']} cuBLAS bf16 {kind} ({base:.1f})" + {"bf16": "", "tf32": " x 0.5 (tf32)", "tf32x3": " x 0.5 (tf32) / 2 (a tf32 product and a bf16 correction product of the same length per multiply-add)"}[path] +
             f": timed region {region_s * 1e3:.0f} ms")
    return base * scale, label, scale


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self._stop, self._t = index, [], threading.Event(), None

    def _run_nvml(self) -> bool:
        """Fast sampling through NVML (read-only queries); returns False if NVML is unavailable."""
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            mx = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            bits = [(nv.nvmlClocksEventReasonHwSlowdown, "hw_slowdown"),
                    (nv.nvmlClocksEventReasonHwThermalSlowdown, "hw_thermal_slowdown"),
                    (nv.nvmlClocksEventReasonSwThermalSlowdown, "sw_thermal_slowdown"),
                    (nv.nvmlClocksEventReasonSwPowerCap, "sw_power_cap")]
        except Exception:
            return False
        while not self._stop.is_set():
            try:
                sm = nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)
                pw = nv.nvmlDeviceGetPowerUsage(h) / 1000.0
                rs = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                self.rows.append([str(sm), str(mx), str(pw)] + ["Active" if rs & b else "Not Active" for b, _ in bits])
            except Exception:
                pass
            self._stop.wait(0.005)
        return True

    def _run(self):
        if self._run_nvml():
            return
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                      "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
                self.rows.append([c.strip() for c in out.strip().split(",")])
            except Exception:
                pass
            self._stop.wait(0.2)

    def __enter__(self):
        self._t = threading.Thread(target=self._run, daemon=True)
        self._t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._t.join(timeout=6)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def algorithmic(cfg, path, inputs=None):
    """Flops / bytes one apply launch must do (what the roofline fraction is computed from).

    Dense apply: 2*J*D*K flop; bytes = W read + W write (+ bf16 shadow) + the K (u, v) pairs.
    Sparse-v scatter apply (SC, fp32 path): 2*J*nnz flop; bytes = W read + W write + U + CSR codes.
    """
    J, D, K = cfg["J"], cfg["D"], cfg["K"]
    es = 2 if path == "bf16" else 4
    if cfg["model"] == "sc" and path == "f32":
        nnz = int(inputs["rowptr"][0][-1]) if inputs is not None else int(cfg["density"] * K * D)
        return dict(flops=2.0 * J * nnz, bytes=2.0 * J * D * 4 + K * J * 4 + nnz * 8.0, sparse=True)
    flops = 2.0 * J * D * K
    bytes_ = 2.0 * J * D * 4 + K * (J + D) * es + (J * D * 2 if path == "bf16" else 0)
    return dict(flops=flops, bytes=bytes_, sparse=False)


# dram__bytes_read.sum + dram__bytes_write.sum of one apply launch, from the ncu captures summarised
# under profiles/ (captured at J = 8192 and scaled by J where the full launch is too large to capture).
NCU_APPLY_TRAFFIC_BYTES = {("C4", "bf16"): 4.03e9, ("C3", "f32"): 6.28e8, ("C1", "tf32"): 2.03e8, ("C2", "tf32"): 1.21e8,
                           ("C1", "f32"): 3.39e8, ("C2", "f32"): 1.95e8}


def oracle_step_time(cfg, inputs, sample_workers: int):
    """Seconds of one oracle step (factors + apply) on the first `sample_workers` workers' samples."""
    from oracle import sfb_oracle as orc
    from sfbgen import batch_of
    model_id = {"mlr": orc.MODEL_MLR, "dml": orc.MODEL_DML, "sc": orc.MODEL_SC}[cfg["model"]]
    n = sample_workers * cfg["B"]
    b = batch_of(inputs, cfg, 0)
    if cfg["model"] == "sc":
        rp = b["rowptr"][:n + 1]
        b = dict(rowptr=rp, idx=b["idx"][:rp[-1]], val=b["val"][:rp[-1]], Xdata=b["Xdata"][:n])
    else:
        b = {k: (v[:n] if hasattr(v, "shape") and v.shape[0] == cfg["K"] else v) for k, v in b.items()}
    t0 = time.perf_counter()
    orc.step(model_id, inputs["W"], b, cfg["eta"], cfg.get("margin", 1.0))
    return time.perf_counter() - t0, n


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def pick_sample_workers(cfg, budget=1.5e12):
    """Workers whose samples make up the oracle's bounded sample.

    budget: fp64 flops of one sampled oracle step.  The reference arm repeats the step `--steps` times, so it
    takes the default (a few seconds per step on the GPU machine's host); the cpu_baseline leg times ONE step and
    asks for more (10-30 s).  The sparse-coding oracle spends its time in per-sample scatter loops, not flops:
    a quarter of the workers there.
    """
    if cfg["model"] == "sc":
        return max(1, cfg["P"] // 4)
    flops_per_worker = 4.0 * cfg["J"] * cfg["D"] * cfg["B"]           # forward + apply, fp64
    return int(max(1, min(cfg["P"], budget // max(flops_per_worker, 1.0))))


def run_reference(args, cfg, inputs):
    """The oracle as the reference arm: each step is one oracle step on a bounded sample."""
    sw = pick_sample_workers(cfg)
    for _ in range(min(args.warmup, 1)):
        oracle_step_time(cfg, inputs, sw)
    t, n = 0.0, 0
    for _ in range(args.steps):
        dt, n = oracle_step_time(cfg, inputs, sw)
        t += dt
    value = n * args.steps / t
    cores = blas_threads()
    sample = f"{sw} of {cfg['P']} workers' samples ({n} of {cfg['K']}) of minibatch 0 at full J x D, per step"
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg, cfg["path"]), "arithmetic": "fp64 CPU oracle on a bounded sample"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "implementation": ORACLE_IMPL, "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }


def max_over_ranks(values, device=None):
    """Element-wise maximum of `values` over all ranks (identity when not distributed)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_throughput(units_per_rank_step, steps, ms, world):
    """Units all ranks processed divided by the (max over ranks) time: replicas => weak scaling."""
    return world * units_per_rank_step * steps / (ms * 1e-3)


def workload_name(cfg, path):
    dens = f" density={cfg['density']}" if cfg["model"] == "sc" else ""
    return (f"{cfg['name']} {cfg['model'].upper()} J={cfg['J']} D={cfg['D']} P={cfg['P']} B={cfg['B']} "
            f"K={cfg['K']}{dens} path={path}")


def run_bsp(args, cfg, inputs, wl, path, rank, world, local_rank, barrier):
    """One job over all ranks: rank r computes the factors of its P / world workers, the worker streams are
    all-gathered in place (NCCL), every rank applies all K pairs to its own copy of W.  K samples per step in
    total, whatever the number of ranks (strong scaling)."""
    import torch
    from paper_1511_08486_b200.bsp import BspSfb, exchange_bytes
    from paper_1511_08486_b200.workload import shard_batch
    dev = wl.W.device
    stream = torch.cuda.current_stream()
    K, eta = cfg["K"], cfg["eta"]
    bsp = BspSfb(wl.ctx, wl.desc, wl.sf_buf)
    shards = [shard_batch(t, cfg["model"], bsp.first, bsp.n_workers, cfg["B"]) for t in wl.batches]
    step_bytes = 4.0 * cfg["J"] * cfg["D"] + wl.ctx.sf_buffer_bytes
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if step_bytes < (252 << 20) else None

    def step(t):
        s = shards[t % wl.pool]
        bsp.step(wl.W, s["X"], s["aux"], eta, clock=t)

    wl.reset()
    for t in range(max(args.warmup, 3)):
        step(t)
    barrier()
    l0 = wl.ctx.launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    ms = 0.0
    with ClockSampler(local_rank) as clocks:
        if flush is None:
            ev[0].record(stream)
            for t in range(args.steps):
                step(args.warmup + t)
            ev[1].record(stream)
            barrier()
            ms = ev[0].elapsed_time(ev[1])
        else:
            for t in range(args.steps):
                flush.fill_(t & 1)
                barrier()
                ev[0].record(stream)
                step(args.warmup + t)
                ev[1].record(stream)
                torch.cuda.synchronize()
                ms += ev[0].elapsed_time(ev[1])
            barrier()
    launches = wl.ctx.launch_count() - l0
    status = wl.ctx.status()

    # stages, timed apart: factors of the shard / exchange / header + apply
    from paper_1511_08486_b200.bsp import all_gather_streams
    st = [0.0, 0.0, 0.0]
    nprof = min(args.steps, 16)
    for t in range(nprof):
        s = shards[t % wl.pool]
        barrier()
        ev[0].record(stream)
        wl.ctx.factors_shard(wl.W, s["X"], s["aux"], wl.sf_buf, bsp.first, bsp.n_workers)
        ev[1].record(stream)
        if bsp.in_group:
            all_gather_streams(wl.sf_buf, bsp.streams_off, bsp.stream_stride, cfg["P"])
        ev[2].record(stream)
        wl.ctx.commit_header(wl.sf_buf, t)
        wl.ctx.apply(wl.W, wl.sf_buf, eta)
        ev[3].record(stream)
        torch.cuda.synchronize()
        for k in range(3):
            st[k] += ev[k].elapsed_time(ev[k + 1]) / nprof

    # end to end: the shard's minibatch starts in pinned host memory, the committed header comes back
    host = [{k: v.cpu().pin_memory() for k, v in s.items() if isinstance(v, torch.Tensor)} for s in shards]
    stage = [{k: torch.empty_like(v, device=dev) for k, v in h.items()} for h in host]
    from paper_1511_08486_b200 import binding as Bd
    stage_aux = [Bd.make_aux(**{k: v for k, v in sg.items() if k != "X"}) for sg in stage]
    h2d = sum(v.numel() * v.element_size() for v in host[0].values())
    header = torch.empty(128, dtype=torch.uint8).pin_memory()

    def e2e_step(t):
        b = t % wl.pool
        for k, v in host[b].items():
            stage[b][k].copy_(v, non_blocking=True)
        bsp.step(wl.W, stage[b].get("X"), stage_aux[b], eta, clock=t)
        header.copy_(wl.sf_buf[:128], non_blocking=True)
    for t in range(3):
        e2e_step(t)
    barrier()
    ev[0].record(stream)
    for t in range(args.steps):
        e2e_step(args.warmup + t)
    ev[1].record(stream)
    barrier()
    e2e_ms = ev[0].elapsed_time(ev[1])
    ms, e2e_ms, st[0], st[1], st[2] = max_over_ranks([ms, e2e_ms, st[0], st[1], st[2]], device=dev)
    if rank != 0:
        return None
    peaks = load_peaks()
    alg = algorithmic(cfg, path, inputs)
    xb = exchange_bytes(cfg["P"], world, bsp.stream_stride)
    out = {
        "metric": METRIC, "value": whole_job_throughput(K, args.steps, ms, 1), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "strong", "vs_baseline": None, "dtype": path, "data": "synthetic",
        "config": {"workload": workload_name(cfg, path), "parallelism": f"bsp sfb: {cfg['P']} workers over {world} gpu(s)",
                   "l2": "per-step footprint larger than L2" if flush is None else "L2 flushed between steps",
                   "eta": eta, "pool": cfg["pool"]},
        "e2e": {"value": whole_job_throughput(K, args.steps, e2e_ms, 1), "unit": UNIT, "h2d_bytes_per_step": h2d * world,
                "d2h_bytes_per_step": 128 * world},
        "gpu_launches": int(launches), "device_status": status,
        "stages_ms": {"factors": st[0], "exchange": st[1], "apply": st[2], "steps_recorded": nprof},
        "exchange_bytes_per_step": xb,
        "clocks": clocks.summary(),
    }
    if alg is not None and not alg["sparse"] and path != "f32":
        peak, label, _ = tensor_peak(peaks, path, ms * 1e-3)
        tf = alg["flops"] / (st[2] * 1e-3) / 1e12
        out["roofline"] = {"bound": "tensor", "achieved": tf, "peak": peak, "unit": "TFLOP/s", "frac": tf / peak,
                           "traffic": None, "kernel": "umma_gemm_kernel (apply)", "peak_source": label}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="C4")
    ap.add_argument("--path", default=None, help="f32 | tf32 | bf16 (default: the configuration's own)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--graph", action="store_true",
                    help="record sfb_step into one CUDA graph per pool minibatch and replay it (launch-bound small "
                         "configurations; the header's clock is then the recorded one)")
    ap.add_argument("--mode", default="replicas", choices=["replicas", "bsp"],
                    help="N > 1: independent replicas of the whole path (default), or ONE job whose P workers are split "
                         "over the ranks with an all-gather of the worker streams per step (sufficient factor broadcasting)")
    for dim in ("J", "D", "P", "B"):
        ap.add_argument(f"--{dim}", type=int, default=None, help=f"override {dim} (smaller cases for profiler captures)")
    ap.add_argument("--compact", action="store_true",
                    help="leave pairs whose u is zero out of the SF buffer (DML: dissimilar pairs beyond the margin)")
    ap.add_argument("--density", type=float, default=None,
                    help="sparse coding: fraction of nonzeros in the codes (default: the configuration's 5 %%)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    from sfbgen import get_config, make_inputs
    cfg = get_config(args.config)
    over = {k: getattr(args, k) for k in ("J", "D", "P", "B") if getattr(args, k) is not None}
    if args.density is not None:
        over["density"] = args.density
    if over:
        from sfbgen import scaled
        cfg = scaled(args.config, **over)
    path = args.path or cfg["path"]
    if args.compact:
        cfg["compact"] = 1

    if args.impl == "reference":
        if rank == 0:
            inputs = make_inputs(cfg)
            print(json.dumps(run_reference(args, cfg, inputs)), flush=True)
        return

    import torch
    import torch.distributed as dist
    from paper_1511_08486_b200.build import build_library
    from paper_1511_08486_b200.workload import DeviceWorkload

    build_library()
    torch.cuda.set_device(local_rank)
    in_group = world > 1 or (args.mode == "bsp" and "RANK" in os.environ)   # bsp under a launcher: NCCL even for one rank
    if in_group:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    inputs = make_inputs(cfg)
    if args.graph:            # capture needs a stream of its own; the context takes the current stream
        torch.cuda.set_stream(torch.cuda.Stream(device=dev))
    wl = DeviceWorkload(cfg, inputs, path=path, device=dev)
    K, eta = cfg["K"], cfg["eta"]
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.mode == "bsp":
        out = run_bsp(args, cfg, inputs, wl, path, rank, world, local_rank, barrier)
        if rank == 0:
            print(json.dumps(out), flush=True)
        wl.close()
        if in_group:
            dist.destroy_process_group()
        return

    # L2 flush buffer for workloads whose per-step footprint is below L2
    step_bytes = 4.0 * cfg["J"] * cfg["D"] + wl.ctx.sf_buffer_bytes
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if step_bytes < (252 << 20) else None

    graphs = []

    def one_step(t):
        if graphs:
            graphs[t % wl.pool].replay()
        else:
            wl.step(t, eta=eta)

    def run_steps(n, t0=0):
        for t in range(n):
            if flush is not None:
                flush.fill_(t & 1)
            one_step(t0 + t)

    # ---- device-resident timing ----------------------------------------------------------------
    wl.reset()
    run_steps(max(args.warmup, 3))
    barrier()
    if args.graph and args.mode == "replicas":
        for b in range(wl.pool):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                wl.step(b, eta=eta)
            graphs.append(g)
        launches_per_step = wl.ctx.launch_count()
        wl.step(0, eta=eta)
        launches_per_step = wl.ctx.launch_count() - launches_per_step      # what one replay launches
        run_steps(3)
        barrier()
    # Stage times come from events recorded inside sfb_step.  When a step is long enough for three event records
    # not to matter (>= 0.2 ms) they are recorded in the SAME pass that gives `value`, so factors + apply add up
    # to ms_per_step and share its power state; for launch-bound steps a second pass records them.
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    run_steps(3, t0=args.warmup)
    ev1.record(stream)
    barrier()
    probe_ms = ev0.elapsed_time(ev1) / 3.0
    stages_same_pass = (not graphs) and probe_ms >= 0.2 and args.steps <= 128
    if stages_same_pass:
        wl.ctx.profile(True)
    l0 = wl.ctx.launch_count()
    with ClockSampler(local_rank) as clocks:
        if flush is None:
            ev0.record(stream)
            run_steps(args.steps, t0=args.warmup)
            ev1.record(stream)
            barrier()
            ms = ev0.elapsed_time(ev1)
        else:   # time each step alone so the flush is outside the timed spans
            ms = 0.0
            for t in range(args.steps):
                flush.fill_(t & 1)
                ev0.record(stream)
                one_step(args.warmup + t)
                ev1.record(stream)
                torch.cuda.synchronize()
                ms += ev0.elapsed_time(ev1)
            barrier()
    launches = wl.ctx.launch_count() - l0 if not graphs else launches_per_step * args.steps
    if stages_same_pass:
        f_ms, a_ms, n_rec = wl.ctx.stage_ms()
        wl.ctx.profile(False)
    status = wl.ctx.status()
    graphs_used = bool(graphs)
    graphs.clear()            # stages and the end-to-end leg below run eagerly

    if not stages_same_pass:
        wl.ctx.profile(True)
        nprof = min(args.steps, 128)
        run_steps(nprof, t0=args.warmup)
        f_ms, a_ms, n_rec = wl.ctx.stage_ms()
        wl.ctx.profile(False)
    f_ms, a_ms = f_ms / max(n_rec, 1), a_ms / max(n_rec, 1)

    # ---- end to end: host buffers in, result out, inside the timed region ------------------------
    host_batches = []
    for t in wl.batches:
        hb = {k: v.cpu().pin_memory() for k, v in t.items() if isinstance(v, torch.Tensor)}
        host_batches.append(hb)
    h2d = sum(v.numel() * v.element_size() for v in host_batches[0].values())
    result_host = torch.empty(128, dtype=torch.uint8).pin_memory()
    d2h = result_host.numel()

    from paper_1511_08486_b200 import binding as Bd
    host_aux = [Bd.make_aux(**{k: v for k, v in hb.items() if k != "X"}) for hb in host_batches]

    def e2e_step(t):   # one C-ABI call: host inputs in, step, committed header (clock, shapes) back to the host
        b = t % wl.pool
        wl.ctx.step_host(wl.W, host_batches[b].get("X"), host_aux[b], wl.sf_buf, eta, clock=t, header_host=result_host)
    for t in range(3):
        e2e_step(t)
    barrier()
    ev0.record(stream)
    for t in range(args.steps):
        e2e_step(args.warmup + t)
    ev1.record(stream)
    barrier()
    e2e_ms = ev0.elapsed_time(ev1)
    clock_of_last = int(np.frombuffer(result_host.numpy().tobytes(), dtype=np.uint32)[7])

    # ---- max over ranks ---------------------------------------------------------------------------
    ms, e2e_ms = max_over_ranks([ms, e2e_ms], device=dev)

    if rank == 0:
        peaks = load_peaks()
        alg = algorithmic(cfg, path, inputs)
        value = whole_job_throughput(K, args.steps, ms, world)
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": {"f32": "f32", "tf32": "tf32", "bf16": "bf16", "tf32x3": "tf32x3 (fp32 operands: tf32 product + bf16 correction product, fp32 accumulate)"}[path],
            "data": "synthetic",
            "config": {"workload": workload_name(cfg, path), "parallelism": f"replicas x{world}" if world > 1 else "1 gpu",
                       "l2": "per-step footprint larger than L2" if flush is None else "L2 flushed between steps",
                       "eta": eta, "pool": cfg["pool"], "cuda_graph": graphs_used, "compact": bool(cfg.get("compact", 0))},
            "e2e": {"value": whole_job_throughput(K, args.steps, e2e_ms, world), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "last_clock_read_back": clock_of_last,
                    "returned": "the 128-byte header the step committed (clock, shapes); W (the worker's local copy of "
                                "the parameters) and the SF buffer stay resident on the device by design"},
            "gpu_launches": int(launches),
            "device_status": status,
            "stages_ms": {"factors": f_ms, "apply": a_ms, "steps_recorded": n_rec,
                          "pass": "the timed region of `value`" if stages_same_pass else "a second pass after it"},
            "clocks": clocks.summary(),
        }
        # the message of the last step: what a full broadcast (every worker to P - 1 peers) would put on the wire,
        # next to what synchronising the full matrix through a server would (push + pull of J x D per worker)
        P_ = cfg["P"]
        sent = wl.ctx.wire_bytes(wl.sf_buf)
        es_ = 2 if path == "bf16" else 4
        out["wire"] = {"sf_buffer_bytes_sent": sent, "compacted": bool(cfg.get("compact", 0)),
                       "full_broadcast_bytes": (P_ - 1) * sent,
                       "full_matrix_sync_bytes": 2 * P_ * cfg["J"] * cfg["D"] * es_}
        applied = wl.ctx.active_pairs()
        if alg is not None and 0 < applied < K:
            # the apply left out pairs whose u is zero: its work is counted on the pairs it multiplied through
            alg["flops_all_pairs"] = alg["flops"]
            out["pairs_applied_last_step"] = applied
        if alg is not None:
            apply_tflops = alg["flops"] * (applied / K if 0 < applied < K else 1.0) / (a_ms * 1e-3) / 1e12
            fwd_tflops = alg["flops"] / (f_ms * 1e-3) / 1e12
            traffic = NCU_APPLY_TRAFFIC_BYTES.get((args.config, path)) if not over else None
            if alg["sparse"]:
                gbs = alg["bytes"] / (a_ms * 1e-3) / 1e9
                out["roofline"] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                   "frac": gbs / peaks["hbm_gbs"], "traffic": traffic, "kernel": "csc_apply_kernel",
                                   "peak_source": f"{peaks['source']} HBM copy bandwidth"}
                # what the counters show as the limiter: every multiply-add takes 4 bytes of u from shared memory
                smem_tbs = 2.0 * alg["flops"] / (a_ms * 1e-3) / 1e12
                out["roofline"]["secondary"] = {"bound": "shared-memory operand reads", "achieved": smem_tbs,
                                                "peak": SMEM_TBS, "unit": "TB/s", "frac": smem_tbs / SMEM_TBS,
                                                "peak_source": "148 SMs x 128 B/clk x 1.965 GHz"}
            elif path == "f32":
                out["roofline"] = {"bound": "alu", "achieved": apply_tflops, "peak": FP32_FMA_TFLOPS, "unit": "TFLOP/s",
                                   "frac": apply_tflops / FP32_FMA_TFLOPS, "traffic": traffic,
                                   "kernel": "sgemm_pipe_kernel<0> (apply)", "peak_source": "148 SMs x 128 FMA lanes x 1.965 GHz"}
            else:
                # the apply is ONE launch per step: its launch duration is the apply stage's event span
                peak, label, scale = tensor_peak(peaks, path, ms * 1e-3)
                out["roofline"] = {"bound": "tensor", "achieved": apply_tflops, "peak": peak, "unit": "TFLOP/s",
                                   "frac": apply_tflops / peak, "traffic": traffic, "kernel": "umma_gemm_kernel (apply)",
                                   "peak_source": label,
                                   "frac_of_burst": apply_tflops / (peaks["bf16"] * scale),
                                   "frac_of_sustained": apply_tflops / (peaks["bf16_sustained"] * scale),
                                   "frac_of_datasheet": apply_tflops / (DATASHEET_BF16_TFLOPS * scale)}
            out["apply_tflops"] = apply_tflops
            out["forward_tflops"] = fwd_tflops
            # the factor stage (forward contraction + finishing passes) against the bound of its contraction
            if alg["sparse"]:
                l2_tbs = 2.0 * alg["flops"] / (f_ms * 1e-3) / 1e12     # every multiply-add gathers 4 bytes of W from L2
                out["roofline_factors"] = {"bound": "l2", "achieved": l2_tbs, "peak": L2_TBS, "unit": "TB/s",
                                           "frac": l2_tbs / L2_TBS, "kernel": "sc_forward_kernel",
                                           "peak_source": "ncu: 17.9 TB/s of L2 reads at lts__throughput 73 %"}
            elif path == "f32":
                out["roofline_factors"] = {"bound": "alu", "achieved": fwd_tflops, "peak": FP32_FMA_TFLOPS,
                                           "unit": "TFLOP/s", "frac": fwd_tflops / FP32_FMA_TFLOPS,
                                           "kernel": "fp32 forward kernels + finishing pass"}
            else:
                peak, label, scale = tensor_peak(peaks, path, ms * 1e-3)
                out["roofline_factors"] = {"bound": "tensor", "achieved": fwd_tflops, "peak": peak,
                                           "unit": "TFLOP/s", "frac": fwd_tflops / peak, "peak_source": label,
                                           "kernel": "umma_gemm_kernel (forward) + finishing pass"}
        if not args.no_cpu_baseline:
            sw = pick_sample_workers(cfg, budget=6e12)
            dt, n = oracle_step_time(cfg, inputs, sw)
            out["cpu_baseline"] = {"value": n / dt, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                   "implementation": ORACLE_IMPL,
                                   "sample": f"one oracle step on {sw} of {cfg['P']} workers' samples ({n} of {K}) at full J x D, {dt:.1f} s"}
        print(json.dumps(out), flush=True)
    wl.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
