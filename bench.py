#!/usr/bin/env python
"""Benchmark of the local-update SGD hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME] [--tau T]

One timed "step" is one communication period of the whole path on the
workload's m replicas: tau local SGD(-momentum) iterations on every replica
(forward, loss, backward, fused update), one model-averaging step, one
evaluation of the synchronized model's training loss on the probe block and
one AdaComm decision.  The metric is replica-steps/s = m * tau * K / time.

Prints ONE JSON line (rank 0).  With --gpus N > 1 (launched by torchrun) every
rank runs an independent copy of the job (the path keeps all replicas of one
job on one GPU and has no cross-GPU step), time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1810_08313_b200 import workloads as wl  # noqa: E402

METRIC = "replica-steps/s (m-replica local SGD); model-avg HBM GB/s vs ~8 TB/s peak"
UNIT = "replica-steps/s"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_BF16_TFLOPS = 2250.0       # dense bf16 tensor peak of the data sheet (context beside the measured peaks)
PROBE_ROWS = 4096


# --------------------------------------------------------------------------
# helpers with no GPU dependency (covered by CPU tests)
# --------------------------------------------------------------------------

def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p.get("bf16_tflops", 0.0)),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", 0.0)), "source": "measured"}
    except Exception:
        return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
                "source": "fallback"}


def workload_config(w: wl.Workload, tau: int) -> dict:
    """The keys of `config` that name the workload; both arms (CUDA and CPU oracle) print the same ones."""
    return {"workload": w.name, "dims": list(w.dims), "m": w.m, "batch": w.batch, "tau": tau,
            "momentum": w.momentum, "lr": w.lr, "dataset_rows": w.n_rows}


def probe_rows_for(w: wl.Workload) -> int:
    n = min(PROBE_ROWS, w.n_rows)
    return max(w.batch, n // w.batch * w.batch)


def layer_shapes(w: wl.Workload):
    return [(w.dims[l + 1], w.dims[l]) for l in range(len(w.dims) - 1)]


def flops_per_replica_step(w: wl.Workload) -> float:
    """forward + weight gradient for every layer, data gradient for all but the first."""
    f = 0.0
    for l, (n_out, n_in) in enumerate(layer_shapes(w)):
        f += 2.0 * w.batch * n_out * n_in * (2 if l == 0 else 3)
    return f


def streamed_update_layers(w: wl.Workload):
    """Layers whose weight update runs on the streaming tensor-core kernel: all of them go into one launch."""
    bf = w.gemm_dtype == "bf16"
    out = []
    for l, (n_out, n_in) in enumerate(layer_shapes(w)):
        last = l == len(w.dims) - 2
        if last and n_out <= 16:
            continue
        if n_out % 128 == 0 and n_in % 128 == 0 and w.batch % (64 if bf else 32) == 0:
            out.append(l)
    return out


def update_state_bytes_per_launch(w: wl.Workload, layer: int) -> float:
    """Bytes of replica state the weight-gradient + update launch must move (all m replicas, all layers of the
    launch): read and write W (8 B per parameter), the same for v when momentum is on, and the bf16 copy of
    W for a bf16 model (2 B): 16 or 18 bytes per parameter per replica-step."""
    return update_bytes_per_launch(w, layer, operands=False)


def update_bytes_per_launch(w: wl.Workload, layer: int, operands: bool = True) -> float:
    """Algorithmic bytes of the weight-gradient + update launch that covers layer `layer` (all m replicas):
    read and write W (and v when momentum is on), write the bf16 copy of W (bf16 models), read the
    two GEMM operands once; summed over the layers that share the launch."""
    bf = w.gemm_dtype == "bf16"
    merged = streamed_update_layers(w)
    layers = merged if layer in merged else [layer]
    total = 0.0
    for l in layers:
        n_out, n_in = layer_shapes(w)[l]
        per_param = 8 + (8 if w.momentum != 0 else 0) + (2 if bf else 0)
        operand = (2 if bf else 4) * w.batch * (n_out + n_in) if operands else 0
        total += float(w.m) * (per_param * n_out * n_in + operand)
    return total


def uses_tensor_cores(w: wl.Workload, cls: str, layer: int) -> bool:
    """Mirror of the library's kernel choice: tcgen05 kernels for tile-sized shapes, CUDA cores otherwise."""
    n_out, n_in = layer_shapes(w)[layer]
    fp32 = w.gemm_dtype != "bf16"
    last = layer == len(w.dims) - 2
    if last and n_out <= 16:
        return False                      # narrow output layer: fused CUDA-core kernels
    def ok(M, N, K):
        return M % 128 == 0 and (N % 64 == 0 and K % 32 == 0 if fp32 else N % 128 == 0 and K % 64 == 0)
    if cls == "fwd":
        return (not last) and ok(w.batch, n_out, n_in)
    if cls == "dx":
        return ok(w.batch, n_in, n_out)
    if cls == "dw":
        return ok(n_out, n_in, w.batch)
    return False


# kernel class -> source file whose hash dates the stored DRAM-traffic counters (profiles/traffic.json)
KERNEL_SOURCE = {"dw": "update_tc.cu", "fwd": "gemm_tc.cu", "dx": "gemm_tc.cu", "avg": "average.cu"}


def stored_traffic(w: wl.Workload, cls: str, layer: int):
    """dram__bytes_read + dram__bytes_write per launch from the committed ncu capture of this kernel on
    this workload, or None when there is none or the kernel's source has changed since it was taken."""
    import hashlib
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            table = json.load(f)
        ent = table.get(f"{w.name}:{cls}{layer}")
        # ("avg", 1) is the step + averaging launch, which lives with the update kernels
        src = os.path.join(ROOT, "paper_1810_08313_b200", "csrc",
                           "update_tc.cu" if (cls, layer) == ("avg", 1) else KERNEL_SOURCE[cls])
        sha = hashlib.sha256(open(src, "rb").read()).hexdigest()[:16]
        if ent and ent.get("source_sha") == sha:
            return float(ent["dram_bytes_per_launch"])
    except Exception:
        pass
    return None


def roofline_for(dom, dur_s: float, w: wl.Workload, peaks, clocks, tau: int = 0):
    """Roofline object of the dominant kernel (class, layer) given its mean launch duration."""
    cls, layer = dom
    ms = dur_s * 1e3
    src = f"of {peaks['source']}"
    traffic = stored_traffic(w, cls, layer)
    if cls == "avg" and layer == 1:
        # last update of a period + averaging in one launch: per streamed parameter, write W, v and the bf16 copy
        # of m replicas (10 m B) and the synchronized copy (8 B); read the old state once (8 B, period of 1) or
        # every replica's own (8 m B)
        merged = streamed_update_layers(w)
        shapes = layer_shapes(w)
        n = float(sum(shapes[l][0] * shapes[l][1] for l in merged))
        sb = 8.0 if w.momentum != 0 else 4.0          # W and v, or W alone
        by = n * ((sb + 2.0) * w.m + sb + (sb if tau == 1 else sb * w.m))
        ach = by / dur_s / 1e9
        return {"kernel": f"weight gradient + update + averaging, layers {merged} in one launch (tcgen05, streaming)",
                "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"], "traffic": traffic if tau != 1 else None, "peak_source": src,
                "ms_per_launch": ms, "bytes_per_launch": by, "frac_of_8TBs": ach / 8000.0}
    if cls == "avg":
        by = 8.0 * w.m * wl.n_params(w.dims, w.has_bias) * (2 if w.momentum != 0 else 1)
        ach = by / dur_s / 1e9
        return {"kernel": "averaging (params + momentum)", "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"],
                "unit": "GB/s", "frac": ach / peaks["hbm_gbs"], "traffic": traffic, "peak_source": src,
                "ms_per_launch": ms}
    tc = uses_tensor_cores(w, cls, layer)
    if cls == "dw" and tc:
        # achieved = the state bytes alone (16 / 18 B per parameter per replica-step); the GEMM operands that the
        # launch also reads once (dZ and the layer inputs) are reported beside it, not counted in the fraction
        by = update_state_bytes_per_launch(w, layer)
        by_all = update_bytes_per_launch(w, layer)
        ach = by / dur_s / 1e9
        merged = streamed_update_layers(w)
        which = f"layers {merged}" if layer in merged and len(merged) > 1 else f"layer {layer}"
        return {"kernel": f"weight gradient + update, {which} in one launch (tcgen05, streaming)", "bound": "hbm",
                "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                "traffic": traffic, "peak_source": src, "ms_per_launch": ms,
                "bytes_per_launch": by, "operand_bytes_per_launch": by_all - by,
                "achieved_with_operands": by_all / dur_s / 1e9, "frac_of_8TBs": ach / 8000.0}
    n_out, n_in = layer_shapes(w)[layer]
    fl = 2.0 * w.m * w.batch * n_out * n_in
    ach = fl / dur_s / 1e12
    if tc and w.gemm_dtype == "bf16":
        peak = peaks["bf16_tflops_sustained"]
        return {"kernel": f"{cls} layer {layer} (tcgen05 bf16)", "bound": "tensor", "achieved": ach, "peak": peak,
                "unit": "TFLOP/s", "frac": ach / peak, "traffic": traffic,
                "peak_source": src + " (sustained bf16)", "ms_per_launch": ms,
                "frac_of_burst": ach / peaks["bf16_tflops"] if peaks.get("bf16_tflops") else None,
                "frac_of_nominal_2250": ach / NOMINAL_BF16_TFLOPS}
    if tc:
        # fp32 operands: three tf32 MMAs per product; tf32 dense peak = bf16 peak x (1.1 / 2.25) nominal ratio
        peak = peaks["bf16_tflops_sustained"] * (1.1 / 2.25) / 3.0
        return {"kernel": f"{cls} layer {layer} (tcgen05 3xTF32)", "bound": "tensor", "achieved": ach, "peak": peak,
                "unit": "TFLOP/s", "frac": ach / peak, "traffic": traffic,
                "peak_source": src + " bf16 sustained x 1.1/2.25 (nominal tf32:bf16) / 3 MMAs per fp32 product",
                "ms_per_launch": ms}
    mhz = clocks.get("sm_mhz") or 1965.0
    peak = fp32_alu_peak_tflops(mhz)
    return {"kernel": f"{cls} layer {layer} (CUDA cores)", "bound": "alu", "achieved": ach, "peak": peak,
            "unit": "TFLOP/s", "frac": ach / peak, "traffic": traffic,
            "peak_source": f"derived: 148 SMs x 128 lanes x 2 x {mhz:.0f} MHz", "ms_per_launch": ms}


def gemm_flops_per_launch(w: wl.Workload, layer: int) -> float:
    n_out, n_in = layer_shapes(w)[layer]
    return 2.0 * w.m * w.batch * n_out * n_in


def fp32_alu_peak_tflops(sm_mhz: float, sms: int = 148) -> float:
    """128 fp32 lanes per SM, one FMA (2 flops) per lane per clock."""
    return sms * 128 * 2 * sm_mhz * 1e6 / 1e12


def aggregate_over_ranks(ms_local: float, units_local: float):
    """(max ms over ranks, total units) with torch.distributed when initialised."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms_local, units_local
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([ms_local], dtype=torch.float64, device=dev)
    u = torch.tensor([units_local], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU every 20 ms.  It is started before the
    warm-up (nvidia-smi needs a few hundred milliseconds to come up) and the samples are cut to the timed
    region by their timestamps; when the region was too short to catch one, the samples of the warm-up
    (the same kernels under the same load) stand in and `window` says so."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None
        self.t_begin = self.t_end = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def mark_begin(self):
        self.t_begin = time.time()

    def mark_end(self):
        self.t_end = time.time()

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        try:
            time.sleep(0.05)
            self.proc.terminate()
            self.proc.wait(timeout=5)
        except Exception:
            pass
        text = open(self.path).read()
        try:
            os.unlink(self.path)
        except OSError:
            pass
        inside = parse_clock_csv(text, self.t_begin, self.t_end)
        if inside["samples"] > 0:
            inside["window"] = "timed region"
            return inside
        both = parse_clock_csv(text)
        both["window"] = "warm-up and timed region (the timed region was shorter than a sampling period)"
        return both


def _smi_time(stamp: str):
    """nvidia-smi's 'YYYY/MM/DD HH:MM:SS.mmm' as seconds since the epoch (local time), or None."""
    import datetime
    try:
        return datetime.datetime.strptime(stamp.strip(), "%Y/%m/%d %H:%M:%S.%f").timestamp()
    except ValueError:
        return None


def parse_clock_csv(text: str, t_begin=None, t_end=None):
    """Median SM clock, maximum clock and the set of throttle reasons seen.  Lines are
    [timestamp,] sm, max, power, hw_slowdown, hw_thermal, sw_thermal, sw_power_cap; with t_begin / t_end
    only lines stamped inside [t_begin, t_end] count."""
    sm, mx, reasons = [], [], set()
    names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
    for line in text.strip().splitlines():
        a = [x.strip() for x in line.split(",")]
        stamp = None
        if len(a) >= 8:
            stamp, a = _smi_time(a[0]), a[1:]
        if len(a) < 7:
            continue
        if t_begin is not None and t_end is not None:
            if stamp is None or not (t_begin <= stamp <= t_end):
                continue
        try:
            sm.append(float(a[0])); mx.append(float(a[1]))
        except ValueError:
            continue
        for name, val in zip(names, a[3:7]):
            if val.lower().startswith("active"):
                reasons.add(name)
    if not sm:
        return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
    return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
            "samples": len(sm)}


# --------------------------------------------------------------------------
# the oracle arm (CPU): --impl reference and the cpu_baseline leg
# --------------------------------------------------------------------------

def oracle_replica_steps_per_s(w: wl.Workload, X, y, x1, tau: int, budget_s: float, max_iters: int):
    """Times the CPU oracle, as it stands, on whole iterations (all m replicas) of the workload plus
    the averaging step every tau iterations.  Returns (replica-steps/s, iterations, seconds)."""
    from oracle import localsgd_oracle as orc
    spec = orc.ModelSpec(w.dims, w.loss, w.has_bias)
    lr, mu = float(np.float32(w.lr)), float(np.float32(w.momentum))
    iters = 0
    t0 = time.perf_counter()
    offs_all = wl.batch_row_offsets(w.seed + 1, max_iters, w.m, X.shape[0], w.batch)
    xs = np.repeat(x1[None], w.m, axis=0).astype(np.float32)
    vs = np.zeros_like(xs)
    t0 = time.perf_counter()
    while iters < max_iters:
        for i in range(w.m):
            r0 = int(offs_all[iters, i])
            _, g = orc.loss_and_grad(spec, xs[i], X[r0:r0 + w.batch], y[r0:r0 + w.batch])
            xn, vn = orc.sgd_momentum_step(xs[i], vs[i], g, lr, mu)
            xs[i] = xn.astype(np.float32); vs[i] = vn.astype(np.float32)
        iters += 1
        if iters % tau == 0:
            orc.average_replicas(xs)
            if mu != 0:
                orc.average_replicas(vs)
        if time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    return w.m * iters / dt, iters, dt


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, w: wl.Workload):
    """The oracle timed on the host cores: each step is one whole iteration (m replica-steps)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_rows = min(w.n_rows, 8192)
    X, y = wl.make_dataset(w, n_rows=n_rows)
    x1 = wl.initial_point(w)
    from oracle import localsgd_oracle as orc
    spec = orc.ModelSpec(w.dims, w.loss, w.has_bias)
    lr, mu = float(np.float32(w.lr)), float(np.float32(w.momentum))
    tau = args.tau
    xs = np.repeat(x1[None], w.m, axis=0).astype(np.float32)
    vs = np.zeros_like(xs)
    total = args.warmup + args.steps
    offs = wl.batch_row_offsets(w.seed + 1, total, w.m, n_rows, w.batch)

    def one_iter(k):
        for i in range(w.m):
            r0 = int(offs[k, i])
            _, g = orc.loss_and_grad(spec, xs[i], X[r0:r0 + w.batch], y[r0:r0 + w.batch])
            xn, vn = orc.sgd_momentum_step(xs[i], vs[i], g, lr, mu)
            xs[i] = xn.astype(np.float32); vs[i] = vn.astype(np.float32)
        if (k + 1) % tau == 0:
            orc.average_replicas(xs)
            if mu != 0:
                orc.average_replicas(vs)

    for k in range(args.warmup):
        one_iter(k)
    t0 = time.perf_counter()
    for k in range(args.warmup, total):
        one_iter(k)
    dt = time.perf_counter() - t0
    value = w.m * args.steps / dt
    cores = cpu_threads()
    sample = f"{args.steps} whole iterations (m={w.m} replica-steps each, averaging every {tau}) of {w.name} on {n_rows} rows"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": dict(workload_config(w, tau), step="one iteration of all m replicas on the CPU oracle, on the "
                                                       f"first {n_rows} dataset rows"),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------
# the CUDA arm
# --------------------------------------------------------------------------

def run_ours(args, w: wl.Workload):
    import torch
    import torch.distributed as dist
    from paper_1810_08313_b200.binding import LocalSGD, adacomm_next_tau, average_flat, block_average_flat

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU implementation")
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl")
    peaks = load_peaks()
    tau, K, W = args.tau, args.steps, args.warmup
    m, B = w.m, w.batch

    # ---- synthetic inputs, resident in HBM before the timed region ----------
    X, y = wl.make_dataset(w)
    x1 = wl.initial_point(w)
    xd = torch.from_numpy(X).cuda()
    if w.gemm_dtype == "bf16":
        xd = xd.to(torch.bfloat16)
    yd = torch.from_numpy(y).cuda()
    total_periods = W + K
    if args.shard:
        # ONE job of w.m replicas dealt out over the ranks (m / N each): local steps need no communication, every
        # averaging step is one all-gather of partial sums over NCCL plus the rank-ordered combining kernel
        from paper_1810_08313_b200.sharded import ShardedLocalSGD
        sh = ShardedLocalSGD(w.m, w.dims, w.loss, w.has_bias, w.gemm_dtype, lr=w.lr, momentum=w.momentum, batch=B,
                             device=f"cuda:{local_rank}")
        eng, m = sh.eng, sh.m
        offs = wl.batch_row_offsets(w.seed + 100, total_periods * tau, w.m, w.n_rows, B)
        offs = np.ascontiguousarray(offs[:, sh.first:sh.first + sh.m])
    else:
        eng = LocalSGD(m, w.dims, w.loss, w.has_bias, w.gemm_dtype, lr=w.lr, momentum=w.momentum, batch=B,
                       device=f"cuda:{local_rank}")
        offs = wl.batch_row_offsets(w.seed + 100 + rank, total_periods * tau, m, w.n_rows, B)
    import dataclasses
    w_r = dataclasses.replace(w, m=m)          # this rank's share, for the per-launch byte and flop counts
    eng.bind_dataset(xd, yd)
    eng.set_params(x1)
    probe = probe_rows_for(w)
    loss_dev = torch.zeros((tau, m), dtype=torch.float32, device="cuda")
    F_0 = eng.eval_loss(0, 0, probe)

    def period(p):
        eng.local_steps(tau, offs[p * tau:(p + 1) * tau], loss_dev, average=True)    # the period and its averaging step
        F_t = eng.eval_loss(0, 0, probe)
        return F_t, adacomm_next_tau(F_t, F_0, tau)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()

    # ---- warm-up, with every kernel class timed to find the dominant one ----
    # (the first period is left out of the per-kernel times: first launches load their kernels lazily)
    period(0)
    eng.profile_begin()
    for p in range(1, W):
        period(p)
    shares_raw = eng.profile_end()
    tot = sum(v[0] for v in shares_raw.values()) or 1.0
    shares = {f"{c}{l}": round(v[0] / tot, 4) for (c, l), v in sorted(shares_raw.items(), key=lambda kv: -kv[1][0])}
    kernel_us = {f"{c}{l}": round(v[0] / v[1] * 1e3, 2) for (c, l), v in shares_raw.items() if v[1]}
    dom = max(shares_raw.items(), key=lambda kv: kv[1][0])[0] if shares_raw else ("dw", 0)

    # ---- timed region ---------------------------------------------------------
    eng.profile_begin([dom[0]], dom[1])
    launches0 = eng.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.mark_begin()
    e0.record()
    F_t, next_tau = 0.0, tau
    for p in range(W, W + K):
        F_t, next_tau = period(p)
    e1.record()
    barrier()
    sampler.mark_end()
    clocks = sampler.stop()
    ms_local = e0.elapsed_time(e1)
    launches = eng.launch_count() - launches0
    dom_ms, dom_n = eng.profile_end().get(dom, (0.0, 0))
    ms, units = aggregate_over_ranks(ms_local, float(m * tau * K))
    value = units / (ms * 1e-3)

    # ---- roofline of the dominant kernel ---------------------------------------
    roofline = roofline_for(dom, dom_ms * 1e-3 / dom_n, w_r, peaks, clocks, tau) if dom_n else None

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms / K, "higher_is_better": True, "scaling": "strong" if args.shard else "weak",
        "vs_baseline": None,
        "dtype": "bf16" if w.gemm_dtype == "bf16" else "f32", "data": "synthetic",
        "config": dict(workload_config(w, tau),
                       step="one period: tau local iterations x m replicas + averaging + probe loss + AdaComm decision",
                       l2="inputs larger than L2: mini-batches are drawn at random from a %.0f MB resident dataset"
                          % (xd.numel() * xd.element_size() / 1e6),
                       multi_gpu=("one job sharded by replica, one all-gather of partial sums per period" if args.shard
                                  else "replicas only: independent jobs, no data-path collective") if world > 1
                       else "single GPU"),
        "clocks": clocks, "gpu_launches": int(launches), "kernel_time_shares": shares,
        "kernel_us_per_launch": kernel_us,
        "last_probe_loss": F_t, "next_tau": next_tau,
    }
    if roofline:
        line["roofline"] = roofline
    # tensor-core GEMMs of the step (forward / data gradient): achieved rate from the per-launch event times
    gemm = {}
    for (c, l), v in shares_raw.items():
        if c in ("fwd", "dx") and v[1] and uses_tensor_cores(w, c, l):
            r = roofline_for((c, l), v[0] * 1e-3 / v[1], w_r, peaks, clocks)
            gemm[f"{c}{l}"] = {"TFLOP/s": round(r["achieved"], 1), "frac": round(r["frac"], 4),
                               "us_per_launch": round(v[0] / v[1] * 1e3, 2)}
    if gemm:
        line["gemm_tensor"] = gemm

    if not args.kernel_only:
        # ---- end to end: mini-batches from pinned host memory, losses back to the host (every rank; the
        # time is the maximum over ranks, the units add up) -------
        e_steps = max(1, min(K, 3))
        xh = torch.empty((tau, m, B, w.dims[0]), dtype=xd.dtype).pin_memory()
        yh = torch.empty((tau, m, B), dtype=yd.dtype).pin_memory()
        lh = torch.zeros((tau, m), dtype=torch.float32).pin_memory()
        o = offs[:tau]
        for s in range(tau):
            for i in range(m):
                r0 = int(o[s, i])
                xh[s, i].copy_(xd[r0:r0 + B].cpu()); yh[s, i].copy_(yd[r0:r0 + B].cpu())
        def e2e_period():
            eng.local_steps_host(tau, xh, yh, lh)
            eng.average()
            F = eng.eval_loss(0, 0, probe)
            return adacomm_next_tau(F, F_0, tau)
        e2e_period()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e_steps):
            e2e_period()
        barrier()
        dt = time.perf_counter() - t0
        e_ms, e_units = aggregate_over_ranks(dt * 1e3, float(m * tau * e_steps))
        line["e2e"] = {"value": e_units / (e_ms * 1e-3), "unit": UNIT,
                       "h2d_bytes_per_step": int(xh.numel() * xh.element_size() + yh.numel() * yh.element_size()),
                       "d2h_bytes_per_step": int(lh.numel() * 4 + 4),
                       "note": "per period; batches copied from pinned host memory inside the timed region; when "
                               "the copies (bytes / host-link rate) take longer than the kernels of a period the "
                               "host link, not the GPU, sets this number"}

    if rank == 0 and world == 1 and not args.kernel_only:
        # ---- averaging bandwidth on the model-sized flat vectors (params + momentum) ----------
        # (each replica's vector starts on a 256-byte boundary, as in the library's own layout; the 10^9
        #  point is run when --avg-1b is given: m = 16 with momentum needs 2 x 64 GB)
        avg = {}
        # the engine's state is no longer needed on the device from here on for the largest point
        for P in [14_706_698, 23_500_000, 1_000_000_000]:
            stride = (P + 63) // 64 * 64
            # 10^9 elements: params + momentum of m replicas are 2 * m * 4 GB; m = 4 (32 GB) always runs when
            # the memory is there, m = 8 and 16 (64 / 128 GB) with --avg-1b
            ms_list = (4, 8, 16) if P < 10 ** 8 else ((4, 8, 16) if args.avg_1b else (4,))
            half = max(ms_list)
            free_b, _ = torch.cuda.mem_get_info()
            while ms_list and 2 * max(ms_list) * stride * 4 > 0.9 * free_b:
                ms_list = ms_list[:-1]
                half = max(ms_list) if ms_list else 0
            if not ms_list:
                avg[f"P{P}"] = "did not fit in free device memory"
                continue
            buf = torch.empty((2 * half, stride), device="cuda", dtype=torch.float32)
            buf.uniform_(-1.0, 1.0)
            for mm in ms_list:
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
                for _ in range(3):
                    average_flat(buf[:mm].view(-1), mm, P, stride); average_flat(buf[half:half + mm].view(-1), mm, P, stride)
                ev[0].record()
                reps = 10 if P < 10 ** 8 else 3
                for _ in range(reps):
                    average_flat(buf[:mm].view(-1), mm, P, stride); average_flat(buf[half:half + mm].view(-1), mm, P, stride)
                ev[1].record()
                torch.cuda.synchronize()
                gbs = 2 * 8.0 * mm * P * reps / (ev[0].elapsed_time(ev[1]) * 1e-3) / 1e9
                avg[f"P{P}_m{mm}"] = {"GB/s": round(gbs, 1), "frac_measured_peak": round(gbs / peaks["hbm_gbs"], 4),
                                      "frac_8TBs": round(gbs / 8000.0, 4)}
            # the same pass with block momentum (Section 5.3): + period-start model and global buffer,
            # 8m + 16 bytes per parameter
            if P < 10 ** 8:
                anc = torch.zeros(2, stride, device="cuda", dtype=torch.float32)
                ub = torch.zeros(2, stride, device="cuda", dtype=torch.float32)
                for mm in (4, 16):
                    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
                    def both():
                        block_average_flat(buf[:mm].view(-1), anc[0], ub[0], mm, P, 0.05, 0.3, stride)
                        block_average_flat(buf[half:half + mm].view(-1), anc[1], ub[1], mm, P, 0.05, 0.3, stride)
                    for _ in range(3):
                        both()
                    ev[0].record()
                    for _ in range(10):
                        both()
                    ev[1].record()
                    torch.cuda.synchronize()
                    gbs = 2 * (8.0 * mm + 16.0) * P * 10 / (ev[0].elapsed_time(ev[1]) * 1e-3) / 1e9
                    avg[f"block_P{P}_m{mm}"] = {"GB/s": round(gbs, 1),
                                                "frac_measured_peak": round(gbs / peaks["hbm_gbs"], 4),
                                                "frac_8TBs": round(gbs / 8000.0, 4)}
                del anc, ub
            del buf
        line["averaging_gbs"] = avg

        # ---- the other workload configurations: a short device-timed run each -------------------------------
        if not args.no_side_configs:
            line["configs"] = {name: side_config(name, args.tau) for name in sorted(wl.WORKLOADS) if name != w.name}

        # ---- measured throughput against the period, beside the runtime model's speed-up (Section 3.2) -----
        if args.tau_sweep:
            sweep = {}
            n_it = 400
            so = wl.batch_row_offsets(w.seed + 999, n_it, m, w.n_rows, B)
            sl = torch.zeros((n_it, m), dtype=torch.float32, device="cuda")
            for t in (1, 2, 5, 20, 100):
                ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
                for rep in range(2):           # first pass warms up
                    torch.cuda.synchronize()
                    ev[0].record()
                    for k0 in range(0, n_it, t):
                        n = min(t, n_it - k0)
                        eng.local_steps(n, so[k0:k0 + n], sl[k0:k0 + n])
                        eng.average()
                    ev[1].record()
                    torch.cuda.synchronize()
                sweep[t] = ev[0].elapsed_time(ev[1]) / n_it          # ms per iteration
            # Y: time of an iteration without averaging, D: time of one averaging, both from the two ends
            # of the sweep (T(tau) = Y + D / tau)
            D_ms = (sweep[1] - sweep[100]) / (1.0 - 1.0 / 100.0)
            Y_ms = sweep[1] - D_ms
            alpha = D_ms / Y_ms
            line["tau_sweep"] = {
                "ms_per_iteration": {str(t): round(v, 5) for t, v in sweep.items()},
                "Y_ms": round(Y_ms, 5), "D_ms": round(D_ms, 5), "alpha": round(alpha, 4),
                "speedup_measured": {str(t): round(sweep[1] / v, 4) for t, v in sweep.items()},
                "speedup_model": {str(t): round((1 + alpha) / (1 + alpha / t), 4) for t in sweep},
                "note": "model: (1 + alpha) / (1 + alpha / tau) with alpha = D / Y fitted at tau = 1 and 100"}

        # ---- the workload's whole job in the native run loop (ls_run): K iterations, AdaComm where configured -------
        # ---- communication period 1 (where AdaComm takes a long run): device-timed iterations, each a local step
        # of every replica plus the averaging step ------------------------------------------------------------
        n1 = 30
        o1 = wl.batch_row_offsets(w.seed + 55, n1, m, w.n_rows, B)
        for k in range(5):
            eng.local_steps(1, o1[k:k + 1], loss_dev[:1], average=True)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
        ev[0].record()
        for k in range(5, n1):
            eng.local_steps(1, o1[k:k + 1], loss_dev[:1], average=True)
        ev[1].record()
        torch.cuda.synchronize()
        ms1 = ev[0].elapsed_time(ev[1]) / (n1 - 5)
        line["tau1"] = {"ms_per_period": round(ms1, 4), "replica_steps_per_s": round(m / (ms1 * 1e-3), 1),
                        "note": "one local step of all replicas + the averaging step per period, inputs resident"}

        logged = {}
        if args.full_run:
            runs = {}
            Kfull = w.n_iters
            fo = wl.batch_row_offsets(w.seed + 7, Kfull, m, w.n_rows, B)
            schedules = [(w.adacomm_tau0, w.adacomm_interval)] if w.adacomm_tau0 else [(t, 0) for t in w.taus]
            for tau0, interval in schedules:
                eng.set_params(x1)
                for i in range(m):
                    eng.set_state(i, None, np.zeros_like(x1))
                torch.cuda.synchronize()
                t0 = time.perf_counter()
                out = eng.run(Kfull, tau0, fo, interval=interval or 0, probe_rows=probe if interval else 0)
                eng.sync()
                dt = time.perf_counter() - t0
                F_end = eng.eval_loss(0, 0, probe)
                taus = out["taus"]
                # run-length form of the period list: [[tau, how many periods in a row], ...]
                rle = []
                for t in taus:
                    if rle and rle[-1][0] == t:
                        rle[-1][1] += 1
                    else:
                        rle.append([int(t), 1])
                runs[f"tau0_{tau0}" + ("_adacomm" if interval else "")] = {
                    "iterations": Kfull, "seconds": round(dt, 4), "replica_steps_per_s": round(m * Kfull / dt, 1),
                    "averaging_steps": len(taus), "periods_rle": rle[:40], "F_0": F_0, "F_end": F_end,
                    "decisions": len(out["decision_k"])}
                if interval:
                    logged[f"tau0_{tau0}_adacomm"] = (tau0, float(out["F_0"]), [float(F) for F in out["decision_F"]],
                                                      [int(t) for t in out["decision_tau"]])
            line["full_run"] = runs

        # ---- the CPU oracle on the host cores, bounded sample -----------------------------------
        if not args.no_cpu_baseline:
            v, iters, dt = oracle_replica_steps_per_s(w, X[:8192], y[:8192], x1, tau, budget_s=args.cpu_budget,
                                                      max_iters=10 * tau)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                    "sample": f"{iters} whole iterations (m={m} replica-steps each) in {dt:.1f} s on "
                                              f"the first 8192 rows"}
            # the oracle's rule on the losses that the native run loop logged: the periods it chose must be
            # the oracle's, bit for bit (Section 4.2)
            from oracle import localsgd_oracle as orc
            for key, (tau0, F0_run, Fs, taus_run) in logged.items():
                want = orc.tau_schedule_from_trace(F0_run, tau0, Fs)
                line["full_run"][key]["tau_trace_bit_exact"] = bool(want == taus_run)
    eng.close()
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def side_config(name: str, tau_default: int, periods: int = 10, warm: int = 3, max_rows: int = 16384):
    """Device-timed replica-steps/s of one of the other workload configurations: `periods` periods at the
    workload's first configured tau (local steps + averaging in one call per period, inputs resident), after
    `warm` untimed ones.  The resident dataset is cut to max_rows rows (still larger than L2 for the MLPs)
    so that the side runs add seconds, not minutes."""
    import torch
    from paper_1810_08313_b200.binding import LocalSGD
    w = wl.WORKLOADS[name]
    tau = int(w.adacomm_tau0 or (tau_default if tau_default in w.taus else w.taus[0]))
    n_rows = min(w.n_rows, max_rows * (2 if w.gemm_dtype == "bf16" else 1))
    X, y = wl.make_dataset(w, n_rows=n_rows)
    xd = torch.from_numpy(X).cuda()
    if w.gemm_dtype == "bf16":
        xd = xd.to(torch.bfloat16)
    yd = torch.from_numpy(y).cuda()
    eng = LocalSGD(w.m, w.dims, w.loss, w.has_bias, w.gemm_dtype, lr=w.lr, momentum=w.momentum, batch=w.batch)
    eng.bind_dataset(xd, yd)
    eng.set_params(wl.initial_point(w))
    offs = wl.batch_row_offsets(w.seed + 5, (warm + periods) * tau, w.m, n_rows, w.batch)
    loss_dev = torch.zeros((tau, w.m), dtype=torch.float32, device="cuda")
    for p in range(warm):
        eng.local_steps(tau, offs[p * tau:(p + 1) * tau], loss_dev, average=True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n0 = eng.launch_count()
    torch.cuda.synchronize()
    e0.record()
    for p in range(warm, warm + periods):
        eng.local_steps(tau, offs[p * tau:(p + 1) * tau], loss_dev, average=True)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    out = {"replica_steps_per_s": round(w.m * tau * periods / (ms * 1e-3), 1), "tau": tau, "periods": periods,
           "ms_per_period": round(ms / periods, 4), "dtype": "bf16" if w.gemm_dtype == "bf16" else "f32",
           "m": w.m, "batch": w.batch, "dims": list(w.dims), "dataset_rows": n_rows,
           "gpu_launches": int(eng.launch_count() - n0), "last_loss": float(loss_dev[-1].mean().item())}
    eng.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3_mlp_bf16", choices=sorted(wl.WORKLOADS))
    ap.add_argument("--replicas", type=int, default=0,
                    help="run the workload with this many replicas instead of its own count (a smaller footprint for "
                         "profiler captures; the line's workload name then ends in @mN)")
    ap.add_argument("--shard", action="store_true",
                    help="with --gpus N: one job whose m replicas are dealt out over the N ranks (m / N each) with one "
                         "NCCL all-gather of partial sums per averaging step, instead of N independent jobs")
    ap.add_argument("--no-side-configs", action="store_true",
                    help="skip the short device-timed runs of the other workload configurations")
    ap.add_argument("--tau", type=int, default=20)
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tau-sweep", action="store_true",
                    help="also time iterations at tau = 1, 2, 5, 20, 100 and compare with the speed-up model of Section 3.2")
    ap.add_argument("--avg-1b", action="store_true", help="add the 10^9-element point to the averaging sweep (128 GB)")
    ap.add_argument("--no-full-run", dest="full_run", action="store_false",
                    help="skip the workload's whole job (its iteration count, tau or AdaComm schedule; a few seconds) in "
                         "the native run loop, reported with its throughput, loss and the periods chosen")
    ap.add_argument("--full-run", dest="full_run", action="store_true", help=argparse.SUPPRESS)
    ap.set_defaults(full_run=True)
    ap.add_argument("--kernel-only", action="store_true",
                    help="only the device-timed region (for profiler runs): no e2e, averaging sweep or CPU baseline")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    w = wl.WORKLOADS[args.workload]
    if args.replicas:
        import dataclasses
        w = dataclasses.replace(w, m=int(args.replicas), name=f"{w.name}@m{int(args.replicas)}")
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
