"""Benchmark: IST training samples/s on one B200 (or N independent replicas).

A "step" is one whole IST round on a synthetic workload: partition + gather, K local SGD steps
of all S subnets, reassemble.  Timed on the device with CUDA events on the library's stream,
after warm-up, bracketed by a barrier and a synchronize; max over ranks.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C3] [--impl reference]

Prints one JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1910_02120_b200 import synth  # noqa: E402

METRIC = "IST training samples/sec (all S subnets, device-timed)"
UNIT = "samples/s"
# DRAM bytes per launch from ncu captures, kept in a tracked file with the hash of the kernel
# source each capture was taken on; a class whose source has changed since reports traffic = null.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.json")
CSRC = os.path.join(ROOT, "paper_1910_02120_b200", "csrc")
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="C3", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dims", default="",
                    help="profiling aid: replace the configuration's layer widths (comma separated); with "
                         "--subnets / --batch a reduced case of the same kernels for ncu captures")
    ap.add_argument("--subnets", type=int, default=0)
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--shard-subnets", action="store_true",
                    help="with --gpus N > 1: split the S subnets over the ranks (one all-gather of the trained "
                         "slices per round, strong scaling) instead of running N independent replicas")
    ap.add_argument("--norm-eps", type=float, default=None,
                    help="standardise hidden pre-activations over the batch (Sec. 2.2) with this epsilon")
    ap.add_argument("--iid", action="store_true",
                    help="independent assignment of neurons to subnets (unequal group sizes) instead of the balanced split")
    ap.add_argument("--local-steps", type=int, default=0,
                    help="override K (local steps per round); makes a small case for profiler captures")
    ap.add_argument("--sweep", action="store_true",
                    help="run the scaling sweep (1024-H-H-100, batch 512, bf16) over H x S x K; one JSON line per point")
    ap.add_argument("--sweep-H", default="2048,8192,32768,65536")
    ap.add_argument("--sweep-S", default="1,2,4,8,16")
    ap.add_argument("--sweep-K", default="1,10,100")
    ap.add_argument("--quick", action="store_true",
                    help="device-timed pass only (no end-to-end, per-class or CPU passes), warm-up as given")
    return ap.parse_args()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


def measured_traffic(workload_name: str, kernel_class: str, work_per_launch_now: float):
    """DRAM bytes per launch of this class from the recorded ncu capture, scaled by the launch's
    algorithmic work in the record's unit (bytes for HBM-bound classes, flop for the contractions;
    the capture may be of a reduced case of the same kernel), or None when there
    is no capture for this workload and class or the kernel source has changed since."""
    import hashlib
    try:
        rec = json.load(open(TRAFFIC_FILE))[workload_name][kernel_class]
        src = open(os.path.join(CSRC, rec["source"]), "rb").read()
    except (OSError, KeyError, ValueError):
        return None
    if hashlib.sha256(src).hexdigest() != rec["source_sha256"]:
        return None
    return rec["dram_bytes_per_launch"] * work_per_launch_now / rec["algorithmic_per_launch"]


def config_dict(w: synth.Workload, n_gpus: int, norm_eps=None, sharded=False, iid=False):
    extra = {} if norm_eps is None else {"normalization": f"per-neuron batch standardisation, eps={norm_eps:g}"}
    if iid:
        extra["partition"] = "independent assignment (unequal subnets)"
    return {
        **extra,
        "workload": f"{w.name}: MLP {'-'.join(map(str, w.layer_dims))}, S={w.S}, batch={w.B}, "
                    f"K={w.K} local steps/round, {w.precision} operands, fp32 masters",
        "samples_per_step": w.samples_per_round,
        "step": "one IST round: partition+gather, K local SGD steps of S subnets, reassemble",
        "inputs": f"{w.x_dist}; distinct batch per subnet per local step",
        "l2": "per-round working set (inputs + full network + packed slices) exceeds the 126 MB L2",
        "parallelism": "single GPU" if n_gpus == 1 else
                       (f"{w.S} subnets split over {n_gpus} GPUs, one all-gather of trained slices per round" if sharded
                        else f"{n_gpus} independent replicas"),
    }


# ---------------------------------------------------------------------------------------------
# algorithmic work per round (all S subnets), used for the roofline fractions
# ---------------------------------------------------------------------------------------------

def spmm_bytes(w: synth.Workload, data, n1: int) -> float:
    """Algorithmic bytes of the sparse first layer over a round (all subnets and local steps).
    Forward, per stored nonzero and subnet: one bf16 weight row of n1 entries + 8 B (column and
    value), and n1 * 2 B of output per batch row.  Backward with the fused update: per nonzero the
    8 B again and the delta row (n1 * 2 B); per distinct touched input row 10 B per weight (fp32
    master read and written, bf16 copy written)."""
    es = 2 if w.precision == "bf16" else 4
    total = 0.0
    rp = np.asarray(data.row_ptr, dtype=np.int64)
    for i in range(w.S * w.K):                       # one (subnet, step) minibatch each
        lo, hi = rp[i * w.B], rp[(i + 1) * w.B]
        nnz = float(hi - lo)
        distinct = float(np.unique(data.col[lo:hi]).size)
        total += nnz * (n1 * es + 8) + w.B * n1 * es            # forward
        total += nnz * (8 + n1 * es) + distinct * n1 * (8 + (2 if es == 2 else 0))   # backward + update
    return total


def work_model(w: synth.Workload, norm=False, data=None):
    d, S, B, K = w.layer_dims, w.S, w.B, w.K
    t = len(d) - 1
    n = [d[0]] + [-(-d[l] // S) for l in range(1, t)] + [d[t]]
    layer_elems = [n[l - 1] * n[l] for l in range(1, t + 1)]          # per subnet
    packed = S * sum(layer_elems)
    dense_first = w.x_dist != "csr"
    fwd = 2 * B * S * sum(layer_elems[(0 if dense_first else 1):])
    dx = 2 * B * S * sum(layer_elems[1:])
    dw = 2 * B * S * sum(layer_elems[(0 if dense_first else 1):])
    opw = 2 if w.precision == "bf16" else 0
    es = 2 if w.precision == "bf16" else 4
    hidden = B * S * sum(n[1:t])                    # hidden pre-activations per local step
    # standardisation: forward reads fp32 z and writes a; backward reads z and d_zh, writes d_z
    norm_bytes = {"norm": hidden * ((4 + es) + (4 + 2 * es)) * K} if norm else {}
    if not dense_first and data is not None:
        norm_bytes["spmm"] = spmm_bytes(w, data, n[1])
    return {
        "packed_elems": packed,
        "flops": {"fwd": fwd * K, "dx": dx * K, "dw_sgd": dw * K},
        # bytes: gather = read fp32 + write fp32 master (+ bf16 copy); scatter = read + write fp32;
        # fused update inside dw_sgd = read + write master (+ bf16 copy)
        "bytes": {"gather": packed * (8 + opw), "scatter": packed * 8,
                  "dw_sgd": packed * (8 + opw) * K, **norm_bytes},
    }


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------

class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        self.skip = 0

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "25", "-i", str(self.gpu)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def mark(self):
        """The timed region starts here: lines written so far belong to the warm-up."""
        try:
            self.skip = sum(1 for l in open(self.f.name) if l.strip())
        except OSError:
            self.skip = 0

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        rows = [l.strip().split(", ") for l in open(self.f.name) if l.strip()][self.skip:]
        os.unlink(self.f.name)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1]))
                mx.append(float(r[2]))
            except ValueError:
                continue
            for name, v in zip(names, r[5:9]):
                if v.strip().lower() == "active":
                    reasons.add(name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ---------------------------------------------------------------------------------------------
# the CPU oracle, timed as it stands on a bounded sample of the workload
# ---------------------------------------------------------------------------------------------

def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


class OracleSample:
    """One bounded sample of a round: the full partition, the slicing of all S subnets, one local
    step on each of `n_sub` subnets, and the reassembly.  The round's throughput is extrapolated
    as S*K*B / (t_partition+slice+reassemble + S*K*t_step)."""

    def __init__(self, w: synth.Workload, n_sub=1, norm_eps=None):
        from oracle import ist_oracle as O
        self.O, self.w, self.n_sub, self.norm_eps = O, w, min(n_sub, w.S), norm_eps
        W, b = synth.make_weights(w.layer_dims, w.seed)
        self.o = O.IstOracle(w.layer_dims, w.S, norm_eps=norm_eps)
        self.o.bind_weights(W, b)
        del W, b
        small = w.scaled(S=self.n_sub, K=1)
        self.data = synth.make_round_inputs(small)

    def run(self, seed):
        o, w = self.o, self.w
        t0 = time.perf_counter()
        o.partition(seed)
        t1 = time.perf_counter()
        X = (self.data.row_ptr, self.data.col, self.data.val) if self.data.is_csr else self.data.X
        for s in range(self.n_sub):
            Ws, bs = o.subnets[s]
            xb, yb = o._batch(X, self.data.y, s, 0)
            self.O.sgd_step(Ws, bs, xb, yb, w.lr, o.dtype, self.norm_eps)
        t2 = time.perf_counter()
        o.reassemble()
        t3 = time.perf_counter()
        fixed = (t1 - t0) + (t3 - t2)
        step = (t2 - t1) / self.n_sub
        est_round = fixed + w.S * w.K * step
        return w.samples_per_round / est_round, t3 - t0

    def describe(self):
        return (f"per step: partition + slicing of all {self.w.S} subnets + 1 local SGD step on "
                f"{self.n_sub} subnet(s) at full width + reassembly, fp64 numpy; round throughput "
                f"extrapolated as S*K*B/(t_fixed + S*K*t_step)")


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    smp = OracleSample(w, norm_eps=args.norm_eps)
    for i in range(args.warmup):
        smp.run(1000 + i)
    vals, secs = [], []
    for i in range(args.steps):
        v, s = smp.run(2000 + i)
        vals.append(v)
        secs.append(s)
    value = float(np.mean(vals))
    cores = oracle_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(secs)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_dict(w, 1, args.norm_eps),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": smp.describe()},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
# multi-rank plumbing: replicas only, no data-path collective
# ---------------------------------------------------------------------------------------------

def max_over_ranks(ms: float, device=None) -> float:
    """Slowest rank's elapsed time (the job is as slow as its slowest replica)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(samples_per_rank_step: int, steps: int, world: int, ms: float) -> float:
    """Whole-job samples/s: every rank processed samples_per_rank_step * steps samples in ms."""
    return world * samples_per_rank_step * steps / (ms * 1e-3)


# ---------------------------------------------------------------------------------------------
# the CUDA path
# ---------------------------------------------------------------------------------------------

def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_1910_02120_b200 import api

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # ---- inputs, resident on the device before timing starts ---------------------------------
    shard = args.shard_subnets and world > 1
    if shard:
        from paper_1910_02120_b200 import sharding
        first, count = sharding.subnet_range(w.S, world, rank)
    ww = w.scaled(seed=w.seed + (0 if shard else 1000 * rank))
    W, b = synth.make_weights(ww.layer_dims, ww.seed)
    Wd = [torch.from_numpy(x).to(dev) for x in W]
    bd = [torch.from_numpy(x).to(dev) for x in b]
    del W, b
    data = synth.make_round_inputs(ww)
    if shard:      # same network and partition everywhere; this rank keeps the rows of its own subnets
        if data.is_csr:
            raise SystemExit("--shard-subnets takes dense inputs")
        data = synth.Batchset(y=data.y[first:first + count].copy(), X=data.X[first:first + count].copy())
    prec = api.IST_BF16 if w.precision == "bf16" else api.IST_FP32
    ctx = api.Ist(w.layer_dims, w.S, prec, w.B, input_is_csr=data.is_csr, device=str(dev),
                  partition_rule=api.IST_PART_IID if args.iid else api.IST_PART_BALANCED)
    ctx.bind_weights(Wd, bd)
    if args.norm_eps is not None:
        ctx.enable_normalization(args.norm_eps)
    if shard:
        ctx.set_subnet_range(first, count)
    n_local = count if shard else w.S
    y_host = torch.from_numpy(data.y.reshape(-1).copy()).pin_memory()
    if data.is_csr:
        host_in = [torch.from_numpy(data.row_ptr.astype(np.int32)).pin_memory(),
                   torch.from_numpy(data.col).pin_memory(), torch.from_numpy(data.val).pin_memory()]
    else:
        xt = torch.from_numpy(data.X.reshape(-1, w.layer_dims[0]))
        if w.precision == "bf16" and w.layer_dims[0] % 8 == 0:
            xt = xt.to(torch.bfloat16)
        host_in = [xt.pin_memory()]
    dev_in = [t.to(dev) for t in host_in]
    y_dev = y_host.to(dev)
    loss_dev = torch.empty(n_local * w.K, dtype=torch.float32, device=dev)
    loss_host = torch.empty(n_local * w.K, dtype=torch.float32).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in host_in) + y_host.numel() * 4
    d2h = loss_host.numel() * 4

    def X_of(ts):
        return tuple(ts) if data.is_csr else ts[0]

    def one_round(r, X, y):
        if shard:
            sharding.sharded_round(ctx, 7000 + r, X, y, w.lr, w.K, w.B, first, count, loss_out=loss_dev)
        else:
            ctx.round(7000 + r, X, y, w.lr, w.K, w.B, loss_out=loss_dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # ---- device-resident timing ---------------------------------------------------------------
    # the clock sampler (an nvidia-smi process) needs a few hundred milliseconds before its first
    # line: it starts before the warm-up rounds, and only the lines written after mark() count
    n_warm = args.warmup if args.quick else max(args.warmup, 3)
    sampler = ClockSampler(local)
    sampler.start()
    for i in range(n_warm):
        one_round(i, X_of(dev_in), y_dev)
    ctx.sync_status()
    barrier()
    sampler.mark()
    launches0 = ctx.kernel_launches()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        one_round(100 + i, X_of(dev_in), y_dev)
    e1.record()
    barrier()
    launches = ctx.kernel_launches() - launches0
    clocks = sampler.stop()
    ms = max_over_ranks(e0.elapsed_time(e1), dev)
    ctx.sync_status()
    per_rank = w.samples_per_round // world if shard else w.samples_per_round   # samples this rank's subnets saw
    value = job_value(per_rank, args.steps, world, ms)
    if args.quick:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                              "warmup": n_warm, "ms_per_step": ms / args.steps, "quick": True,
                              "gpu_launches": launches, "config": config_dict(w, world, args.norm_eps, shard, args.iid)}))
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- end to end: host buffers in, loss out, copies inside the timed region ------------------
    # Every round's X and y come from pinned host memory and its loss array goes back to the host.
    # Two device staging sets: the copy of round i+1 (copy stream) overlaps the compute of round i.
    stages = [([torch.empty_like(t, device=dev) for t in host_in], torch.empty_like(y_host, device=dev))
              for _ in range(2)]
    copy_stream = torch.cuda.Stream(device=dev)
    main_stream = torch.cuda.current_stream(dev)
    copied = [torch.cuda.Event() for _ in range(2)]
    consumed = [torch.cuda.Event() for _ in range(2)]

    def e2e_rounds(n, seed0):
        for i in range(n):
            xs, ys = stages[i % 2]
            with torch.cuda.stream(copy_stream):
                if i >= 2:
                    copy_stream.wait_event(consumed[i % 2])     # round i-2 has finished with this set
                for dst, src in zip(xs, host_in):
                    dst.copy_(src, non_blocking=True)
                ys.copy_(y_host, non_blocking=True)
                copied[i % 2].record(copy_stream)
            main_stream.wait_event(copied[i % 2])
            one_round(seed0 + i, X_of(xs), ys)
            consumed[i % 2].record(main_stream)
            loss_host.copy_(loss_dev, non_blocking=True)

    e2e_rounds(2, 0)
    barrier()
    e0.record()
    copy_stream.wait_event(e0)          # the first copy starts inside the timed region
    e2e_rounds(args.steps, 200)
    e1.record()
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1), dev)
    e2e_value = job_value(per_rank, args.steps, world, ms_e2e)

    # ---- per-kernel-class device times (separate pass, events around each class) ---------------
    ctx.profile(True)
    prof_rounds = min(args.steps, 3)
    for i in range(prof_rounds):
        one_round(300 + i, X_of(dev_in), y_dev)
    prof = ctx.profile_read()
    ctx.profile(False)
    ctx.sync_status()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk = peaks()
    wm = work_model(w, norm=args.norm_eps is not None, data=data if data.is_csr else None)
    if shard:      # this rank ran the local steps of its own subnets only; gather / scatter cover all S
        for k in ("fwd", "dx", "dw_sgd"):
            wm["flops"][k] = wm["flops"][k] * count // w.S
        for k in ("dw_sgd", "norm"):
            if k in wm["bytes"]:
                wm["bytes"][k] = wm["bytes"][k] * count // w.S
    tensor_peak = pk["bf16_tflops_sustained"] if w.precision == "bf16" else None
    kernels = {}
    for name, (n, t_ms) in prof.items():
        if n == 0:
            continue
        ent = {"launches_per_step": n / prof_rounds, "ms_per_step": t_ms / prof_rounds}
        sec = t_ms * 1e-3 / prof_rounds
        if name in wm["flops"] and sec > 0:
            ent["tflops"] = wm["flops"][name] / sec / 1e12
        if name in wm["bytes"] and sec > 0:
            ent["gbs"] = wm["bytes"][name] / sec / 1e9
        kernels[name] = ent
    # Which roofline bounds each class: x*W and delta*W^T are dense contractions (tensor cores);
    # a^T*delta with the fused update moves 10 bytes per weight for 2*B flop, so HBM bounds it, like
    # gather and scatter.  The fp32 path runs its contractions on the CUDA cores.
    dominant = max(kernels, key=lambda k: kernels[k]["ms_per_step"])
    dk = kernels[dominant]
    # the recorded ncu captures are of the plain configurations: no traffic figure for a variant
    variant = bool(args.iid or args.norm_eps is not None or shard or args.dims or args.subnets or args.batch)
    tensor_classes = ("fwd", "dx") if tensor_peak else ()
    if dominant in tensor_classes:
        roof = {"kernel": dominant, "bound": "tensor", "achieved": dk["tflops"], "peak": tensor_peak,
                "unit": "TFLOP/s", "frac": dk["tflops"] / tensor_peak,
                "traffic": None if variant else measured_traffic(w.name, dominant, wm["flops"][dominant] / dk["launches_per_step"]),
                "peak_source": pk["_source"] + " (sustained bf16)",
                "flops_per_launch": wm["flops"][dominant] / dk["launches_per_step"],
                "avg_launch_ms": dk["ms_per_step"] / dk["launches_per_step"]}
    elif dominant in wm["bytes"] and (tensor_peak or dominant not in wm["flops"]):
        gbs = dk["gbs"]
        roof = {"kernel": dominant, "bound": "hbm", "achieved": gbs, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": gbs / pk["hbm_gbs"], "peak_source": pk["_source"],
                "bytes_per_launch": wm["bytes"][dominant] / dk["launches_per_step"],
                "traffic": None if variant else measured_traffic(w.name, dominant, wm["bytes"][dominant] / dk["launches_per_step"]),
                "avg_launch_ms": dk["ms_per_step"] / dk["launches_per_step"]}
    elif dominant in wm["flops"]:
        # fp32 CUDA-core contraction: 148 SMs x 128 FMA lanes x 2 flop x max clock
        alu_peak = 148 * 128 * 2 * pk.get("sm_max_mhz", 1965.0) * 1e6 / 1e12
        roof = {"kernel": dominant, "bound": "alu", "achieved": dk["tflops"], "peak": alu_peak,
                "unit": "TFLOP/s", "frac": dk["tflops"] / alu_peak, "traffic": None,
                "peak_source": "derived: 148 SMs x 128 lanes x 2 x max SM clock"}
    else:
        roof = {"kernel": dominant, "bound": "latency", "achieved": None, "peak": None, "unit": None,
                "frac": None, "traffic": None}
    for name, ent in kernels.items():      # fraction of the relevant measured peak, per class
        if name in tensor_classes and "tflops" in ent:
            ent["frac_of_bf16_peak"] = ent["tflops"] / tensor_peak
        elif "gbs" in ent:
            ent["frac_of_hbm_peak"] = ent["gbs"] / pk["hbm_gbs"]

    cpu = None
    if world == 1 and not args.no_cpu_baseline and not args.iid:
        smp = OracleSample(w, n_sub=2, norm_eps=args.norm_eps)
        t0 = time.perf_counter()
        vals = []
        while len(vals) < 2 or (time.perf_counter() - t0 < 10 and len(vals) < 6):
            vals.append(smp.run(9000 + len(vals))[0])
        cpu = {"value": float(np.mean(vals)), "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
               "sample": smp.describe() + f"; {len(vals)} samples"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": n_warm, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "strong" if shard else "weak", "vs_baseline": None, "dtype": w.precision.replace("fp", "f"),
        "data": "synthetic",
        "config": config_dict(w, world, args.norm_eps, shard, args.iid), "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e / args.steps},
        "gpu_launches": launches, "roofline": roof, "kernels": kernels, "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """Scaling sweep: device-timed whole rounds at every (H, S, K); weights and inputs are drawn on
    the device (same distributions as synth.py) so that the 17 GB networks need no host copy."""
    import torch
    from paper_1910_02120_b200 import api
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    pk = peaks()
    gen = torch.Generator(device=dev)
    for H in [int(x) for x in args.sweep_H.split(",")]:
        dims = (1024, H, H, 100)
        gen.manual_seed(BASE_SWEEP_SEED + H)
        Wd = []
        for l in range(3):
            bound = (6.0 / dims[l]) ** 0.5
            Wd.append((torch.rand(dims[l], dims[l + 1], device=dev, generator=gen) * 2 - 1) * bound)
        bd = [torch.zeros(dims[l + 1], device=dev) for l in range(3)]
        for S in [int(x) for x in args.sweep_S.split(",")]:
            ctx = api.Ist(dims, S, api.IST_BF16, 512, device=str(dev))
            ctx.bind_weights(Wd, bd)
            for K in [int(x) for x in args.sweep_K.split(",")]:
                w = synth.c5(H, S, K)
                X = torch.randn(S * K * 512, 1024, device=dev, generator=gen).to(torch.bfloat16)
                y = torch.randint(0, 100, (S * K * 512,), device=dev, dtype=torch.int32, generator=gen)
                loss = torch.empty(S * K, device=dev)
                ctx.round(1, X, y, w.lr, K, 512, loss_out=loss)
                ctx.sync_status()
                reps = 3 if K >= 10 else 10
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for r in range(reps):
                    ctx.round(2 + r, X, y, w.lr, K, 512, loss_out=loss)
                e1.record()
                torch.cuda.synchronize(dev)
                ctx.sync_status()
                ms = e0.elapsed_time(e1) / reps
                wm = work_model(w)
                flops = sum(wm["flops"].values())
                print(json.dumps({"sweep": "C5", "H": H, "S": S, "K": K, "ms_per_round": ms,
                                  "samples_per_s": w.samples_per_round / (ms * 1e-3),
                                  "gemm_tflops_over_round": flops / (ms * 1e-3) / 1e12,
                                  "frac_of_bf16_peak": flops / (ms * 1e-3) / 1e12 / pk["bf16_tflops_sustained"],
                                  "update_gbs_over_round": wm["bytes"]["dw_sgd"] / (ms * 1e-3) / 1e9,
                                  "mean_loss": float(loss.mean().item())}), flush=True)
                del X, y, loss
            ctx.close()
            del ctx
            torch.cuda.empty_cache()
        del Wd, bd
        torch.cuda.empty_cache()


BASE_SWEEP_SEED = 4321


def main():
    args = parse_args()
    if args.sweep:
        run_sweep(args)
        return
    w = synth.WORKLOADS[args.config]
    if args.local_steps > 0:
        w = w.scaled(K=args.local_steps, name=w.name + f"-K{args.local_steps}")
    if args.dims:
        w = w.scaled(layer_dims=tuple(int(x) for x in args.dims.split(",")), name=w.name + "-reduced")
    if args.subnets > 0:
        w = w.scaled(S=args.subnets)
    if args.batch > 0:
        w = w.scaled(B=args.batch)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
