#!/usr/bin/env python
"""Benchmark of the RanDeS hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload vit_l14] [--storage f32]
    python bench.py --impl reference ...        # the CPU oracle on a bounded sample

One step = one pass of the whole hot path over one synthetic weight set:
compress all K task models into M, retrieve every task once, then stream-add
`--swap` further models and remove them again.  The headline value is the
algorithmic bytes of the step (what the method must move) divided by the
device time of the step, summed over GPUs.  Rank 0 prints one JSON line.
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
sys.path.insert(0, ROOT)

from paper_2505_11204_b200 import workloads as wl  # noqa: E402

FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
WORKLOADS = {"toy": wl.toy, "vit_b32": wl.vit_b32, "gpt2_small": wl.gpt2_small, "flan_t5_base": wl.flan_t5_base,
             "vit_l14": wl.vit_l14}


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vit_l14", choices=sorted(WORKLOADS))
    ap.add_argument("--storage", default=None, choices=["f32", "bf16"])
    ap.add_argument("--tasks", type=int, default=None, help="number of task models K (default: the workload's)")
    ap.add_argument("--context", default="flip", choices=["flip", "gauss"],
                    help="gauss: the Gaussian-like diagonal context of the paper's RD ablation instead of the +-1 flip")
    ap.add_argument("--swap", type=int, default=5, help="models streamed in and out per step")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "rows"],
                    help="with N GPUs: every rank runs the whole workload (weak scaling, default), or every rank holds "
                         "one row slice of every layer (strong scaling); neither needs a collective on the data path")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip timing the CPU oracle")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--check-ranks", action="store_true",
                    help="only bring up the N ranks (nccl with GPUs, gloo without), count them and print "
                         '{"n_gpus": N, "ranks_joined": N}: a check of the launch plumbing, no kernel runs')
    ap.add_argument("--reference-budget-s", type=float, default=240.0,
                    help="--impl reference: wall-clock budget of the timed steps; fewer steps are timed (and the "
                         "line says so) when the requested number would not fit")
    return ap.parse_args(argv)


# --------------------------------------------------------------------------------- ranks
def rank_env(args):
    """(rank, world, local_rank) of this process, after checking them against --gpus.

    Launched by torch.distributed.run the environment carries WORLD_SIZE; it must equal --gpus.
    Launched plainly with --gpus N > 1, bench.py starts the N ranks itself (launch_ranks)."""
    world = os.environ.get("WORLD_SIZE")
    if world is None:
        if args.gpus != 1:
            raise SystemExit("bench.py: --gpus %d needs %d ranks; none were started" % (args.gpus, args.gpus))
        return 0, 1, 0
    world = int(world)
    if world != args.gpus:
        raise SystemExit("bench.py: --gpus %d but WORLD_SIZE=%d: start one rank per GPU (or drop WORLD_SIZE and let "
                         "bench.py start them)" % (args.gpus, world))
    return int(os.environ.get("RANK", "0")), world, int(os.environ.get("LOCAL_RANK", "0"))


def launch_ranks(args, argv):
    """`python bench.py --gpus N` without a launcher: run N ranks of this script on this node through
    torch.distributed.run (rendezvous on 127.0.0.1, a free port) and return its exit code."""
    import socket

    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(args.gpus),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


def check_ranks(args):
    """Bring the ranks up, count them with one all-reduce, print the count: nothing else runs."""
    import torch
    import torch.distributed as dist

    rank, world, local = rank_env(args)
    joined = 1
    if world > 1:
        if torch.cuda.is_available():
            torch.cuda.set_device(local)
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
            t = torch.ones(1, dtype=torch.float64, device="cuda")
        else:
            dist.init_process_group("gloo")
            t = torch.ones(1, dtype=torch.float64)
        dist.all_reduce(t)
        joined = int(t.item())
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"n_gpus": world, "ranks_joined": joined, "backend": "nccl" if torch.cuda.is_available() else "gloo",
                          "check": "ranks only; no kernel was launched"}))
    return 0 if joined == world else 1


def make_workload(args) -> wl.Workload:
    w = WORKLOADS[args.workload]()
    if args.storage is not None:
        w = w.with_storage(wl.BF16 if args.storage == "bf16" else wl.F32)
    if args.tasks is not None:
        w = w.with_tasks(args.tasks)
    if getattr(args, "context", "flip") == "gauss":
        w = w.with_gaussian_context()
    return w


def step_bytes(w: wl.Workload, n_swap: int, out_bytes: int = 4):
    """Algorithmic bytes of each operation of one step (M is fp32)."""
    s = 2 if w.storage == wl.BF16 else 4
    P, K = w.n_params, w.n_tasks
    b = {
        "compress": (K * s + s + 4) * P,
        "retrieve": (4 + s + out_bytes) * P,          # per call; K calls per step
        "add": (8 + 2 * s) * P,                       # per call; n_swap calls per step
        "remove": (8 + 2 * s) * P,
    }
    total = b["compress"] + K * b["retrieve"] + n_swap * (b["add"] + b["remove"])
    return b, total


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def kernel_source_hash():
    import hashlib

    h = hashlib.sha256()
    for name in ("randes_kernels.cu", "randes_group.cu", "randes_device.cuh"):
        with open(os.path.join(ROOT, "paper_2505_11204_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def read_traffic():
    """DRAM traffic figures taken with ncu (profiles/traffic.txt); empty once the kernels changed."""
    out = {}
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.txt")) as f:
            for line in f:
                if line.startswith("#") or not line.strip():
                    continue
                k, v = line.split()[:2]
                out[k] = v
        if out.get("source_sha256") != kernel_source_hash():
            return {}
        return {k: float(v) for k, v in out.items() if k != "source_sha256"}
    except Exception:
        return {}


def max_over_ranks(values, world, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity when world == 1)."""
    if world <= 1:
        return list(values)
    import torch
    import torch.distributed as dist

    t = torch.tensor(values, dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def aggregate_value(total_bytes_per_rank: float, ms_per_step_max: float, world: int) -> float:
    """Whole-job GB/s: every rank moves total_bytes per step; time is the slowest rank's."""
    return world * total_bytes_per_rank / (ms_per_step_max * 1e-3) / 1e9


def aggregate_value_sliced(total_bytes_whole_model: float, ms_per_step_max: float) -> float:
    """Whole-job GB/s when the ranks hold row slices of one model: its bytes once, over the slowest rank's time."""
    return total_bytes_whole_model / (ms_per_step_max * 1e-3) / 1e9


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def config_dict(w, args):
    """What was run -- the same dict from both arms for the same flags (what differs between them goes into `note`)."""
    return {"workload": "%s-shaped synthetic weights, K=%d tasks, %d layers, %.1f M params; step = compress + %d retrieves + %d adds + %d removes"
                        % (w.name, w.n_tasks, w.n_layers, w.n_params / 1e6, w.n_tasks, args.swap, args.swap),
            "storage": "bf16" if w.storage == wl.BF16 else "f32", "lambda": w.lam,
            **({"context": "Gaussian-like diagonal (the RD ablation of Section 5.5)"} if getattr(args, "context", "flip") == "gauss" else {}),
            "l2": ("inputs exceed L2: every call streams at least %.2f GB" if (4 + 4) * w.n_params > 2 * 126e6 else
                   "working set of %.3f GB fits in L2: latency-bound, not a roofline case")
                  % ((4 + (2 if w.storage == wl.BF16 else 4)) * w.n_params / 1e9)}


# --------------------------------------------------------------------------------- CPU oracle legs
def run_oracle_step(ro, ws, base, tasks, extra, n_swap):
    K = ws.n_tasks
    M = ro.compress(ws.spec, ws.storage, ws.task_ids, ws.seeds, base, tasks)
    for t, s in zip(ws.task_ids, ws.seeds):
        ro.retrieve(ws.spec, ws.storage, wl.F32, t, s, ws.lam, base, M)
    for j in range(n_swap):
        ro.add_model(ws.spec, ws.storage, K + j, ws.seeds[0] + K + j, base, extra[j], M)
    for j in range(n_swap):
        ro.remove_model(ws.spec, ws.storage, K + j, ws.seeds[0] + K + j, base, extra[j], M)
    return M


def time_oracle(w: wl.Workload, n_swap: int, steps: int, warmup: int, budget_s: float, models=None):
    """The CPU oracle, as it stands, on the WHOLE workload: `warmup` untimed steps, then up to `steps` timed ones
    (fewer when they would not fit `budget_s` of wall clock; the result says how many ran).  `models` =
    (base, [K + n_swap models]) as host arrays, when the caller already holds them."""
    from oracle import randes_oracle as ro

    K = w.n_tasks
    if models is None:
        ids = list(w.task_ids) + [K + j for j in range(n_swap)]
        models = wl.model_set(w, ids, threads=os.cpu_count() or 1)
    base, all_models = models
    tasks, extra = all_models[:K], all_models[K:]
    t_first = None
    for _ in range(warmup):
        t0 = time.perf_counter()
        run_oracle_step(ro, w, base, tasks, extra, n_swap)
        t_first = time.perf_counter() - t0
    ran, t_sum = 0, 0.0
    while ran < steps:
        est = t_first if ran == 0 else t_sum / ran
        if ran >= 1 and est is not None and t_sum + est > budget_s:
            break
        t0 = time.perf_counter()
        run_oracle_step(ro, w, base, tasks, extra, n_swap)
        t_sum += time.perf_counter() - t0
        ran += 1
    dt = t_sum / max(ran, 1)
    _, total = step_bytes(w, n_swap)
    return {"value": total / dt / 1e9, "unit": "GB/s", "cores": ro.num_threads(), "kind": "oracle",
            "sample": "the whole workload (%s: all %d layers, %.1f M params, K=%d, swap=%d): %d warm-up + %d timed step(s), %.2f s per step"
                      % (w.name, w.n_layers, w.n_params / 1e6, K, n_swap, warmup, ran, dt),
            "ms_per_step": dt * 1e3, "steps_timed": ran, "warmup_run": warmup}


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return 0
    w = make_workload(args)
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    r = time_oracle(w, args.swap, steps, warmup, args.reference_budget_s)
    note = "CPU oracle on the whole workload; %d warm-up step(s), %d of the %d requested steps timed" % (warmup, r["steps_timed"], steps)
    if r["steps_timed"] < steps:
        note += " (the rest would have exceeded the %.0f s budget of this arm)" % args.reference_budget_s
    line = {
        "impl": "reference", "metric": "hot_path_algorithmic_bandwidth", "value": r["value"], "unit": "GB/s",
        "n_gpus": args.gpus, "steps": steps, "warmup": warmup, "steps_timed": r["steps_timed"], "ms_per_step": r["ms_per_step"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32" if w.storage == wl.F32 else "bf16 storage, f32 arithmetic", "data": "synthetic",
        "config": config_dict(w, args), "note": note,
        "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
        "e2e": {"value": r["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def check_linear_sample(c):
    """Compare the kept block of randes_linear's output with the CPU oracle (fp64 from the definition) within the
    tolerance of the GPU tests, sqrt(2 cols + 2) 2^-24 sum_c |x| (|W_0| + |lambda M|).  Runs in the baseline leg."""
    import numpy as np

    from oracle import randes_oracle as ro

    wq = c["workload"]
    t = wq.task_ids[c["task"]]
    s_ = wq.seeds[c["task"]]
    y_ref, y_abs = ro.linear(wq.spec, wq.storage, t, s_, c["lam"], c["layer"], c["x"], c["base"], c["M"], m_dtype=wl.BF16)
    cols = wq.cols[c["layer"]]
    tol = np.sqrt(2.0 * cols + 2.0) * 2.0 ** -24 * y_abs + 1e-30
    err = np.abs(c["y"].astype(np.float64) - y_ref)
    return {"checked": bool((err <= tol).all()), "checked_outputs": int(err.size), "worst_error_over_tolerance": float((err / tol).max()),
            "check": "%d sampled token rows x all %d features against the CPU oracle" % (len(c["tokens"]), y_ref.shape[1])}


def time_bf16_storage(w, n_swap, dev, stream, peak, peak_kind, world, barrier):
    """compress / retrieve / add / remove of the same workload with bf16 weights (fp32 superposition and output).
    Values are drawn on the device (seeded; the kernels have no data-dependent branches)."""
    import torch

    from paper_2505_11204_b200 import randes

    wb = w.with_storage(wl.BF16)
    K = wb.n_tasks
    offs, total_el = [], 0
    for r, c in zip(wb.rows, wb.cols):
        offs.append(total_el)
        total_el += (r * c + 63) // 64 * 64
    views = lambda flat: [flat[o:o + r * c].view(r, c) for o, r, c in zip(offs, wb.rows, wb.cols)]
    g = torch.Generator(device=dev).manual_seed(977)
    base32 = torch.randn(total_el, device=dev, generator=g) * 0.02
    shared = torch.randn(total_el, device=dev, generator=g)
    flats = [base32.to(torch.bfloat16)]
    for _ in range(K + 1):
        d = wb.scale * (0.5 * shared + (0.75 ** 0.5) * torch.randn(total_el, device=dev, generator=g))
        flats.append((base32 + d).to(torch.bfloat16))
        del d
    del base32, shared
    vs = [views(f) for f in flats]
    p_base, p_tasks, p_new = randes.ptr_array(vs[0]), randes.ptr_array(vs[1:1 + K]), randes.ptr_array(vs[1 + K])
    plan = randes.Plan.from_workload(wb, max_tasks=K + 1, device=dev)
    M = plan.new_superposition()
    out = plan.new_output(wl.F32)
    p_out = randes.ptr_array(out)
    sh = stream.cuda_stream
    b, _ = step_bytes(wb, n_swap)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    spans = {"compress": [], "retrieve": [], "add": [], "remove": []}
    for rep in range(3 + 10):
        e = [ev() for _ in range(5)]
        e[0].record(stream)
        randes.randes_compress(plan.handle, p_base, p_tasks, M, sh)
        e[1].record(stream)
        for t in wb.task_ids:
            randes.randes_retrieve(plan.handle, t, wb.lam, wl.F32, p_base, M, p_out, sh)
        e[2].record(stream)
        randes.randes_add_model(plan.handle, K, wb.seeds[0] + K, p_base, p_new, M, sh)
        e[3].record(stream)
        randes.randes_remove_model(plan.handle, K, p_base, p_new, M, sh)
        e[4].record(stream)
        if rep >= 3:
            for j, n in enumerate(("compress", "retrieve", "add", "remove")):
                spans[n].append((e[j], e[j + 1]))
    barrier()
    res = {"storage": "bf16", "superposition": "f32", "output": "f32", "tasks": K, "params_M": wb.n_params / 1e6,
           "timed": "10 rounds of compress + K retrieves + add + remove after 3 warm-up rounds"}
    calls = {"compress": 1, "retrieve": K, "add": 1, "remove": 1}
    for n, sp in spans.items():
        ms = max_over_ranks([sum(a.elapsed_time(z) for a, z in sp) / (len(sp) * calls[n])], world, dev)[0]
        gbs = b[n] / (ms * 1e-3) / 1e9
        res[n] = {"ms_per_call": ms, "GBps": gbs, "Gparams_per_s": wb.n_params / (ms * 1e-3) / 1e9,
                  "frac_of_%s_peak" % peak_kind: gbs / peak, "frac_of_nominal_8TBps": gbs / NOMINAL_HBM_GBS,
                  "bytes_per_param": b[n] / wb.n_params}
    plan.close()
    return res


# --------------------------------------------------------------------------------- GPU legs
def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist

    from paper_2505_11204_b200 import build, randes

    rank, world, local = rank_env(args)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if not os.path.exists(randes.LIB_PATH):
        if rank == 0:
            build.build_library()
        if world > 1:
            dist.barrier()
    randes.lib()

    w_whole = make_workload(args)
    sliced = args.shard == "rows" and world > 1
    # row slices: the transforms move data across layers and flip by column, never across rows, so a slice is a
    # complete, smaller problem (synthetic values are drawn per slice; they do not influence speed)
    w = wl.row_slice(w_whole, rank, world)[0] if sliced else w_whole
    K, n_swap = w.n_tasks, args.swap
    ids = list(w.task_ids) + [K + j for j in range(n_swap)]
    swap_seeds = [w.seeds[0] + K + j for j in range(n_swap)]
    want_e2e = not args.no_e2e
    e2e_skipped = None
    if want_e2e:
        # the end-to-end leg keeps every model of the step in pinned host memory, once per rank
        try:
            import psutil

            s_b = 2 if w.storage == wl.BF16 else 4
            need = world * (len(ids) + 1) * w.n_params * s_b * 1.25    # every model of the step, plus slack
            avail = psutil.virtual_memory().available
            if need > 0.8 * avail:
                want_e2e = False
                e2e_skipped = "not measured: %d ranks would pin %.0f GB of host memory, %.0f GB available" % (
                    world, need / 1e9, avail / 1e9)
        except ImportError:
            pass

    # ---- inputs: generated on the host (seeded), one flat arena per model (pinned when the
    #      end-to-end leg needs it again), copied to a flat device arena; layers are views
    tdt = torch.bfloat16 if w.storage == wl.BF16 else torch.float32
    offs, total_el = [], 0
    for r, c in zip(w.rows, w.cols):
        offs.append(total_el)
        total_el += (r * c + 63) // 64 * 64           # 256-byte aligned layer starts

    def views(flat):
        return [flat[o:o + r * c].view(r, c) for o, r, c in zip(offs, w.rows, w.cols)]

    def host_arena(arrs):
        flat = torch.zeros(total_el, dtype=tdt, pin_memory=want_e2e)
        for v, a in zip(views(flat), arrs):
            v.copy_(torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(a))
        return flat

    base_np, models_np = wl.model_set(w, ids, threads=max(1, (os.cpu_count() or 1) // world))
    h_flat = [host_arena(base_np)] + [host_arena(m) for m in models_np]     # [0] = W_0, [1 + i] = model i
    del base_np, models_np

    def device_set():
        flats = [torch.empty(total_el, dtype=tdt, device=dev) for _ in h_flat]
        vs = [views(f) for f in flats]
        return {"flat": flats, "base": vs[0], "models": vs[1:], "p_base": randes.ptr_array(vs[0]),
                "p_tasks": randes.ptr_array(vs[1:1 + K]), "p_swap": [randes.ptr_array(m) for m in vs[1 + K:]]}

    dset = device_set()
    for dst, src in zip(dset["flat"], h_flat):
        dst.copy_(src, non_blocking=True)
    torch.cuda.synchronize()
    d_base, d_models = dset["base"], dset["models"]
    if not want_e2e:
        del h_flat

    plan = randes.Plan.from_workload(w, max_tasks=K + n_swap, device=dev)
    M = plan.new_superposition()
    out = plan.new_output(wl.F32)
    p_base, p_tasks, p_swap = dset["p_base"], dset["p_tasks"], dset["p_swap"]
    p_out = randes.ptr_array(out)
    stream = torch.cuda.current_stream(dev)
    sh = stream.cuda_stream
    names = ["compress", "retrieve", "add", "remove"]

    def step(events=None):
        def mark():
            if events is not None:
                e = torch.cuda.Event(enable_timing=True)
                e.record(stream)
                events.append(e)
        mark()
        randes.randes_compress(plan.handle, p_base, p_tasks, M, sh)
        mark()
        for t in w.task_ids:
            randes.randes_retrieve(plan.handle, t, w.lam, wl.F32, p_base, M, p_out, sh)
        mark()
        for j in range(n_swap):
            randes.randes_add_model(plan.handle, K + j, swap_seeds[j], p_base, p_swap[j], M, sh)
        mark()
        for j in range(n_swap):
            randes.randes_remove_model(plan.handle, K + j, p_base, p_swap[j], M, sh)
        mark()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    barrier()
    def timed_run():
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
            time.sleep(0.3)
        launches0 = randes.randes_launch_count()
        evs = []
        t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t_begin.record(stream)
        for _ in range(args.steps):
            step(evs)
        t_end.record(stream)
        barrier()
        launches = randes.randes_launch_count() - launches0
        clocks = sampler.stop() if rank == 0 else None
        return evs, t_begin.elapsed_time(t_end), launches, clocks

    def clocks_bad(c):
        if not c or c.get("sm_mhz") is None:
            return False
        bad = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"} & set(c["reasons"])
        stuck = c["sm_mhz"] < 0.6 * c["sm_max_mhz"] and not c["reasons"]
        return bool(bad) or stuck

    evs, total_ms, launches, clocks = timed_run()
    flag = torch.tensor([1.0 if (rank == 0 and clocks_bad(clocks)) else 0.0], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(flag, op=dist.ReduceOp.MAX)
    if float(flag[0]) > 0:      # throttled or clock-locked: measure once more
        first = clocks
        evs, total_ms, launches, clocks = timed_run()
        if rank == 0:
            clocks["remeasured_after"] = first

    op_ms = {n: 0.0 for n in names}
    for s_i in range(args.steps):
        e = evs[s_i * 5:(s_i + 1) * 5]
        for j, n in enumerate(names):
            op_ms[n] += e[j].elapsed_time(e[j + 1])
    red = max_over_ranks([total_ms] + [op_ms[n] for n in names], world, dev)
    total_ms, op_ms = red[0], {n: red[1 + j] for j, n in enumerate(names)}

    b, total_bytes = step_bytes(w, n_swap)
    ms_per_step = total_ms / args.steps
    whole_bytes = step_bytes(w_whole, n_swap)[1]
    value = aggregate_value_sliced(whole_bytes, ms_per_step) if sliced else aggregate_value(total_bytes, ms_per_step, world)
    peak, peak_kind = measured_peak()
    calls = {"compress": 1, "retrieve": K, "add": n_swap, "remove": n_swap}
    ops = {}
    for n in names:
        c = calls[n] * args.steps
        if c == 0:
            continue
        ms = op_ms[n] / c
        gbs = b[n] / (ms * 1e-3) / 1e9
        ops[n] = {"ms_per_call": ms, "GBps": gbs, "Gparams_per_s": w.n_params / (ms * 1e-3) / 1e9,
                  "frac_of_%s_peak" % peak_kind: gbs / peak, "frac_of_nominal_8TBps": gbs / NOMINAL_HBM_GBS,
                  "share_of_step": op_ms[n] / total_ms}
    # dominant kernel = the kernel instantiation with the largest share of the step
    shares = {"retrieve_kernel": op_ms["retrieve"],
              "accumulate_kernel<single task> (add, remove)": op_ms.get("add", 0.0) + op_ms.get("remove", 0.0),
              "compress_group_kernel + accumulate_kernel<compress>": op_ms["compress"]}
    dom = max(shares, key=shares.get)
    rd = args.context == "gauss"          # every call then runs the general-context kernels: no ncu traffic figure applies
    traffic_tbl = {} if rd else read_traffic()
    if dom == "retrieve_kernel":
        dom_bytes, dom_ms = b["retrieve"], ops["retrieve"]["ms_per_call"]
        traffic = traffic_tbl.get("retrieve_kernel_bytes_per_param")
        traffic = traffic * w.n_params if traffic and w.storage == wl.F32 else None
    elif dom.startswith("accumulate_kernel<single"):
        dom_bytes, dom_ms = b["add"], (op_ms["add"] + op_ms["remove"]) / (2 * n_swap * args.steps)
        traffic = traffic_tbl.get("accumulate_kernel_single_bytes_per_param")
        traffic = traffic * w.n_params if traffic and w.storage == wl.F32 else None
    else:
        dom_bytes, dom_ms = b["compress"], ops["compress"]["ms_per_call"]
        traffic = traffic_tbl.get("compress_kernels_traffic_over_algorithmic")
        traffic = traffic * dom_bytes if traffic and w.storage == wl.F32 else None
    achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
    if rd:
        dom = {"retrieve_kernel": "context_retrieve_kernel", "accumulate_kernel<single task> (add, remove)": "context_accumulate_kernel<one task> (add, remove)",
               "compress_group_kernel + accumulate_kernel<compress>": "context_accumulate_kernel<compress>"}[dom]
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak,
                "peak_source": "%s copy bandwidth (MEASURED_PEAKS.json)" % peak_kind if peak_kind == "measured"
                               else "fallback copy bandwidth",
                "unit": "GB/s", "frac": achieved / peak, "traffic": traffic,
                "traffic_source": "ncu dram bytes on the ViT-B/32-shaped case scaled by parameter count (profiles/)"
                                  if traffic else "none valid for the current kernel sources",
                "share_of_step": max(shares.values()) / total_ms,
                "per_kernel": {k: {"achieved": ops[k]["GBps"], "frac": ops[k]["GBps"] / peak, "bytes_per_launch": b[k]}
                               for k in ops}}

    # ---- beyond the step: all K tasks rebuilt in one launch (batched retrieve), timed alone
    extras = {}
    nb = min(K, 32)
    if nb >= 2 and not rd:                 # (batched retrieve, the Gram matrix and the fused linear layer are not offered under that context)
        try:
            b_outs = [plan.new_output(wl.F32) for _ in range(nb)]
            p_bout = randes.ptr_array(b_outs)
            b_ids = list(w.task_ids[:nb])
            for _ in range(2):
                randes.randes_retrieve_batch(plan.handle, b_ids, w.lam, wl.F32, p_base, M, p_bout, sh)
            barrier()
            a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = 5
            a.record(stream)
            for _ in range(reps):
                randes.randes_retrieve_batch(plan.handle, b_ids, w.lam, wl.F32, p_base, M, p_bout, sh)
            z.record(stream)
            barrier()
            ms = max_over_ranks([a.elapsed_time(z)], world, dev)[0] / reps
            s_el = 2 if w.storage == wl.BF16 else 4
            byts = (s_el + 4 + nb * 4) * w.n_params      # W_0 once, M once (repeats served by L2), nb outputs
            extras["retrieve_batch"] = {"tasks": nb, "ms_per_call": ms, "ms_per_model": ms / nb,
                                        "Gparams_per_s": nb * w.n_params / (ms * 1e-3) / 1e9,
                                        "GBps": byts / (ms * 1e-3) / 1e9, "frac_of_%s_peak" % peak_kind: byts / (ms * 1e-3) / 1e9 / peak,
                                        "speedup_per_model_vs_retrieve": ops["retrieve"]["ms_per_call"] / (ms / nb)}
            del b_outs, p_bout
            torch.cuda.empty_cache()
        except torch.OutOfMemoryError:
            extras["retrieve_batch"] = None

    # ---- the step's n_swap models added in one pass over M instead of one pass each, timed alone
    if n_swap >= 2:
        p_swap_all = randes.ptr_array(dset["models"][K:])
        swap_ids = [K + j for j in range(n_swap)]
        evs = []
        for rep in range(2 + 5):
            a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            randes.randes_add_models(plan.handle, swap_ids, swap_seeds, p_base, p_swap_all, M, sh)
            z.record(stream)
            for j in range(n_swap):
                randes.randes_remove_model(plan.handle, K + j, p_base, p_swap[j], M, sh)
            if rep >= 2:
                evs.append((a, z))
        barrier()
        ms = max_over_ranks([sum(a.elapsed_time(z) for a, z in evs) / len(evs)], world, dev)[0]
        s_el = 2 if w.storage == wl.BF16 else 4
        byts = (n_swap * s_el + s_el + 8) * w.n_params      # n_swap models, W_0 (repeats served by L2), M in and out
        extras["add_models"] = {"models": n_swap, "ms_per_call": ms, "ms_per_model": ms / n_swap,
                                "GBps": byts / (ms * 1e-3) / 1e9, "frac_of_%s_peak" % peak_kind: byts / (ms * 1e-3) / 1e9 / peak,
                                "speedup_per_model_vs_add": ops["add"]["ms_per_call"] / (ms / n_swap)}

    # ---- interference diagnostics: the Gram matrix of the K transformed deltas (one pass over all K + 1 models), timed alone
    if K <= 32 and not rd:
        try:
            gram = torch.empty(K, K, dtype=torch.float64, device=dev)
            g_bytes = randes.randes_delta_gram_scratch_bytes(plan.handle)
            g_scratch = torch.empty(g_bytes // 8, dtype=torch.float64, device=dev)
            spans = []
            for rep in range(1 + 3):
                a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                randes.randes_delta_gram(plan.handle, p_base, p_tasks, gram, g_scratch, g_bytes, sh)
                z.record(stream)
                if rep >= 1:
                    spans.append((a, z))
            barrier()
            ms = max_over_ranks([sum(a.elapsed_time(z) for a, z in spans) / len(spans)], world, dev)[0]
            s_el = 2 if w.storage == wl.BF16 else 4
            byts = (K + 1) * s_el * w.n_params
            cos, mean_cos = randes.randes_pairwise_cosines(gram)
            extras["delta_gram"] = {"tasks": K, "ms_per_call": ms, "GBps": byts / (ms * 1e-3) / 1e9,
                                    "frac_of_%s_peak" % peak_kind: byts / (ms * 1e-3) / 1e9 / peak,
                                    "mean_pairwise_cosine_after_transform": mean_cos,
                                    "interference_norm_task0": randes.randes_interference_norm(gram, 0, w.lam),
                                    "note": "fp64 tensor-core products (mma.m8n8k4), bound by the fp64 pipe; the synthetic deltas have cosine 0.25 before the transforms"}
            del gram, g_scratch
        except torch.OutOfMemoryError:
            extras["delta_gram"] = None

    # ---- adapter deltas (Section 5.8): the tasks' tensors already hold the deltas (base = NULL), only the layers that carry
    #      an adapter are in the plan; rank-16 deltas materialised beforehand, here random values of that shape
    if args.workload == "flan_t5_base":
        try:
            wa = wl.subset(w, wl.flan_t5_lora_targets(w), w.name + ":adapter-targets")
            g_a = torch.Generator(device=dev).manual_seed(4321)
            a_tasks = [[(torch.randn(r, c, device=dev, generator=g_a) * 1e-4).to(tdt) for r, c in zip(wa.rows, wa.cols)] for _ in range(K + 1)]
            plan_a = randes.Plan.from_workload(wa, max_tasks=K + 1, device=dev)
            M_a = plan_a.new_superposition()
            pa = randes.ptr_array(a_tasks[:K])
            pa_new = randes.ptr_array(a_tasks[K])
            t_c, t_a = [], []
            for rep in range(2 + 5):
                e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                e0.record(stream)
                randes.randes_compress(plan_a.handle, None, pa, M_a, sh)
                e1.record(stream)
                randes.randes_add_model(plan_a.handle, 1000, 77, None, pa_new, M_a, sh)
                e2.record(stream)
                randes.randes_remove_model(plan_a.handle, 1000, None, pa_new, M_a, sh)
                if rep >= 2:
                    t_c.append((e0, e1)); t_a.append((e1, e2))
            barrier()
            ms_c = max_over_ranks([sum(x.elapsed_time(y) for x, y in t_c) / len(t_c)], world, dev)[0]
            ms_a = max_over_ranks([sum(x.elapsed_time(y) for x, y in t_a) / len(t_a)], world, dev)[0]
            s_el = 2 if w.storage == wl.BF16 else 4
            extras["adapter_deltas"] = {"layers": wa.n_layers, "params_M": wa.n_params / 1e6, "tasks": K,
                                        "compress_ms": ms_c, "compress_GBps": (K * s_el + 4) * wa.n_params / (ms_c * 1e-3) / 1e9,
                                        "add_ms": ms_a, "add_GBps": (8 + s_el) * wa.n_params / (ms_a * 1e-3) / 1e9,
                                        "note": "tasks given as deltas (no base): compress moves K*s + 4 bytes per parameter, add 8 + s"}
            plan_a.close()
            del a_tasks, M_a
            torch.cuda.empty_cache()
        except torch.OutOfMemoryError:
            extras["adapter_deltas"] = None

    lin_check = None
    # ---- a linear layer on the retrieved weight, the weight never written (tensor cores): the largest
    #      repeated matrix of the set, bf16 weights and a bf16 superposition, 8192 tokens, timed alone
    class NotOffered(Exception):
        pass

    try:
        if rd:
            raise NotOffered
        reps_by_group = {}
        for l, g in enumerate(w.group):
            if w.rows[l] > 1 and w.cols[l] % 8 == 0:
                reps_by_group.setdefault(g, []).append(l)
        cand = [ls for ls in reps_by_group.values() if len(ls) > 1] or list(reps_by_group.values())
        grp = max(cand, key=lambda ls: w.rows[ls[0]] * w.cols[ls[0]])[:4]
        wl_lin = wl.subset(w, grp, w.name + ":linear").with_storage(wl.BF16).with_tasks(min(K, 4))
        g_lin = torch.Generator(device=dev).manual_seed(1234)
        lin_base = [(torch.randn(r, c, device=dev, generator=g_lin) * 0.02).to(torch.bfloat16) for r, c in zip(wl_lin.rows, wl_lin.cols)]
        lin_tasks = [[(b.float() + 1e-3 * torch.randn(b.shape, device=dev, generator=g_lin)).to(torch.bfloat16) for b in lin_base]
                     for _ in range(wl_lin.n_tasks)]
        plan_lin = randes.Plan.from_workload(wl_lin, max_tasks=wl_lin.n_tasks, device=dev, m_dtype=wl.BF16)
        M_lin = plan_lin.compress(lin_base, lin_tasks)
        n_tok = 8192
        rows_l, cols_l = wl_lin.rows[0], wl_lin.cols[0]
        x_lin = torch.randn(n_tok, cols_l, device=dev, generator=g_lin).to(torch.bfloat16)
        y_lin = torch.empty(n_tok, rows_l, device=dev, dtype=torch.float32)
        pb_lin = randes.ptr_array(lin_base)
        for _ in range(3):
            randes.randes_linear(plan_lin.handle, 0, w.lam, 0, x_lin, n_tok, pb_lin, M_lin, y_lin, sh)
        barrier()
        # a sampled block of this output (both 128-token halves of the first and the last block of tokens, every
        # feature) is kept, with the operands, for the comparison with the CPU oracle in the baseline leg
        tok = sorted(set(t for t in (0, 1, 127, 128, 129, 255, n_tok // 2, n_tok - 256, n_tok - 129, n_tok - 128, n_tok - 1) if 0 <= t < n_tok))
        u16 = lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)
        lin_check = {"workload": wl_lin, "task": 0, "layer": 0, "lam": w.lam, "tokens": tok,
                     "x": u16(x_lin[tok].contiguous()), "y": y_lin[tok].cpu().numpy(), "base": [u16(b) for b in lin_base],
                     "M": [u16(plan_lin.slot(M_lin, l)) for l in range(wl_lin.n_layers)]}
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 20
        a.record(stream)
        for i in range(reps):
            randes.randes_linear(plan_lin.handle, i % wl_lin.n_tasks, w.lam, i % len(grp), x_lin, n_tok, pb_lin, M_lin, y_lin, sh)
        z.record(stream)
        barrier()
        ms = max_over_ranks([a.elapsed_time(z)], world, dev)[0] / reps
        flops = 4.0 * n_tok * rows_l * cols_l            # two products of 2 * tokens * rows * cols each
        try:
            with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
                tc_peak, tc_kind = float(json.load(f)["bf16_tflops"]), "measured burst"
        except Exception:
            tc_peak, tc_kind = 1590.0, "fallback"
        extras["linear"] = {"layer_shape": [rows_l, cols_l], "tokens": n_tok, "ms_per_call": ms, "TFLOPs": flops / (ms * 1e-3) / 1e12,
                            "bound": "tensor", "peak_TFLOPs": tc_peak, "peak_source": "%s bf16 GEMM (MEASURED_PEAKS.json)" % tc_kind
                            if tc_kind != "fallback" else "fallback bf16 GEMM",
                            "frac": flops / (ms * 1e-3) / 1e12 / tc_peak, "giveups": randes.randes_linear_giveups(), "checked": None,
                            "note": "y = x W_0^T + lambda (x D) M^T, bf16 operands, fp32 accumulators; flops count both products"}
        plan_lin.close()
        del lin_base, lin_tasks, M_lin, x_lin, y_lin
        torch.cuda.empty_cache()
    except (torch.OutOfMemoryError, NotOffered):
        extras["linear"] = None

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region.
    #      Every step copies all its inputs from pinned host memory and all its results back.
    #      Copies and kernels are pipelined: the next step's inputs arrive in a second set of
    #      device buffers while this step computes, and retrieved models leave through two
    #      alternating output buffers.
    e2e = None
    if want_e2e:
        del out, p_out
        sets = [dset, device_set()]
        out_el = sum((r * c + 63) // 64 * 64 for r, c in zip(w.rows, w.cols))
        o_flat = [torch.empty(out_el, dtype=torch.float32, device=dev) for _ in range(2)]
        o_ptrs = [randes.ptr_array(views(f)) for f in o_flat]
        h_out = [torch.empty(out_el, dtype=torch.float32, pin_memory=True) for _ in range(2)]
        h_M = torch.empty_like(M, device="cpu").pin_memory()
        s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        ev = lambda: torch.cuda.Event()
        ev_in, ev_set_free = [ev(), ev()], [ev(), ev()]
        ev_ret, ev_out_free, ev_m_free = [ev(), ev()], [ev(), ev()], ev()
        for e_ in ev_set_free + ev_out_free + [ev_m_free]:
            e_.record(stream)

        def e2e_step(i):
            k = i % 2
            ds = sets[k]
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_set_free[k])
                for dst, src in zip(ds["flat"], h_flat):
                    dst.copy_(src, non_blocking=True)
                ev_in[k].record(s_in)
            stream.wait_event(ev_in[k])
            stream.wait_event(ev_m_free)
            randes.randes_compress(plan.handle, ds["p_base"], ds["p_tasks"], M, sh)
            for n_t, ti in enumerate(w.task_ids):
                bfr = n_t % 2
                stream.wait_event(ev_out_free[bfr])
                randes.randes_retrieve(plan.handle, ti, w.lam, wl.F32, ds["p_base"], M, o_ptrs[bfr], sh)
                ev_ret[bfr].record(stream)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_ret[bfr])
                    h_out[bfr].copy_(o_flat[bfr], non_blocking=True)
                    ev_out_free[bfr].record(s_out)
            for j in range(n_swap):
                randes.randes_add_model(plan.handle, K + j, swap_seeds[j], ds["p_base"], ds["p_swap"][j], M, sh)
            for j in range(n_swap):
                randes.randes_remove_model(plan.handle, K + j, ds["p_base"], ds["p_swap"][j], M, sh)
            ev_set_free[k].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_set_free[k])
                h_M.copy_(M, non_blocking=True)
                ev_m_free.record(s_out)

        e2e_step(0)
        stream.wait_stream(s_out)
        barrier()
        a, z = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        s_in.wait_event(a)
        for i in range(args.e2e_steps):
            e2e_step(i + 1)
        stream.wait_stream(s_out)
        stream.wait_stream(s_in)
        z.record(stream)
        barrier()
        e2e_ms = max_over_ranks([a.elapsed_time(z)], world, dev)[0] / args.e2e_steps
        s_b = 2 if w.storage == wl.BF16 else 4
        e2e = {"value": aggregate_value_sliced(whole_bytes, e2e_ms) if sliced else aggregate_value(total_bytes, e2e_ms, world),
               "unit": "GB/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": (1 + K + n_swap) * w.n_params * s_b,
               "d2h_bytes_per_step": (K + 1) * w.n_params * 4, "steps": args.e2e_steps,
               "note": "copies and kernels pipelined over three streams; PCIe-bound"}
        del h_out, h_M, sets, o_flat

    plan.close()
    del d_models, d_base, M, dset
    torch.cuda.empty_cache()

    # ---- the same workload with the weights stored as bf16 (fp32 superposition, fp32 output), timed alone
    if w.storage == wl.F32 and args.workload != "toy":
        try:
            extras["bf16_storage"] = time_bf16_storage(w, n_swap, dev, stream, peak, peak_kind, world, barrier)
        except torch.OutOfMemoryError:
            extras["bf16_storage"] = None
        torch.cuda.empty_cache()

    # ---- the CPU oracle beside it: the whole workload, one warm-up step and two timed ones (rank 0, one GPU only);
    #      the sampled block of the linear layer's output is compared with the oracle here as well
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        host_models = None
        if want_e2e:
            def layers_np(flat):
                vs = views(flat)
                return [v.view(torch.int16).numpy().view(np.uint16) if v.dtype == torch.bfloat16 else v.numpy() for v in vs]
            host_models = (layers_np(h_flat[0]), [layers_np(f) for f in h_flat[1:]])
        cpu = time_oracle(w, n_swap, 2, 1, 120.0, models=host_models)
        cpu = {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample")}
        del host_models
        if lin_check is not None and extras.get("linear"):
            extras["linear"].update(check_linear_sample(lin_check))
    if want_e2e:
        del h_flat

    if rank == 0:
        line = {
            "metric": "hot_path_algorithmic_bandwidth", "value": value, "unit": "GB/s", "n_gpus": world,
            "steps": args.steps, "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "strong" if sliced else "weak", "vs_baseline": None,
            "dtype": "f32" if w.storage == wl.F32 else "bf16 storage, f32 arithmetic", "data": "synthetic",
            "config": config_dict(w_whole, args),
            "note": ("every rank holds one row slice of every layer (1/%d of the rows); per-call figures under "
                     "'ops' are rank 0's slice; no collective on the data path" % world) if sliced else
                    "every rank runs the whole workload on its own GPU; no collective on the data path",
            "Gparams_per_s": {n: ops[n]["Gparams_per_s"] for n in ops},
            "ops": ops, "extras": extras, "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e if e2e is not None else ({"value": None, "note": e2e_skipped} if e2e_skipped else None), "gpu_launches": int(launches),
            "clocks": clocks,
            "paper_context": "the paper times retrieval only: 658.19 ms per CLIP ViT-L/14 model and 292.70 ms per "
                             "ViT-B/32 model on an Intel Xeon Gold 6448Y CPU (other hardware; context, not a target)",
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main(argv=None):
    argv = sys.argv[1:] if argv is None else list(argv)
    args = parse_args(argv)
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be at least 1")
    if args.impl == "reference":
        return run_reference(args)       # rank 0 alone works, whatever started it
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return launch_ranks(args, argv)
    if args.check_ranks:
        return check_ranks(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
