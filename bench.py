#!/usr/bin/env python
"""Benchmark of the ASI hot path: compress + compressed weight gradient per layer-step.

  python bench.py --gpus N --steps K --warmup W            # CUDA path (one rank per GPU)
  python bench.py --impl reference --steps K --warmup W    # the fp64 CPU oracle, as it stands

One "step" is one training step of the workload: every trained layer's activation is compressed
(forward order), then every layer's weight gradient is computed from the compressed form (backward
order).  Throughput is layer-steps per second over all ranks.  Inputs are seeded synthetic tensors
shaped like the fine-tuning workload; the timed loop rotates over several distinct input sets whose
total size exceeds the L2 cache.  Prints ONE JSON line on rank 0.
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
sys.path.insert(0, ROOT)

from asi_inputs.configs import get_config, make_stream  # noqa: E402

METRIC = "asi_compress_wgrad_layer_steps_per_s"
UNIT = "layer-steps/s"
WORKLOADS = {0: "single-conv(8x32x16x16,r=4,8,8,8)", 1: "resnet18-last4-convs(B=64,224px,90%-energy-ranks)",
             2: "mobilenetv2-last5(B=128,80%-energy-ranks)", 3: "resnet34-all-3x3-shapes(B=128,90%-energy-ranks)",
             4: "vit-base-mlp(B=32,N=197,bf16-in)"}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=4000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=1, help="0-based workload index (default: ResNet-18 last 4 convs)")
    ap.add_argument("--sets", type=int, default=8, help="distinct input sets rotated through the timed loop")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="budget of the CPU-baseline leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch kernels directly instead of replaying CUDA graphs")
    ap.add_argument("--timed-only", action="store_true",
                    help="only the device-resident timed loop (no end-to-end, per-kernel or CPU legs)")
    return ap.parse_args()


# ------------------------------------------------------------------------------------------------
# CPU oracle legs (the only places this file touches oracle/)
# ------------------------------------------------------------------------------------------------
def _oracle_layer_step(O, L, A, dY, U_prev):
    S, U = O.asi_compress(A, U_prev)
    if L.kind == "linear":
        dW = O.linear_wgrad_factored(S, U, dY)
    else:
        dW = O.conv_wgrad_factored(S, U, dY, L.k, L.k, L.stride, L.pad, L.groups)
    return U, dW


def oracle_inputs(cfg, n_sets):
    data = []
    for li, L in enumerate(cfg.layers):
        st = make_stream(cfg, li)
        U0 = [u.astype(np.float64) for u in st.u_prev0()]
        sets = []
        for _ in range(n_sets):
            A, dY = st.next()
            sets.append((A.astype(np.float64), dY.astype(np.float64)))
        data.append((L, U0, sets))
    return data


def cpu_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def run_cpu_baseline(cfg, seconds):
    """Times the oracle, unmodified, on whole steps of the workload until `seconds` elapse."""
    from oracle import asi_oracle as O
    data = oracle_inputs(cfg, 2)
    U = [d[1] for d in data]
    done, t0, i = 0, time.perf_counter(), 0
    while True:
        for li, (L, _, sets) in enumerate(data):
            A, dY = sets[i % len(sets)]
            U[li], _ = _oracle_layer_step(O, L, A, dY, U[li])
            done += 1
        i += 1
        el = time.perf_counter() - t0
        if el >= seconds or i >= 1000:
            break
    return {"value": done / el, "unit": UNIT, "cores": cpu_cores(), "kind": "oracle",
            "sample": f"{i} whole steps ({done} layer-steps) of the same workload in {el:.1f} s, "
                      f"fp64 NumPy (BLAS threads = available cores)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import asi_oracle as O
    cfg = get_config(args.config)
    data = oracle_inputs(cfg, 2)
    U = [d[1] for d in data]
    nl = len(data)
    # bounded sample: as many layers of the step as keep the whole run within ~2 minutes
    t0 = time.perf_counter()
    for li, (L, _, sets) in enumerate(data):
        U[li], _ = _oracle_layer_step(O, L, sets[0][0], sets[0][1], U[li])
    t_step = time.perf_counter() - t0
    budget = 120.0
    per_step = max(1, min(nl, int(budget / max(1e-9, (args.steps + args.warmup) * t_step / nl))))

    def one_step(i):
        n = 0
        for li in range(per_step):
            L, _, sets = data[(i * per_step + li) % nl]
            A, dY = sets[i % len(sets)]
            U[(i * per_step + li) % nl], _ = _oracle_layer_step(O, L, A, dY, U[(i * per_step + li) % nl])
            n += 1
        return n

    for i in range(args.warmup):
        one_step(i)
    done, t0 = 0, time.perf_counter()
    for i in range(args.steps):
        done += one_step(i)
    el = time.perf_counter() - t0
    val = done / el
    sample = f"{per_step} of {nl} layers per step, {args.steps} steps, fp64 NumPy oracle on host cores"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * el / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": WORKLOADS[args.config]},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cpu_cores(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi polled in a child process; rows are stamped with the host clock on arrival so the
    ones that fall inside the timed region can be picked out afterwards."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows, self.proc, self.thr = [], None, None
        self.gpu = gpu_index

    def start(self, wait_s=4.0):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-i", str(self.gpu),
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thr = threading.Thread(target=self._read, daemon=True)
        self.thr.start()
        t0 = time.monotonic()
        while not self.rows and time.monotonic() - t0 < wait_s:     # first row: the poller is up
            time.sleep(0.02)

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.monotonic(), line.strip()))

    def stop(self, t_begin=None, t_end=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        inside = [r for t, r in self.rows if t_begin is not None and t_begin <= t <= t_end]
        window = "timed region"
        if len(inside) < 3:                   # region shorter than a few polls: use every row under load
            inside = [r for t, r in self.rows if t_begin is None or t >= t_begin - 1.0]
            window = "warm-up and timed region"
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in inside:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 6:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "window": window}


# ------------------------------------------------------------------------------------------------
# CUDA path
# ------------------------------------------------------------------------------------------------
def args_key(args):
    return f"config{args.config}"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2505_05086_b200 import binding
    from paper_2505_05086_b200.replicas import job_throughput
    from paper_2505_05086_b200.runner import LayerRunner

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the ASI path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    binding.lib()

    cfg = get_config(args.config)
    nl = len(cfg.layers)
    runners, acts, dys, host = [], [], [], []
    for li, L in enumerate(cfg.layers):
        st = make_stream(cfg, li)
        r = LayerRunner("linear" if L.kind == "linear" else "conv", L.dims, L.ranks, L.cout, k=L.k,
                        stride=L.stride, pad=L.pad, groups=L.groups, bf16=cfg.bf16, device=dev)
        r.set_factors(st.u_prev0())
        a_l, d_l, h_l = [], [], []
        for s in range(args.sets):
            A, dY = st.next()
            a_l.append(r.to_device(A))
            d_l.append(r.to_device(dY))
            if s < 2:
                h_l.append((a_l[-1].cpu().pin_memory(), d_l[-1].cpu().pin_memory()))
        runners.append(r)
        acts.append(a_l)
        dys.append(d_l)
        host.append(h_l)
    elem = 2 if cfg.bf16 else 4
    set_bytes = sum(r.plan.info.act_elems * elem + r.plan.info.dy_elems * elem for r in runners)
    stream = torch.cuda.Stream(device=dev)
    side = [torch.cuda.Stream(device=dev) for _ in range(nl)]

    def step(i):
        s = i % args.sets
        for li in range(nl):
            runners[li].compress(acts[li][s], stream)
        for li in reversed(range(nl)):
            runners[li].wgrad(dys[li][s], stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    launches_per_step = sum(r.plan.launch_count(0) + r.plan.launch_count(1) for r in runners)
    if args.sets % 2:
        raise SystemExit("--sets must be even (the two factor buffers of a layer alternate every step)")

    # One CUDA graph per input set: the layers of a step are independent of one another (each compress
    # reads only its own layer's activation, each wgrad its own dY), so every layer is its own branch.
    graphs = None
    with torch.cuda.stream(stream):
        for i in range(max(2, min(args.warmup, args.sets))):
            step(i)
    torch.cuda.synchronize()
    if not args.no_graph:
        graphs = []
        for s in range(args.sets):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                cur = torch.cuda.current_stream()
                for li in range(nl):
                    side[li].wait_stream(cur)
                    runners[li].compress(acts[li][s], side[li])
                for li in reversed(range(nl)):
                    runners[li].wgrad(dys[li][s], side[li])
                for li in range(nl):
                    cur.wait_stream(side[li])
            graphs.append(g)

    def run_step(i):
        if graphs is None:
            step(i)
        else:
            graphs[i % args.sets].replay()

    # ---- device-resident timing --------------------------------------------------------------
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    with torch.cuda.stream(stream):
        for i in range(args.warmup):
            run_step(i)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t_begin = time.monotonic()
        e0.record(stream)
        for i in range(args.steps):
            run_step(args.warmup + i)
        e1.record(stream)
        barrier()
        t_end = time.monotonic()
        ms = e0.elapsed_time(e1)
    clocks = sampler.stop(t_begin, t_end) if rank == 0 else None
    for r in runners:
        if not r.ok():
            raise SystemExit("device status: the timed loop reported an error (rank-deficient iterate or timeout)")
    value, ms = job_throughput(nl * args.steps, ms, dev)       # max over ranks, whole-job aggregate

    if args.timed_only:
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                              "warmup": args.warmup, "ms_per_step": ms / args.steps, "timed_only": True,
                              "launch": "direct" if graphs is None else "cuda-graph", "clocks": clocks}))
        if world > 1:
            dist.destroy_process_group()
        return

    # the same steps launched kernel by kernel on one stream (no graph), for comparison
    k_serial = max(10, min(args.steps, 300))
    with torch.cuda.stream(stream):
        barrier()
        e0.record(stream)
        for i in range(k_serial):
            step(i)
        e1.record(stream)
        barrier()
        serial_value = nl * k_serial / (e0.elapsed_time(e1) * 1e-3)

    # ---- end to end from pinned host buffers --------------------------------------------------
    arenas = [torch.empty(r.plan.step_host_arena_bytes(), dtype=torch.uint8, device=dev) for r in runners]
    hU = [[torch.empty(r.plan.info.u_elems).pin_memory() for _ in range(2)] for r in runners]
    for li, r in enumerate(runners):
        hU[li][0].copy_(r.U[r.cur].cpu())
    hS = [torch.empty(r.plan.info.core_elems).pin_memory() for r in runners]
    hW = [torch.empty(r.plan.info.dw_elems).pin_memory() for r in runners]
    sh = int(stream.cuda_stream)

    def step_host(i):
        for li, r in enumerate(runners):
            A, dY = host[li][i % 2]
            up, un = hU[li][i % 2], hU[li][(i + 1) % 2]
            r.plan.step_host(A.data_ptr(), dY.data_ptr(), up.data_ptr(), un.data_ptr(), hS[li].data_ptr(),
                             hW[li].data_ptr(), arenas[li].data_ptr(), arenas[li].numel(), sh)

    k_e2e = max(4, min(args.steps, 40))
    k_e2e += k_e2e % 2
    with torch.cuda.stream(stream):
        for i in range(4):
            step_host(i)
        barrier()
        e0.record(stream)
        for i in range(k_e2e):
            step_host(i)
        e1.record(stream)
        barrier()
        ms_e2e = e0.elapsed_time(e1)
    e2e_value, ms_e2e = job_throughput(nl * k_e2e, ms_e2e, dev)
    h2d = sum((r.plan.info.act_elems + r.plan.info.dy_elems) * elem + r.plan.info.u_elems * 4 for r in runners)
    d2h = sum((r.plan.info.u_elems + r.plan.info.core_elems + r.plan.info.dw_elems) * 4 for r in runners)
    e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
           "d2h_bytes_per_step": int(d2h), "steps": k_e2e}

    # ---- per-kernel timing for the roofline ---------------------------------------------------
    peak, peak_kind = load_peaks()
    fam = {}
    n_prof_steps = 6
    for name, kid in binding.KERNEL_IDS.items():
        n_pairs = 4096
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(2 * n_pairs)]
        for e in evs:
            e.record(stream)                      # materialise the handles
        torch.cuda.synchronize()
        keep = binding.profile_begin(kid, [e.cuda_event for e in evs])
        with torch.cuda.stream(stream):
            for i in range(n_prof_steps):
                torch.cuda._sleep(3_000_000)      # hold the stream so the launches below queue up behind it:
                step(i)                           # the events then bracket device time, not host launch latency
        n, nbytes = binding.profile_end()
        torch.cuda.synchronize()
        del keep
        n_rec = min(n, n_pairs)
        if n_rec == 0:
            continue
        tot_ms = sum(evs[2 * j].elapsed_time(evs[2 * j + 1]) for j in range(n_rec))
        fam[name] = {"launches_per_step": n / n_prof_steps, "ms_per_step": tot_ms / n_prof_steps * (n / n_rec),
                     "alg_bytes_per_step": nbytes / n_prof_steps}
    top = max(fam, key=lambda k: fam[k]["ms_per_step"])
    f = fam[top]
    achieved = f["alg_bytes_per_step"] / (f["ms_per_step"] * 1e-3) / 1e9
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if os.path.exists(tpath):                     # DRAM bytes per launch from the committed ncu capture
        traffic = json.load(open(tpath)).get(args_key(args), {}).get(top)
    roofline = {"kernel": top, "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                "avg_launch_us": 1e3 * f["ms_per_step"] / f["launches_per_step"],
                "alg_bytes_per_launch": f["alg_bytes_per_step"] / f["launches_per_step"],
                "families": {k: {"us_per_step": round(1e3 * v["ms_per_step"], 2),
                                 "launches_per_step": v["launches_per_step"]} for k, v in fam.items()}}

    if world > 1:
        dist.barrier()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOADS[args.config], "layers": nl,
                   "ranks": [list(L.ranks) for L in cfg.layers], "in_dtype": "bf16" if cfg.bf16 else "f32",
                   "l2_policy": f"inputs larger than L2: {args.sets} rotating input sets, "
                                f"{args.sets * set_bytes / 1e6:.0f} MB of act+dY",
                   "launch": ("direct launches on one stream" if graphs is None else
                              "CUDA-graph replay, one graph per input set, one branch per layer"),
                   "single_stream_direct_launch_value": serial_value,
                   "multi_gpu": "replicas only (one independent copy of the workload per GPU)"},
        "activation_GBps": sum(r.plan.info.act_elems * elem for r in runners) * args.steps / (ms * 1e-3) / 1e9,
        "e2e": e2e, "gpu_launches": int(launches_per_step * args.steps), "clocks": clocks, "roofline": roofline,
    }
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = run_cpu_baseline(cfg, args.cpu_seconds)
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
