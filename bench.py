#!/usr/bin/env python
"""Benchmark of the ASI hot path: compress + compressed weight gradient per layer-step.

  python bench.py --gpus N --steps K --warmup W            # CUDA path (one rank per GPU)
  python bench.py --impl reference --steps K --warmup W    # the fp64 CPU oracle, as it stands

One "step" is one training step of a workload: every trained layer's activation is compressed
(forward order), then every layer's weight gradient is computed from the compressed form (backward
order).  Throughput is layer-steps per second over all ranks.  Inputs are seeded synthetic tensors
shaped like the fine-tuning workloads; the timed loop rotates over distinct input sets whose total
size exceeds the L2 cache.

The headline line is measured on the largest single-GPU workload (the ResNet-34-shaped sweep); the
other four workloads are measured in the same invocation and reported under "per_config".  Every
entry carries a roofline: compulsory bytes (|A| + |dY| + |dW| of every layer) against the measured
HBM peak, useful flops (the paper's overhead and speed-up cost models, as multiply-adds x 2, plus
the core products) against the peak of the unit that runs them, the slower of the two as the bound.
Prints ONE JSON line on rank 0.
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
             2: "mobilenetv2-last5(B=128,80%-energy-ranks)", 3: "resnet34-all-conv-shapes(B=128,90%-energy-ranks)",
             4: "vit-base-mlp(B=32,N=197,bf16-in)", 5: "llm-tokens(B=8,N=512,D=2048,rank20,bf16-in)"}
HEADLINE = 3                  # the largest workload that fits one GPU
L2_BYTES = 126e6
N_SM, FMA_PER_SM_CLK = 148, 128


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=None,
                    help="0-based workload index: measure only this one (default: all, headline = the sweep)")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="budget of the CPU-baseline leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch kernels directly instead of replaying CUDA graphs")
    ap.add_argument("--timed-only", action="store_true",
                    help="only the device-resident timed loop (no end-to-end, per-kernel or CPU legs)")
    ap.add_argument("--min-timed-ms", type=float, default=250.0,
                    help="the block of --steps steps is repeated until this much device time has been timed")
    return ap.parse_args()


# ------------------------------------------------------------------------------------------------
# cost models (closed forms of the paper; no method arithmetic)
# ------------------------------------------------------------------------------------------------
def layer_costs(L, bf16):
    """Compulsory bytes and useful flops of one layer-step.  Flops: compress = 2 x (2 N sum r_m, the
    overhead model's two products per mode, + the core products in mode order), wgrad = 2 x C_ASI."""
    eb = 2 if bf16 else 4
    dims, r = L.dims, L.ranks
    N = int(np.prod(dims))
    dy = int(np.prod(L.dy_shape))
    dw = int(np.prod(L.dw_shape))
    macs_modes = [2.0 * N * rm for rm in r]
    core, lead, rest = 0.0, 1.0, float(N)
    for d, rm in zip(dims, r):
        core += lead * rest * rm
        lead *= rm
        rest /= d
    if L.kind == "conv":
        B, C, H, W = dims
        Ho, Wo = L.out_hw
        r1, r2, r3, r4 = r
        wg = (r1 * B * L.cout * Ho * Wo + r1 * r2 * r3 * r4 * H + r1 * r2 * r4 * H * W +
              r1 * r2 * L.cout * Ho * Wo * L.k * L.k + r2 * L.cout * C * L.k * L.k / L.groups * L.groups)
    else:
        lead_dims, Din = dims[:-1], dims[-1]
        wg, lead, rest = 0.0, 1.0, float(np.prod(lead_dims[1:])) * L.cout
        for m, d in enumerate(lead_dims):
            wg += lead * r[m] * d * rest
            lead *= r[m]
            if m + 1 < len(lead_dims):
                rest /= lead_dims[m + 1]
        wg += lead * r[-1] * L.cout + r[-1] * L.cout * Din
    # contractions the library runs on the tensor cores: bf16 token layers, factor width 16..64 (a multiple of 4)
    tc = 0.0
    if bf16 and L.kind == "linear":
        for m, rm in enumerate(r):
            if rm % 4 == 0 and 16 <= rm <= 64 and m >= 1:
                tc += macs_modes[m]
    return {"act_bytes": N * eb, "dy_bytes": dy * eb, "dw_bytes": dw * 4,
            "flops": 2.0 * (sum(macs_modes) + core + wg), "flops_tensor": 2.0 * tc}


def roofline_for(step_costs, t_step_s, hbm_peak_gbs, peak_kind, fp32_peak_tf, tensor_peak_tf):
    nbytes = sum(c["act_bytes"] + c["dy_bytes"] + c["dw_bytes"] for c in step_costs)
    fl = sum(c["flops"] for c in step_costs)
    fl_tc = sum(c["flops_tensor"] for c in step_costs)
    t_hbm = nbytes / (hbm_peak_gbs * 1e9)
    t_alu = (fl - fl_tc) / (fp32_peak_tf * 1e12) + fl_tc / (tensor_peak_tf * 1e12)
    bound = "hbm" if t_hbm >= t_alu else "alu"
    out = {"bound": bound, "step_bytes": nbytes, "step_flops": fl, "t_hbm_us": 1e6 * t_hbm, "t_alu_us": 1e6 * t_alu,
           "step_us": 1e6 * t_step_s, "step_frac": max(t_hbm, t_alu) / t_step_s,
           "step_frac_hbm": t_hbm / t_step_s, "peak_kind": f"of {peak_kind}",
           "fp32_peak_tflops": fp32_peak_tf, "note": "step_frac = slower of (compulsory bytes / HBM peak) and "
           "(useful flops / peak of the unit that runs them), divided by the measured step time"}
    return out


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


def oracle_inputs(cfg, n_sets, layers=None):
    data = []
    for li, L in enumerate(cfg.layers):
        if layers is not None and li not in layers:
            continue
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


def _time_oracle(O, data, seconds):
    """Runs layer-steps round-robin over `data` until `seconds` elapse; returns seconds per whole step
    of the workload, extrapolating by activation elements when not every layer was reached."""
    U = [d[1] for d in data]
    per_layer = [[] for _ in data]
    t_start, i = time.perf_counter(), 0
    while True:
        for li, (L, _, sets) in enumerate(data):
            A, dY = sets[i % len(sets)]
            t0 = time.perf_counter()
            U[li], _ = _oracle_layer_step(O, L, A, dY, U[li])
            per_layer[li].append(time.perf_counter() - t0)
            if time.perf_counter() - t_start >= seconds and i == 0 and li + 1 < len(data):
                break
        i += 1
        if time.perf_counter() - t_start >= seconds or i >= 1000:
            break
    elems = [float(np.prod(d[0].dims)) for d in data]
    done = [li for li in range(len(data)) if per_layer[li]]
    t_done = sum(float(np.median(per_layer[li])) for li in done)
    t_step = t_done * sum(elems) / sum(elems[li] for li in done)
    n_calls = sum(len(x) for x in per_layer)
    return t_step, len(done), n_calls, time.perf_counter() - t_start


def run_cpu_baseline(cfg, seconds):
    """Times the oracle, unmodified, on the workload's layers: all host cores, then one core."""
    from oracle import asi_oracle as O
    data = oracle_inputs(cfg, 1)
    nl = len(data)
    t_step, n_done, n_calls, el = _time_oracle(O, data, seconds)
    out = {"value": nl / t_step, "unit": UNIT, "cores": cpu_cores(), "kind": "oracle",
           "sample": f"{n_calls} layer-steps over {n_done} of the {nl} layers of the workload in {el:.1f} s "
                     f"(median per layer; a whole step = {t_step:.2f} s"
                     f"{', extrapolated by activation elements' if n_done < nl else ''}), fp64 NumPy, "
                     f"BLAS threads = available cores"}
    try:
        from threadpoolctl import threadpool_limits
        with threadpool_limits(limits=1):
            t1, n1, c1, el1 = _time_oracle(O, data, max(4.0, seconds / 2))
        out["single_core_value"] = nl / t1
        out["single_core_sample"] = (f"{c1} layer-steps over {n1} of {nl} layers in {el1:.1f} s with BLAS limited "
                                     f"to one thread")
    except Exception as e:                                   # threadpoolctl missing: say so, keep the main figure
        out["single_core_value"] = None
        out["single_core_sample"] = f"not measured ({type(e).__name__})"
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import asi_oracle as O
    ci = HEADLINE if args.config is None else args.config
    cfg = get_config(ci)
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
    sample = f"{per_step} of {nl} layers per step (round-robin), {args.steps} steps, fp64 NumPy oracle on host cores"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * el / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": WORKLOADS[ci]},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cpu_cores(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi polled in a child process; rows are stamped with the host clock on arrival so the
    ones that fall inside a timed region can be picked out afterwards."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows, self.proc, self.thr = [], None, None
        self.gpu = gpu_index

    def start(self, wait_s=4.0):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-i", str(self.gpu),
                 "-lms", "25"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
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

    def window(self, t_begin, t_end):
        inside = [r for t, r in self.rows if t_begin <= t <= t_end]
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
                "reasons": sorted(reasons), "samples": len(sm), "window": "timed region"}

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()


# ------------------------------------------------------------------------------------------------
# CUDA path
# ------------------------------------------------------------------------------------------------
def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d.get("bf16_tflops_sustained", d.get("bf16_tflops", 1400.0))), "measured"
    return 6650.0, 1400.0, "fallback"


class Workload:
    """Device-resident inputs, runners and CUDA graphs of one configuration."""

    def __init__(self, ci, dev, use_graph, torch, n_host_sets=0):
        from paper_2505_05086_b200.binding import ASI_FLAG_SHARE_SM
        from paper_2505_05086_b200.runner import LayerRunner, StepRunner
        self.ci, self.cfg, self.torch = ci, get_config(ci), torch
        cfg = self.cfg
        self.nl = len(cfg.layers)
        self.costs = [layer_costs(L, cfg.bf16) for L in cfg.layers]
        self.set_bytes = sum(c["act_bytes"] + c["dy_bytes"] for c in self.costs)
        sets = int(np.ceil(3.0 * L2_BYTES / self.set_bytes))
        self.sets = max(2, min(8, sets + sets % 2))
        self.runners, self.acts, self.dys, self.host = [], [], [], []
        self.graph_runners = []
        for li, L in enumerate(cfg.layers):
            st = make_stream(cfg, li)
            r = LayerRunner("linear" if L.kind == "linear" else "conv", L.dims, L.ranks, L.cout, k=L.k,
                            stride=L.stride, pad=L.pad, groups=L.groups, bf16=cfg.bf16, device=dev)
            r.set_factors(st.u_prev0())
            if use_graph:
                # the graph runs the layers side by side: its plans leave room on every SM for the neighbours
                g = LayerRunner("linear" if L.kind == "linear" else "conv", L.dims, L.ranks, L.cout, k=L.k,
                                stride=L.stride, pad=L.pad, groups=L.groups, bf16=cfg.bf16, device=dev,
                                flags=ASI_FLAG_SHARE_SM)
                g.set_factors(st.u_prev0())
                self.graph_runners.append(g)
            a_l, d_l, h_l = [], [], []
            for s in range(self.sets):
                A, dY = st.next()
                a_l.append(r.to_device(A))
                d_l.append(r.to_device(dY))
                if s < n_host_sets:
                    h_l.append((a_l[-1].cpu().pin_memory(), d_l[-1].cpu().pin_memory()))
            self.runners.append(r)
            self.acts.append(a_l)
            self.dys.append(d_l)
            self.host.append(h_l)
        self.stream = torch.cuda.Stream(device=dev)
        # the whole step through the batched entry points (one call forward, one call backward)
        self.step = StepRunner(self.runners)
        # for the graph every layer is a branch of its own (the layers of a step are independent of one another):
        # measured faster than the batched launches on one branch, whose kernel stages run one after the other
        self.side = [torch.cuda.Stream(device=dev) for _ in range(self.nl)]
        self.launches_per_step = (self._count_launches() if not use_graph else
                                  sum(r.plan.launch_count(0) + r.plan.launch_count(1) for r in self.graph_runners))
        with torch.cuda.stream(self.stream):
            for i in range(2):
                self.step_direct(i)
        torch.cuda.synchronize()
        self.graphs = None
        if use_graph:
            # One CUDA graph per input set.  The layers of a step are independent of one another (each compress
            # reads only its own layer's activation, each wgrad its own dY), so every layer is its own branch.
            self.graphs = []
            for s in range(self.sets):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=self.stream):
                    cur = torch.cuda.current_stream()
                    for li in range(self.nl):
                        self.side[li].wait_stream(cur)
                        self.graph_runners[li].compress(self.acts[li][s], self.side[li])
                    for li in reversed(range(self.nl)):
                        self.graph_runners[li].wgrad(self.dys[li][s], self.side[li])
                    for li in range(self.nl):
                        cur.wait_stream(self.side[li])
                self.graphs.append(g)

    def _count_launches(self):
        """Kernel launches of one step through the batched entry points: fused layers of one variant
        (map size, rank bucket) share three compress launches and, per rank bucket, one wgrad launch."""
        n, cvar, wvar = 0, {}, {}
        for r in self.runners:
            pl, d = r.plan, r.dims
            if pl.launch_count(0) == 3:
                key = (d[2], 4 if max(r.ranks) <= 4 else 8)
                cvar[key] = cvar.get(key, 0) + 1
            else:
                n += pl.launch_count(0)
            if pl.launch_count(1) == 1:
                key = 4 if max(r.ranks) <= 4 else 8
                wvar[key] = wvar.get(key, 0) + 1
            else:
                n += pl.launch_count(1)
        n += sum(3 * -(-c // 8) for c in cvar.values()) + sum(-(-c // 8) for c in wvar.values())
        return n

    def step_direct(self, i, only=None):
        s = i % self.sets
        if only != "wgrad":
            self.step.compress([self.acts[li][s] for li in range(self.nl)], self.stream)
        if only != "compress":
            self.step.wgrad([self.dys[li][s] for li in range(self.nl)], self.stream)

    def run_step(self, i):
        if self.graphs is None:
            self.step_direct(i)
        else:
            self.graphs[i % self.sets].replay()

    def ok(self):
        return all(r.ok() for r in self.runners) and all(r.ok() for r in self.graph_runners)

    def free(self):
        self.graphs = None
        self.runners = self.graph_runners = self.acts = self.dys = self.host = None
        self.torch.cuda.empty_cache()


def time_blocks(wl, steps, warmup, min_ms, barrier, torch, fn=None):
    """Blocks of `steps` steps, each bracketed by CUDA events on the launching stream, repeated until
    `min_ms` of device time have been timed (at least 3 blocks).  Returns per-block milliseconds and
    the host-clock window of the timed region."""
    fn = fn or wl.run_step
    with torch.cuda.stream(wl.stream):
        for i in range(max(3, warmup)):
            fn(i)
        barrier()
        probe0, probe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        probe0.record(wl.stream)
        for i in range(steps):
            fn(i)
        probe1.record(wl.stream)
        torch.cuda.synchronize()
        est = max(1e-3, probe0.elapsed_time(probe1))
        n_blocks = int(max(3, min(400, np.ceil(min_ms / est))))
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_blocks + 1)]
        barrier()
        t_begin = time.monotonic()
        evs[0].record(wl.stream)
        k = 0
        for b in range(n_blocks):
            for i in range(steps):
                fn(k)
                k += 1
            evs[b + 1].record(wl.stream)
        barrier()
        t_end = time.monotonic()
    return [evs[b].elapsed_time(evs[b + 1]) for b in range(n_blocks)], (t_begin, t_end)


def kernel_families(wl, binding, torch, n_prof_steps=4):
    """Per kernel family: device time per launch (CUDA events recorded by the library around each
    launch on its own stream) and the bytes each launch must move at least."""
    fam = {}
    for name, kid in binding.KERNEL_IDS.items():
        n_pairs = 1024
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(2 * n_pairs)]
        for e in evs:
            e.record(wl.stream)                      # materialise the handles
        torch.cuda.synchronize()
        keep = binding.profile_begin(kid, [e.cuda_event for e in evs])
        with torch.cuda.stream(wl.stream):
            for i in range(n_prof_steps):
                torch.cuda._sleep(3_000_000)          # hold the stream so the launches below queue up behind it:
                wl.step_direct(i)                     # the events then bracket device time, not host launch latency
        n, nbytes = binding.profile_end()
        torch.cuda.synchronize()
        del keep
        n_rec = min(n, n_pairs)
        if n_rec == 0:
            continue
        tot_ms = sum(evs[2 * j].elapsed_time(evs[2 * j + 1]) for j in range(n_rec))
        fam[name] = {"launches_per_step": n / n_prof_steps, "ms_per_step": tot_ms / n_prof_steps * (n / n_rec),
                     "alg_bytes_per_step": nbytes / n_prof_steps}
    return fam


def measure_config(ci, args, dev, world, rank, barrier, torch, binding, job_throughput, sampler, peaks, headline):
    hbm_peak, tensor_peak, peak_kind = peaks
    wl = Workload(ci, dev, not args.no_graph, torch, n_host_sets=2 if (headline and not args.timed_only) else 0)
    cfg = wl.cfg
    blocks, (t_begin, t_end) = time_blocks(wl, args.steps, args.warmup, args.min_timed_ms, barrier, torch)
    if not wl.ok():
        raise SystemExit(f"device status: the timed loop of workload {ci} reported an error "
                         f"(rank-deficient iterate or expired wait)")
    ms_block = float(np.median(blocks))
    value, ms_block = job_throughput(wl.nl * args.steps, ms_block, dev)     # max over ranks, whole-job aggregate
    ms_step = ms_block / args.steps
    clocks = sampler.window(t_begin, t_end) if (rank == 0 and sampler is not None) else None
    sm_max = (clocks or {}).get("sm_max_mhz") or 1965.0
    fp32_peak_tf = N_SM * FMA_PER_SM_CLK * 2 * sm_max * 1e6 / 1e12
    roof = roofline_for(wl.costs, ms_step * 1e-3, hbm_peak, peak_kind, fp32_peak_tf, tensor_peak)
    entry = {"workload": WORKLOADS[ci], "dtype": "bf16-in/f32" if cfg.bf16 else "f32", "layers": wl.nl,
             "ms_per_step": ms_step, "value": value, "timed_blocks": len(blocks),
             "timed_ms_total": float(sum(blocks)), "block_ms_min_med_max": [float(min(blocks)), ms_block, float(max(blocks))],
             "input_sets": wl.sets, "input_bytes_rotated": wl.sets * wl.set_bytes,
             "gpu_launches_per_step": wl.launches_per_step, "clocks": clocks, "roofline": roof}
    if args.timed_only:
        wl.free()
        return entry, None
    # the same steps launched kernel by kernel on one stream (no graph)
    b2, _ = time_blocks(wl, max(5, min(args.steps, 50)), 3, 60.0, barrier, torch, fn=wl.step_direct)
    entry["single_stream_value"] = wl.nl * max(5, min(args.steps, 50)) / (float(np.median(b2)) * 1e-3)
    # compress alone: the activation bandwidth the metric names, |A| sizeof(in) / t_compress
    b3, _ = time_blocks(wl, max(5, min(args.steps, 50)), 3, 60.0, barrier, torch,
                        fn=lambda i: wl.step_direct(i, only="compress"))
    t_c = float(np.median(b3)) * 1e-3 / max(5, min(args.steps, 50))
    entry["activation_GBps"] = sum(c["act_bytes"] for c in wl.costs) / t_c / 1e9
    entry["compress_us_per_step_single_stream"] = 1e6 * t_c
    # dominant kernel family against the HBM roofline
    fam = kernel_families(wl, binding, torch)
    extra = None
    if fam:
        top = max(fam, key=lambda k: fam[k]["ms_per_step"])
        f = fam[top]
        achieved = f["alg_bytes_per_step"] / (f["ms_per_step"] * 1e-3) / 1e9
        traffic = None
        tpath = os.path.join(ROOT, "profiles", "ncu_traffic.json")
        if os.path.exists(tpath):                     # DRAM bytes per launch from the committed ncu capture
            traffic = json.load(open(tpath)).get(f"config{ci}", {}).get(top)
        entry["roofline"].update({
            "kernel": top, "achieved": achieved, "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak,
            "traffic": traffic, "avg_launch_us": 1e3 * f["ms_per_step"] / f["launches_per_step"],
            "alg_bytes_per_launch": f["alg_bytes_per_step"] / f["launches_per_step"],
            "families": {k: {"us_per_step": round(1e3 * v["ms_per_step"], 2),
                             "launches_per_step": v["launches_per_step"]} for k, v in fam.items()}})
    if headline:
        extra = wl
    else:
        wl.free()
    return entry, extra


def measure_e2e(wl, args, dev, barrier, torch, job_throughput):
    """The same metric end to end through asi_step_host: pinned host buffers in, results back."""
    cfg = wl.cfg
    elem = 2 if cfg.bf16 else 4
    runners = wl.runners
    arenas = [torch.empty(r.plan.step_host_arena_bytes(), dtype=torch.uint8, device=dev) for r in runners]
    hU = [[torch.empty(r.plan.info.u_elems).pin_memory() for _ in range(2)] for r in runners]
    for li, r in enumerate(runners):
        hU[li][0].copy_(r.U[r.cur].cpu())
    hS = [torch.empty(r.plan.info.core_elems).pin_memory() for r in runners]
    hW = [torch.empty(r.plan.info.dw_elems).pin_memory() for r in runners]
    sh = int(wl.stream.cuda_stream)

    def step_host(i):
        for li, r in enumerate(runners):
            A, dY = wl.host[li][i % 2]
            up, un = hU[li][i % 2], hU[li][(i + 1) % 2]
            r.plan.step_host(A.data_ptr(), dY.data_ptr(), up.data_ptr(), un.data_ptr(), hS[li].data_ptr(),
                             hW[li].data_ptr(), arenas[li].data_ptr(), arenas[li].numel(), sh)

    k_e2e = max(4, min(args.steps, 10))
    k_e2e += k_e2e % 2
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(wl.stream):
        for i in range(4):
            step_host(i)
        barrier()
        e0.record(wl.stream)
        for i in range(k_e2e):
            step_host(i)
        e1.record(wl.stream)
        barrier()
        ms_e2e = e0.elapsed_time(e1)
    for li, r in enumerate(runners):
        if r.plan.step_host_status(arenas[li].data_ptr(), sh) != 0:
            raise SystemExit("device status: the end-to-end loop reported an error")
    e2e_value, ms_e2e = job_throughput(wl.nl * k_e2e, ms_e2e, dev)
    h2d = sum((r.plan.info.act_elems + r.plan.info.dy_elems) * elem + r.plan.info.u_elems * 4 for r in runners)
    d2h = sum((r.plan.info.u_elems + r.plan.info.core_elems + r.plan.info.dw_elems) * 4 for r in runners)
    return {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
            "steps": k_e2e, "api": "asi_step_host (pinned host buffers, copies inside the timed region)"}


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2505_05086_b200 import binding
    from paper_2505_05086_b200.replicas import job_throughput

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

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peaks = load_peaks()
    head_ci = HEADLINE if args.config is None else args.config
    # replicas (N > 1) measure the headline workload only: every rank would otherwise regenerate all inputs
    others = [] if (args.config is not None or world > 1) else [c for c in (0, 1, 2, 4, 5) if c != head_ci]
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler is not None:
        sampler.start()
    head, wl = measure_config(head_ci, args, dev, world, rank, barrier, torch, binding, job_throughput, sampler,
                              peaks, headline=True)
    e2e = None
    if wl is not None:
        e2e = measure_e2e(wl, args, dev, barrier, torch, job_throughput)
        wl.free()
    per_config = [head]
    for ci in others:
        try:
            get_config(ci)
        except ValueError:
            continue
        entry, _ = measure_config(ci, args, dev, world, rank, barrier, torch, binding, job_throughput, sampler,
                                  peaks, headline=False)
        per_config.append(entry)
    if sampler is not None:
        sampler.stop()
    if world > 1:
        dist.barrier()
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    cfg = get_config(head_ci)
    roof = dict(head["roofline"])
    out = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOADS[head_ci], "layers": head["layers"],
                   "ranks": [list(L.ranks) for L in cfg.layers], "in_dtype": "bf16" if cfg.bf16 else "f32",
                   "l2_policy": f"inputs larger than L2: {head['input_sets']} rotating input sets, "
                                f"{head['input_bytes_rotated'] / 1e6:.0f} MB of act+dY",
                   "launch": ("asi_compress_batched + asi_wgrad_batched on one stream" if args.no_graph else
                              "CUDA-graph replay, one graph per input set, one branch per layer, plans with ASI_FLAG_SHARE_SM"),
                   "single_stream_launch": "asi_compress_batched + asi_wgrad_batched, one call each per step",
                   "timing": f"{head['timed_blocks']} blocks of {args.steps} steps, {head['timed_ms_total']:.0f} ms "
                             f"of device time; ms_per_step = median block / steps",
                   "single_stream_direct_launch_value": head.get("single_stream_value"),
                   "multi_gpu": "replicas only (one independent copy of the workload per GPU)"},
        "gpu_launches": int(head["gpu_launches_per_step"] * args.steps * head["timed_blocks"]),
        "clocks": head["clocks"], "roofline": roof, "per_config": per_config,
    }
    if "activation_GBps" in head:
        out["activation_GBps"] = head["activation_GBps"]
    if e2e is not None:
        out["e2e"] = e2e
    if world == 1 and not args.no_cpu_baseline and not args.timed_only:
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
