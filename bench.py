#!/usr/bin/env python
"""Benchmark of the XConv hot path: sketch (S = Z^T X) + weight-gradient estimate, layers per second.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--r R] [--impl xconv|reference]

One step is one pass of the hot path over one synthetic layer batch: xconv_sketch, xconv_backprobe and
xconv_contract (the last two are exactly xconv_wgrad) through the C ABI, inputs resident in HBM.  The
line printed by rank 0 carries the whole-job throughput, the same metric end to end from pinned host
buffers (`e2e`), the roofline of the dominant kernel (`roofline`), the float64 oracle timed on the
host cores (`cpu_baseline`), the time of every phase launched alone (`phases`: sketch, back-probe,
contraction, and `wgrad` = the estimator as one call with L not counted in its algorithmic bytes)
and, as context, torch's exact cuDNN weight gradient.
With N > 1 every rank owns its own batch shard (same Z everywhere) and the dW estimates are summed
with one NCCL all-reduce per step (weak scaling); `--gpus N` without a launcher starts the N ranks itself.
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

import numpy as np

METRIC = "sketch+wgrad layers/s"
UNIT = "layers/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
FP32_ALU_TFLOPS_DERIVED = 148 * 128 * 2 * 1.965e9 / 1e12   # 148 SMs x 128 FMA lanes x 2 flop x max SM clock (context)
PHASE_STREAM_BYTES = 200 << 20                         # a phase that streams this much per launch evicts its own inputs
L2_ROTATE_BYTES = 300 << 20                            # tensors of a step below this: rotate through copies


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


def layer_work(c, r):
    """Algorithmic bytes and flops per launch of each phase (what the method must move and compute)."""
    s = 4 if c["dtype"] == "f32" else 2
    N = c["H"] * c["W"]
    B, Cin, Cout = c["B"], c["Cin"], c["Cout"]
    T = 9
    return {
        "sketch": dict(bytes=s * (B + r) * Cin * N + 4 * r * B, flops=2.0 * r * B * Cin * N),
        # the two launches of the estimator, each charged the L it writes or reads ("L charged": diagnostics)
        "backprobe": dict(bytes=s * (B + r) * Cout * N + 4 * r * B, flops=2.0 * r * B * Cout * N),
        "contract": dict(bytes=s * r * (Cin + Cout) * N + 4 * T * Cin * Cout, flops=2.0 * T * r * Cout * Cin * N),
        # the estimator as one unit of work: reads dY, Z and S, writes dW; L is not counted (what a kernel that
        # never wrote L would move), so any round trip of L is overhead charged to the implementation
        "wgrad": dict(bytes=s * (B * Cout * N + r * Cin * N) + 4 * r * B + 4 * T * Cout * Cin,
                      flops=2.0 * r * Cout * N * (B + T * Cin)),
    }


# DRAM bytes (read + write) of one launch of the dominant kernel, from the ncu capture summarised in
# profiles/ (None where the kernel has changed since, or was never captured).
NCU_TRAFFIC = {   # (config, r, phase): bytes; profiles/tc_gemm_kernel_config*.md, profiles/simt_kernels_config2_r64.md
    (5, 64, "sketch"): 235.9e6, (5, 64, "backprobe"): 221.4e6, (5, 64, "contract"): 55.0e6,
    (5, 16, "contract"): 12.9e6, (5, 256, "contract"): 205.8e6,
    (4, 64, "sketch"): 339.6e6, (4, 64, "backprobe"): 277.1e6, (4, 64, "contract"): 545.5e6,
    (3, 32, "sketch"): 79.1e6, (3, 32, "backprobe"): 53.2e6, (3, 32, "contract"): 53.8e6,
    (2, 64, "sketch"): 50.4e6, (2, 64, "backprobe"): 33.6e6, (2, 64, "contract"): 33.6e6,
}


def ncu_traffic(cfg, r, phase):
    return NCU_TRAFFIC.get((cfg, r, phase))


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for row in self.rows:
            try:
                sm.append(float(row[0])); mx.append(float(row[1]))
            except Exception:
                continue
            for n, v in zip(names, row[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------------- oracle legs

_ORACLE_INPUTS = {}


def oracle_sample_time(cfg, r, frac=8, impl="numpy"):
    """The float64 oracle, as it stands, on a bounded sample of the workload: the sketch of B/frac
    samples plus the estimator for Cout/frac output channels (all probes, input channels and pixels).
    Both costs are linear in the sliced axis, so the layer time is frac x the sample time."""
    from oracle import xconv_oracle as O
    from paper_2106_06998_b200 import inputs
    c = inputs.layer_shape(cfg)
    if frac <= 0:       # about 0.3 s of oracle time per GFLOP-pair on a few cores: aim at 10-20 s
        est = 2.0 * r * c["Cout"] * c["H"] * c["W"] * (c["B"] + 9 * c["Cin"]) / 4e9
        frac = 1
        while est / frac > 16 and frac < 64:
            frac *= 2
    Bs, Ms = max(1, c["B"] // frac), max(1, c["Cout"] // frac)
    key = (cfg, r, frac)
    if key not in _ORACLE_INPUTS:            # drawn once per run, outside the timed calls
        g = np.random.Generator(np.random.PCG64(1))
        _ORACLE_INPUTS.clear()
        _ORACLE_INPUTS[key] = (inputs.draw(c["x"], (Bs, c["Cin"], c["H"], c["W"]), 11, c["dtype"]),
                               inputs.draw("normal", (c["B"], Ms, c["H"], c["W"]), 12, c["dtype"], c["dy_var"] ** 0.5),
                               inputs.draw(c["z"], (r, c["Cin"], c["H"], c["W"]), 13, c["dtype"]),
                               g.standard_normal((r, c["B"])))
    X, dY, Z, S = _ORACLE_INPUTS[key]
    if impl == "c":                          # the same formulas as plain C loop nests (oracle/xconv_oracle.c)
        from oracle import c_oracle as O
        O.lib()
    t0 = time.perf_counter()
    O.sketch(X, Z)
    t1 = time.perf_counter()
    O.wgrad_estimate(S, dY, Z)
    t2 = time.perf_counter()
    sample = (f"sketch of B/{frac}={Bs} samples + estimator for Cout/{frac}={Ms} output channels "
              f"(all r, Cin, pixels); layer time = {frac} x sample time")
    return frac * (t2 - t0), frac * (t1 - t0), frac * (t2 - t1), sample


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
    except Exception:
        n = 1
    return min(n, len(os.sched_getaffinity(0)))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2106_06998_b200 import inputs
    c = inputs.layer_shape(args.config)
    times = []
    sample = ""
    frac = args.oracle_frac
    if frac <= 0:
        # every step times the oracle on a slice of the layer; the slice shrinks with the number of steps
        # asked for, so that the whole run stays within a few minutes (about 0.3 s of oracle time per
        # GFLOP-pair on a few cores; at most a 16th of the layer: on smaller slices the oracle's fixed costs take
        # over and the layer time extrapolated from the slice comes out too long)
        est = 2.0 * args.r * c["Cout"] * c["H"] * c["W"] * (c["B"] + 9 * c["Cin"]) / 4e9
        per_step = min(16.0, 150.0 / max(1, args.warmup + args.steps))
        frac = 1
        while est / frac > per_step and frac < 16:
            frac *= 2
    for i in range(args.warmup + args.steps):
        t, _, _, sample = oracle_sample_time(args.config, args.r, frac=frac)
        if i >= args.warmup:
            times.append(t)
    t = float(np.mean(times))              # layer time: frac x the time of one step's sample
    val = 1.0 / t
    cfg_line = workload_config(args, c, 0)
    cfg_line["layers_per_step"] = 1.0 / frac
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / frac, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": cfg_line,
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                             "sample": sample + f"; a step is one sample = 1/{frac} layer, value = layers_per_step / step time"},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_config(args, c, copies=1):
    es = 4 if c["dtype"] == "f32" else 2
    step_mb = es * c["H"] * c["W"] * (c["B"] * (c["Cin"] + c["Cout"]) + args.r * (c["Cin"] + c["Cout"])) / 1e6
    l2 = ("not applicable: the oracle runs on the host" if copies == 0 else
          f"the tensors of one step ({step_mb:.0f} MB) exceed the 126 MB L2" if copies == 1 else
          f"steps rotate through {copies} copies of the tensors of one step ({step_mb:.0f} MB each) at different "
          f"addresses, {copies * step_mb:.0f} MB in all, so that no step finds its inputs in the 126 MB L2")
    return {"workload": f"config {args.config}: 3x3 conv layer B={c['B']} Cin={c['Cin']} Cout={c['Cout']} "
                        f"{c['H']}x{c['W']} {c['dtype']} storage, {c['z']} probes, r={args.r}",
            "r": args.r, "layout": "channels_last", "accumulate": "f32", "l2": l2}


# ----------------------------------------------------------------------------------- GPU arm

def run_xconv(args):
    import torch
    import torch.distributed as dist

    import __graft_entry__ as entry
    from paper_2106_06998_b200 import binding as xb
    from paper_2106_06998_b200 import dp, inputs

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        # NCCL's communicator lines (topology, NVLS, channels) stay visible, on stderr: stdout carries the JSON line
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        os.environ.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
        dist.init_process_group("nccl", device_id=dev)
    entry.build()

    cfg, r = args.config, args.r
    c = inputs.layer_shape(cfg)
    tdt = torch.float32 if c["dtype"] == "f32" else torch.bfloat16
    B, Cin, Cout, H, W = c["B"], c["Cin"], c["Cout"], c["H"], c["W"]
    # seeded synthetic inputs of the workload's recipe, drawn on the host; each rank its own batch
    # shard (X, dY differ per rank), the same probes Z on every rank
    lay = inputs.make_layer(cfg, r, tensors=("Z",))
    Z = xb.to_device(lay["Z"], c["dtype"], dev)
    hX = inputs.draw(c["x"], (B, Cin, H, W), inputs.seed_for(cfg, r, "X") + 7919 * rank, c["dtype"])
    hdY = inputs.draw("normal", (B, Cout, H, W), inputs.seed_for(cfg, r, "dY") + 7919 * rank, c["dtype"],
                      c["dy_var"] ** 0.5)
    X, dY = xb.to_device(hX, c["dtype"], dev), xb.to_device(hdY, c["dtype"], dev)
    del lay

    class Layer:
        """Buffers and the timed step of one (config, r) workload.  A layer whose tensors (X, dY, Z, L) fit
        the 126 MB L2 is held in several copies at different addresses and the steps rotate through them,
        so that every step finds its inputs in HBM, not in L2."""

        def __init__(self, r_, Z_, zero_blocks=None):
            self.r = r_
            self.zero_blocks = zero_blocks        # kept alive: the descriptor holds its address
            self.desc = xb.make_desc(B, Cin, Cout, H, W, r_, tdt, zero_blocks=zero_blocks)
            self.S = torch.empty((r_, B), dtype=torch.float32, device=dev)
            self.dW = torch.empty((Cout, Cin, 3, 3), dtype=torch.float32, device=dev, memory_format=torch.channels_last)
            set_bytes = X.element_size() * (X.numel() + dY.numel() + Z_.numel() + r_ * Cout * H * W)
            self.copies = 1 if set_bytes >= L2_ROTATE_BYTES else min(64, -(-L2_ROTATE_BYTES // set_bytes) + 1)
            self.sets = []
            for i in range(self.copies):
                self.sets.append((X if i == 0 else X.clone(), dY if i == 0 else dY.clone(), Z_ if i == 0 else Z_.clone(),
                                  torch.empty((r_, Cout, H, W), dtype=tdt, device=dev, memory_format=torch.channels_last)))
            self.ws = torch.empty(max(xb.workspace_bytes(self.desc, xb.OP_SKETCH),
                                      xb.workspace_bytes(self.desc, xb.OP_WGRAD)), dtype=torch.uint8, device=dev)
            self.launches = 0
            self.count = 0

        def step(self, events=None):
            X_, dY_, Z_, L_ = self.sets[self.count % self.copies]
            self.count += 1
            if events:
                events[0].record()
            xb.sketch_into(self.desc, X_, Z_, self.S, self.ws)
            self.launches += xb.last_launch_count()
            if events:
                events[1].record()
            xb.backprobe_into(self.desc, self.S, dY_, L_, self.ws)
            self.launches += xb.last_launch_count()
            if events:
                events[2].record()
            xb.contract_into(self.desc, L_, Z_, self.dW, self.ws)
            self.launches += xb.last_launch_count()
            if events:
                events[3].record()
            dp.allreduce_dw(self.dW)

        def measure(self, steps, warmup, sampler=None, phase_events=True):
            """W warm-up steps, then exactly `steps` timed steps between barriers and synchronisations;
            returns (total ms as the max over ranks, mean per-phase ms or None, clock record).
            With phase_events an event is recorded between the three calls of every step: that gives
            the per-phase times but costs about 15 us per step, because an event between two kernels
            keeps the second from starting its preamble under the tail of the first."""
            for _ in range(max(3, warmup)):
                self.step()
            torch.cuda.synchronize()
            if xb.workspace_status(self.ws) != 0:
                raise SystemExit("a device-side wait ran out during warm-up")
            ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
            t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if sampler is not None:
                sampler.start()
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()
            self.launches = 0
            t_begin.record()
            for i in range(steps):
                self.step(ev[i] if phase_events else None)
            t_end.record()
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
            total = t_begin.elapsed_time(t_end)
            clk = sampler.stop() if sampler is not None else None
            if world > 1:
                t = torch.tensor([total], device=dev)
                dist.all_reduce(t, op=dist.ReduceOp.MAX)
                total = float(t.item())
            if xb.workspace_status(self.ws) != 0:
                raise SystemExit("a device-side wait ran out during the timed region")
            ph = None
            if phase_events:
                ph = {n: float(np.mean([ev[i][k].elapsed_time(ev[i][k + 1]) for i in range(steps)]))
                      for k, n in enumerate(("sketch", "backprobe", "contract"))}
            return total, ph, clk

        def measure_graph(self, steps):
            """The same step captured once into a CUDA graph and replayed `steps` times (the library allocates nothing
            and never synchronises, so its calls can be captured): ms per step, or None if capture is unavailable.
            One tensor set: for layers below L2's size the replays find their inputs in L2, so only the launch-bound
            layers gain from it."""
            try:
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    self.count = 0
                    self.step()
                torch.cuda.current_stream().wait_stream(side)
                graph = torch.cuda.CUDAGraph()
                self.count = 0
                with torch.cuda.graph(graph):
                    self.step()
                for _ in range(3):
                    graph.replay()
                a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a_.record()
                for _ in range(steps):
                    graph.replay()
                b_.record()
                torch.cuda.synchronize()
                if xb.workspace_status(self.ws) != 0:
                    return None
                return a_.elapsed_time(b_) / steps
            except Exception:
                return None

        def phase_call(self, name, i):
            """One launch of one phase on the i-th tensor set (through the C ABI, as in the step)."""
            X_, dY_, Z_, L_ = self.sets[i % len(self.sets)]
            if name == "sketch":
                xb.sketch_into(self.desc, X_, Z_, self.S, self.ws)
            elif name == "backprobe":
                xb.backprobe_into(self.desc, self.S, dY_, L_, self.ws)
            elif name == "contract":
                xb.contract_into(self.desc, L_, Z_, self.dW, self.ws)
            else:
                xb.wgrad_into(self.desc, self.S, dY_, Z_, self.dW, self.ws)

        def measure_phase(self, name, steps):
            """Average duration of one phase (its main kernel and its helper kernels): `steps` launches of
            that call back to back between two CUDA events on the launching stream, after warm-up.  No event
            sits between two launches, so consecutive launches overlap preamble and tail exactly as the calls
            of a step do.  A phase that moves less than PHASE_STREAM_BYTES per launch rotates through enough
            tensor sets at different addresses that no launch finds its inputs in the 126 MB L2."""
            es = X.element_size()
            per = {"sketch": es * (X.numel() + self.sets[0][2].numel()),
                   "backprobe": es * (dY.numel() + self.sets[0][3].numel()),
                   "contract": es * (self.sets[0][2].numel() + self.sets[0][3].numel()),
                   "wgrad": es * (dY.numel() + self.sets[0][2].numel())}[name]
            need = 1 if per >= PHASE_STREAM_BYTES else min(64, -(-L2_ROTATE_BYTES // per) + 1)
            while len(self.sets) < need:      # more copies of the tensors, made outside the timed region
                X0, dY0, Z0, L0 = self.sets[0]
                self.sets.append((X0, dY0, Z0.clone(), torch.empty_like(L0)) if name == "contract"
                                 else (X0.clone(), dY0.clone(), Z0.clone(), torch.empty_like(L0)))
            if name == "contract":            # every L the region reads holds this layer's back-probe
                for i in range(need):
                    xb.backprobe_into(self.desc, self.S, self.sets[i][1], self.sets[i][3], self.ws)
            for i in range(max(3, need)):
                self.phase_call(name, i)
            torch.cuda.synchronize()
            a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a_.record()
            for i in range(steps):
                self.phase_call(name, i % need)
            b_.record()
            torch.cuda.synchronize()
            if xb.workspace_status(self.ws) != 0:
                raise SystemExit(f"a device-side wait ran out while timing {name}")
            return a_.elapsed_time(b_) / steps, need

        def measure_phases(self, steps):
            out, sets = {}, {}
            for n in ("sketch", "backprobe", "contract", "wgrad"):
                out[n], sets[n] = self.measure_phase(n, steps)
            del self.sets[max(1, self.copies):]
            torch.cuda.empty_cache()
            return out, sets

    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        gpu_id = str(local)
    layer = Layer(r, Z)
    # the timed region of the headline number: K steps, nothing but the three calls in the stream
    total_ms, _, clocks = layer.measure(args.steps, args.warmup, ClockSampler(gpu_id) if rank == 0 else None,
                                        phase_events=False)
    ms_step = total_ms / args.steps
    n_launch = layer.launches
    # every phase on its own: K launches back to back between two events (the roofline numbers), and the K
    # steps once more with an event between the calls (diagnostic: the events keep the kernels from overlapping)
    n_phase = max(5, min(args.steps, 100))
    phase_ms, phase_sets = layer.measure_phases(n_phase)
    total_ev_ms, phase_ev_ms, _ = layer.measure(n_phase, 3, None, phase_events=True)
    graph_ms = layer.measure_graph(n_phase) if world == 1 else None
    desc, S, dW = layer.desc, layer.S, layer.dW
    launches = [n_launch]

    # ---- end to end from pinned host buffers through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        pX, pdY, pZ = X.cpu().pin_memory(), dY.cpu().pin_memory(), Z.cpu().pin_memory()
        pS = torch.empty((r, B), dtype=torch.float32).pin_memory()
        pdW = torch.empty((Cout, Cin, 3, 3), dtype=torch.float32).contiguous(memory_format=torch.channels_last).pin_memory()
        arena = torch.empty(xb.host_arena_bytes(desc), dtype=torch.uint8, device=dev)
        n_e2e = max(2, min(args.steps, 5))
        for _ in range(2):
            xb.xconv_sketch_wgrad_host(desc, pX, pdY, pZ, pS, pdW, arena)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            xb.xconv_sketch_wgrad_host(desc, pX, pdY, pZ, pS, pdW, arena)   # synchronises before returning
        t_e2e = torch.tensor([(time.perf_counter() - t0) / n_e2e], device=dev)
        if world > 1:
            dist.all_reduce(t_e2e, op=dist.ReduceOp.MAX)
        es = X.element_size()
        e2e = {"value": world / float(t_e2e.item()), "unit": UNIT,
               "h2d_bytes_per_step": (X.numel() + dY.numel() + Z.numel()) * es,
               "d2h_bytes_per_step": (S.numel() + dW.numel()) * 4, "steps": n_e2e,
               "note": "xconv_sketch_wgrad_host: pinned host buffers, copies and sync inside the call"}
        del pX, pdY, pZ, arena

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of every phase (live CUDA-event times: K launches of the phase back to back)
    peaks, peak_src = load_peaks()
    tensor_peak = peaks["bf16_tflops"] if total_ms < 2000 else peaks["bf16_tflops_sustained"]
    fma_tflops = xb.measure_fma_rate(dev)              # measured FP32 FMA rate: the ceiling of the FP32-FMA kernels

    def phase_table(r_, desc_, ph_ms):
        work = layer_work(c, r_)
        eng = {"sketch": xb.engine_for(desc_, xb.OP_SKETCH), "backprobe": xb.engine_for(desc_, xb.OP_BACKPROBE),
               "contract": xb.engine_for(desc_, xb.OP_CONTRACT), "wgrad": xb.engine_for(desc_, xb.OP_WGRAD)}
        out = {}
        for n, ms in ph_ms.items():
            gbs = work[n]["bytes"] / (ms * 1e-3) / 1e9
            tfs = work[n]["flops"] / (ms * 1e-3) / 1e12
            comp_peak = tensor_peak if eng[n] == "tcgen05_bf16" else fma_tflops
            t_mem, t_comp = work[n]["bytes"] / (peaks["hbm_gbs"] * 1e9), work[n]["flops"] / (comp_peak * 1e12)
            bound = "hbm" if t_mem >= t_comp else ("tensor" if eng[n] == "tcgen05_bf16" else "alu")
            out[n] = {"ms": ms, "engine": eng[n], "GBps": gbs, "TFLOPps": tfs, "bound": bound,
                      "peak": peaks["hbm_gbs"] if bound == "hbm" else comp_peak,
                      "roofline_ms": 1e3 * max(t_mem, t_comp),
                      "frac": (gbs / peaks["hbm_gbs"]) if bound == "hbm" else tfs / comp_peak}
            if n in ("backprobe", "contract"):
                out[n]["note"] = "L charged to this launch (diagnostic); the estimator as a whole is `wgrad`"
        return out

    phases = phase_table(r, desc, phase_ms)
    kernels = {n: phase_ms[n] for n in ("sketch", "backprobe", "contract")}
    dom = max(kernels, key=kernels.get)
    d = phases[dom]
    low = min(("sketch", "wgrad"), key=lambda n: phases[n]["frac"])
    roofline = {"kernel": dom + " (tc_gemm_kernel and its reduce/cast helper, timed together)", "bound": d["bound"],
                "achieved": d["GBps"] if d["bound"] == "hbm" else d["TFLOPps"], "peak": d["peak"],
                "unit": "GB/s" if d["bound"] == "hbm" else "TFLOP/s", "frac": d["frac"],
                "traffic": ncu_traffic(cfg, r, dom),
                "peak_source": f"of {peak_src}" + ("" if d["bound"] != "alu" else
                                                   " (FP32 FMA rate measured by xconv_measure_fma_rate; derived "
                                                   f"148 SMs x 128 FMA x 2 x 1.965 GHz = {FP32_ALU_TFLOPS_DERIVED:.1f})"),
                "timing": f"{n_phase} launches of the phase back to back between two CUDA events",
                "furthest_below": {"phase": low, "bound": phases[low]["bound"], "frac": phases[low]["frac"],
                                   "note": "of the two units of the method (sketch; estimator = back-probe + "
                                           "contraction with L not counted), the one furthest below its roofline"}}

    # ---- the rest of the layer API on the same tensors: forward (conv + sketch) and exact dX
    full = None
    if not args.no_context:
        Wt = xb.to_device(inputs.draw("normal", (Cout, Cin, 3, 3), inputs.seed_for(cfg, r, "W"), c["dtype"],
                                      (2.0 / (Cin * 9)) ** 0.5), c["dtype"], dev)
        Y = torch.empty((B, Cout, H, W), dtype=tdt, device=dev, memory_format=torch.channels_last)
        dX = torch.empty((B, Cin, H, W), dtype=tdt, device=dev, memory_format=torch.channels_last)
        wsf = torch.empty(max(xb.workspace_bytes(desc, xb.OP_FORWARD), xb.workspace_bytes(desc, xb.OP_DGRAD)),
                          dtype=torch.uint8, device=dev)

        def _time(f, n=20, name=None):
            if name:
                torch.cuda.nvtx.range_push("api_" + name)          # a handle for profilers
            try:
                return _time_inner(f, n)
            finally:
                if name:
                    torch.cuda.nvtx.range_pop()

        def _time_inner(f, n):
            for _ in range(3):
                f()
            a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a_.record()
            for _ in range(n):
                f()
            b_.record()
            torch.cuda.synchronize()
            return a_.elapsed_time(b_) / n

        # Algorithm 1 with only the seed kept: Z redrawn inside the sketch kernel / into the workspace
        wss = torch.empty(max(xb.workspace_bytes(desc, xb.OP_SKETCH_SEEDED), xb.workspace_bytes(desc, xb.OP_WGRAD_SEEDED)),
                          dtype=torch.uint8, device=dev)
        S2 = torch.empty_like(S)
        full = {"forward_ms": _time(lambda: xb.forward_into(desc, X, Wt, Z, Y, S, wsf)),
                "dgrad_ms": _time(lambda: xb.dgrad_into(desc, dY, Wt, dX, wsf)),
                "wgrad_ms": _time(lambda: xb.wgrad_into(desc, S, dY, Z, dW, layer.ws), name="wgrad"),
                "sketch_seeded_ms": _time(lambda: xb.sketch_seeded_into(desc, X, 12345, S2, wss), name="sketch_seeded"),
                "wgrad_seeded_ms": _time(lambda: xb.wgrad_seeded_into(desc, S, dY, 12345, dW, wss), name="wgrad_seeded"),
                "conv_engine": xb.engine_for(desc, xb.OP_FORWARD),
                "note": "xconv_forward = conv + sketch; xconv_dgrad = exact dX; xconv_wgrad = back-probe + contraction "
                        "in one call; *_seeded: probes redrawn from a seed instead of read from memory; not part of the metric"}
        del Y, dX, wsf, wss

    # ---- the other probe counts of this workload's sweep (shorter runs), same step and timing
    sweep = []
    if not args.no_sweep and world == 1:
        for r2 in c["r"]:
            if r2 == r:
                continue
            Z2 = xb.to_device(inputs.make_layer(cfg, r2, tensors=("Z",))["Z"], c["dtype"], dev)
            lay2 = Layer(r2, Z2)
            n2 = max(5, min(args.steps, 30))
            tot2, _, _ = lay2.measure(n2, 3, None, phase_events=False)
            ph2, _ = lay2.measure_phases(n2)
            sweep.append({"r": r2, "ms_per_step": tot2 / n2, "value": 1e3 * n2 / tot2, "phases": phase_table(r2, lay2.desc, ph2)})
            del lay2, Z2
            torch.cuda.empty_cache()

    # ---- the same step with Gaussian probing vectors (the workload names no distribution; Rademacher is the primary run)
    gaussian = None
    if not args.no_sweep and world == 1 and c["z"] != "gaussian":
        Zg = xb.to_device(inputs.draw("gaussian", (r, Cin, H, W), inputs.seed_for(cfg, r, "Z") + 17, c["dtype"]), c["dtype"], dev)
        layg = Layer(r, Zg)
        ng = max(5, min(args.steps, 30))
        totg, _, _ = layg.measure(ng, 3, None, phase_events=False)
        phg, _ = layg.measure_phases(ng)
        gaussian = {"r": r, "z": "gaussian", "ms_per_step": totg / ng, "value": 1e3 * ng / totg,
                    "phases_ms": {k: v for k, v in phg.items()}}
        del layg, Zg
        torch.cuda.empty_cache()

    # ---- block-sparse probes (Eq. 7) on this workload: the contraction told which 64-channel blocks of Z are zero
    block_sparse = None
    if (not args.no_sweep and world == 1 and tdt != torch.float32 and Cin % 64 == 0 and Cout % 64 == 0
            and Cin % min(256, Cin) == 0 and r <= B):
        block_sparse = []
        n3 = max(5, min(args.steps, 30))
        tile = min(256, Cin) // 64          # 64-channel blocks per column tile of the contraction

        def sparse_case(r3, Z3, pg, whole_tiles):
            gen = torch.Generator(device="cpu").manual_seed(inputs.seed_for(cfg, r3, "Z") + int(1000 * pg) + whole_tiles)
            if whole_tiles:                 # the blocks of a probing vector inside a column tile are kept or dropped together
                keep = (torch.rand((r3, Cin // 64 // tile), generator=gen) < pg).repeat_interleave(tile, dim=1).to(dev)
            else:
                keep = (torch.rand((r3, Cin // 64), generator=gen) < pg).to(dev)
            Zs = (Z3 * keep.repeat_interleave(64, dim=1)[:, :, None, None].to(tdt)).contiguous(memory_format=torch.channels_last)
            zb = xb.xconv_zero_blocks(Zs)
            lay3 = Layer(r3, Zs, zero_blocks=zb)
            used = xb.zero_blocks_used(lay3.desc)
            xb.sketch_into(lay3.desc, X, Zs, lay3.S, lay3.ws)
            torch.cuda.nvtx.range_push(f"zb_r{r3}_p{pg}_w{int(whole_tiles)}")      # a handle for profilers
            t3, _ = lay3.measure_phase("contract", n3)
            torch.cuda.nvtx.range_pop()
            listed = float((zb.view(r3, -1, tile) == 0).any(dim=2).float().mean())
            del lay3
            torch.cuda.empty_cache()
            return {"r": r3, "p_block": pg, "blocks": "256 channels" if whole_tiles else "64 channels",
                    "zero_share": float(zb.float().mean()), "probes_read_share": listed, "skipping": used, "contract_ms": t3}

        for pg in (1.0, 0.5, 0.25, 0.125):
            block_sparse.append(sparse_case(r, Z, pg, True))
        for pg in (0.5, 0.125):
            block_sparse.append(sparse_case(r, Z, pg, False))
        if 256 in c["r"] and r != 256:
            Z256 = xb.to_device(inputs.make_layer(cfg, 256, tensors=("Z",))["Z"], c["dtype"], dev)
            for pg in (1.0, 0.5):
                block_sparse.append(sparse_case(256, Z256, pg, True))
            del Z256
            torch.cuda.empty_cache()

    cpu = None
    if not args.no_cpu:
        t, ts, tw, sample = oracle_sample_time(cfg, r, frac=args.oracle_frac)
        c_loops = None
        try:                                 # the second statement of the oracle, timed on the same sample
            tc_, _, _, _ = oracle_sample_time(cfg, r, frac=args.oracle_frac, impl="c")
            from oracle import c_oracle
            c_loops = {"value": 1.0 / tc_, "unit": UNIT, "cores": c_oracle.threads(), "kind": "oracle, plain C loop nests with OpenMP"}
        except Exception as e:               # no gcc or no OpenMP on this host
            c_loops = {"unavailable": type(e).__name__}
        cpu = {"value": 1.0 / t, "unit": UNIT, "cores": host_threads(), "kind": "oracle", "sample": sample, "c_loops": c_loops,
               "sketch_s": ts, "wgrad_s": tw}

    context = {}
    if not args.no_context:
        try:
            Wt = torch.empty((Cout, Cin, 3, 3), dtype=tdt, device=dev).contiguous(memory_format=torch.channels_last)
            f = lambda: torch.ops.aten.convolution_backward(dY, X, Wt, None, [1, 1], [1, 1], [1, 1], False, [0, 0],
                                                            1, [False, True, False])
            for _ in range(3):
                f()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(5):
                f()
            b.record(); torch.cuda.synchronize()
            context["torch_cudnn_exact_wgrad_ms"] = a.elapsed_time(b) / 5
        except Exception as e:      # context only
            context["torch_cudnn_exact_wgrad_ms"] = f"unavailable: {type(e).__name__}"
        context["paper"] = ("no timing table; text: up to 10x over im2col on a Xeon E3-1270 v6 for large images "
                            "and batches at small r, competitive with cuDNN on an RTX 2000 Ada (Section 5.4)")
    es = X.element_size()
    line = {"metric": METRIC, "value": world * 1e3 / ms_step, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32" if c["dtype"] == "f32" else "bf16",
            "data": "synthetic", "config": workload_config(args, c, layer.copies), "clocks": clocks, "e2e": e2e,
            "gpu_launches": launches[0], "roofline": roofline, "cpu_baseline": cpu, "phases": phases,
            "phase_timing": {"launches_per_phase": n_phase, "tensor_sets_per_phase": phase_sets,
                             "fp32_fma_tflops_measured": fma_tflops,
                             "with_events_between_calls_ms": dict(phase_ev_ms, step=total_ev_ms / n_phase),
                             "step_replayed_from_a_cuda_graph_ms": graph_ms,
                             "note": "phases and roofline: each call timed alone, K launches back to back between two "
                                     "CUDA events; with_events_between_calls_ms: the step with an event between its "
                                     "three calls, which keeps a kernel's preamble from overlapping the previous "
                                     "kernel's tail (diagnostic)"},
            "sweep": sweep, "gaussian_probes": gaussian, "layer_api": full,
            "block_sparse": None if block_sparse is None else {
                "cases": block_sparse,
                "dense_contract_ms": {str(r): phases["contract"]["ms"],
                                      **{str(e["r"]): e["phases"]["contract"]["ms"] for e in sweep if e["r"] == 256}},
                "note": "xconv_contract with desc.zero_blocks (Eq. 7): blocks of Z kept with probability p_block and named "
                        "to the contraction when zero; per column tile of 256 channels it reads and multiplies only the "
                        "probing vectors with a non-zero block there (probes_read_share), so blocks of 256 channels are "
                        "skipped in proportion and independent 64-channel blocks only where all four of a tile are zero"},
            "memory_ratio": {"elements": Cin * H * W / r, "stored_bytes": Cin * H * W * es / (4.0 * r)},
            "context": context}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def spawn_ranks(n):
    """`python bench.py --gpus N` started without a launcher: run the same command line as N ranks of one node
    under torch.distributed.run (rendezvous on 127.0.0.1) and hand back its exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), "--", os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="xconv", choices=["xconv", "reference"])
    ap.add_argument("--config", type=int, default=5)
    ap.add_argument("--r", type=int, default=64)
    ap.add_argument("--oracle-frac", type=int, default=0, help="slice of the layer the oracle is timed on (0: pick for ~10-20 s)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-context", action="store_true")
    ap.add_argument("--no-sweep", action="store_true")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_xconv(args)


if __name__ == "__main__":
    main()
