#!/usr/bin/env python
"""Benchmark of the mixed-adapter LoRA linear layer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

A step is one pass of the whole hot path over one synthetic batch: the token-segmentation pass
followed by lora_mixed_linear (decode kernels for T <= 16, else shrink + tcgen05 GEMM with the
fused expand).  The primary workload is the 7B-class q_proj decode batch (8 tokens, 5 resident
adapter entries); its metric is algorithmic HBM GB/s.  The same line carries, under "prefill",
the 2048-token post-publish prefill batch in TFLOP/s.  Steps rotate through R distinct
(W0, adapter table, x) sets so that successive steps never find their weights in L2, and are
replayed from CUDA graphs so that launch gaps do not dominate microsecond kernels.

Multi-GPU: the layer has no exchange step, so N ranks run N independent replicas (weak scaling);
`value` is the sum over ranks divided by the slowest rank's time.

--impl reference times the fp64 CPU oracle (test infrastructure, untuned) on the host cores on
a bounded sample per step.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2608_15241_b200 import workloads as wl

L2_BYTES = 126e6
WORKLOADS = {
    "decode_q_proj": dict(make=wl.decode_q_proj, kind="decode", metric="mixed-LoRA linear HBM GB/s (decode)",
                          unit="GB/s", dtype="bf16"),
    "prefill_q_proj": dict(make=wl.prefill_q_proj, kind="prefill", metric="mixed-LoRA linear TFLOP/s (prefill)",
                           unit="TFLOP/s", dtype="bf16"),
    "mlp_up_gate": dict(make=wl.mlp_up_gate, kind="prefill", metric="mixed-LoRA linear TFLOP/s (prefill)",
                        unit="TFLOP/s", dtype="bf16"),
}


def ncu_traffic(workload):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary, or None."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        return json.load(open(path)).get(workload, {}).get("bytes")
    except (OSError, ValueError):
        return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=p["hbm_gbs"], tensor_burst=p["bf16_tflops"], tensor_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm=6650.0, tensor_burst=1590.0, tensor_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while a region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid: str | None):
        self.rows = []
        self.proc = None
        self.uuid = uuid

    def start(self):
        cmd = ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50"]
        if self.uuid:
            cmd += ["-i", self.uuid]
        try:
            self.proc = subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.06)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, pw = [], [], set(), []
        for ts, line in self.rows:
            if ts < t0 or ts > t1 + 0.06:
                continue
            f = [v.strip() for v in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------------

class Rotation:
    """R resident sets of one workload: distinct W0 / x / adapter tables, same shapes and values
    distribution (set 0 is the seeded workload itself, the others are row-rolled copies)."""

    def __init__(self, w, device, min_bytes):
        import torch
        from paper_2608_15241_b200.binding import Table, lml_tokens_workspace_bytes as b_tokens_ws
        self.w = w
        self.device = device
        per_set = w.bytes()
        self.R = max(2, int(math.ceil(min_bytes / per_set)))
        dev = lambda b: torch.from_numpy(np.ascontiguousarray(b).view(np.int16)).view(torch.bfloat16).to(device)
        x0, W00 = dev(w.x), dev(w.W0)
        A0 = [dev(e.A) for e in w.entries]
        B0 = [dev(e.B) for e in w.entries]
        self.sets = []
        G = len(w.entries) + 1
        for i in range(self.R):
            tbl = Table(w.d_in, w.d_out, max_slots=len(w.entries), device=torch.device(device).index or 0)
            roll = lambda t: t if i == 0 else torch.roll(t, shifts=i, dims=0).contiguous()
            slots = [tbl.register_adapter(e.adapter_id, e.version, roll(a), roll(b), e.scale)
                     for e, a, b in zip(w.entries, A0, B0)]
            tok = np.array([slots[e] if e >= 0 else -1 for e in w.token_entry], np.int32)
            s = dict(table=tbl, x=x0 if i == 0 else roll(x0), W0=roll(W00),
                     tok=torch.from_numpy(tok).to(device),
                     perm=torch.empty(w.T, dtype=torch.int32, device=device),
                     so=torch.empty(G + 1, dtype=torch.int32, device=device),
                     ids=torch.empty(G, dtype=torch.int32, device=device),
                     y=torch.empty((w.T, w.d_out), dtype=torch.bfloat16, device=device),
                     slots=slots)
            s["ws"] = torch.empty(max(tbl.workspace_bytes(w.T, max(G, w.G)), b_tokens_ws(tbl.handle, w.T)), dtype=torch.uint8,
                                  device=device)
            # pre-segmented form (segments as the workload states them) for the layer-only loop
            s["so_pre"] = torch.from_numpy(w.seg_offsets).to(device)
            s["ids_pre"] = torch.from_numpy(np.array([slots[e] if e >= 0 else -1 for e in w.seg_entry], np.int32)).to(device)
            s["perm_pre"] = None if w.perm is None else torch.from_numpy(w.perm).to(device)
            self.sets.append(s)
        torch.cuda.synchronize()

    def step(self, i):
        """Whole hot path from one slot id per token: token segmentation + layer, through the call a
        serving loop makes (lora_mixed_linear_tokens).  Up to 16 tokens that is one launch (the decode
        kernel binds every row to its slot itself); above, the segmentation kernel, the row gather, the
        shrink kernel and the GEMM."""
        from paper_2608_15241_b200 import binding as b
        s = self.sets[i % self.R]
        t = s["table"]
        b.lora_mixed_linear_tokens(t.handle, s["x"].data_ptr(), s["W0"].data_ptr(), self.w.T, s["tok"].data_ptr(),
                                   s["y"].data_ptr(), s["ws"].data_ptr(), s["ws"].numel(), b._stream(None))
        return t.last_launch_count()

    def layer_only(self, i):
        """lora_mixed_linear on pre-segmented input: the launches the roofline figure refers to."""
        from paper_2608_15241_b200 import binding as b
        s = self.sets[i % self.R]
        t = s["table"]
        b.lora_mixed_linear(t.handle, s["x"].data_ptr(), s["W0"].data_ptr(), self.w.T, s["so_pre"].data_ptr(),
                            s["ids_pre"].data_ptr(), self.w.G, 0 if s["perm_pre"] is None else s["perm_pre"].data_ptr(),
                            s["y"].data_ptr(), s["ws"].data_ptr(), s["ws"].numel(), b._stream(None))
        return t.last_launch_count()

    def prepare_dual(self):
        """Second binding for the dual-version call: every segment takes its neighbour's entry."""
        import torch
        from paper_2608_15241_b200.binding import lml_dual_workspace_bytes
        w = self.w
        for s in self.sets:
            other = np.roll(w.seg_entry, 1)
            s["ids_b"] = torch.from_numpy(np.array([s["slots"][e] if e >= 0 else -1 for e in other], np.int32)).to(self.device)
            s["y_b"] = torch.empty_like(s["y"])
            s["ws_dual"] = torch.empty(lml_dual_workspace_bytes(s["table"].handle, w.T, w.G), dtype=torch.uint8,
                                       device=self.device)
        torch.cuda.synchronize()

    def dual_only(self, i):
        """Both bindings in one call (shared base product)."""
        from paper_2608_15241_b200 import binding as b
        s = self.sets[i % self.R]
        t = s["table"]
        b.lora_mixed_linear_dual(t.handle, s["x"].data_ptr(), s["W0"].data_ptr(), self.w.T, s["so_pre"].data_ptr(),
                                 s["ids_pre"].data_ptr(), s["ids_b"].data_ptr(), self.w.G,
                                 0 if s["perm_pre"] is None else s["perm_pre"].data_ptr(), s["y"].data_ptr(),
                                 s["y_b"].data_ptr(), s["ws_dual"].data_ptr(), s["ws_dual"].numel(), b._stream(None))
        return t.last_launch_count()

    def two_singles(self, i):
        """The same two outputs by two ordinary calls."""
        from paper_2608_15241_b200 import binding as b
        s = self.sets[i % self.R]
        t = s["table"]
        n = 0
        for ids, y in ((s["ids_pre"], s["y"]), (s["ids_b"], s["y_b"])):
            b.lora_mixed_linear(t.handle, s["x"].data_ptr(), s["W0"].data_ptr(), self.w.T, s["so_pre"].data_ptr(),
                                ids.data_ptr(), self.w.G, 0 if s["perm_pre"] is None else s["perm_pre"].data_ptr(),
                                y.data_ptr(), s["ws"].data_ptr(), s["ws"].numel(), b._stream(None))
            n += t.last_launch_count()
        return n

    def prepare_backward(self):
        """Transposed tables (for dx), an upstream gradient and gradient buffers for the backward pass."""
        import torch
        from paper_2608_15241_b200.binding import Table, lml_backward_workspace_bytes
        w = self.w
        dev = lambda b: torch.from_numpy(np.ascontiguousarray(b).view(np.int16)).view(torch.bfloat16).to(self.device)
        from paper_2608_15241_b200 import workloads as wl
        dy0 = dev(wl.normal_bf16(4242, 1, (w.T, w.d_out), 1.0))
        A0 = [dev(e.A) for e in w.entries]
        B0 = [dev(e.B) for e in w.entries]
        for i, s in enumerate(self.sets):
            tT = Table(w.d_out, w.d_in, max_slots=len(w.entries), device=torch.device(self.device).index or 0)
            roll = lambda t: t if i == 0 else torch.roll(t, shifts=i, dims=0).contiguous()
            slots_T = [tT.register_adapter_transposed(e.adapter_id, e.version, roll(a), roll(b), e.scale)
                       for e, a, b in zip(w.entries, A0, B0)]
            s["table_T"] = tT
            s["ids_T"] = torch.from_numpy(np.array([slots_T[e] if e >= 0 else -1 for e in w.seg_entry], np.int32)).to(self.device)
            s["W0T"] = s["W0"].t().contiguous()
            s["dy"] = roll(dy0)
            s["dx"] = torch.empty((w.T, w.d_in), dtype=torch.bfloat16, device=self.device)
            s["dA"] = torch.zeros((tT.max_slots, 64, w.d_in), dtype=torch.float32, device=self.device)
            s["dB"] = torch.zeros((tT.max_slots, w.d_out, 64), dtype=torch.float32, device=self.device)
            s["ws_bwd"] = torch.empty(max(lml_backward_workspace_bytes(s["table"].handle, w.T, w.G),
                                          tT.workspace_bytes(w.T, w.G)), dtype=torch.uint8, device=self.device)
        torch.cuda.synchronize()

    def backward_dx(self, i):
        """dx = dy.W0 + s (dy.B).A: the layer on the transposed table."""
        from paper_2608_15241_b200 import binding as b
        s = self.sets[i % self.R]
        t = s["table_T"]
        b.lora_mixed_linear(t.handle, s["dy"].data_ptr(), s["W0T"].data_ptr(), self.w.T, s["so_pre"].data_ptr(),
                            s["ids_T"].data_ptr(), self.w.G, 0, s["dx"].data_ptr(), s["ws_bwd"].data_ptr(),
                            s["ws_bwd"].numel(), b._stream(None))
        return t.last_launch_count()

    def backward_adapters(self, i):
        from paper_2608_15241_b200 import binding as b
        s = self.sets[i % self.R]
        b.lora_mixed_linear_backward_adapters(s["table"].handle, s["table_T"].handle, s["x"].data_ptr(), s["dy"].data_ptr(),
                                              self.w.T, s["so_pre"].data_ptr(), s["ids_pre"].data_ptr(),
                                              s["ids_T"].data_ptr(), self.w.G, s["dA"].data_ptr(), s["dB"].data_ptr(),
                                              s["ws_bwd"].data_ptr(), s["ws_bwd"].numel(), b._stream(None))
        return s["table"].last_launch_count()

    def close(self):
        for s in self.sets:
            s["table"].close()
            if "table_T" in s:
                s["table_T"].close()


def timed_graph_loop(fn, R, steps, warmup, stream, min_warm_seconds=0.0):
    """Time exactly `steps` calls fn(i) replayed from CUDA graphs of R consecutive calls.
    Returns (seconds, kernel launches inside the timed region, (t0, t1) wall clock)."""
    import torch
    launches_per = [0] * R
    # One graph holds several rounds over the R input sets (at least 64 calls when the run is long enough): consecutive
    # calls inside a graph overlap as programmatic dependents, consecutive graph launches do not.
    Rg = R * max(1, min(-(-64 // R), steps // R)) if steps >= R else R
    with torch.cuda.stream(stream):
        for i in range(R):          # eager pass: allocations, lazy init
            launches_per[i] = fn(i)
        stream.synchronize()
        g_full = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_full, stream=stream):
            for i in range(Rg):
                fn(i)
        tail = steps % Rg
        g_tail = None
        if tail:
            g_tail = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_tail, stream=stream):
                for i in range(tail):
                    fn(i)
        warm_replays = max(1, -(-warmup // Rg))
        t_w = time.time()
        n = 0
        while n < warm_replays or time.time() - t_w < min_warm_seconds:
            g_full.replay()
            n += 1
            if n % 16 == 0:
                stream.synchronize()
        stream.synchronize()
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0 = time.time()
        ev0.record(stream)
        for _ in range(steps // Rg):
            g_full.replay()
        if g_tail is not None:
            g_tail.replay()
        ev1.record(stream)
        torch.cuda.synchronize()
        t1 = time.time()
        barrier()
    launches = (steps // R) * sum(launches_per) + sum(launches_per[:steps % R])
    return ev0.elapsed_time(ev1) / 1e3, launches, (t0, t1)


def timed_e2e_loop(rot, steps, warmup, stream):
    """Host buffers in, host buffer out, through lora_mixed_linear_host; copies inside the timed region."""
    import torch
    from paper_2608_15241_b200 import binding as b
    w = rot.w
    hosts = []
    for s in rot.sets:          # all R sets: successive steps never find their weights in L2
        xh = s["x"].cpu().pin_memory()
        yh = torch.empty((w.T, w.d_out), dtype=torch.bfloat16).pin_memory()
        so = s["so_pre"].cpu().pin_memory()
        ids = s["ids_pre"].cpu().pin_memory()
        pm = None if s["perm_pre"] is None else s["perm_pre"].cpu().pin_memory()
        ws = torch.empty(b.lml_host_workspace_bytes(s["table"].handle, w.T, w.G), dtype=torch.uint8, device=rot.device)
        hosts.append((s, xh, yh, so, ids, pm, ws))
    h2d = w.T * w.d_in * 2 + (w.G + 1) * 4 + w.G * 4 + (w.T * 4 if w.perm is not None else 0)
    d2h = w.T * w.d_out * 2

    def call(i):
        s, xh, yh, so, ids, pm, ws = hosts[i % len(hosts)]
        b.lora_mixed_linear_host(s["table"].handle, xh.data_ptr(), s["W0"].data_ptr(), w.T, so.data_ptr(),
                                 ids.data_ptr(), w.G, 0 if pm is None else pm.data_ptr(), yh.data_ptr(),
                                 ws.data_ptr(), ws.numel(), b._stream(None))

    if w.T <= 16:
        # A decode step is replayed from CUDA graphs, as a serving loop replays its decode steps: every replay still
        # pulls that step's inputs out of pinned host memory and writes its result there.
        def counted(i):
            call(i)
            return 1
        secs, _, _ = timed_graph_loop(counted, len(hosts), steps, max(3, warmup), stream)
        return secs, h2d, d2h
    with torch.cuda.stream(stream):
        for i in range(max(3, warmup)):
            call(i)
        stream.synchronize()
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for i in range(steps):
            call(i)
        ev1.record(stream)
        torch.cuda.synchronize()
        barrier()
    return ev0.elapsed_time(ev1) / 1e3, h2d, d2h


_DIST = {"on": False, "device": "cuda"}


def barrier():
    if _DIST["on"]:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(v: float) -> float:
    """Slowest rank's time: the job is as fast as its slowest replica."""
    if not _DIST["on"]:
        return v
    import torch
    import torch.distributed as dist
    t = torch.tensor([v], dtype=torch.float64, device=_DIST["device"])
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, steps: int, units_per_step: float, local_seconds: float) -> float:
    """Replicas only: every rank processes `steps` batches of its own; the job's throughput is all
    ranks' units over the slowest rank's time."""
    return world * steps * units_per_step / max_over_ranks(local_seconds)


def units_of(w, kind):
    return w.bytes() / 1e9 if kind == "decode" else w.flops() / 1e12   # GB or TFLOP per step


def run_workload(name, steps, warmup, device, world, peaks, want_cpu_baseline, e2e_steps,
                 extras=("dual", "backward", "context", "e2e", "shuffled")):
    import torch
    spec = WORKLOADS[name]
    w = spec["make"]()
    kind = spec["kind"]
    rot = Rotation(w, device, 4 * L2_BYTES)
    stream = torch.cuda.Stream(device=device)
    uuid = None
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(device).uuid)
    except Exception:
        pass
    sampler = ClockSampler(uuid)
    sampler.start()
    t_load0 = time.time()
    secs, launches, (t0, t1) = timed_graph_loop(rot.step, rot.R, steps, warmup, stream, min_warm_seconds=0.4)
    clocks = sampler.stop(t_load0, t1)
    unit_per_step = units_of(w, kind)
    value = whole_job_value(world, steps, unit_per_step, secs)
    secs = max_over_ranks(secs)

    # the layer's own launches (pre-segmented input): what the roofline fraction is computed from
    # (its length does not follow --steps: a kernel time from a handful of calls is not a measurement)
    ksteps = max(rot.R, 2000 if kind == "decode" else (200 if w.flops() < 2e11 else 60))
    ksecs, klaunches, _ = timed_graph_loop(rot.layer_only, rot.R, ksteps, max(3 * rot.R, 20), stream)
    per_launch = ksecs / ksteps
    achieved = unit_per_step / per_launch
    if kind == "decode":
        roof = {"bound": "hbm", "kernel": "decode_main_kernel (LoRA shrink runs on three of its warps)",
                "achieved": achieved, "peak": peaks["hbm"], "unit": "GB/s", "frac": achieved / peaks["hbm"],
                "peak_source": peaks["source"], "frac_of_nominal_8TBs": achieved / 8000.0, "traffic": None,
                "us_per_launch": per_launch * 1e6}
    else:
        roof = {"bound": "tensor", "kernel": "lora_gemm_sm100_kernel (the LoRA shrink runs inside it)",
                "achieved": achieved, "peak": peaks["tensor_burst"], "unit": "TFLOP/s",
                "frac": achieved / peaks["tensor_burst"], "peak_source": peaks["source"] + " burst",
                "frac_of_sustained": achieved / peaks["tensor_sustained"], "frac_of_nominal_2250": achieved / 2250.0,
                "traffic": None, "us_per_launch": per_launch * 1e6}

    dual = None
    if w.G >= 1 and "dual" in extras:
        # the same tokens under two bindings: one call with a shared base product (decode: one launch, W0 out of HBM
        # once) against two ordinary calls
        rot.prepare_dual()
        dsteps = max(rot.R, min(steps, 100)) if kind != "decode" else max(rot.R, min(10 * steps, 1200))
        d_secs, _, _ = timed_graph_loop(rot.dual_only, rot.R, dsteps, 3, stream)
        t_secs, _, _ = timed_graph_loop(rot.two_singles, rot.R, dsteps, 3, stream)
        dual = {"us_per_call": d_secs / dsteps * 1e6, "two_single_calls_us": t_secs / dsteps * 1e6}
    backward = None
    if kind != "decode" and w.G >= 1 and w.perm is None and "backward" in extras:
        # the training task's pass through the layer: dx (the layer on the transposed table) and the adapter gradients
        rot.prepare_backward()
        bsteps = max(rot.R, min(steps, 100))
        x_secs, _, _ = timed_graph_loop(rot.backward_dx, rot.R, bsteps, 3, stream)
        a_secs, _, _ = timed_graph_loop(rot.backward_adapters, rot.R, bsteps, 3, stream)
        backward = {"dx_us": x_secs / bsteps * 1e6, "adapter_gradients_us": a_secs / bsteps * 1e6}
    # context: spread of the layer-only time over repeats, one call alone (launch to completion seen from the
    # host), and the plain library GEMM of the same base shape (harness only: not a target, not part of the path)
    reps = []
    rsteps = max(rot.R, min(ksteps, 400 if kind == "decode" else 60))
    for _ in range(5 if "context" in extras else 1):
        r_secs, _, _ = timed_graph_loop(rot.layer_only, rot.R, rsteps, 3, stream)
        reps.append(r_secs / rsteps * 1e6)
    lat = []
    with torch.cuda.stream(stream):
        for i in range(40 if "context" in extras else 3):
            stream.synchronize()
            t_a = time.perf_counter()
            rot.layer_only(i)
            stream.synchronize()
            lat.append((time.perf_counter() - t_a) * 1e6)
    mm_us = None
    try:
        if "context" not in extras:
            raise RuntimeError("skipped")
        with torch.cuda.stream(stream):
            outs = [torch.empty((w.T, w.d_out), dtype=torch.bfloat16, device=device) for _ in range(2)]
            def mm(i):
                s_ = rot.sets[i % rot.R]
                torch.matmul(s_["x"], s_["W0"].t(), out=outs[i & 1])
                return 1
            mm_secs, _, _ = timed_graph_loop(mm, rot.R, rsteps, 3, stream)
            mm_us = mm_secs / rsteps * 1e6
    except Exception:
        mm_us = None
    context = {"layer_only_us_min": min(reps), "layer_only_us_median": float(np.median(reps)), "repeats": len(reps),
               "single_call_latency_us_median": float(np.median(lat)), "single_call_latency_us_min": min(lat),
               "torch_matmul_base_only_us": mm_us,
               "l2_bytes": int(getattr(torch.cuda.get_device_properties(device), "L2_cache_size", 0))}
    roof["traffic"] = ncu_traffic(name)
    roof["algorithmic"] = w.bytes() if kind == "decode" else w.flops()
    e2e = None
    if "e2e" in extras:
        esecs, h2d, d2h = timed_e2e_loop(rot, e2e_steps, 3, stream)
        esecs = max_over_ranks(esecs)
        e2e = {"value": world * e2e_steps * unit_per_step / esecs, "unit": spec["unit"], "steps": e2e_steps,
               "ms_per_step": esecs / e2e_steps * 1e3, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "host_buffer_sets": rot.R,
               "timing": "CUDA-graph replay of the host-buffer call" if w.T <= 16 else "one host-buffer call after the other"}

    # quick sampled parity of the last timed step against the oracle (rank 0)
    out = {"metric": spec["metric"], "value": value, "unit": spec["unit"], "ms_per_step": secs / steps * 1e3,
           "gpu_launches": launches, "roofline": roof, "clocks": clocks, "context": context,
           "config": {"workload": name, "tokens": w.T, "d_in": w.d_in, "d_out": w.d_out,
                      "resident_entries": len(w.entries), "segments": w.G, "rotation_sets": rot.R,
                      "l2_policy": f"inputs larger than L2: {rot.R} distinct weight/activation sets "
                                   f"({rot.R * w.bytes() / 1e6:.0f} MB) visited round-robin",
                      "timing": "CUDA-graph replay of R-step chunks, CUDA events on the launch stream"}}
    if clocks and clocks.get("sm_mhz"):
        # time x clock: comparable across power states (the long prefill loops run under the 1 kW cap at a lower SM clock)
        out["us_per_step_times_sm_ghz"] = secs / steps * 1e6 * clocks["sm_mhz"] / 1e3
    if e2e:
        out["e2e"] = e2e
    if dual:
        out["dual_version_call"] = dual
    if backward:
        out["backward"] = backward
    if want_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(w, kind, spec["unit"], budget_s=6.0 if "context" in extras else 2.0)
        out["parity_sample"] = sampled_parity(rot)
    rot.close()
    del rot
    torch.cuda.empty_cache()
    if kind != "decode" and "shuffled" in extras:
        # the same batch with its rows in arrival order: per-token ids through the segmentation pass, the
        # row gather and the scatter epilogue, all inside the timed step
        ws = wl.mlp_up_gate(shuffled=True) if name == "mlp_up_gate" else wl.shuffle_rows(w)
        rot_s = Rotation(ws, device, 4 * L2_BYTES)
        ssteps = max(rot_s.R, min(steps, 200 if ws.flops() < 2e11 else 60))
        s_secs, s_launches, _ = timed_graph_loop(rot_s.step, rot_s.R, ssteps, max(3 * rot_s.R, 10), stream)
        s_secs = max_over_ranks(s_secs)
        out["shuffled_rows"] = {"ms_per_step": s_secs / ssteps * 1e3, "value": world * ssteps * units_of(ws, kind) / s_secs,
                                "unit": spec["unit"], "steps": ssteps, "launches_per_step": s_launches // ssteps,
                                "frac_of_measured_burst": units_of(ws, kind) / (s_secs / ssteps) / peaks["tensor_burst"]}
        if want_cpu_baseline:
            out["shuffled_rows"]["parity_sample"] = sampled_parity(rot_s)
        rot_s.close()
        del rot_s
        torch.cuda.empty_cache()
    return out


def sampled_parity(rot):
    import torch
    import oracle
    w = rot.w
    s = rot.sets[0]
    rot.step(0)
    torch.cuda.synchronize()
    y = s["y"].view(torch.int16).cpu().numpy().view(np.uint16)
    rng = np.random.default_rng(0)
    pos = np.unique(rng.integers(0, w.T, size=min(w.T, 8))).astype(np.int32)
    ref, _ = oracle.forward_workload(w, positions=pos)
    rows = pos if w.perm is None else w.perm[pos]
    r = oracle.compare(y, ref, rows=rows)
    r["rows"] = int(len(pos))
    return r


def cpu_baseline(w, kind, unit, budget_s):
    """The oracle as it stands on the host cores, on a bounded sample of the workload: a spread of
    token rows (all output columns), repeated if the whole workload is smaller than the budget, so
    that the sample is about budget_s x cores seconds of CPU work."""
    import oracle
    cores = oracle.threads()
    probe = np.array([0], dtype=np.int32)
    t = time.time()
    oracle.forward_workload(w, positions=probe, nthreads=1)
    per_row = max(time.time() - t, 1e-4)
    rows = int(min(w.T, max(cores, budget_s * cores / per_row)))
    pos = np.unique(np.linspace(0, w.T - 1, rows).astype(np.int32))
    repeats = int(max(1, min(200, budget_s * cores / (per_row * len(pos)))))
    t = time.time()
    for _ in range(repeats):
        oracle.forward_workload(w, positions=pos)
    secs = (time.time() - t) / repeats
    frac = len(pos) / w.T
    v = units_of(w, kind) * frac / secs
    return {"value": v, "unit": unit, "cores": cores, "kind": "oracle",
            "single_thread_value": units_of(w, kind) / (per_row * w.T),   # one row on one thread, scaled by rows
            "sample": f"{len(pos)} of {w.T} token rows (all output columns) x {repeats} passes, "
                      f"{secs * repeats:.1f} s wall on {cores} threads, scaled by rows"}


def run_layer_sweep(device, peaks, steps, only=None, parity=False, tokens=None):
    """The decoder-layer sweep (three distinct projection shapes x five token counts), one cell after
    the other: microseconds per call of lora_mixed_linear_tokens and the fraction of the bound that
    holds for the cell (the slower of bytes / HBM peak and flops / tensor peak)."""
    import torch
    stream = torch.cuda.Stream(device=device)
    cells = []
    for proj, same_as in (("q", "q k v o"), ("gate", "gate up"), ("down", "down")):
        for T in (tokens or (sorted({t_ for _, t_ in only}) if only else wl.SWEEP_TOKENS)):
            if only and (proj, T) not in only:
                continue
            w = wl.layer_sweep(proj, T)
            rot = Rotation(w, device, 3 * L2_BYTES)
            n = max(rot.R, min(steps, 400 if T <= 16 else (100 if T <= 1024 else 30)))
            secs, launches, _ = timed_graph_loop(rot.step, rot.R, n, 3 * rot.R, stream)
            us = secs / n * 1e6
            t_hbm = w.bytes() / (peaks["hbm"] * 1e9)
            t_tensor = w.flops() / (peaks["tensor_burst"] * 1e12)
            cells.append({"projections": same_as, "d_in": w.d_in, "d_out": w.d_out, "tokens": T, "segments": w.G,
                          "us_per_call": us, "launches_per_call": launches // n, "GB/s": w.bytes() / secs * n / 1e9,
                          "TFLOP/s": w.flops() / secs * n / 1e12, "bound": "hbm" if t_hbm >= t_tensor else "tensor",
                          "frac_of_bound": max(t_hbm, t_tensor) / (secs / n)})
            if parity:
                r = sampled_parity(rot)
                cells[-1]["parity_sample"] = {"ok": r["ok"], "rows": r["rows"], "rel_fro": r["rel_fro"],
                                              "worst_tol_ratio": r["worst_tol_ratio"]}
            rot.close()
            del rot
            torch.cuda.empty_cache()
    return cells


def run_multi_decode(device, peaks, want_parity, calls=600):
    """Several projections of one decode step in one lora_mixed_linear_multi call: q/k/v (3 x 4096 x 4096) and
    gate/up (2 x 11008 x 4096) of a 7B-class layer, 8 tokens of 4 agents, 5 resident entries of rank 16 per
    projection.  Per cell: microseconds per call, algorithmic GB/s and fraction of the measured HBM peak, against
    the same projections as one call each."""
    import torch
    from paper_2608_15241_b200 import binding as b
    from paper_2608_15241_b200.binding import Table
    stream = torch.cuda.Stream(device=device)
    dev = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)
    cells = []
    for name, Ns in (("decode_qkv", (4096, 4096, 4096)), ("decode_gate_up", (11008, 11008))):
        K, T, n_ad, rank = 4096, 8, 5, 16
        P = len(Ns)
        x_bits = wl.normal_bf16(5, 1, (T, K), 1.0)
        W_bits = [wl.normal_bf16(5, 10 + p, (n, K), 0.02) for p, n in enumerate(Ns)]
        ents = [[wl.AdapterEntry(a, 1, rank, 2.0, wl.normal_bf16(5, 100 + 10 * p + a, (rank, K), 0.02),
                                 wl.normal_bf16(5, 300 + 10 * p + a, (n, rank), 0.02)) for a in range(n_ad)]
                for p, n in enumerate(Ns)]
        tok_np = np.array([0, 0, 1, 1, 2, 2, 3, 3], np.int32)     # 4 agents x 2 tokens; the fifth entry is resident, unused
        used = 4
        nbytes = sum(2.0 * K * n + 2.0 * T * n + used * 2.0 * rank * (K + n) for n in Ns) + 2.0 * T * K + 4.0 * T * P
        R = max(2, int(math.ceil(3 * L2_BYTES / nbytes)))
        x0, W0s = dev(x_bits), [dev(w) for w in W_bits]
        A0 = [[dev(e.A) for e in pe] for pe in ents]
        B0 = [[dev(e.B) for e in pe] for pe in ents]
        tok = torch.from_numpy(tok_np).to(device)
        sets = []
        for i in range(R):
            roll = lambda t_: t_ if i == 0 else torch.roll(t_, shifts=i, dims=0).contiguous()
            tabs = [Table(K, n, n_ad, device=torch.device(device).index or 0) for n in Ns]
            for p, t in enumerate(tabs):
                for a in range(n_ad):
                    t.register_adapter(a, 1, roll(A0[p][a]), roll(B0[p][a]), 2.0)
            s_ = dict(tabs=tabs, h=[t.handle for t in tabs], x=roll(x0), W=[roll(w) for w in W0s],
                      ys=[torch.empty((T, n), dtype=torch.bfloat16, device=device) for n in Ns])
            s_["ws"] = torch.empty(b.lml_multi_workspace_bytes(s_["h"], T), dtype=torch.uint8, device=device)
            sets.append(s_)
        torch.cuda.synchronize()

        def multi(i):
            s_ = sets[i % R]
            b.lora_mixed_linear_multi(s_["h"], s_["x"].data_ptr(), [w.data_ptr() for w in s_["W"]], T, [tok.data_ptr()] * P,
                                      [y.data_ptr() for y in s_["ys"]], s_["ws"].data_ptr(), s_["ws"].numel(), b._stream(None))
            return sum(t.last_launch_count() for t in s_["tabs"])

        def separate(i):
            s_ = sets[i % R]
            for p in range(P):
                b.lora_mixed_linear_tokens(s_["h"][p], s_["x"].data_ptr(), s_["W"][p].data_ptr(), T, tok.data_ptr(),
                                           s_["ys"][p].data_ptr(), s_["ws"].data_ptr(), s_["ws"].numel(), b._stream(None))
            return P

        n = max(R, calls)
        m_secs, m_launches, _ = timed_graph_loop(multi, R, n, 3 * R, stream)
        s_secs, _, _ = timed_graph_loop(separate, R, n, 3 * R, stream)
        cell = {"workload": name, "projections": P, "d_in": K, "d_out": list(Ns), "tokens": T,
                "us_per_call": m_secs / n * 1e6, "launches_per_call": m_launches // n,
                "GB/s": nbytes / (m_secs / n) / 1e9, "frac_of_measured_hbm": nbytes / (m_secs / n) / 1e9 / peaks["hbm"],
                "one_call_per_projection_us": s_secs / n * 1e6, "algorithmic_bytes": nbytes, "rotation_sets": R}
        if want_parity:
            import oracle
            multi(0)
            torch.cuda.synchronize()
            worst = {"ok": True, "rel_fro": 0.0, "worst_tol_ratio": 0.0}
            for p in range(P):
                ref, _ = oracle.forward(x_bits, W_bits[p], ents[p], np.arange(T + 1, dtype=np.int32), tok_np)
                r = oracle.compare(sets[0]["ys"][p].view(torch.int16).cpu().numpy().view(np.uint16), ref)
                worst = {"ok": worst["ok"] and r["ok"], "rel_fro": max(worst["rel_fro"], r["rel_fro"]),
                         "worst_tol_ratio": max(worst["worst_tol_ratio"], r["worst_tol_ratio"])}
            worst["rows"] = T * P
            cell["parity"] = worst
        cells.append(cell)
        for s_ in sets:
            for t in s_["tabs"]:
                t.close()
        del sets
        torch.cuda.empty_cache()
    return cells


def run_reference(args):
    """The reference arm of this tier: the fp64 oracle on host cores, a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    if args.workload not in WORKLOADS:      # the sweep has no single metric: the reference arm times the headline workload
        args.workload = "decode_q_proj"
    spec = WORKLOADS[args.workload]
    w = spec["make"]()
    kind = spec["kind"]
    cores = oracle.threads()
    t = time.time()
    oracle.forward_workload(w, positions=np.array([0], np.int32), nthreads=1)
    per_row = max(time.time() - t, 1e-4)
    total = args.steps + args.warmup
    budget = min(2.0, 150.0 / max(total, 1))                       # seconds of wall clock per step
    rows = int(max(1, min(w.T, budget * cores / per_row)))
    # when even one row per step is too slow, shrink the sample along output columns as well
    col_frac = min(1.0, budget * cores / per_row) if rows == 1 else 1.0
    n_cols = max(8, int(w.d_out * col_frac) // 8 * 8)
    W0s = w.W0[:n_cols]
    ents = [wl.AdapterEntry(e.adapter_id, e.version, e.rank, e.scale, e.A, e.B[:n_cols]) for e in w.entries]
    pos = np.unique(np.linspace(0, w.T - 1, rows).astype(np.int32))

    def step():
        oracle.forward(w.x, W0s, ents, w.seg_offsets, w.seg_entry, w.perm, positions=pos)

    for _ in range(args.warmup):
        step()
    t = time.time()
    for _ in range(args.steps):
        step()
    secs = time.time() - t
    frac = (len(pos) / w.T) * (n_cols / w.d_out)
    value = args.steps * units_of(w, kind) * frac / secs
    sample = f"{len(pos)} of {w.T} token rows x {n_cols} of {w.d_out} output columns per step, scaled by the fraction"
    line = {"impl": "reference", "metric": spec["metric"], "value": value, "unit": spec["unit"], "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": secs / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "tokens": w.T, "d_in": w.d_in, "d_out": w.d_out},
            "cpu_baseline": {"value": value, "unit": spec["unit"], "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": spec["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20000)
    ap.add_argument("--warmup", type=int, default=2000)
    ap.add_argument("--workload", default="decode_q_proj", choices=sorted(WORKLOADS) + ["layer_sweep", "multi_decode"],
                    help="layer_sweep: per-cell timings of the decoder-layer sweep (1 GPU, its own JSON line)")
    ap.add_argument("--sweep-cells", default="", help="layer_sweep: only these cells, e.g. q:128,down:16 (projections q, gate, down)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-secondary", action="store_true", help="skip the prefill line object")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the layer has no CPU path")
    import __graft_entry__ as entry
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(device))
        _DIST["on"] = True
    if rank == 0:
        entry.build()
    barrier()
    peaks = measured_peaks()
    warmup = max(3, args.warmup)
    if args.workload == "multi_decode":
        if rank == 0:
            print(json.dumps({"metric": "several projections of one decode step in one lora_mixed_linear_multi call", "unit": "us",
                              "n_gpus": 1, "dtype": "bf16", "data": "synthetic", "peak_source": peaks["source"],
                              "cells": run_multi_decode(device, peaks, True, calls=max(8, min(args.steps, 600)))}), flush=True)
        barrier()
        return
    if args.workload == "layer_sweep":
        only = {(c.split(":")[0], int(c.split(":")[1])) for c in args.sweep_cells.split(",") if c} or None
        if rank == 0:
            print(json.dumps({"metric": "decoder-layer sweep, per-cell time of lora_mixed_linear_tokens", "unit": "us",
                              "n_gpus": 1, "dtype": "bf16", "data": "synthetic", "peak_source": peaks["source"],
                              "cells": run_layer_sweep(device, peaks, args.steps, only)}), flush=True)
        barrier()
        return
    primary = run_workload(args.workload, args.steps, warmup, device, world, peaks, rank == 0,
                           e2e_steps=max(3, min(args.steps, 200)))
    line = {"metric": primary.pop("metric"), "value": primary.pop("value"), "unit": primary.pop("unit"),
            "n_gpus": world, "steps": args.steps, "warmup": warmup, "ms_per_step": primary.pop("ms_per_step"),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic"}
    line.update(primary)
    if not args.no_secondary and args.workload == "decode_q_proj":
        # the other configurations of the workload, each an object of its own in the same line
        psteps = max(3, min(args.steps, 400))
        sec = run_workload("prefill_q_proj", psteps, max(3, min(warmup, 40)), device, world, peaks, rank == 0,
                           e2e_steps=max(3, min(psteps, 50)))
        sec["steps"] = psteps
        line["prefill"] = sec
        msteps = max(3, min(args.steps, 100))
        sec = run_workload("mlp_up_gate", msteps, max(3, min(warmup, 10)), device, world, peaks, rank == 0,
                           e2e_steps=3, extras=("dual", "shuffled"))
        sec["steps"] = msteps
        line["mlp_up_gate"] = sec
        if rank == 0:
            line["multi_projection_decode"] = run_multi_decode(device, peaks, True)
            line["layer_sweep"] = {"what": "us per lora_mixed_linear_tokens call (segmentation included) and fraction of the "
                                           "cell's bound = max(bytes / measured HBM peak, flops / measured burst tensor peak) / time; "
                                           "16 adapters of rank 16, two of them in two versions (18 resident entries), Zipf(1.1) binding",
                                   "cells": run_layer_sweep(device, peaks, 200, parity=True)}
            line["few_blocks_of_16_tokens"] = {"what": "the same sweep at 32 and 64 tokens: blocks of 16 on the decode kernel in one launch "
                                                       "(launches_per_call 1) or, where that loses, one launch that binds the tokens in their "
                                                       "order and computes the shrink, then the GEMM (launches_per_call 2)",
                                               "cells": run_layer_sweep(device, peaks, 200, parity=True, tokens=(32, 64))}
        barrier()
    if rank == 0:
        print(json.dumps(line), flush=True)
    if _DIST["on"]:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
