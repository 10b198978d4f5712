#!/usr/bin/env python
"""Benchmark of the VQ-decode linear-layer hot path on B200.

A step = one pass of the whole hot path (stream indices, stage codebooks, unpack, look up,
multiply-accumulate, reduce + store) over one batch of synthetic activations for every layer
of one benchmark configuration (default: the Llama-2-70B-shaped layer set, 2-D VQ with 4-bit
indices and int8 codebooks, batch 1: the largest single-GPU workload).  Layers that read the same
activations in a transformer block (q/k/v, gate/up) go through one grouped call.  Metric:
compressed bytes (indices + codebooks + scales + activations + outputs) moved per second, i.e.
achieved HBM bandwidth on the compressed representation.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import vq_synth  # noqa: E402

METRIC = "vq_decode_gemv_compressed_byte_hbm_bandwidth"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


def layer_bytes(spec: vq_synth.LayerSpec, stride: int, batch: int) -> int:
    """Algorithmic bytes of one layer call: everything stored for W plus activations and outputs."""
    idx = spec.N * stride
    if int(spec.int8) == 2:   # int4 codebooks: two entries' values per byte, one fp16 scale per row and 128 columns
        cb = spec.n_blocks * spec.entries * spec.d // 2
        sc = spec.N * (spec.K // 128) * 2
    else:
        cb = spec.n_blocks * spec.entries * spec.d * (1 if spec.int8 else 2)
        sc = spec.n_blocks * 2 if spec.int8 else 0
    return idx + cb + sc + 2 * batch * (spec.K + spec.N)


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------
class ClockSampler:
    """Polls NVML for SM clock and throttle reasons while the timed region runs."""

    BAD = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20}
    NOTE = {"sw_power_cap": 0x4}

    def __init__(self, uuid: str):
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _poll(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                    else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for name, bit in {**self.BAD, **self.NOTE}.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv:
            self._stop.clear()
            self._thread = threading.Thread(target=self._poll, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread:
            self._stop.set()
            self._thread.join()
            self._thread = None

    def summary(self, source: str):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0, "source": "nvml unavailable"}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples), "source": source}


# ------------------------------------------------------------------------------------------
# the CUDA arm
# ------------------------------------------------------------------------------------------
GROUPS = (("q", "k", "v"), ("gate", "up"))   # projections of a transformer block that read the same activations


def call_groups(specs):
    """Layer indices per library call: adjacent q/k/v and gate/up layers of one format and K form a
    group (at most 4 members), everything else is a call of its own."""
    out, i = [], 0
    while i < len(specs):
        name = specs[i].name.split(".")[-1]
        grp = next((g for g in GROUPS if name == g[0]), None)
        members = [i]
        if grp:
            for j, want in enumerate(grp[1:], start=1):
                if i + j < len(specs) and specs[i + j].name.split(".")[-1] == want and specs[i + j].K == specs[i].K:
                    members.append(i + j)
                else:
                    break
        out.append(members)
        i += len(members)
    return out


class DeviceSet:
    """R distinct device copies of every layer of a configuration, so that a layer's bytes have
    been evicted from L2 by the time its copy is read again."""

    def __init__(self, cfg_name: str, batch: int, device, max_copies=None):
        import torch
        import paper_2402_15319_b200 as vq
        self.vq, self.torch = vq, torch
        conf = vq_synth.CONFIGS[cfg_name]
        self.cfg_name, self.batch, self.device = cfg_name, batch, device
        self.batch_built = batch
        self.batch_host = batch   # the host-side buffers keep the constructor's batch
        self.specs = conf["layers"]
        self.fmts, self.host, self.bytes_per_layer = [], [], []
        for lid, spec in enumerate(self.specs):
            fmt = vq.VQFormat(spec.N, spec.K, spec.d, spec.b, spec.Br, spec.Bc, int(spec.int8))
            info = vq.vq_pack_info(fmt)
            L = vq_synth.make_layer(spec, info.row_stride_bytes, conf["seed"], lid)
            X = vq_synth.make_x(spec, conf["seed"], batch, lid)
            self.fmts.append(fmt)
            self.host.append((L, X))
            self.bytes_per_layer.append(layer_bytes(spec, info.row_stride_bytes, batch))
        self.groups = call_groups(self.specs)
        # a group's members read ONE activation tensor (the first member's): count it once
        shared_x = sum(2 * batch * self.specs[i].K for g in self.groups for i in g[1:])
        self.step_bytes = int(sum(self.bytes_per_layer)) - shared_x
        self.n_weights = sum(s.n_weights for s in self.specs)
        self.copies = max(2, -(-2 * L2_BYTES // self.step_bytes))
        if max_copies:
            self.copies = min(self.copies, max_copies)
        self.dev = []  # [copy][layer] -> (idx, cb, scale)
        base = []
        for (L, X) in self.host:
            base.append((torch.from_numpy(L.idx).to(device), torch.from_numpy(L.cb).to(device),
                         None if L.scale is None else torch.from_numpy(L.scale).to(device)))
        self.dev.append(base)
        for _ in range(1, self.copies):
            self.dev.append([tuple(None if t is None else t.clone() for t in lay) for lay in base])
        self.X = [torch.from_numpy(X).to(device) for (_, X) in self.host]
        self.Y = [torch.empty((batch, s.N), dtype=torch.float16, device=device) for s in self.specs]
        self.ws = [torch.zeros(vq.vq_workspace_bytes(f, batch), dtype=torch.uint8, device=device) for f in self.fmts]
        self.group_fmt, self.group_ws = {}, {}
        for g in self.groups:
            if len(g) > 1:
                sp = self.specs[g[0]]
                gf = vq.VQFormat(sum(self.specs[i].N for i in g), sp.K, sp.d, sp.b, sp.Br, sp.Bc, int(sp.int8))
                self.group_fmt[g[0]] = gf
                self.group_ws[g[0]] = torch.zeros(vq.vq_workspace_bytes(gf, batch), dtype=torch.uint8, device=device)
        # host side of the end-to-end path
        self.hX = [torch.from_numpy(X).pin_memory() for (_, X) in self.host]
        self.hY = [torch.empty((batch, s.N), dtype=torch.float16).pin_memory() for s in self.specs]
        self.ws_host = [torch.zeros(vq.vq_workspace_bytes_host(f, batch), dtype=torch.uint8, device=device) for f in self.fmts]
        self.group_ws_host = {i: torch.zeros(vq.vq_workspace_bytes_grouped_host(gf, len(g), batch), dtype=torch.uint8, device=device)
                              for g in self.groups if len(g) > 1 for i, gf in [(g[0], self.group_fmt[g[0]])]}
        # a group's activations cross the host boundary once
        self.h2d = sum(int(self.hX[g[0]].numel()) * 2 for g in self.groups)
        self.d2h = sum(int(y.numel()) * 2 for y in self.hY)

    def step(self, copy: int):
        vq = self.vq
        for g in self.groups:
            i = g[0]
            if len(g) == 1:
                idx, cb, sc = self.dev[copy][i]
                vq.vq_gemm_small_batch(self.fmts[i], idx, cb, sc, self.X[i], self.Y[i], self.batch, self.ws[i])
            else:
                members = [(self.dev[copy][j][0], self.dev[copy][j][1], self.dev[copy][j][2], self.Y[j], self.specs[j].N) for j in g]
                vq.vq_gemm_small_batch_grouped(self.group_fmt[i], members, self.X[i], self.batch, self.group_ws[i])

    def set_batch(self, batch: int):
        """Same weights, another batch size (activations, outputs and workspaces are remade)."""
        torch, vq = self.torch, self.vq
        conf = vq_synth.CONFIGS[self.cfg_name]
        self.batch = batch
        self.X = [torch.from_numpy(vq_synth.make_x(s, conf["seed"], batch, lid)).to(self.device) for lid, s in enumerate(self.specs)]
        self.Y = [torch.empty((batch, s.N), dtype=torch.float16, device=self.device) for s in self.specs]
        self.ws = [torch.zeros(vq.vq_workspace_bytes(f, batch), dtype=torch.uint8, device=self.device) for f in self.fmts]
        for i in list(self.group_fmt):
            self.group_ws[i] = torch.zeros(vq.vq_workspace_bytes(self.group_fmt[i], batch), dtype=torch.uint8, device=self.device)
        per_layer = [b - 2 * self.batch_built * (s.K + s.N) + 2 * batch * (s.K + s.N) for b, s in zip(self.bytes_per_layer, self.specs)]
        self.bytes_per_layer, self.batch_built = per_layer, batch
        self.step_bytes = int(sum(per_layer)) - sum(2 * batch * self.specs[i].K for g in self.groups for i in g[1:])

    def step_host(self, copy: int):
        """The same calls as step() with host activations and outputs (built for the batch of the constructor)."""
        vq = self.vq
        for g in self.groups:
            i = g[0]
            if len(g) == 1:
                idx, cb, sc = self.dev[copy][i]
                vq.vq_gemm_small_batch_host(self.fmts[i], idx, cb, sc, self.hX[i], self.hY[i], self.batch_host, self.ws_host[i])
            else:
                members = [(self.dev[copy][j][0], self.dev[copy][j][1], self.dev[copy][j][2], self.hY[j], self.specs[j].N) for j in g]
                vq.vq_gemm_small_batch_grouped_host(self.group_fmt[i], members, self.hX[i], self.batch_host, self.group_ws_host[i])
        self.torch.cuda.synchronize()

    def launches_per_step(self) -> int:
        """Library kernels one step launches (a grouped call launches one kernel, or one per member)."""
        n = 0
        for g in self.groups:
            n += 1 if len(g) == 1 else self.vq.vq_grouped_kernel_launches(self.group_fmt[g[0]], len(g), self.batch)
        return n

    def call_names(self):
        return ["+".join(self.specs[i].name.split(".")[-1] for i in g) for g in self.groups]

    def call_bytes(self, gi: int) -> int:
        g = self.groups[gi]
        return int(sum(self.bytes_per_layer[i] for i in g) - sum(2 * self.batch * self.specs[i].K for i in g[1:]))

    def time_calls(self, reps: int = 10):
        """Every library call of the step alone in a graph (its copies round-robin, cold cache):
        [(name, us, bytes, GB/s)]."""
        torch, vq = self.torch, self.vq
        out = []
        for gi, g in enumerate(self.groups):
            def one(copy, g=g):
                i = g[0]
                if len(g) == 1:
                    idx, cb, sc = self.dev[copy][i]
                    vq.vq_gemm_small_batch(self.fmts[i], idx, cb, sc, self.X[i], self.Y[i], self.batch, self.ws[i])
                else:
                    members = [(self.dev[copy][j][0], self.dev[copy][j][1], self.dev[copy][j][2], self.Y[j], self.specs[j].N) for j in g]
                    vq.vq_gemm_small_batch_grouped(self.group_fmt[i], members, self.X[i], self.batch, self.group_ws[i])
            nbytes = self.call_bytes(gi)
            rounds = max(1, -(-2 * L2_BYTES // max(1, nbytes * self.copies)))   # enough calls to outrun the L2
            one(0)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                for _ in range(rounds):
                    for c in range(self.copies):
                        one(c)
            graph.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / (reps * rounds * self.copies)
            out.append((self.call_names()[gi], us, nbytes, nbytes / us / 1e3))
        return out

    def graph(self, n_steps: int, first_copy: int = 0):
        torch = self.torch
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for s in range(n_steps):
                self.step((first_copy + s) % self.copies)
        return g


def time_steps(ds: DeviceSet, steps: int, warmup: int, barrier=None):
    """Times exactly `steps` steps as CUDA-graph replays (one graph = one round over all copies)."""
    torch = ds.torch
    chunk = ds.copies
    ds.step(0)
    torch.cuda.synchronize()
    g_full = ds.graph(chunk)
    rem = steps % chunk
    g_rem = ds.graph(rem) if rem else None
    for _ in range(max(1, -(-warmup // chunk))):
        g_full.replay()
    torch.cuda.synchronize()
    if barrier:
        barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps // chunk):
        g_full.replay()
    if g_rem:
        g_rem.replay()
    e1.record()
    torch.cuda.synchronize()
    if barrier:
        barrier()
    return e0.elapsed_time(e1)  # ms


def time_e2e(ds: DeviceSet, steps: int, warmup: int):
    torch = ds.torch
    for s in range(max(3, min(warmup, 10))):
        ds.step_host(s % ds.copies)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for s in range(steps):
        ds.step_host(s % ds.copies)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1)


class OracleWork:
    """Host copies of a configuration for the CPU oracle; a pass covers the first rows of each layer."""

    def __init__(self, cfg_name: str, batch: int):
        from oracle import vq_oracle as orc
        self.orc = orc
        conf = vq_synth.CONFIGS[cfg_name]
        self.cfg_name, self.batch = cfg_name, batch
        self.total_w = sum(s.n_weights for s in conf["layers"])
        self.work = []
        for lid, spec in enumerate(conf["layers"]):
            f = orc.Fmt(spec.N, spec.K, spec.d, spec.b, spec.Br, spec.Bc, spec.int8)
            L = vq_synth.make_layer(spec, f.stride, conf["seed"], lid)
            X = vq_synth.make_x(spec, conf["seed"], batch, lid)
            self.work.append((f, L, X, spec))

    def run(self, max_weights: float, threads: int):
        """One bounded pass; returns (seconds, algorithmic bytes covered, description)."""
        frac = min(1.0, max_weights / self.total_w)
        t0 = time.perf_counter()
        nbytes = 0.0
        for f, L, X, spec in self.work:
            n_rows = max(1, int(round(spec.N * frac)))
            rows = None if n_rows >= spec.N else np.arange(n_rows, dtype=np.int32)
            self.orc.gemm(f, L.idx, L.cb, L.scale, X, rows=rows, threads=threads)
            nbytes += layer_bytes(spec, f.stride, self.batch) * n_rows / spec.N
        dt = time.perf_counter() - t0
        desc = (f"{self.cfg_name} batch {self.batch}: first {frac * 100:.2f}% of the rows of every layer "
                f"(about {int(self.total_w * frac)} of {self.total_w} weights) per pass, fp64 oracle as it stands")
        return dt, nbytes, desc


ORACLE_WEIGHTS_PER_SEC_PER_THREAD = 15e6  # sizing guess only; the timing itself is measured


def run_reference(args):
    from oracle import vq_oracle as orc
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    orc.build()
    threads = orc.hardware_threads() or os.cpu_count() or 1
    # bounded sample per step so that the whole run ends within a few minutes
    per_step_s = min(3.0, max(0.02, 150.0 / (args.steps + args.warmup)))
    max_w = per_step_s * ORACLE_WEIGHTS_PER_SEC_PER_THREAD * threads
    ow = OracleWork(args.config, args.batch)
    for _ in range(args.warmup):
        ow.run(max_w, threads)
    t, nbytes, desc = 0.0, 0.0, ""
    for _ in range(args.steps):
        dt, nb, desc = ow.run(max_w, threads)
        t += dt
        nbytes += nb
    val = nbytes / t / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.config} batch {args.batch}", "sample_per_step": desc},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def dram_traffic_note(cfg_name: str):
    """Average DRAM bytes (read + write) per launch of the dominant kernel, from the committed ncu
    summary (profiles/dram_traffic.json); None when no capture of the current kernel exists."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.json")) as f:
            entry = json.load(f).get(cfg_name)
        return None if not entry or not entry.get("current", False) else float(entry["avg_bytes_per_launch"])
    except Exception:
        return None


KERNEL_OF = {"cfg1": "rowcb_kernel<LdsTbl<false>,1>", "cfg2": "rowcb_kernel<PrmtI8,1>",
             "cfg3": "blockcb_kernel<2,6,1> (q/k/v and gate/up as grouped launches)",
             "cfg4": "blockcb_kernel<4,8,NB>", "cfg5": "stream_kernel<RowD2B4<int8>,NB,R,CW,CPS>",
             "llama3_8b": "blockcb_kernel<2,6,NB,warp-private tables>",
             "llama3_8b_int4cb": "blockcb_kernel<2,6,NB,warp-private tables, int4 codebooks>",
             "llama3_8b_d2b5_4x256": "warptab_kernel<5,NB>"}


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """Slowest rank's time: the whole job is done when the last replica is."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(step_bytes_per_rank: int, world: int, ms_per_step: float) -> float:
    """Replicas only: every rank moves step_bytes_per_rank per step; value = all ranks' bytes / slowest time."""
    return world * step_bytes_per_rank / (ms_per_step * 1e-3) / 1e9


PROBE_POLICY = {"cfg1": 0, "cfg2": 1, "cfg3": 3, "cfg5": 0}   # decode-loop probe that matches a configuration's kernel


def measure_ceilings(device, torch, vq, sm_mhz: float):
    """What this GPU allows before any kernel design: a plain read of 1 GiB, and the look-up +
    multiply-accumulate loops of the kernels on data that already sits in shared memory (8 warps per
    SM, no global traffic).  The decode-loop rates are turned into GB/s of compressed bytes with each
    configuration's stored bytes per weight and the SM clock `sm_mhz`."""
    out = {"sm_mhz_used": sm_mhz}
    buf = torch.empty(1 << 30, dtype=torch.uint8, device=device)
    buf.random_(0, 255)
    sink = torch.zeros(4, dtype=torch.uint8, device=device)
    for _ in range(2):
        vq.vq_probe_read(buf, sink)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        vq.vq_probe_read(buf, sink)
    e1.record()
    torch.cuda.synchronize()
    out["read_peak_GBps"] = 5 * buf.numel() / (e0.elapsed_time(e1) * 1e-3) / 1e9
    del buf
    sms = torch.cuda.get_device_properties(device).multi_processor_count
    scratch = torch.zeros(8 * sms + 128 * sms * 8 + 1024, dtype=torch.uint8, device=device)
    names = {0: "2-D 4-bit per-row codebooks (two row tiles per warp)", 1: "1-D 4-bit int8 codebooks (register look-up)",
             2: "uniform INT4 g128", 3: "2-D 6-bit shared codebooks (two row tiles per warp)"}
    loops = {}
    for pol in (0, 1, 2, 3):
        vq.vq_probe_decode_loop(pol, 8, 1, 50, scratch)
        clocks, weights = vq.vq_probe_decode_loop(pol, 8, 1, 2000, scratch)
        loops[pol] = {"policy": names[pol], "weights_per_clk_per_sm": weights / clocks,
                      "Tweights_per_s": weights / clocks * sms * sm_mhz * 1e6 / 1e12}
    out["decode_loop"] = loops
    per_cfg = {}
    for cfg, pol in PROBE_POLICY.items():
        conf = vq_synth.CONFIGS[cfg]
        nbytes = sum(layer_bytes(sp, vq.vq_pack_info(vq.VQFormat(sp.N, sp.K, sp.d, sp.b, sp.Br, sp.Bc, int(sp.int8))).row_stride_bytes, 1)
                     for sp in conf["layers"])
        nw = sum(sp.n_weights for sp in conf["layers"])
        per_cfg[cfg] = {"bytes_per_weight": nbytes / nw, "decode_loop_GBps": loops[pol]["Tweights_per_s"] * 1e3 * nbytes / nw}
    per_cfg["int4g128"] = {"bytes_per_weight": 4.125 / 8, "decode_loop_GBps": loops[2]["Tweights_per_s"] * 1e3 * 4.125 / 8}
    out["per_config"] = per_cfg
    return out


def time_int4g128(cfg_name: str, batch: int, device, torch, vq):
    """The uniform INT4 group-128 yard-stick on the shapes of a configuration: us per layer set and
    GB/s over its own bytes (nibbles + fp16 scale per 128 columns + x + y), cold cache."""
    conf = vq_synth.CONFIGS[cfg_name]
    layers, set_bytes = [], 0
    for lid, spec in enumerate(conf["layers"]):
        if spec.K % 128:
            return None
        q, sc = vq_synth.make_int4g128(spec.N, spec.K, conf["seed"], lid)
        X = vq_synth.make_x(spec, conf["seed"], batch, lid)
        nbytes = q.size + sc.size * 2 + 2 * batch * (spec.N + spec.K)
        set_bytes += nbytes
        layers.append((spec, torch.from_numpy(q).to(device), torch.from_numpy(sc).to(device), torch.from_numpy(X).to(device),
                       torch.empty((batch, spec.N), dtype=torch.float16, device=device),
                       torch.zeros(vq.vq_int4g128_workspace_bytes(spec.N, batch), dtype=torch.uint8, device=device)))
    copies = max(2, -(-2 * L2_BYTES // set_bytes))
    dev = [layers] + [[(sp, q.clone(), sc.clone(), X, Y, ws) for (sp, q, sc, X, Y, ws) in layers] for _ in range(copies - 1)]

    def step(c):
        for sp, q, sc, X, Y, ws in dev[c]:
            vq.vq_int4g128_gemm_small_batch(sp.N, sp.K, q, sc, X, Y, batch, ws)
    step(0)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for c in range(copies):
            step(c)
    for _ in range(2):
        g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(10):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (10 * copies)
    return {"us_per_step": us, "GBps": set_bytes / us / 1e3, "bytes": set_bytes}


def time_transfer_decode(device, torch, vq, N: int = 11008, K: int = 4096, reps: int = 5):
    """The transfer + decode experiment of App. B on a gate_proj-shaped layer: time to read one stored
    layer and write it out as fp16, for FP16 / INT8 / INT4-g128 storage and for three VQ formats
    (the format points of cfg3, cfg5 and cfg4).  Latencies relative to INT4, as the paper's table."""
    n_out = max(2, min(6, (2 * L2_BYTES) // (2 * N * K) + 1))
    outs = [torch.empty((N, K), dtype=torch.float16, device=device) for _ in range(n_out)]

    def timed(call):
        for w in outs:
            call(w)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for w in outs:
                call(w)
        g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (reps * n_out)

    rows = {}
    w16 = torch.from_numpy(vq_synth.normal(21, 1, N * K).astype(np.float16).reshape(N, K)).to(device)
    rows["fp16"] = {"bits_per_weight": 16.0, "us": timed(lambda w: vq.vq_unpack_uniform(vq.VQ_UNPACK_FP16, N, K, w16, None, w))}
    del w16
    q8 = torch.from_numpy(vq_synth.random_bytes(21, 2, N * K).reshape(N, K).view(np.int8)).to(device)
    s8 = torch.from_numpy((0.001 + 0.003 * vq_synth.uniform01(21, 3, N)).astype(np.float16)).to(device)
    rows["int8_row"] = {"bits_per_weight": 8.0 + 16.0 / K, "us": timed(lambda w: vq.vq_unpack_uniform(vq.VQ_UNPACK_INT8_ROW, N, K, q8, s8, w))}
    del q8
    q4, s4 = vq_synth.make_int4g128(N, K, 21)
    q4, s4 = torch.from_numpy(q4).to(device), torch.from_numpy(s4).to(device)
    rows["int4_g128"] = {"bits_per_weight": 4.125, "us": timed(lambda w: vq.vq_unpack_uniform(vq.VQ_UNPACK_INT4_G128, N, K, q4, s4, w))}
    del q4
    for name, src in (("vq_2d_3.125", "cfg3"), ("vq_2d_2.125", "cfg5"), ("vq_4d_2.125", "cfg4")):
        t = vq_synth.CONFIGS[src]["layers"][0]
        spec = vq_synth.LayerSpec(name, N, K, t.d, t.b, t.Br, t.Bc, t.int8, cb_sigma=t.cb_sigma)
        fmt = vq.VQFormat(N, K, spec.d, spec.b, spec.Br, spec.Bc, vq.VQ_CB_INT8_SCALED if spec.int8 else vq.VQ_CB_FP16)
        info = vq.vq_pack_info(fmt)
        L = vq_synth.make_layer(spec, info.row_stride_bytes, 21, 4)
        idx, cb = torch.from_numpy(L.idx).to(device), torch.from_numpy(L.cb).to(device)
        sc = None if L.scale is None else torch.from_numpy(L.scale).to(device)
        rows[name] = {"bits_per_weight": 8.0 * info.total_bytes / (N * K),
                      "us": timed(lambda w: vq.vq_decode_weights(fmt, idx, cb, sc, w))}
    base = rows["int4_g128"]
    for r in rows.values():
        r["rel_footprint"] = r["bits_per_weight"] / base["bits_per_weight"]
        r["rel_latency"] = r["us"] / base["us"]
        r["GBps"] = (r["bits_per_weight"] / 8.0 + 2.0) * N * K / r["us"] / 1e3
    return {"layer": f"{N}x{K}", "output": "fp16 [N][K]", "rows": rows}


def time_assign(device, torch, vq, cfg_name: str = "cfg3", N: int = 11008, K: int = 4096, reps: int = 5):
    """E-step (Eq. 5) on a gate_proj-shaped dense matrix against the codebooks of a configuration's
    format: us per call, vectors per second, and the arithmetic rate against the fp32 lanes of the
    GPU (SM count x 128 lanes x SM clock, one operation per lane and clock)."""
    t = vq_synth.CONFIGS[cfg_name]["layers"][0]
    spec = vq_synth.LayerSpec("assign", N, K, t.d, t.b, t.Br, t.Bc, t.int8, cb_sigma=t.cb_sigma)
    fmt = vq.VQFormat(N, K, spec.d, spec.b, spec.Br, spec.Bc, vq.VQ_CB_INT8_SCALED if spec.int8 else vq.VQ_CB_FP16)
    info = vq.vq_pack_info(fmt)
    L = vq_synth.make_layer(spec, info.row_stride_bytes, 22, 0)
    W = (spec.cb_sigma * vq_synth.normal(22, 40, N * K)).astype(np.float16).reshape(N, K)
    h = (0.25 + 2.0 * vq_synth.uniform01(22, 41, K)).astype(np.float32)
    d_W, d_h = torch.from_numpy(W).to(device), torch.from_numpy(h).to(device)
    cb = torch.from_numpy(L.cb).to(device)
    sc = None if L.scale is None else torch.from_numpy(L.scale).to(device)
    d_idx = torch.empty((N, info.row_stride_bytes), dtype=torch.uint8, device=device)
    vq.vq_assign_indices(fmt, d_W, cb, sc, d_h, d_idx)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        vq.vq_assign_indices(fmt, d_W, cb, sc, d_h, d_idx)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / reps
    Q = torch.empty((N, K), dtype=torch.float16, device=device)
    vq.vq_decode_weights(fmt, d_idx, cb, sc, Q)
    torch.cuda.synchronize()
    err = (d_W.double() - Q.double()).pow(2).mean().item()
    sqnr = 10.0 * np.log10(d_W.double().pow(2).mean().item() / err)
    vectors = N * K // spec.d
    ops = vectors * (1 << spec.b) * (4 * spec.d + 2)   # per (vector, centroid): d sub, 2d mul, d-1 add, compare, 2 selects
    props = torch.cuda.get_device_properties(device)
    sm_mhz = props.clock_rate / 1e3 if hasattr(props, "clock_rate") else 1965.0
    peak = props.multi_processor_count * 128 * sm_mhz * 1e6
    return {"layer": f"{N}x{K}", "format": f"d={spec.d} b={spec.b} {spec.Br}x{spec.Bc}", "us": us,
            "Gvectors_per_s": vectors / us / 1e3, "alu_ops_per_s": ops / us * 1e6, "alu_peak_ops_per_s": peak,
            "alu_frac": ops / us * 1e6 / peak, "sqnr_db_random_codebook": sqnr}


def time_normalized(device, torch, vq, N: int = 14336, K: int = 4096, block_cols: int = 32, copies: int = 6, reps: int = 5):
    """Block-wise normalisation applied at decode (paper appendix on blockwise data normalization) on a
    gate_proj-shaped layer of the deployed format (2-D, 6-bit, int8 codebook per 32x256 block): batch-1 product and
    weight materialisation, each over `copies` device copies of the layer (cold cache), beside the same calls
    without normalisation."""
    spec = vq_synth.LayerSpec("norm", N, K, 2, 6, 32, 256, True)
    fmt = vq.VQFormat(N, K, 2, 6, 32, 256, vq.VQ_CB_INT8_SCALED)
    info = vq.vq_pack_info(fmt)
    L = vq_synth.make_layer(spec, info.row_stride_bytes, 31, 0)
    codes, lut = vq_synth.make_norm(spec, block_cols, 32)
    dev = [tuple(torch.from_numpy(a).to(device) for a in (L.idx, L.cb, L.scale, codes, lut)) for _ in range(copies)]
    X = torch.from_numpy(vq_synth.make_x(spec, 33, 1)).to(device)
    Y = torch.empty((1, N), dtype=torch.float16, device=device)
    W = torch.empty((N, K), dtype=torch.float16, device=device)
    ws = torch.zeros(vq.vq_workspace_bytes(fmt, 1), dtype=torch.uint8, device=device)

    def timed(call):
        call(0)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for r in range(reps):
            for c in range(copies):
                call(c)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (reps * copies)

    nbytes = info.total_bytes + codes.nbytes + lut.nbytes + 2 * (N + K)
    g_us = timed(lambda c: vq.vq_gemm_small_batch_normalized(fmt, *dev[c], block_cols, X, Y, 1))
    p_us = timed(lambda c: vq.vq_gemm_small_batch(fmt, dev[c][0], dev[c][1], dev[c][2], X, Y, 1, ws))
    d_us = timed(lambda c: vq.vq_decode_weights_normalized(fmt, *dev[c], block_cols, W))
    q_us = timed(lambda c: vq.vq_decode_weights(fmt, dev[c][0], dev[c][1], dev[c][2], W))
    return {"layer": f"{N}x{K}", "format": "d=2 b=6 32x256 int8", "norm_block_cols": block_cols,
            "gemm_b1_us": g_us, "gemm_b1_GBps": nbytes / g_us / 1e3, "gemm_b1_plain_us": p_us,
            "decode_us": d_us, "decode_plain_us": q_us}


def time_decode(ds, reps: int = 3):
    """vq_decode_weights on the largest layer of the set: (us, GB/s over indices + codebooks + fp16 output)."""
    torch, vq = ds.torch, ds.vq
    i = max(range(len(ds.specs)), key=lambda j: ds.specs[j].n_weights)
    spec, fmt = ds.specs[i], ds.fmts[i]
    outs = [torch.empty((spec.N, spec.K), dtype=torch.float16, device=ds.device) for _ in range(max(2, min(6, (2 * L2_BYTES) // (2 * spec.n_weights) + 1)))]
    idx, cb, sc = ds.dev[0][i]
    for w in outs:
        vq.vq_decode_weights(fmt, idx, cb, sc, w)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()   # replayed, so that small layers are not timed at the host's launch rate
    with torch.cuda.graph(graph):
        for c, w in enumerate(outs):
            lay = ds.dev[c % ds.copies][i]
            vq.vq_decode_weights(fmt, lay[0], lay[1], lay[2], w)
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / (reps * len(outs))
    nbytes = ds.bytes_per_layer[i] - 2 * ds.batch * (spec.K + spec.N) + 2 * spec.n_weights
    return {"layer": spec.name, "us": us, "GBps": nbytes / us / 1e3, "bytes": nbytes}


def run_ours(args):
    import torch
    import paper_2402_15319_b200 as vq
    vq.load()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    peak, peak_src = measured_peaks()
    if args.ceilings:   # the micro-benchmarks alone; the SM clock is the median polled while they run
        if rank == 0:
            sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid))
            sampler.start()
            t_end = time.time() + 1.0
            while time.time() < t_end:
                measure_ceilings(dev, torch, vq, 1965.0)
            sampler.stop()
            clocks = sampler.summary("polled during the micro-benchmarks")
            print(json.dumps({"metric": "ceilings", "peak_GBps": peak, "peak_source": peak_src, "clocks": clocks,
                              **measure_ceilings(dev, torch, vq, float(clocks.get("sm_mhz") or 1965.0))}))
        return
    ds = DeviceSet(args.config, args.batch, dev)
    if args.decode_only:   # vq_decode_weights alone on the configuration's largest layer (profiling runs)
        dec = time_decode(ds)
        dec["frac_of_measured"] = dec["GBps"] / peak
        if rank == 0:
            print(json.dumps({"metric": "vq_decode_weights_bandwidth", "unit": "GB/s", "value": dec["GBps"], "config": args.config, **dec}))
        return
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid))
    sampler.start()
    ms = time_steps(ds, args.steps, args.warmup, barrier)
    sampler.stop()
    clock_src = "polled during the timed region"
    if len(sampler.samples) < 3:  # region shorter than a few polls: repeat the identical loop for the clock record
        sampler.start()
        t_end = time.time() + 0.5
        while time.time() < t_end:
            time_steps(ds, args.steps, 0)
        sampler.stop()
        clock_src = "timed region too short to poll; polled during immediate repeats of the same loop"
    ms = max_over_ranks(ms, dist, dev)
    ms_per_step = ms / args.steps
    value = whole_job_gbs(ds.step_bytes, world, ms_per_step)

    e2e_steps = max(5, min(args.steps, 200))
    ms_e2e = time_e2e(ds, e2e_steps, args.warmup) if not args.no_e2e else float("nan")
    ms_e2e = max_over_ranks(ms_e2e, dist, dev)
    e2e_val = whole_job_gbs(ds.step_bytes, world, ms_e2e / e2e_steps)

    launches_per_step = ds.launches_per_step()
    step_gbs = ds.step_bytes / (ms_per_step * 1e-3) / 1e9  # one GPU's kernels
    # the dominant kernel: every library call of the step timed alone (CUDA events, graph replay, cold cache)
    calls = ds.time_calls()
    dom = max(calls, key=lambda c: c[1])
    traffic = dram_traffic_note(args.config)
    clocks = sampler.summary(clock_src)
    sp0 = ds.specs[0]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": f"{args.config}: {sp0.name.split('.')[0]} layer set ({len(ds.specs)} layers, "
                        f"{ds.n_weights} weights), d={sp0.d}, {sp0.b}-bit indices, "
                        f"{'int4 (+scale per row and 128 columns)' if int(sp0.int8) == 2 else 'int8+scale' if sp0.int8 else 'fp16'} codebook per {sp0.Br}x{sp0.Bc} block, batch {args.batch}",
            "calls_per_step": ds.call_names(),
            "grouping": "q/k/v and gate/up read one activation tensor each (the first member's) through vq_gemm_small_batch_grouped; "
                        "that tensor is counted once in bytes_per_step",
            "bytes_per_step": ds.step_bytes, "us_per_layer_set": ms_per_step * 1e3,
            "cold_cache": f"{ds.copies} distinct device copies of every layer visited round-robin "
                          f"({ds.copies * ds.step_bytes / 2**20:.0f} MiB > 2 x L2); inputs larger than L2, no flush",
            "launch": "CUDA graph of one round over all copies, replayed",
            "pct_of_nominal_8TBps": 100 * step_gbs / NOMINAL_HBM_GBS,
            "frac_of_measured_whole_step": step_gbs / peak,
            "parallelism": "replicas only (one GPU per process, no collective)" if world > 1 else "single GPU",
        },
        "clocks": clocks,
        "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": ds.h2d, "d2h_bytes_per_step": ds.d2h,
                "steps": e2e_steps, "ms_per_step": ms_e2e / e2e_steps,
                "what": "the step's calls with host buffers (vq_gemm_small_batch_grouped_host for q/k/v and gate/up, vq_gemm_small_batch_host for o and down): activations read from pinned host memory, kernels, outputs written back to pinned host memory, stream synchronised every step; compressed weights resident in HBM"},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": {
            "bound": "hbm", "kernel": f"{KERNEL_OF.get(args.config, 'vq gemm kernel')}: call '{dom[0]}' (largest share of the step: "
                                      f"{100 * dom[1] / sum(c[1] for c in calls):.0f}% of the summed call times)",
            "achieved": dom[3], "peak": peak, "unit": "GB/s", "frac": dom[3] / peak, "peak_source": peak_src,
            "algorithmic_bytes_per_launch": dom[2], "avg_launch_us": dom[1], "traffic": traffic,
            "calls_alone": [{"call": c[0], "us": c[1], "bytes": c[2], "GBps": c[3], "frac": c[3] / peak} for c in calls],
        },
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import vq_oracle as orc
        orc.build()
        threads = orc.hardware_threads() or os.cpu_count() or 1
        dt, nbytes, desc = OracleWork(args.config, args.batch).run(12.0 * ORACLE_WEIGHTS_PER_SEC_PER_THREAD * threads, threads)
        line["cpu_baseline"] = {"value": nbytes / dt / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": desc, "seconds": dt}
    if rank == 0 and world == 1 and not args.no_per_config:
        del ds
        torch.cuda.empty_cache()
        sm_mhz = clocks.get("sm_mhz") or 1965.0
        ceil = measure_ceilings(dev, torch, vq, float(sm_mhz))
        line["ceilings"] = ceil
        per, i4 = {}, {}
        cfgs = list(vq_synth.CONFIGS) if args.all_configs else ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"]
        for cfg in cfgs:
            d2 = None
            for b in vq_synth.CONFIGS[cfg]["batches"]:
                if d2 is None:
                    d2 = DeviceSet(cfg, b, dev)
                else:
                    d2.set_batch(b)
                st = max(d2.copies * 10, 100)
                m = time_steps(d2, st, d2.copies * 3) / st
                gbs = d2.step_bytes / (m * 1e-3) / 1e9
                row = {"us": round(m * 1e3, 2), "GBps": round(gbs, 1), "frac": round(gbs / peak, 4), "launches": d2.launches_per_step()}
                lim = ceil["per_config"].get(cfg)
                if lim and b <= 8:
                    row["ceilings_GBps"] = {"hbm": round(peak, 1), "read": round(ceil["read_peak_GBps"], 1),
                                            "decode_loop": round(lim["decode_loop_GBps"], 1)}
                per[f"{cfg}.b{b}"] = row
                if args.all_configs and b == vq_synth.CONFIGS[cfg]["batches"][0]:
                    dec = time_decode(d2)
                    dec["frac_of_measured"] = dec["GBps"] / peak
                    per[f"{cfg}.decode_weights"] = dec
            del d2
            torch.cuda.empty_cache()
            r = time_int4g128(cfg, vq_synth.CONFIGS[cfg]["batches"][0], dev, torch, vq)
            if r:
                i4[cfg] = {"us": round(r["us_per_step"], 2), "GBps": round(r["GBps"], 1), "frac": round(r["GBps"] / peak, 4)}
            torch.cuda.empty_cache()
        line["per_config"] = per
        line["int4g128"] = {"what": "uniform INT4 group-128 GEMV (4.125 bits per weight) on each configuration's layer shapes, "
                                    "one call per layer, batch = the configuration's first", "decode_loop_ceiling_GBps":
                            round(ceil["per_config"]["int4g128"]["decode_loop_GBps"], 1), **i4}
        if args.all_configs:
            line["transfer_decode"] = time_transfer_decode(dev, torch, vq)
            line["assign"] = time_assign(dev, torch, vq)
            line["normalized"] = time_normalized(dev, torch, vq)
    if rank == 0:
        print(json.dumps(line))
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def spawn_replicas(args):
    """`--gpus N` without a launcher: start N local ranks (one per GPU) of this same command."""
    import socket
    import subprocess
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=40)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg5", choices=sorted(vq_synth.CONFIGS))
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--all-configs", action="store_true", help="per_config also covers llama3_8b and vq_decode_weights; adds transfer_decode and assign")
    ap.add_argument("--no-per-config", action="store_true", help="skip per_config, int4g128 and ceilings (profiling runs)")
    ap.add_argument("--ceilings", action="store_true", help="run the ceiling micro-benchmarks alone and print them")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--decode-only", action="store_true", help="time vq_decode_weights on the configuration's largest layer and exit")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end loop (profiling runs)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_replicas(args))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
