#!/usr/bin/env python
"""Benchmark of the BCQ GEMV hot path: per-token time of all linear layers of a decoder stack.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one token at batch 1: every linear layer of the stack (6 per decoder layer) once,
each with its own packed weights resident in HBM (the stack is far larger than L2, so every
launch streams its weights from DRAM).  Prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2407_02891_b200 import synth

# name -> (hidden, ffn, layers, q, group, description)
WORKLOADS = {
    "opt30b_q3_g128": dict(hidden=7168, ffn=28672, layers=48, q=3, group=128),
    "opt30b_q2_g128": dict(hidden=7168, ffn=28672, layers=48, q=2, group=128),
    "opt6.7b_q3_g128": dict(hidden=4096, ffn=16384, layers=32, q=3, group=128),
    "opt66b_q2_g128": dict(hidden=9216, ffn=36864, layers=64, q=2, group=128),
    "opt66b_q2_row": dict(hidden=9216, ffn=36864, layers=64, q=2, group=0),
    # Llama-2-70B-shaped layers (GQA: fused k/v of 2 x 1024 rows, gated FFN); 8 of them so that the
    # operands (3 GB) are far larger than L2.  Use --batch 1|2|4|8|16 for the small-batch sweep.
    "llama70b_q3_g128": dict(family="llama", hidden=8192, ffn=28672, kv=2048, layers=8, q=3, group=128),
}
DEFAULT_WORKLOAD = "opt30b_q3_g128"
# DRAM bytes per launch of the dominant kernel: the per-shape dram__bytes_read + dram__bytes_write figures of
# the ncu capture summarised under profiles/ (a small text file, one "key value" pair per line); they hold
# only for the library revision they were taken on.
NCU_TRAFFIC_FILE = os.path.join(ROOT, "profiles", "lut_gemv_kernel_opt30b_q3_g128.traffic.txt")
METRIC = "BCQ GEMV us/token (sum of all linear layers of the decoder stack, bs=1)"
UNIT = "us/token"


def layer_shapes(w):
    """(name, N, K) of the six linear layers of one decoder layer (OPT, or Llama-2 with GQA).

    With w["fuse"] the projections that read the same activation are stacked into one product
    (q/k/v; gate/up): the same weights and the same arithmetic in fewer, longer launches."""
    h, f = w["hidden"], w["ffn"]
    if w.get("family") == "llama":
        if w.get("fuse"):
            return [("qkv", h + w["kv"], h), ("o", h, h), ("gate_up", 2 * f, h), ("down", h, f)]
        return [("q", h, h), ("kv", w["kv"], h), ("o", h, h), ("gate", f, h), ("up", f, h), ("down", h, f)]
    if w.get("fuse"):
        return [("qkv", 3 * h, h), ("out", h, h), ("fc1", f, h), ("fc2", h, f)]
    return [("q", h, h), ("k", h, h), ("v", h, h), ("out", h, h), ("fc1", f, h), ("fc2", h, f)]


def algorithmic_bytes(N, K, q, group, B=1):
    """Packed planes + fp16 alphas + fp16 offsets + x + y."""
    G = 1 if group == 0 else K // group
    return q * N * K // 8 + 2 * q * N * G + 2 * N * G + 2 * B * K + 2 * B * N


def ncu_traffic_per_launch(lib_version, workload, shapes_per_step):
    """Mean DRAM bytes per launch over one step from the tracked ncu figures, or None when they were taken on
    another library revision or workload.  shapes_per_step: {"NxK": launches per step}."""
    try:
        kv = {}
        with open(NCU_TRAFFIC_FILE) as f:
            for line in f:
                line = line.split("#")[0].split()
                if len(line) == 2:
                    kv[line[0]] = line[1]
        if int(kv["lib_version"]) != lib_version or kv["workload"] != workload:
            return None
        total = sum(float(kv["dram_bytes_" + s]) * n for s, n in shapes_per_step.items())
        return total / sum(shapes_per_step.values())
    except (OSError, KeyError, ValueError):
        return None


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ---------------------------------------------------------------------------------------------
# clocks during the timed region
# ---------------------------------------------------------------------------------------------

class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int, period=0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None
        self.period = period

    def _run(self):
        while not self._stop.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                mask = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def max_over_ranks(value: float, world: int, device) -> float:
    """The slowest rank's time: replicas run independently, the job is as slow as its slowest rank.
    A barrier, then an all-reduce(MAX) of one scalar -- the only collective of the multi-GPU path."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    dist.barrier()
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_metric(ms_per_step: float, world: int) -> float:
    """us/token of the whole job: `world` replicas each finish one token per step (weak scaling)."""
    return ms_per_step * 1e3 / world


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# ---------------------------------------------------------------------------------------------
# the stack on the device
# ---------------------------------------------------------------------------------------------

class Stack:
    """All packed layers of the workload, resident on one GPU, plus per-shape x and per-layer y."""

    def __init__(self, wname, w, device, B=1):
        import torch
        from paper_2407_02891_b200 import binding as bq

        self.bq, self.torch, self.device = bq, torch, device
        self.w, self.wname, self.B = w, wname, B
        q, group = w["q"], w["group"]
        self.items = []       # (desc, packed, alpha, z, x, y, ws)
        self.bytes = 0
        scales, xs, wss = {}, {}, {}
        distinct = []
        for (pname, N, K) in layer_shapes(w):
            if (N, K) not in distinct:
                distinct.append((N, K))
        # the activations of a token: one vector (B vectors) per distinct input width K (projections of equal K
        # read the same vector, as q/k/v or gate/up do), side by side in ONE device buffer, so that the
        # end-to-end leg can bring a token's activations in with a single copy
        widths = []
        for (_, K) in distinct:
            if K not in widths:
                widths.append(K)
        x_np = [synth.activations(f"{wname}/K{K}", B, K).reshape(-1) for K in widths]
        self.x_host_all = torch.from_numpy(np.concatenate(x_np))
        self.x_all = self.x_host_all.to(device)
        xk, off = {}, 0
        for K, xv in zip(widths, x_np):
            xk[K] = self.x_all[off:off + xv.size]            # 16-byte aligned: K is a multiple of 512
            off += xv.size
        for (N, K) in distinct:
            a, z = synth.scale_rows(f"{wname}/{N}x{K}", N, K, q, group)
            dt = bq.desc(N, K, q, group, bq.LAYOUT_TILED)
            scales[(N, K)] = (torch.from_numpy(a).to(device), torch.from_numpy(z).to(device))
            xs[(N, K)] = xk[K]
            wss[(N, K)] = bq.new_workspace(dt, B, device=device)
        self.names = []       # generator names of every item, for the parity check
        for layer in range(w["layers"]):
            for (pname, N, K) in layer_shapes(w):
                dc = bq.desc(N, K, q, group, bq.LAYOUT_CANONICAL)
                dt = dc.with_layout(bq.LAYOUT_TILED)
                canon = synth.planes_device(f"{wname}/L{layer}/{pname}", N, K, q, device).reshape(-1)
                ad, zd = scales[(N, K)]
                packed, at, zt = bq.empty_operands(dt, device)      # every layer owns its operands
                bq.repack(dc, canon, ad, zd, dt, packed, at, zt)
                y = torch.zeros(B * N, dtype=torch.float16, device=device)
                self.items.append((dt, packed, at, zt, xs[(N, K)], y, wss[(N, K)], (N, K)))
                self.names.append(f"{wname}/L{layer}/{pname}")
                self.bytes += algorithmic_bytes(N, K, q, group, B)
            torch.cuda.synchronize(device)
        self.graph = None

    def launch_one(self, it):
        (d, packed, a, z, x, y, ws, _) = it
        if self.B == 1:
            self.bq.gemv(d, packed, a, z, x, y, ws)
        else:
            self.bq.gemm_smallbatch(d, packed, a, z, x, y, self.B, ws)

    def launch_all(self):
        for it in self.items:
            self.launch_one(it)

    # ---- the projections that read the same activation, one launch each (bcq_gemv_multi) --------------
    def grouped_launches(self):
        """[[item indices]]: q/k/v (OPT), q + fused k/v and gate + up (Llama-2) share their activation."""
        together = [{"q", "kv"}, {"gate", "up"}] if self.w.get("family") == "llama" else [{"q", "k", "v"}]
        per_layer = len(layer_shapes(self.w))
        names = [n for (n, _, _) in layer_shapes(self.w)]
        out = []
        for layer in range(self.w["layers"]):
            base, i = layer * per_layer, 0
            while i < per_layer:
                grp = next((g for g in together if names[i] in g), None)
                j = i + 1
                while grp is not None and j < per_layer and names[j] in grp:
                    j += 1
                out.append(list(range(base + i, base + j)))
                i = j
        return out

    def launch_grouped(self, groups, ws_multi):
        bq = self.bq
        for g in groups:
            if len(g) == 1:
                self.launch_one(self.items[g[0]])
                continue
            its = [self.items[i] for i in g]
            d0 = its[0][0]
            d = bq.desc(sum(it[0].N for it in its), d0.K, d0.q, d0.group, bq.LAYOUT_TILED)
            layers = [bq.Layer(it[0], it[1], it[2], it[3]) for it in its]
            bq.gemv_multi(d, layers, its[0][4], [it[5] for it in its], ws_multi[(d.N, d.K)])

    def time_dequant(self, steps):
        """us per token of the ablation without lookup tables (bcq_gemv_dequant) on the same operands."""
        torch, bq = self.torch, self.bq

        def launch():
            for (d, packed, a, z, x, y, ws, _) in self.items:
                bq.gemv_dequant(d, packed, a, z, x, y)

        launch()
        torch.cuda.synchronize(self.device)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            launch()
        g.replay()
        torch.cuda.synchronize(self.device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            g.replay()
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1) * 1e3 / steps

    def time_grouped(self, steps):
        """us per token with those projections launched together; None when nothing is grouped."""
        torch, bq = self.torch, self.bq
        groups = self.grouped_launches()
        if self.B != 1 or self.w.get("fuse") or all(len(g) == 1 for g in groups):
            return None
        ws_multi = {}
        for g in groups:
            if len(g) > 1:
                its = [self.items[i] for i in g]
                d0 = its[0][0]
                d = bq.desc(sum(it[0].N for it in its), d0.K, d0.q, d0.group, bq.LAYOUT_TILED)
                if (d.N, d.K) not in ws_multi:
                    ws_multi[(d.N, d.K)] = bq.new_workspace(d, 1, device=self.device)
        self.launch_grouped(groups, ws_multi)
        torch.cuda.synchronize(self.device)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.launch_grouped(groups, ws_multi)
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize(self.device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            g.replay()
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1) * 1e3 / steps, len(groups)

    def launches_per_step(self):
        """Kernel launches of one step: one per layer, except where the default plan of the batch is the
        lookup-table kernel, which takes two columns per launch (one with per-row scales)."""
        n = 0
        for it in self.items:
            plan = self.bq.plan_default(it[0], self.B)
            per_launch = 2 if self.bq.scales_in_tiles(it[0]) else 1
            n += -(-self.B // per_launch) if (self.B > 1 and plan.kernel == 1) else 1
        return n

    def capture(self):
        torch = self.torch
        self.launch_all()                      # first launches configure the kernels before capture
        torch.cuda.synchronize(self.device)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.launch_all()
        self.graph = g

    def step(self):
        self.graph.replay()

    def time_steps(self, steps):
        """Device time of `steps` graph replays, in ms (CUDA events on the launching stream)."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            self.graph.replay()
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1)

    def per_shape_us(self, reps=3):
        """Mean device time per launch of each distinct shape: all launches of the shape, every one on its own
        weights, captured in a CUDA graph (plain launches from Python would time the host, not the device)."""
        torch = self.torch
        out = {}
        shapes = sorted({it[7] for it in self.items})
        for s in shapes:
            its = [it for it in self.items if it[7] == s]
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for it in its:
                    self.launch_one(it)
            g.replay()
            torch.cuda.synchronize(self.device)
            best = None
            for _ in range(reps):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                g.replay()
                e1.record()
                e1.synchronize()
                t = e0.elapsed_time(e1) * 1e3 / len(its)
                best = t if best is None else min(best, t)
            N, K = s
            b = algorithmic_bytes(N, K, self.w["q"], self.w["group"], self.B)
            out[f"{N}x{K}"] = {"us": round(best, 3), "gbs": round(b / best * 1e-3, 1), "launches": len(its)}
        return out

    def parity(self, rows_per_shape=48):
        """Sampled output rows of the LAST launch of every distinct shape (what the timed replays left in y),
        recomputed by the CPU oracle from inputs regenerated on the host."""
        import oracle

        q, group = self.w["q"], self.w["group"]
        worst, rows_checked, per_shape = 0.0, 0, {}
        last = {}
        for idx, it in enumerate(self.items):
            last[it[7]] = idx
        for (N, K), idx in last.items():
            name = self.names[idx]
            y = self.items[idx][5].cpu().numpy().astype(np.float64).reshape(self.B, N)
            r = synth.u64(name + "/bench_rows", 0, rows_per_shape) % np.uint64(N)
            rows = np.unique(np.concatenate([r.astype(np.int64), [0, N - 1]]))
            a, z = synth.scale_rows(f"{self.wname}/{N}x{K}", N, K, q, group)
            X = synth.activations(f"{self.wname}/K{K}", self.B, K)
            ref = oracle.forward_planes(synth.plane_rows(name, N, K, q, rows), a[:, rows], z[rows], X, group)
            err = float(np.abs(y[:, rows] - ref).max() / np.abs(ref).max()) if np.isfinite(y).all() else float("inf")
            per_shape[f"{N}x{K}"] = err
            worst = max(worst, err)
            rows_checked += len(rows)
        return {"max_rel_err": worst, "tol": 5e-3, "rows": rows_checked, "per_shape": per_shape,
                "ok": bool(worst <= 5e-3),
                "what": "sampled rows of the last launch of every distinct shape after the timed replays, "
                        "against the fp64 CPU oracle on regenerated inputs"}

    def e2e_steps(self, steps):
        """The same token end to end: the token's activations come from pinned host memory (one copy), the
        products run through bcq_gemv as in the timed region (the captured graph), the last layer's output
        goes back to pinned host memory (one copy), and the host waits for it."""
        torch = self.torch
        xh = self.x_host_all.pin_memory()
        last_y = self.items[-1][5]
        yh = torch.zeros(last_y.numel(), dtype=torch.float16).pin_memory()
        h2d = xh.numel() * xh.element_size()
        d2h = yh.numel() * yh.element_size()

        def one():
            self.x_all.copy_(xh, non_blocking=True)
            self.graph.replay()
            yh.copy_(last_y, non_blocking=True)
            torch.cuda.current_stream().synchronize()

        for _ in range(3):
            one()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(self.device)
        e0.record()
        for _ in range(steps):
            one()
        e1.record()
        e1.synchronize()
        return e0.elapsed_time(e1) / steps, h2d, d2h


# ---------------------------------------------------------------------------------------------
# the oracle, timed on the host cores (CPU baseline / reference arm)
# ---------------------------------------------------------------------------------------------

class OracleSample:
    """One decoder layer of the workload (6 products) for the CPU oracle, generated once on the host."""

    def __init__(self, wname, w):
        import oracle

        self.oracle, self.wname, self.w = oracle, wname, w
        q, group = self.w["q"], self.w["group"]
        self.data = []
        for (pname, N, K) in layer_shapes(self.w):
            p = synth.planes(f"{wname}/L0/{pname}", N, K, q)
            a, z = synth.scale_rows(f"{wname}/{N}x{K}", N, K, q, group)
            x = synth.activations(f"{wname}/K{K}", 1, K)
            self.data.append((p, a, z, x))
        self.cores = oracle.num_threads()

    def layer_seconds(self):
        t0 = time.perf_counter()
        for (p, a, z, x) in self.data:
            self.oracle.forward_planes(p, a, z, x, self.w["group"])
        return time.perf_counter() - t0

    def us_per_token(self, budget_s=12.0, max_reps=48):
        """Time the oracle on the layer as often as fits the budget; scale the median to the stack."""
        times, t_start = [], time.perf_counter()
        while len(times) < max_reps:
            times.append(self.layer_seconds())
            if time.perf_counter() - t_start + times[-1] > budget_s:
                break
        sample = (f"{len(times)} x one decoder layer (6 products) of {self.wname}, fp64 bit-plane form, "
                  f"median x {self.w['layers']} layers")
        return float(np.median(times)) * self.w["layers"] * 1e6, sample


# ---------------------------------------------------------------------------------------------

def spawn_replicas(n: int) -> int:
    """`python bench.py --gpus N` run plainly: start the N replicas (one process per GPU) the way the
    contract launches them, and pass their output through.  Fails cleanly when the box has fewer GPUs."""
    import subprocess

    import torch
    have = torch.cuda.device_count()
    if have < n:
        sys.stderr.write(f"bench.py: --gpus {n} asked for, {have} visible: nothing measured\n")
        return 2
    port = 29500 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def run_search(args):
    """--search: the search over BCchoice and the re-explored scale (bcq_grid_search) on one OPT-30B-shaped
    projection; a second benchmark beside the per-token line, with its own roofline (tensor cores)."""
    import torch
    from paper_2407_02891_b200 import binding as bq

    N = K = 7168
    T, n_bits, q, group, n_scales = args.search_tokens, 5, 3, 128, 8
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    W = (0.05 * synth.normal("search/W", 0, N * K)).reshape(N, K).astype(np.float16)
    X = synth.activations("search/X", T, K)
    Wd, Xd = torch.from_numpy(W).to(device), torch.from_numpy(X).to(device)
    parts, s = bq.partitions(n_bits, q), bq.reexplore_factors(n_bits, n_scales)
    for _ in range(max(3, args.warmup)):
        out = bq.grid_search(N, K, q, group, Wd, Xd, n_bits, parts, s)
    torch.cuda.synchronize(device)
    steps = min(args.steps, 20)
    with ClockSampler(physical_gpu_index(0)) as clocks:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            out = bq.grid_search(N, K, q, group, Wd, Xd, n_bits, parts, s)
        e1.record()
        e1.synchronize()
    ms = e0.elapsed_time(e1) / steps
    flops = 2.0 * N * K * T * len(parts) * n_scales
    peak = 1590.0
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak_kind = "fallback"
    if os.path.exists(path):
        with open(path) as f:
            peak, peak_kind = float(json.load(f)["bf16_tflops"]), "measured (bf16 burst; fp16 runs at the same rate)"
    # parity on sampled rows (rows are independent): the oracle on the same weights, inputs and candidates
    import oracle
    rows = np.unique(synth.u64("search/rows", 0, 24) % np.uint64(N)).astype(np.int64)
    ref_rows, _, _ = oracle.grid_search(W[rows], X, group, n_bits, list(parts), s)
    got = out[1].cpu().numpy().astype(np.float64)[:, :, rows]
    rel = float(np.abs(got - ref_rows).max() / np.abs(ref_rows).max())
    status = bq.lib().bcq_poll_status()
    print(json.dumps({
        "metric": "GPTQT search over BCchoice and scale factor, ms per layer", "value": ms, "unit": "ms", "n_gpus": 1,
        "steps": steps, "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16 operands, f32 accumulate (tcgen05)", "data": "synthetic",
        "config": {"workload": f"search_{N}x{K}_T{T}_n{n_bits}_q{q}_g{group}", "candidates": int(len(parts)),
                   "scale_factors": n_scales, "tokens": T},
        "clocks": clocks.summary(), "gpu_launches": steps * (n_scales + 2 * ((n_scales + 7) // 8) + 1),   # quantiser per factor; errors and sums per 8 factors; argmin
        "roofline": {"bound": "tensor", "achieved": round(flops / ms / 1e9, 1), "peak": peak, "unit": "TFLOP/s",
                     "frac": round(flops / ms / 1e9 / peak, 4), "peak_kind": peak_kind, "traffic": None,
                     "kernel": "search_error_kernel", "flops_per_step": flops},
        "parity": {"max_rel_err": rel, "tol": 5e-3, "rows": int(len(rows)), "ok": bool(rel <= 5e-3 and status == 0),
                   "what": "per-row errors of all candidates on sampled rows against the fp64 oracle"},
        "best": [int(v) for v in out[2].cpu().numpy()]}))
    if not (rel <= 5e-3 and status == 0):
        sys.exit(1)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-parity", action="store_true", help="skip the sampled-row oracle check of the timed outputs")
    ap.add_argument("--batch", type=int, default=1, help="activation vectors per product (1..16)")
    ap.add_argument("--fuse", action="store_true",
                    help="stack the projections that share an activation (q/k/v, gate/up) into one product each; "
                         "not the default workload: a second number beside it")
    ap.add_argument("--layers", type=int, default=0, help="override the number of decoder layers (profiling)")
    ap.add_argument("--search", action="store_true",
                    help="time bcq_grid_search on a 7168 x 7168 projection instead of the per-token step")
    ap.add_argument("--search-tokens", type=int, default=128, help="calibration tokens T of --search (16..256)")
    ap.add_argument("--profile", action="store_true",
                    help="for runs under ncu: plain launches instead of a CUDA graph, warm-up as given, "
                         "no per-shape, e2e or CPU legs; the printed number is not a benchmark value")
    args = ap.parse_args()
    if args.search:
        return run_search(args)

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        sys.exit(spawn_replicas(args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    w = dict(WORKLOADS[args.workload])
    if args.layers > 0:
        w["layers"] = args.layers
    if args.fuse:
        w["fuse"] = True
    config = {"workload": args.workload,
              "shapes": ", ".join(f"{n}:{N}x{K}" for (n, N, K) in layer_shapes(w)) + " per layer",
              "hidden": w["hidden"], "ffn": w["ffn"], "layers": w["layers"], "q": w["q"], "group": w["group"],
              "batch": args.batch, "fused_projections": bool(args.fuse),
              "cache": "inputs larger than L2 (every launch reads its own weights)", "parallelism": "replicas only"}

    if args.impl == "reference":
        if rank != 0:
            return
        # each step is one decoder layer of the stack (a bounded sample), scaled to the whole stack
        smp = OracleSample(args.workload, w)
        steps, warmup = min(args.steps, 20), min(args.warmup, 2)
        for _ in range(warmup):
            smp.layer_seconds()
        t0 = time.perf_counter()
        for _ in range(steps):
            smp.layer_seconds()
        v = (time.perf_counter() - t0) / steps * w["layers"] * 1e6
        cores = smp.cores
        sample = (f"one decoder layer (6 products) of {args.workload} per step, {steps} steps timed, "
                  f"scaled x {w['layers']} layers")
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": v / 1e3, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": "each step: " + sample},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}))
        return

    import torch

    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    from paper_2407_02891_b200 import binding as bq
    bq.lib()   # fail loudly if the CUDA library is missing

    stack = Stack(args.workload, w, device, args.batch)
    if args.profile:
        for _ in range(args.warmup):
            stack.launch_all()
        torch.cuda.synchronize(device)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            stack.launch_all()
        e1.record()
        e1.synchronize()
        print(json.dumps({"profile_run": True, "config": config, "launches": len(stack.items) * args.steps,
                          "ms_per_step_not_a_bench_value": e0.elapsed_time(e1) / args.steps}))
        return
    stack.capture()
    for _ in range(max(3, args.warmup)):
        stack.step()
    torch.cuda.synchronize(device)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize(device)
    with ClockSampler(physical_gpu_index(local)) as clocks:
        ms = stack.time_steps(args.steps)
        torch.cuda.synchronize(device)
    ms = max_over_ranks(ms, world, device)
    ms_per_step = ms / args.steps
    launches_per_step = stack.launches_per_step()

    parity = stack.parity() if rank == 0 and not args.no_parity else None   # what the timed replays left in y
    per_shape = stack.per_shape_us()
    grouped = None
    if world == 1:
        got = stack.time_grouped(args.steps)
        if got is not None:
            gp = stack.parity() if not args.no_parity else None       # the grouped launches wrote the same y tensors
            grouped = {"value": got[0], "unit": UNIT, "launches_per_step": got[1],
                       "achieved_gbs": round(stack.bytes / (got[0] * 1e-6) / 1e9, 1),
                       "frac": round(stack.bytes / (got[0] * 1e-6) / 1e9 / measured_peak_gbs()[0], 4),
                       "what": "the same token with the projections that read the same activation (q/k/v; gate/up) "
                               "launched together through bcq_gemv_multi: same weights, same outputs, fewer launches; "
                               "a second number, not the headline",
                       "parity_max_rel_err": None if gp is None else gp["max_rel_err"]}
            if gp is not None and not gp["ok"]:
                parity = gp
    ablation = None
    if world == 1 and args.batch == 1 and not args.fuse:
        us = stack.time_dequant(max(2, min(args.steps, 10)))
        ap_ = stack.parity() if not args.no_parity else None      # the ablation wrote the same y tensors
        ablation = {"value": us, "unit": UNIT, "ratio_to_value": round(us / (ms_per_step * 1e3), 2),
                    "parity_max_rel_err": None if ap_ is None else ap_["max_rel_err"],
                    "what": "the same token through bcq_gemv_dequant: every weight dequantised to fp16 and multiplied, no "
                            "lookup tables, same operands and bytes; the paper quotes 1.24x for binary-coded weights over "
                            "a 3-bit linear kernel on OPT-30B (RTX A5000): context, other hardware"}
        if ap_ is not None and not ap_["ok"]:
            parity = ap_
    e2e = None
    if not args.no_e2e:
        e_ms, h2d, d2h = stack.e2e_steps(max(3, min(args.steps, 50)))
        e_ms = max_over_ranks(e_ms, world, device)
        e2e = {"value": replica_metric(e_ms, world), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "api": "per token: one copy of the token's activations from pinned host memory, every product through "
                      "bcq_gemv / bcq_gemm_smallbatch (the captured graph of the timed region), one copy of the last "
                      "layer's output to pinned host memory, stream synchronise"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak_gbs()
    achieved = stack.bytes / (ms_per_step * 1e-3) / 1e9
    shapes_per_step = {}
    for it in stack.items:
        key = f"{it[7][0]}x{it[7][1]}"
        shapes_per_step[key] = shapes_per_step.get(key, 0) + 1
    traffic = (ncu_traffic_per_launch(bq.lib().bcq_version(), args.workload, shapes_per_step)
               if args.batch == 1 and not args.fuse else None)
    out = {
        "metric": METRIC, "value": replica_metric(ms_per_step, world), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 accumulate, f16 lookup tables (fp16 x, y, scales)" if args.batch <= 3 else
        "f32 accumulate, f16 tensor-core operands (fp16 x, y, scales)", "data": "synthetic", "config": config,
        "tokens_per_s": world * 1e3 / ms_per_step,
        "clocks": clocks.summary(),
        "gpu_launches": launches_per_step * args.steps,
        "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                     "frac": round(achieved / peak, 4), "frac_of_nominal_8000": round(achieved / 8000.0, 4),
                     "peak_kind": peak_kind,
                     "traffic": traffic,
                     "kernel": f"lut_gemv_kernel<{w['q']}>" if args.batch <= 3 else f"mma_gemm_kernel<{w['q']}>",
                     "algorithmic_bytes_per_launch": stack.bytes // launches_per_step,
                     "launches_per_step": launches_per_step},
        "per_shape": per_shape,
        "e2e": e2e,
        "parity": parity,
        "grouped_projections": grouped,
        "dequant_ablation": ablation,
    }
    if not args.no_cpu_baseline and args.batch == 1:
        smp = OracleSample(args.workload, w)
        v, sample = smp.us_per_token()
        out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": smp.cores, "kind": "oracle", "sample": sample}
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()
    if parity is not None and not parity["ok"]:
        sys.stderr.write("bench.py: the timed outputs do not match the oracle within the tolerance\n")
        sys.exit(1)


if __name__ == "__main__":
    main()
