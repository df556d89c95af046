#!/usr/bin/env python
"""Throughput of the DPSGD gradient-privatisation step (examples/s through per-example weight
gradients + clip + noise) on synthetic inputs, with the roofline fraction of the dominant kernel
and the float64 CPU oracle timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload small_cnn|flat|sweep|per_layer]
    python bench.py --impl reference ...        # times the CPU oracle on a bounded sample

One "step" is one pass of the whole path over one batch: for `small_cnn` 256 examples through
four weight-gradient calls, one clip-accumulate and one noise-average.  Rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2109_12191_b200.sharding import allreduce_accumulator  # noqa: E402  (pure host helper, no CUDA needed)

METRIC = "examples/s through per-example wgrad+clip+noise"
UNIT = "examples/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm=float(d["hbm_gbs"]), bf16=float(d["bf16_tflops"]), bf16_sustained=float(d["bf16_tflops_sustained"]),
                    source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


def source_fingerprint():
    """sha1 over the CUDA sources: ncu traffic figures are only quoted while the kernels they were taken on are unchanged."""
    import glob
    import hashlib
    h = hashlib.sha1()
    for path in sorted(glob.glob(os.path.join(ROOT, "paper_2109_12191_b200", "csrc", "*.cu*"))):
        with open(path, "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def recorded_traffic(workload, call_name):
    """DRAM bytes (read + write) per launch of `call_name` from the committed ncu capture, or None when there is no
    capture for it or the sources have changed since it was taken."""
    path = os.path.join(ROOT, "profiles", f"traffic_{workload}.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        rec = json.load(f)
    if rec.get("source_sha1") != source_fingerprint():
        return None
    return rec.get("dram_bytes_per_launch", {}).get(call_name)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- workloads (device side)
class SmallCnn:
    """The small-CNN workload: 3 convs + classifier on 32x32x3, B=256, fp32, whole-model clip C=1.5, sigma=1."""
    name = "small_cnn"

    def __init__(self, torch, rank, dist=None, world=1):
        from paper_2109_12191_b200 import synth
        from paper_2109_12191_b200.step import GlobalClipStep
        self.torch, self.synth, self.dist, self.world = torch, synth, dist, world
        self.cfg = synth.small_cnn()
        self.layers, self.B = self.cfg["layers"], self.cfg["B"]
        self.lanes = int(os.environ.get("DP_BENCH_LANES", "4")) if world == 1 else 1
        # layers whose per-example gradients outweigh their inputs (conv3, the classifier) are not materialised
        self.recompute = os.environ.get("DP_BENCH_RECOMPUTE", "auto")
        # fp32 inputs; tensor-core layers take them as tf32 (one pass, the precision class the accuracy bounds name)
        # or, with --precision f32, as three products of a hi/lo split
        self.precision = PRECISION
        self.dtype_name = "tf32" if PRECISION == "tf32" else "f32 (3 x tf32 on tensor cores)"
        self.step_obj = GlobalClipStep(self.layers, self.B, PRECISION, self.cfg["C"], self.cfg["sigma"], lanes=self.lanes,
                                       recompute=self.recompute)
        self.examples_per_step = self.B
        # inputs rotate over several sets so that consecutive steps never find their inputs in L2
        self.n_sets = 3
        g = torch.Generator(device="cuda"); g.manual_seed(1000 + rank)
        self.sets = [[(torch.randn(l.x_shape(self.B), device="cuda", generator=g),
                       torch.randn(l.dy_shape(self.B), device="cuda", generator=g)) for l in self.layers]
                     for _ in range(self.n_sets)]
        self.in_bytes = sum(x.numel() * 4 + y.numel() * 4 for x, y in self.sets[0])
        self.host_sets = None
        self.call_names = [f"wgrad:{l.name}" for l in self.layers] + ["clip_accumulate", "noise_average"]

    def describe(self):
        return {"workload": "small_cnn: conv3x3 3->32 s1, 32->64 s2, 64->128 s2, dense 8192->10 (all with bias) on 32x32x3, "
                            "B=256 fp32 inputs, global clip C=1.5, sigma=1.0, |B|=256",
                "precision": ("tensor-core layers round the fp32 inputs to tf32 (nearest even), one pass" if self.precision == "tf32"
                              else "tensor-core layers run three split-tf32 passes"),
                "examples_per_step": self.B, "params": self.step_obj.P,
                "l2": f"inputs rotate over {self.n_sets} resident sets ({self.n_sets * self.in_bytes / 1e6:.0f} MB) and "
                      f"{sum(self.step_obj.P_l[i] for i in self.step_obj._kept) * self.B * 4 / 1e6:.0f} MB of per-example gradients are written and re-read per step",
                "streams": self.lanes,
                "recomputed_layers": [self.layers[i].name for i in sorted(self.step_obj.recompute)]}

    def run(self, i, rec=None):
        st = self.step_obj
        ins = self.sets[i % self.n_sets]
        st.begin()
        k = len(ins)
        if rec is None:
            st.wgrad_all(ins)                              # forked over the step object's streams
            st.clip_accumulate(inputs=ins)
        else:                                              # one call after the other, so that each can be timed
            for li, (X, dY) in enumerate(ins):
                rec.start(li); st.wgrad(li, X, dY); rec.stop(li)
            if st.recompute:
                rec.start(k); st.clip_factors(); st.scale_kept(); rec.stop(k)
                for li in sorted(st.recompute):            # second pass, booked on the layer's own line
                    rec.start(li); st.wgrad_scaled(li, *ins[li]); rec.stop(li)
                st.chunks_done += 1
            else:
                rec.start(k); st.clip_accumulate(); rec.stop(k)
        allreduce_accumulator(st.acc, self.dist)          # N > 1: the one exchange of the step
        if rec: rec.start(k + 1)
        st.finish(seed=0, step=i, world=self.world)
        if rec: rec.stop(k + 1)

    def parts_of(self, call):
        return 2 if call in self.step_obj.recompute else 1

    def capture(self):
        """One CUDA graph per input set, each holding a whole step (the noise step index is baked in: it does
        not change the work)."""
        t = self.torch
        self.graphs = []
        for k in range(self.n_sets):
            g = t.cuda.CUDAGraph()
            with t.cuda.graph(g):
                self.run(k)
            self.graphs.append(g)

    def run_graphed(self, i):
        self.graphs[i % self.n_sets].replay()

    def algorithmic_bytes(self, call):
        """Bytes each call must move per step.  A materialised layer reads its inputs and writes its per-example
        gradients, which the clip call reads back; a recomputed layer reads its inputs twice (norm pass, clipped-sum
        pass) and touches its accumulator."""
        st = self.step_obj
        if call < len(self.layers):
            l = self.layers[call]
            x = math.prod(l.x_shape(self.B)) * 4
            y = math.prod(l.dy_shape(self.B)) * 4
            if call in st.recompute:
                return 2 * (x + y) + 2 * (l.n_weight + l.n_bias) * 4
            return x + y + (l.n_weight + l.n_bias) * self.B * 4
        if call == len(self.layers):
            kept = sum(st.P_l[i] for i in st._kept)
            return kept * self.B * 4 + 2 * kept * 4
        return 2 * st.P * 4

    def e2e_prepare(self):
        t = self.torch
        self.host_sets = [[(x.cpu().pin_memory(), y.cpu().pin_memory()) for x, y in s] for s in self.sets]
        self.stage = [(t.empty_like(x), t.empty_like(y)) for x, y in self.sets[0]]
        self.host_out = t.empty(self.step_obj.P, dtype=t.float32).pin_memory()
        return self.in_bytes, self.step_obj.P * 4

    def e2e_run(self, i):
        st = self.step_obj
        hs = self.host_sets[i % self.n_sets]
        for (dx, dy), (hx, hy) in zip(self.stage, hs):
            dx.copy_(hx, non_blocking=True); dy.copy_(hy, non_blocking=True)
        st.begin()
        st.wgrad_all(self.stage)
        st.clip_accumulate(inputs=self.stage)
        allreduce_accumulator(st.acc, self.dist)
        out = st.finish(seed=0, step=i, world=self.world)
        self.host_out.copy_(out, non_blocking=True)

    def cpu_sample(self, budget_s):
        """The oracle on the first examples of one batch: wgrad + norms + clip + sum + noise + average."""
        import numpy as np
        import oracle
        n = self.B
        ins = [self.synth.layer_inputs(l, n, "f32", 1, li, 0) for li, l in enumerate(self.layers)]
        reps, t0 = 0, time.perf_counter()
        while reps < 16 and (reps == 0 or time.perf_counter() - t0 < budget_s):
            groups = []
            for l, i in zip(self.layers, ins):
                if l.kind == "conv":
                    dW, db = oracle.conv_wgrad(i["X"], i["dY"], l.R, l.S, l.stride, l.pad, bias=l.bias)
                else:
                    dW, db = oracle.dense_wgrad(i["X"], i["dY"], bias=l.bias)
                groups += [dW.reshape(n, -1), db.reshape(n, -1)]
            oracle.privatise([groups], self.cfg["C"], self.cfg["sigma"], "global", 0, 0)
            reps += 1
        dt = time.perf_counter() - t0
        return n * reps / dt, f"one whole batch of {n} examples, whole path (wgrad, norms, clip, sum, noise, average), repeated {reps} times"


class FlatGrad:
    """The flat workload: flattened ResNet-50 gradients, P=25,557,032, B=64 per chunk, 16 chunks, C=1, sigma=1."""
    name = "flat"
    e2e_cap = 8          # an end-to-end step copies 105 GB from the host: a few of them are enough

    def __init__(self, torch, rank, dist=None, world=1):
        from paper_2109_12191_b200 import synth
        from paper_2109_12191_b200.step import FlatClipStep
        self.torch, self.synth, self.dist, self.world = torch, synth, dist, world
        self.cfg = synth.resnet50_flat()
        self.P, self.B, self.G = self.cfg["P"], self.cfg["B"], self.cfg["G"]
        if os.environ.get("DPSTEP_FLAT_PARAMS"):          # reduced P for profiler captures (same kernels, fewer bytes held)
            self.P = int(os.environ["DPSTEP_FLAT_PARAMS"])
        # --variant: "per_example_noise" (the paper's own form of the noise), "microN" (clip the mean of N examples) or
        # "norms_supplied" (the squared norms come in with the gradients, as they do from the weight-gradient
        # epilogues, so the chunk is read once instead of twice)
        self.variant = VARIANT
        micro = int(self.variant[5:]) if self.variant.startswith("micro") else 1
        self.step_obj = FlatClipStep(self.P, self.B, self.cfg["C"], self.cfg["sigma"],
                                     per_example_noise=(self.variant == "per_example_noise"), micro=micro)
        self.examples_per_step = self.B * self.G
        g = torch.Generator(device="cuda"); g.manual_seed(2000 + rank)
        self.bufs = []
        for _ in range(2):                                   # two resident chunks (13 GB), alternated
            t = torch.empty((self.B, self.P), device="cuda")
            t.normal_(0.0, self.cfg["grad_std"], generator=g)
            self.bufs.append(t)
        self.supplied = None
        if self.variant == "norms_supplied":                 # set-up, outside every timed region
            self.supplied = [(t.double() ** 2).sum(1, keepdim=True).float().contiguous() if self.P < 1 << 22
                             else torch.stack([(row.double() ** 2).sum() for row in t]).float().reshape(self.B, 1).contiguous()
                             for t in self.bufs]
        self.call_names = ["clip_accumulate(norms supplied)" if self.supplied else "clip_accumulate(norms computed)", "noise_average"]

    def describe(self):
        return {"workload": f"flat: ResNet-50 (GroupNorm) flattened per-example gradients, P={self.P:,} fp32 ~N(0,1e-6), "
                            "B=64 per chunk x 16 chunks = |B| 1024, global clip C=1.0, sigma=1.0; "
                            + ("squared norms supplied with the gradients" if self.supplied else "norms computed by the library")
                            + ("" if self.variant == "plain" else f"; variant {self.variant}"),
                "examples_per_step": self.examples_per_step, "params": self.P,
                "l2": "each chunk is 6.54 GB, far larger than L2; two resident chunks alternate"}

    def run(self, i, rec=None):
        st = self.step_obj
        st.begin(total_batch=self.B * self.G * self.world, seed=0, step=i)
        for c in range(self.G):
            if rec: rec.start(0)
            st.chunk(self.bufs[c & 1], self.supplied[c & 1] if self.supplied else None)
            if rec: rec.stop(0)
        allreduce_accumulator(st.acc, self.dist)
        if rec: rec.start(1)
        st.finish(seed=0, step=i, world=self.world)
        if rec: rec.stop(1)

    def algorithmic_bytes(self, call):
        if call == 0:                                         # norm pass (unless supplied) + clip pass, accumulator r+w
            return (1 if self.supplied else 2) * self.B * self.P * 4 + 2 * self.P * 4
        return 2 * self.P * 4

    def roofline(self, dom, avg_ms_per_chunk, peaks):
        """Per-example noise draws B*P normals per chunk and is bound by integer and transcendental arithmetic: about
        45 instructions per normal (a quarter of a ten-round Philox block, half a Box-Muller pair, the scaled add), so
        the ceiling is SMs x 128 lanes x SM clock / 45 normals per second."""
        if self.variant != "per_example_noise" or dom != 0:
            return None
        peak = 148 * 128 * 1.965e9 / 45.0 / 1e9
        got = self.B * self.P / (avg_ms_per_chunk / 1e3) / 1e9
        return {"bound": "alu", "achieved": round(got, 1), "peak": round(peak, 1), "peak_source": "derived: 148 SMs x 128 lanes x 1.965 GHz / 45 instructions per normal",
                "unit": "Gnormal/s", "frac": round(got / peak, 4)}

    def e2e_prepare(self):
        t = self.torch
        self.host_chunk = t.empty((self.B, self.P), dtype=t.float32).pin_memory()
        self.host_chunk.copy_(self.bufs[0])
        self.host_out = t.empty(self.P, dtype=t.float32).pin_memory()
        return self.B * self.P * 4 * self.G, self.P * 4

    def e2e_run(self, i):
        st = self.step_obj
        st.begin(total_batch=self.B * self.G * self.world, seed=0, step=i)
        for c in range(self.G):
            self.bufs[c & 1].copy_(self.host_chunk, non_blocking=True)
            st.chunk(self.bufs[c & 1], self.supplied[c & 1] if self.supplied else None)
        allreduce_accumulator(st.acc, self.dist)
        self.host_out.copy_(st.finish(seed=0, step=i, world=self.world), non_blocking=True)

    def cpu_sample(self, budget_s):
        import numpy as np
        import oracle
        n, P = 8, self.P
        G = self.synth.normal_f32((n, P), 3, 0, 0, scale=self.cfg["grad_std"])
        t0 = time.perf_counter()
        acc, _, _ = oracle.clipped_sum([G], self.cfg["C"], "global")
        oracle.noise_average(acc[0], 0, self.cfg["sigma"], self.cfg["C"], n, 0, 0)
        dt = time.perf_counter() - t0
        return n / dt, f"{n} examples of one 64-example chunk at full P (norms, clip, sum) plus one noise+average pass"


class PerLayer:
    """The per-layer workload: ResNet-50 (GroupNorm) per-layer clipping over all 161 tensors, bf16 inputs, B=32 per chunk,
    32 chunks, C_l = C/sqrt(161), clip + accumulate fused into the weight-gradient call."""
    name = "per_layer"
    dtype_name = "bf16"

    def __init__(self, torch, rank, dist=None, world=1):
        from paper_2109_12191_b200 import synth, binding
        from paper_2109_12191_b200.step import PerLayerClipStep
        self.torch, self.synth, self.dist, self.world, self.b = torch, synth, dist, world, binding
        self.cfg = self.config(synth)
        self.layers, self.B, self.G = self.cfg["layers"], self.cfg["B"], self.cfg["G"]
        self.lanes = int(os.environ.get("DP_BENCH_LANES", "4")) if world == 1 else 1
        self.step_obj = PerLayerClipStep(self.layers, self.B, "bf16", self.cfg["C"], self.cfg["sigma"], lanes=self.lanes)
        self.examples_per_step = self.B * self.G
        g = torch.Generator(device="cuda"); g.manual_seed(4000 + rank)
        self.inputs = []
        for l in self.layers:                             # one resident chunk of inputs (2.8 GB), reused by every chunk
            X = torch.empty(l.x_shape(self.B), device="cuda", dtype=torch.bfloat16).normal_(generator=g)
            dY = torch.empty(l.dy_shape(self.B), device="cuda", dtype=torch.bfloat16).normal_(generator=g)
            self.inputs.append((X, dY))
        self.in_bytes = sum((x.numel() + y.numel()) * 2 for x, y in self.inputs)
        self.call_names = ["wgrad:conv (tensor core)", "wgrad:conv (cuda core)", "wgrad:norm_affine", "wgrad:dense", "noise_average"]
        self.kind_of = []
        for l, d in zip(self.layers, self.step_obj.descs):
            if l.kind == "conv":
                self.kind_of.append(0 if binding.dp_wgrad_uses_tensor_cores(d, binding.DP_EPI_CLIP_ACCUM) else 1)
            else:
                self.kind_of.append(2 if l.kind == "norm" else 3)
        self.flops_tc = sum(l.flops() for l, k in zip(self.layers, self.kind_of) if k == 0) * self.B
        self.bytes_kind = [sum((x.numel() + y.numel()) * 2 for (x, y), k in zip(self.inputs, self.kind_of) if k == kk) for kk in range(4)]

    model = "ResNet-50"

    @staticmethod
    def config(synth):
        return synth.resnet50_per_layer()

    def describe(self):
        n_conv = sum(l.kind == "conv" for l in self.layers)
        L = self.step_obj.L
        return {"workload": f"{self.name}: {self.model} (GroupNorm 32) at 224x224, all {L} parameter tensors ({n_conv} conv, "
                            f"{n_conv}x2 norm, fc weight + bias), bf16 X/dY ~N(0,1), B=32 per chunk x 32 chunks = |B| 1024, "
                            f"C=1.0 (C_l = C/sqrt({L})), sigma=1.0; clip + accumulate fused into dp_per_example_wgrad",
                "examples_per_step": self.examples_per_step, "params": self.step_obj.P,
                "l2": f"one chunk of inputs is {self.in_bytes / 1e9:.2f} GB, far larger than L2",
                "streams": self.lanes}

    def run(self, i, rec=None):
        """With a recorder the calls run one after the other on one stream so that each can be timed; otherwise the
        chunk's calls are spread over the step object's lanes."""
        st = self.step_obj
        st.begin()
        for c in range(self.G):
            if rec is None:
                st.chunk_calls(self.inputs)
            else:
                for li, (X, dY) in enumerate(self.inputs):
                    k = self.kind_of[li]
                    rec.start(k)
                    st.wgrad(li, X, dY)
                    rec.stop(k)
            st.chunks_done += 1
        if rec: rec.start(4)
        st.finish(seed=0, step=i)
        if rec: rec.stop(4)

    def capture(self):
        """One CUDA graph holding one chunk (all 107 layer calls); a step replays it G times, then adds the noise."""
        t, st = self.torch, self.step_obj
        self.chunk_graph = t.cuda.CUDAGraph()
        with t.cuda.graph(self.chunk_graph):
            st.chunk_calls(self.inputs)

    def run_graphed(self, i):
        st = self.step_obj
        st.begin()
        for c in range(self.G):
            self.chunk_graph.replay()
            st.chunks_done += 1
        st.finish(seed=0, step=i)

    def algorithmic_bytes(self, call):
        return self.bytes_kind[call] if call < 4 else 2 * self.step_obj.P * 4

    def roofline(self, dom, avg_ms_total_per_chunk, peaks):
        """Tensor-core convs are reported against the bf16 tensor peak (flops counted once although the two-pass
        scheme executes them twice); everything else against HBM."""
        if dom != 0:
            return None
        tf = self.flops_tc / (avg_ms_total_per_chunk / 1e3) / 1e12
        return {"bound": "tensor", "achieved": round(tf, 1), "peak": peaks["bf16_sustained"], "unit": "TFLOP/s",
                "frac": round(tf / peaks["bf16_sustained"], 4)}

    def e2e_prepare(self):
        t = self.torch
        self.host_inputs = [(x.cpu().pin_memory(), y.cpu().pin_memory()) for x, y in self.inputs]
        self.host_sum = t.empty(1, dtype=t.float32).pin_memory()
        return self.in_bytes * self.G, 4 * self.step_obj.P

    def e2e_run(self, i):
        st = self.step_obj
        st.begin()
        for c in range(self.G):
            for li, ((X, dY), (hx, hy)) in enumerate(zip(self.inputs, self.host_inputs)):
                X.copy_(hx, non_blocking=True); dY.copy_(hy, non_blocking=True)
                st.wgrad(li, X, dY)
            st.chunks_done += 1
        acc_w, acc_b = st.finish(seed=0, step=i)
        for a in acc_w:
            a.cpu()

    def cpu_sample(self, budget_s):
        import oracle
        import math
        n = 2
        picks = [l for l in self.layers if l.kind == "conv" and l.H <= 14][:3] + [l for l in self.layers if l.kind == "norm" and l.H <= 28][:3]
        t0 = time.perf_counter(); flops = 0
        for li, l in enumerate(picks):
            inp = self.synth.layer_inputs(l, n, "bf16", 4, li, 0)
            if l.kind == "conv":
                dW, _ = oracle.conv_wgrad(inp["X"], inp["dY"], l.R, l.S, l.stride, l.pad, bias=False)
                groups = [dW.reshape(n, -1)]
            else:
                dg, dbt = oracle.norm_affine_wgrad(inp["X"], inp["dY"])
                groups = [dg, dbt]
            oracle.clipped_sum(groups, 1.0 / math.sqrt(161), "per_layer")
            flops += l.flops() * n
        dt = time.perf_counter() - t0
        total = sum(l.flops() for l in self.layers)
        return (flops / dt) / total, (f"{n} examples through {len(picks)} layers (3 convs, 3 norm layers), scaled to one example's "
                                      f"{total / 1e9:.2f} Gflop by the flop ratio")


class PerLayer101(PerLayer):
    """The same path on ResNet-101 (GroupNorm), the second model of the paper's throughput comparison: 314 tensors."""
    name = "per_layer_r101"
    model = "ResNet-101"

    @staticmethod
    def config(synth):
        return synth.resnet101_per_layer()


WORKLOADS = {"small_cnn": SmallCnn, "flat": FlatGrad, "per_layer": PerLayer, "per_layer_r101": PerLayer101}
VARIANT = "plain"
PRECISION = "tf32"


class CallTimer:
    """CUDA-event pairs around each C-ABI call, recorded on the stream the kernels are launched on."""

    def __init__(self, torch, n_calls):
        self.torch, self.n = torch, n_calls
        self.pairs = [[] for _ in range(n_calls)]
        self._open = {}

    def start(self, k):
        e = self.torch.cuda.Event(enable_timing=True)
        e.record()
        self._open[k] = e

    def stop(self, k):
        e = self.torch.cuda.Event(enable_timing=True)
        e.record()
        self.pairs[k].append((self._open.pop(k), e))

    def totals_ms(self):
        return [sum(a.elapsed_time(b) for a, b in p) for p in self.pairs]

    def counts(self):
        return [len(p) for p in self.pairs]


def run_ours(args):
    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    import __graft_entry__
    if rank == 0:
        __graft_entry__.build()
    if dist:
        dist.barrier()
    from paper_2109_12191_b200 import binding as b

    wl = WORKLOADS[args.workload](torch, rank, dist, world)
    steps, warmup = args.steps, max(args.warmup, 3)

    def barrier():
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing
    for i in range(warmup):
        wl.run(i)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    # The step's launch sequence is static, so on one GPU it is captured into CUDA graphs and replayed; per-call
    # event timing (for the roofline) cannot be taken inside a replay and uses a separate un-captured pass below.
    graphed = args.graph != "off" and world == 1 and hasattr(wl, "capture")
    launches_per_step = None
    if graphed:
        c0 = b.dp_debug_launch_count()
        wl.run(0)
        launches_per_step = b.dp_debug_launch_count() - c0
        torch.cuda.synchronize()
        wl.capture()
        for i in range(3):
            wl.run_graphed(i)
        barrier()
    rec = CallTimer(torch, len(wl.call_names))
    launches0 = b.dp_debug_launch_count()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(steps):
        if graphed:
            wl.run_graphed(warmup + i)
        else:
            wl.run(warmup + i, rec)
    t_end.record()
    barrier()
    launches = (launches_per_step * steps) if graphed else (b.dp_debug_launch_count() - launches0)
    clocks = sampler.stop() if rank == 0 else None
    ms = t_start.elapsed_time(t_end)
    if graphed:
        for i in range(min(steps, args.profile_steps)):
            wl.run(warmup + i, rec)
        barrier()
    if dist:
        t = torch.tensor([ms], device="cuda"); dist.all_reduce(t, op=dist.ReduceOp.MAX); ms = t.item()
    value = wl.examples_per_step * steps * world / (ms / 1e3)

    # ---- end to end: pinned host inputs -> device, the step, result -> host, every step
    h2d, d2h = wl.e2e_prepare()
    e2e_steps = max(3, min(steps, args.e2e_steps, getattr(wl, "e2e_cap", steps)))
    for i in range(2):
        wl.e2e_run(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(e2e_steps):
        wl.e2e_run(i)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    if dist:
        t = torch.tensor([e2e_ms], device="cuda"); dist.all_reduce(t, op=dist.ReduceOp.MAX); e2e_ms = t.item()
    e2e_value = wl.examples_per_step * e2e_steps * world / (e2e_ms / 1e3)

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant call (largest share of device time)
    peaks = measured_peaks()
    totals, counts = rec.totals_ms(), rec.counts()
    dom = max(range(len(totals)), key=lambda k: totals[k])
    parts = wl.parts_of(dom) if hasattr(wl, "parts_of") else 1   # a call timed in two parts (two passes) counts once
    avg_ms = totals[dom] * parts / counts[dom]
    achieved = wl.algorithmic_bytes(dom) / (avg_ms / 1e3) / 1e9
    roofline = {"bound": "hbm", "kernel": wl.call_names[dom], "achieved": round(achieved, 1), "peak": peaks["hbm"],
                "peak_source": peaks["source"], "unit": "GB/s", "frac": round(achieved / peaks["hbm"], 4),
                "avg_ms_per_launch": round(avg_ms, 5), "algorithmic_bytes": wl.algorithmic_bytes(dom),
                "traffic": recorded_traffic(wl.name, wl.call_names[dom]),
                "shares": {n: round(t / sum(totals), 4) for n, t in zip(wl.call_names, totals)}}
    if hasattr(wl, "roofline"):
        own = wl.roofline(dom, totals[dom] / (max(1, counts[-1]) * wl.G), peaks)
        if own:
            roofline.update(own)

    cpu = None
    if not args.no_cpu_baseline:
        import oracle
        v, sample = wl.cpu_sample(10.0)
        cpu = {"value": round(v, 3), "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample}

    line = {"metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": round(ms / steps, 5), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": getattr(wl, "dtype_name", "f32"), "data": "synthetic", "config": dict(wl.describe(), parallelism=("single GPU" if world == 1 else f"batch sharded over {world} GPUs, one all-reduce of the accumulator per step")),
            "e2e": {"value": round(e2e_value, 1), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps},
            "gpu_launches": int(launches), "launch_mode": ("CUDA graph replay" if graphed else "stream launches"), "clocks": clocks, "roofline": roofline, "cpu_baseline": cpu}
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


def run_reference(args):
    """The oracle, as it stands, on this machine's host cores; each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import __graft_entry__
    import oracle
    oracle.build()

    class _NoTorch:
        pass
    cls = WORKLOADS[args.workload]
    wl = cls.__new__(cls)
    from paper_2109_12191_b200 import synth
    wl.synth = synth
    if args.workload == "small_cnn":
        wl.cfg = synth.small_cnn(); wl.layers = wl.cfg["layers"]; wl.B = wl.cfg["B"]
        config = {"workload": "small_cnn (CPU oracle, whole batches)", "examples_per_step": 256}
    else:
        wl.cfg = synth.resnet50_flat(); wl.P, wl.B, wl.G = wl.cfg["P"], wl.cfg["B"], wl.cfg["G"]
        config = {"workload": "flat (CPU oracle on a sample)", "examples_per_step": 8}
    steps, warmup = max(1, min(args.steps, 5)), min(args.warmup, 1)
    for _ in range(warmup):
        wl.cpu_sample(1.0)
    vals, sample = [], ""
    t0 = time.perf_counter()
    for _ in range(steps):
        v, sample = wl.cpu_sample(5.0)
        vals.append(v)
    dt = time.perf_counter() - t0
    v = statistics.mean(vals)
    line = {"impl": "reference", "metric": METRIC, "value": round(v, 3), "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
            "steps": steps, "warmup": warmup, "ms_per_step": round(dt / steps * 1e3, 3), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
            "cpu_baseline": {"value": round(v, 3), "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": round(v, 3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def run_sweep(args):
    """The layer sweep (or any layer list): time dp_per_example_wgrad per layer with both epilogues.
    L2 is flushed (a 512 MB buffer is overwritten) before every timed launch."""
    import torch
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    import __graft_entry__
    __graft_entry__.build()
    from paper_2109_12191_b200 import binding as b, synth
    from paper_2109_12191_b200.step import layer_desc
    peaks = measured_peaks()
    layers = synth.resnet50_sweep()["layers"]
    if args.workload == "sweep_all":
        layers = [l for l in synth.resnet50_gn_layers() if l.kind != "norm"]
    if args.workload == "sweep_all_r101":
        layers = [l for l in synth.resnet101_gn_layers() if l.kind != "norm"]
    if args.layers:
        layers = [layers[int(i)] for i in args.layers.split(",")]
    Bn, dtype = 32, "bf16"
    flush = torch.empty(512 * 1024 * 1024 // 4, dtype=torch.float32, device="cuda")
    rows, reps = [], max(3, args.steps or 10)
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    for l in layers:
        X = torch.randn(l.x_shape(Bn), device="cuda", generator=g).to(torch.bfloat16)
        dY = torch.randn(l.dy_shape(Bn), device="cuda", generator=g).to(torch.bfloat16)
        G_w = torch.empty((Bn, l.n_weight), device="cuda")
        sq = torch.empty((Bn, 1), device="cuda")
        row = {"layer": l.name, "M": l.Kout, "N": l.R * l.S * l.Cin, "K": l.OH * l.OW}
        in_bytes = (X.numel() + dY.numel()) * 2
        flops = l.flops() * Bn
        for epi, tag, out_bytes in ((b.DP_EPI_STORE_NORM, "store", G_w.numel() * 4), (b.DP_EPI_NORM_ONLY, "norm", 0)):
            d = layer_desc(l, Bn, dtype, b.DP_IMPL_AUTO, 0)
            ws = torch.empty(max(b.dp_workspace_bytes(d, epi), 256), dtype=torch.uint8, device="cuda")
            call = lambda: b.check(b.dp_per_example_wgrad(d, X, dY, G_w, None, sq, 1, epi, 0.0, None, None, None, ws))
            for _ in range(3):
                call()
            times = []
            for _ in range(reps):
                flush.fill_(1.0)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(); call(); e1.record()
                torch.cuda.synchronize()
                times.append(e0.elapsed_time(e1))
            b.check(b.dp_wgrad_check(ws))
            ms = statistics.median(times)
            t_hbm = (in_bytes + out_bytes) / (peaks["hbm"] * 1e9) * 1e3
            t_tc = flops / (peaks["bf16"] * 1e12) * 1e3
            row[tag] = {"ms": round(ms, 4), "tflops": round(flops / ms / 1e9, 1), "gbs": round((in_bytes + out_bytes) / ms / 1e6, 1),
                        "bound": "hbm" if t_hbm > t_tc else "tensor", "frac_of_bound": round(max(t_hbm, t_tc) / ms, 3),
                        "tc": bool(b.dp_wgrad_uses_tensor_cores(d, epi)), "ex_per_s": round(Bn / ms * 1e3, 1)}
        rows.append(row)
        del X, dY, G_w
    tot_store = sum(r["store"]["ms"] for r in rows)
    tot_norm = sum(r["norm"]["ms"] for r in rows)
    print(json.dumps({"metric": METRIC, "unit": UNIT, "workload": args.workload, "B": Bn, "dtype": "bf16", "peaks": peaks,
                      "store_total_ms": round(tot_store, 3), "norm_total_ms": round(tot_norm, 3),
                      "store_ex_per_s": round(Bn / tot_store * 1e3, 1), "norm_ex_per_s": round(Bn / tot_norm * 1e3, 1),
                      "layers": rows}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="small_cnn", choices=sorted(WORKLOADS) + ["sweep", "sweep_all", "sweep_all_r101"])
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--graph", default="auto", choices=["auto", "on", "off"], help="replay the step from CUDA graphs (single GPU)")
    ap.add_argument("--profile-steps", type=int, default=20, help="un-captured steps timed per call for the roofline")
    ap.add_argument("--layers", default="", help="sweep workloads: comma-separated layer indices")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--precision", default="tf32", choices=["tf32", "f32"],
                    help="small_cnn: how tensor-core layers take the fp32 inputs (one tf32 pass | three split-tf32 passes)")
    ap.add_argument("--variant", default="plain", help="flat workload: plain | norms_supplied | per_example_noise | micro2 | micro4 ...")
    args = ap.parse_args()
    global VARIANT, PRECISION
    VARIANT = args.variant
    PRECISION = args.precision
    if args.workload.startswith("sweep"):
        return run_sweep(args)
    # the small-CNN step lasts ~0.16 ms: 6000 steps give the clock sampler (200 ms period) several readings under load
    defaults = {"small_cnn": (6000, 10), "flat": (40, 3), "per_layer": (4, 3), "per_layer_r101": (3, 3)}
    if args.steps is None:
        args.steps = defaults[args.workload][0]
    if args.warmup is None:
        args.warmup = defaults[args.workload][1]
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
