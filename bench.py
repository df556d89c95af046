#!/usr/bin/env python
"""Throughput of the DPSGD gradient-privatisation step (examples/s through per-example weight
gradients + clip + noise) on synthetic inputs, with the roofline fraction of the dominant kernel
and the float64 CPU oracle timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W]     # headline: per-layer ResNet-50; other workloads as "legs"
    python bench.py --workload small_cnn|flat|per_layer|per_layer_r101|sweep|sweep_all ...   # one workload only
    python bench.py --impl reference ...                    # times the CPU oracle on a bounded sample

One "step" is one pass of the whole path over one batch: for the headline workload 1024 examples (32 chunks of 32)
through 107 fused weight-gradient + clip calls per chunk and one noise-average.  Rank 0 prints one JSON line; with
no --workload it carries the per-layer ResNet-50 workload in `value` / `config` / `roofline` and, on one GPU, the
flat-gradient (norms computed and norms supplied), small-CNN and layer-sweep workloads under `legs`.  Every timed
region lasts at least a second: the K steps are repeated `repeats` times when K of them are shorter than that.
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
                    sm_max_mhz=float(d.get("sm_max_mhz", 1965.0)), source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, sm_max_mhz=1965.0, source="fallback")


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
        self.lanes = int(os.environ.get("DP_BENCH_LANES", "4"))
        from paper_2109_12191_b200 import binding
        # the two tensor-core convolutions run side by side on their own streams: each is told to take half of the SMs
        # (a call that spreads over all of them makes the other wait for its turn)
        self.sm_target = int(os.environ.get("DP_BENCH_SM_TARGET", str(torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count // 2)))
        binding.check(binding.dp_set_sm_target(self.sm_target))
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
                "streams": self.lanes, "sm_target": self.sm_target,
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
        self._finish(i, rec, k + 1)

    def _finish(self, i, rec=None, slot=None):
        allreduce_accumulator(self.step_obj.acc, self.dist)   # N > 1: the one exchange of the step
        if rec: rec.start(slot)
        self.step_obj.finish(seed=0, step=i, total_batch=self.B * self.world)
        if rec: rec.stop(slot)

    def parts_of(self, call):
        return 2 if call in self.step_obj.recompute else 1

    def capture(self):
        """One CUDA graph per input set holding the step up to the clipped sum.  The exchange between ranks and the
        noise call stay outside: a captured noise call would freeze its step index and repeat the same draw."""
        t, st = self.torch, self.step_obj
        self.graphs = []
        for k in range(self.n_sets):
            g = t.cuda.CUDAGraph()
            with t.cuda.graph(g):
                st.begin()
                st.wgrad_all(self.sets[k])
                st.clip_accumulate(inputs=self.sets[k])
            self.graphs.append(g)

    def run_graphed(self, i):
        self.graphs[i % self.n_sets].replay()
        self._finish(i)

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
        out = st.finish(seed=0, step=i, total_batch=self.B * self.world)
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
        st.finish(seed=0, step=i, total_batch=self.B * self.G * self.world)
        if rec: rec.stop(1)

    def algorithmic_bytes(self, call):
        if call == 0:                                         # norm pass (unless supplied) + clip pass, accumulator r+w
            return (1 if self.supplied else 2) * self.B * self.P * 4 + 2 * self.P * 4
        return 2 * self.P * 4

    def roofline(self, dom, totals, prof_steps, peaks):
        """Per-example noise draws B*P normals per chunk and is bound by integer and transcendental arithmetic: 54
        thread instructions per normal (a quarter of a ten-round Philox block, half a Box-Muller pair, the scaled add;
        counted by ncu: smsp__thread_inst_executed.sum = 27.63 G for 512 M normals), so the ceiling is
        SMs x 128 lanes x SM clock / 54 normals per second."""
        if self.variant != "per_example_noise" or dom != 0:
            return None
        avg_ms_per_chunk = totals[0] / (prof_steps * self.G)
        props = self.torch.cuda.get_device_properties(self.torch.cuda.current_device())
        sms, ghz = props.multi_processor_count, peaks.get("sm_max_mhz", 1965.0) / 1e3
        peak = sms * 128 * ghz * 1e9 / 54.0 / 1e9
        got = self.B * self.P / (avg_ms_per_chunk / 1e3) / 1e9
        return {"bound": "alu", "achieved": round(got, 1), "peak": round(peak, 1),
                "peak_source": f"derived: {sms} SMs x 128 lanes x {ghz:.3f} GHz / 54 thread instructions per normal (ncu count)",
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
        self.host_out.copy_(st.finish(seed=0, step=i, total_batch=self.B * self.G * self.world), non_blocking=True)

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
        only = os.environ.get("DP_BENCH_ONLY")           # experiments: time one layer kind alone ("conv", "norm")
        if only:
            self.layers = [l for l in self.layers if l.kind == only]
        # the layer calls of a chunk run side by side on 16 streams; the SM target (here: all SMs, which still switches
        # the library's tiling from "fastest single call" to "least SM time") is set for that
        self.lanes = int(os.environ.get("DP_BENCH_LANES", "16"))
        self.sm_target = int(os.environ.get("DP_BENCH_SM_TARGET", str(torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count)))
        binding.check(binding.dp_set_sm_target(self.sm_target))
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

    @classmethod
    def workload_text(cls, layers, L):
        n_conv = sum(l.kind == "conv" for l in layers)
        return (f"{cls.name}: {cls.model} (GroupNorm 32) at 224x224, all {L} parameter tensors ({n_conv} conv, "
                f"{n_conv}x2 norm, fc weight + bias), bf16 X/dY ~N(0,1), B=32 per chunk x 32 chunks = |B| 1024, "
                f"C=1.0 (C_l = C/sqrt({L})), sigma=1.0; clip + accumulate fused into dp_per_example_wgrad")

    def describe(self):
        return {"workload": self.workload_text(self.layers, self.step_obj.L),
                "examples_per_step": self.examples_per_step, "params": self.step_obj.P,
                "l2": f"one chunk of inputs is {self.in_bytes / 1e9:.2f} GB, far larger than L2",
                "streams": self.lanes, "sm_target": self.sm_target}

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
        allreduce_accumulator(st.acc, self.dist)
        if rec: rec.start(4)
        st.finish(seed=0, step=i, total_batch=self.B * self.G * self.world)
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
        allreduce_accumulator(st.acc, self.dist)
        st.finish(seed=0, step=i, total_batch=self.B * self.G * self.world)

    def algorithmic_bytes(self, call):
        return self.bytes_kind[call] if call < 4 else 2 * self.step_obj.P * 4

    def class_times_ms(self, reps=20):
        """ms per chunk of each kind of layer call on its own, in the launch mode of the timed region (the chunk's calls
        of that kind captured into a CUDA graph over the step object's streams, replayed `reps` times between two events)."""
        t, st, out = self.torch, self.step_obj, []
        for kind in range(4):
            only = {li for li, k in enumerate(self.kind_of) if k == kind}
            if not only:
                out.append(0.0)
                continue
            g = t.cuda.CUDAGraph()
            with t.cuda.graph(g):
                st.chunk_calls(self.inputs, only=only)
            for _ in range(3):
                g.replay()
            e0, e1 = t.cuda.Event(enable_timing=True), t.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                g.replay()
            e1.record()
            t.cuda.synchronize()
            out.append(e0.elapsed_time(e1) / reps)
        return out

    def roofline(self, dom, totals, prof_steps, peaks):
        """Tensor-core convs are reported against the sustained bf16 tensor peak (they are timed inside a long step;
        flops counted once even where a two-pass scheme executes them twice); the normalisation layers against HBM;
        and the whole chunk against the sum over layers of max(HBM time, tensor time) at the measured peaks."""
        per_chunk = self.class_times_ms()                                 # ms per chunk of each call class, replayed alone
        dom = max(range(4), key=lambda k: per_chunk[k])
        gn_gbs = self.bytes_kind[2] / (per_chunk[2] / 1e3) / 1e9 if per_chunk[2] > 0 else 0.0
        ceiling_ms = 0.0
        for l, (x, y), k in zip(self.layers, self.inputs, self.kind_of):
            t_hbm = (x.numel() + y.numel()) * 2 / (peaks["hbm"] * 1e9) * 1e3
            t_tc = (l.flops() * self.B / (peaks["bf16_sustained"] * 1e12) * 1e3) if k == 0 else 0.0
            ceiling_ms += max(t_hbm, t_tc)
        extra = {"norm_affine": {"bound": "hbm", "achieved": round(gn_gbs, 1), "peak": peaks["hbm"], "unit": "GB/s",
                                 "frac": round(gn_gbs / peaks["hbm"], 4), "algorithmic_bytes": self.bytes_kind[2],
                                 "avg_ms_per_chunk": round(per_chunk[2], 5)},
                 "chunk_ceiling": {"ms_at_measured_peaks": round(ceiling_ms, 4), "ms_classes_alone": round(sum(per_chunk[:4]), 4),
                                   "frac": round(ceiling_ms / max(sum(per_chunk[:4]), 1e-9), 4)},
                 "class_ms_per_chunk": {n: round(v, 4) for n, v in zip(self.call_names[:4], per_chunk)},
                 "how": "each kind of layer call captured alone into a CUDA graph over the same streams and replayed; "
                        "`shares` come from the eager one-stream pass and include host launch gaps"}
        if dom != 0:
            return extra
        tf = self.flops_tc / (per_chunk[0] / 1e3) / 1e12
        n_tc = max(1, sum(1 for k in self.kind_of if k == 0))
        return dict(extra, bound="tensor", kernel="wgrad:conv (tensor core): the chunk's %d fused clip calls" % n_tc,
                    achieved=round(tf, 1), peak=peaks["bf16_sustained"], unit="TFLOP/s",
                    frac=round(tf / peaks["bf16_sustained"], 4), algorithmic_flops=self.flops_tc,
                    algorithmic_bytes=self.bytes_kind[0], avg_ms_per_launch=round(per_chunk[0], 5),
                    launch="one launch = the chunk's tensor-core calls replayed as one graph")

    def e2e_prepare(self):
        t = self.torch
        self.host_inputs = [(x.cpu().pin_memory(), y.cpu().pin_memory()) for x, y in self.inputs]
        self.host_out = t.empty(self.step_obj.acc.numel(), dtype=t.float32).pin_memory()
        return self.in_bytes * self.G, 4 * self.step_obj.acc.numel()

    def e2e_run(self, i):
        st = self.step_obj
        st.begin()
        for c in range(self.G):
            for li, ((X, dY), (hx, hy)) in enumerate(zip(self.inputs, self.host_inputs)):
                X.copy_(hx, non_blocking=True); dY.copy_(hy, non_blocking=True)
                st.wgrad(li, X, dY)
            st.chunks_done += 1
        allreduce_accumulator(st.acc, self.dist)
        st.finish(seed=0, step=i, total_batch=self.B * self.G * self.world)
        self.host_out.copy_(st.acc, non_blocking=True)      # the whole noised, averaged gradient (all 161 tensors)

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


MIN_TIMED_MS = float(os.environ.get("DP_BENCH_MIN_MS", "1000"))   # every timed region lasts at least this long (profiler captures shorten it)


class Env:
    """What every measurement needs: torch, the binding, the process group (or None) and this rank's place in it."""

    def __init__(self):
        import torch
        self.torch = torch
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
        torch.cuda.set_device(self.local)
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local))
            self.dist = dist
        import __graft_entry__
        if self.rank == 0:
            __graft_entry__.build()
        self.barrier()
        from paper_2109_12191_b200 import binding
        self.b = binding

    def barrier(self):
        if self.dist:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def max_over_ranks(self, v):
        if not self.dist:
            return v
        t = self.torch.tensor([v], device="cuda", dtype=self.torch.float64)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return t.item()

    def close(self):
        if self.dist:
            self.dist.destroy_process_group()


def measure(env, wl, steps, warmup, args, want_e2e=True, want_cpu=True):
    """Times one workload.  Returns the result dict on rank 0 (None elsewhere)."""
    torch, b = env.torch, env.b
    warmup = max(warmup, 3)
    for i in range(warmup):
        wl.run(i)
    env.barrier()
    # The step's launch sequence is static, so it is captured into CUDA graphs and replayed (all ranks alike; the
    # exchange between ranks and the noise call stay outside the graphs); per-call event timing (for the roofline)
    # cannot be taken inside a replay and uses a separate un-captured pass below.
    graphed = args.graph != "off" and hasattr(wl, "capture")
    c0 = b.dp_debug_launch_count()
    wl.run(0)
    launches_per_step = b.dp_debug_launch_count() - c0
    torch.cuda.synchronize()
    if graphed:
        wl.capture()
    go = wl.run_graphed if graphed else wl.run
    for i in range(3):
        go(i)
    env.barrier()
    # how often the K steps must be repeated for the timed region to last a second
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    probe = max(1, min(steps, 3))
    p0.record()
    for i in range(probe):
        go(i)
    p1.record()
    env.barrier()
    est_ms = env.max_over_ranks(p0.elapsed_time(p1) / probe)
    repeats = max(1, int(math.ceil(MIN_TIMED_MS * 1.1 / max(est_ms * steps, 1e-3))))
    sampler = ClockSampler(env.local)
    if env.rank == 0:
        sampler.start()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    env.barrier()
    t_start.record()
    for i in range(steps * repeats):
        go(warmup + i)
    t_end.record()
    env.barrier()
    clocks = sampler.stop() if env.rank == 0 else None
    ms = env.max_over_ranks(t_start.elapsed_time(t_end))
    if hasattr(wl.step_obj, "check"):
        wl.step_obj.check()                                  # a bounded wait that gave up would invalidate the timing
    value = wl.examples_per_step * steps * repeats * env.world / (ms / 1e3)

    # per-call timing: every call in order on one stream, event pairs around each
    rec = CallTimer(torch, len(wl.call_names))
    est_run_ms = est_ms * (1.6 if graphed else 1.0)
    prof_steps = max(1, min(steps, args.profile_steps, int(math.ceil(300.0 / max(est_run_ms, 1e-3)))))
    for i in range(prof_steps):
        wl.run(warmup + i, rec)
    env.barrier()

    e2e = None
    if want_e2e:
        # end to end: pinned host inputs -> device, the step, result -> host, every step
        h2d, d2h = wl.e2e_prepare()
        e2e_steps = max(2, min(steps, args.e2e_steps, getattr(wl, "e2e_cap", steps)))
        wl.e2e_run(0)
        env.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(e2e_steps):
            wl.e2e_run(i)
        e1.record()
        env.barrier()
        e2e_ms = env.max_over_ranks(e0.elapsed_time(e1))
        e2e = {"value": round(wl.examples_per_step * e2e_steps * env.world / (e2e_ms / 1e3), 1), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps}
    if env.rank != 0:
        return None

    # roofline of the dominant call (largest share of device time in the per-call pass)
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
        own = wl.roofline(dom, totals, prof_steps, peaks)
        if own:
            roofline.update(own)

    cpu = None
    if want_cpu and not args.no_cpu_baseline:
        import oracle
        v, sample = wl.cpu_sample(10.0)
        cpu = {"value": round(v, 3), "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample}

    return {"value": round(value, 1), "unit": UNIT, "steps": steps, "repeats": repeats, "warmup": warmup,
            "ms_per_step": round(ms / (steps * repeats), 5), "timed_ms": round(ms, 2),
            "dtype": getattr(wl, "dtype_name", "f32"),
            "config": dict(wl.describe(), parallelism=("single GPU" if env.world == 1 else
                                                       f"batch sharded over {env.world} GPUs, one all-reduce of the accumulator per step")),
            "e2e": e2e, "gpu_launches": int(launches_per_step * steps * repeats),
            "launch_mode": ("CUDA graph replay" if graphed else "stream launches"), "clocks": clocks,
            "roofline": roofline, "cpu_baseline": cpu}


def release(env, wl):
    del wl
    import gc
    gc.collect()
    env.torch.cuda.empty_cache()


def line_of(env, res):
    """The contract's JSON line from a measure() result."""
    line = {"metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": env.world, "steps": res["steps"],
            "warmup": res["warmup"], "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": res["dtype"], "data": "synthetic"}
    for k in ("config", "e2e", "gpu_launches", "launch_mode", "repeats", "timed_ms", "clocks", "roofline", "cpu_baseline"):
        line[k] = res[k]
    return line


def run_ours(args):
    global VARIANT
    env = Env()
    names = [args.workload] if args.workload != "all" else ["per_layer"]
    head = None
    for name in names:
        VARIANT = args.variant
        wl = WORKLOADS[name](env.torch, env.rank, env.dist, env.world)
        steps = args.steps if args.steps is not None else DEFAULT_STEPS[name][0]
        warmup = args.warmup if args.warmup is not None else DEFAULT_STEPS[name][1]
        if args.chunks and hasattr(wl, "G"):
            wl.G = args.chunks
            wl.examples_per_step = wl.B * wl.G
        head = measure(env, wl, steps, warmup, args, want_e2e=not args.no_e2e)
        release(env, wl)
    legs = {}
    if args.workload == "all" and env.world == 1 and args.legs != "off":
        # the other workloads, device-resident timing only; each with its own clock samples and roofline
        for key, name, variant in (("flat", "flat", "plain"), ("flat_norms_supplied", "flat", "norms_supplied"),
                                   ("small_cnn", "small_cnn", "plain")):
            VARIANT = variant
            wl = WORKLOADS[name](env.torch, env.rank, env.dist, env.world)
            st, wu = DEFAULT_STEPS[name]
            res = measure(env, wl, st, wu, args, want_e2e=False, want_cpu=False)
            release(env, wl)
            legs[key] = {k: res[k] for k in ("value", "unit", "ms_per_step", "steps", "repeats", "timed_ms", "dtype",
                                             "config", "gpu_launches", "launch_mode", "clocks", "roofline")}
        legs["sweep"] = sweep(env, "sweep", "", reps=150)
    if env.rank == 0:
        line = line_of(env, head)
        if legs:
            line["legs"] = legs
        print(json.dumps(line))
    env.close()


def run_reference(args):
    """The oracle, as it stands, on this machine's host cores; each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import __graft_entry__
    import oracle
    oracle.build()

    name = "per_layer" if args.workload == "all" else args.workload
    cls = WORKLOADS[name]
    wl = cls.__new__(cls)
    from paper_2109_12191_b200 import synth
    wl.synth = synth
    if name == "small_cnn":
        wl.cfg = synth.small_cnn(); wl.layers = wl.cfg["layers"]; wl.B = wl.cfg["B"]
        config = {"workload": "small_cnn (CPU oracle, whole batches)", "examples_per_step": 256}
    elif name == "flat":
        wl.cfg = synth.resnet50_flat(); wl.P, wl.B, wl.G = wl.cfg["P"], wl.cfg["B"], wl.cfg["G"]
        config = {"workload": "flat (CPU oracle on a sample)", "examples_per_step": 8}
    else:
        wl.cfg = cls.config(synth); wl.layers = wl.cfg["layers"]
        config = {"workload": cls.workload_text(wl.layers, wl.cfg["L"]), "examples_per_step": 1024,
                  "sampled": "the CPU oracle runs a sample of layers on two examples, scaled to one example by the flop ratio"}
    steps, warmup = max(1, min(args.steps or 3, 5)), min(args.warmup or 1, 1)
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


def sweep(env, which, layer_sel, reps):
    """The layer sweep (or any layer list): dp_per_example_wgrad per layer with the three epilogues, one call per timing.
    L2 is flushed (a 512 MB buffer is overwritten) before every timed call."""
    torch, b = env.torch, env.b
    from paper_2109_12191_b200 import synth
    from paper_2109_12191_b200.step import layer_desc
    peaks = measured_peaks()
    layers = synth.resnet50_sweep()["layers"]
    if which == "sweep_all":
        layers = synth.resnet50_gn_layers()
    if which == "sweep_all_r101":
        layers = synth.resnet101_gn_layers()
    if layer_sel:                                          # indices or layer names
        by_name = {l.name: l for l in layers}
        layers = [by_name[i] if i in by_name else layers[int(i)] for i in layer_sel.split(",")]
    b.check(b.dp_set_sm_target(int(os.environ.get("DP_BENCH_SM_TARGET", "0"))))
    Bn, dtype = 32, "bf16"
    flush = torch.empty(512 * 1024 * 1024 // 4, dtype=torch.float32, device="cuda")
    rows = []
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    sampler = ClockSampler(env.local)
    sampler.start()
    t_wall = time.perf_counter()
    for l in layers:
        X = torch.randn(l.x_shape(Bn), device="cuda", generator=g).to(torch.bfloat16)
        dY = torch.randn(l.dy_shape(Bn), device="cuda", generator=g).to(torch.bfloat16)
        G_w = torch.empty((Bn, l.n_weight), device="cuda")
        G_b = torch.empty((Bn, l.n_bias), device="cuda") if l.n_bias else None
        acc_w = torch.zeros(l.n_weight, device="cuda")
        acc_b = torch.zeros(l.n_bias, device="cuda") if l.n_bias else None
        sq = torch.empty((Bn, 1), device="cuda")
        row = {"layer": l.name, "kind": l.kind, "M": l.Kout, "N": l.R * l.S * l.Cin, "K": l.OH * l.OW}
        in_bytes = (X.numel() + dY.numel()) * 2
        flops = l.flops() * Bn
        for epi, tag, out_bytes in ((b.DP_EPI_STORE_NORM, "store", G_w.numel() * 4), (b.DP_EPI_NORM_ONLY, "norm", 0),
                                    (b.DP_EPI_CLIP_ACCUM, "clip", 2 * acc_w.numel() * 4)):
            d = layer_desc(l, Bn, dtype, b.DP_IMPL_AUTO, 0)
            ws = torch.empty(max(b.dp_workspace_bytes(d, epi), 256), dtype=torch.uint8, device="cuda")
            b.check(b.dp_workspace_init(ws))
            c0 = b.dp_debug_launch_count()
            call = lambda: b.check(b.dp_per_example_wgrad(d, X, dY, G_w, G_b, sq, 1, epi, 1.0, acc_w, acc_b, None, ws))
            call()
            launches = b.dp_debug_launch_count() - c0
            for _ in range(2):
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
            bound = "hbm" if t_hbm > t_tc else "tensor"
            row[tag] = {"ms": round(ms, 4), "launches": int(launches), "tflops": round(flops / ms / 1e9, 1),
                        "gbs": round((in_bytes + out_bytes) / ms / 1e6, 1), "bound": bound,
                        "peak": peaks["hbm"] if bound == "hbm" else peaks["bf16"], "frac": round(max(t_hbm, t_tc) / ms, 3),
                        "algorithmic_bytes": in_bytes + out_bytes, "algorithmic_flops": flops,
                        "tc": bool(b.dp_wgrad_uses_tensor_cores(d, epi)), "ex_per_s": round(Bn / ms * 1e3, 1)}
        rows.append(row)
        del X, dY, G_w
    clocks = sampler.stop()
    tot = {t: sum(r[t]["ms"] for r in rows) for t in ("store", "norm", "clip")}
    top = max(rows, key=lambda r: r["norm"]["ms"])
    return {"value": round(Bn / tot["norm"] * 1e3, 1), "unit": UNIT, "ms_per_step": round(tot["norm"], 4),
            "what": "examples/s through the listed layers' weight-gradient calls with the fused norm epilogue, one call per "
                    "timing, median of `reps`; store_ / clip_ give the same with the gradients stored resp. clipped and summed",
            "store_ex_per_s": round(Bn / tot["store"] * 1e3, 1), "clip_ex_per_s": round(Bn / tot["clip"] * 1e3, 1),
            "B": Bn, "dtype": "bf16", "reps": reps, "wall_s": round(time.perf_counter() - t_wall, 2),
            "l2": "a 512 MB buffer is overwritten before every timed call", "clocks": clocks,
            "roofline": dict(top["norm"], kernel=f"wgrad:{top['layer']} (norm epilogue; the slowest row)", traffic=None,
                             peak_source=peaks["source"], unit="GB/s" if top["norm"]["bound"] == "hbm" else "TFLOP/s",
                             achieved=top["norm"]["gbs"] if top["norm"]["bound"] == "hbm" else top["norm"]["tflops"]),
            "layers": rows}


def run_sweep(args):
    env = Env()
    out = sweep(env, args.workload, args.layers, max(3, args.steps or 30))
    print(json.dumps(dict({"metric": METRIC, "workload": args.workload, "peaks": measured_peaks()}, **out)))
    env.close()


DEFAULT_STEPS = {"small_cnn": (6000, 10), "flat": (40, 3), "per_layer": (20, 3), "per_layer_r101": (10, 3)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all", choices=["all"] + sorted(WORKLOADS) + ["sweep", "sweep_all", "sweep_all_r101"],
                    help="all: the per-layer ResNet-50 workload as the headline, the others as legs of the same line")
    ap.add_argument("--legs", default="on", choices=["on", "off"], help="with --workload all on one GPU: also time the other workloads")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--graph", default="auto", choices=["auto", "on", "off"], help="replay the step from CUDA graphs")
    ap.add_argument("--profile-steps", type=int, default=20, help="un-captured steps timed per call for the roofline (at most)")
    ap.add_argument("--layers", default="", help="sweep workloads: comma-separated layer indices")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the end-to-end (host buffers) measurement")
    ap.add_argument("--chunks", type=int, default=0, help="per_layer workloads: chunks per step (profiler captures only; 0 = the workload's 32)")
    ap.add_argument("--precision", default="tf32", choices=["tf32", "f32"],
                    help="small_cnn: how tensor-core layers take the fp32 inputs (one tf32 pass | three split-tf32 passes)")
    ap.add_argument("--variant", default="plain", help="flat workload: plain | norms_supplied | per_example_noise | micro2 | micro4 ...")
    args = ap.parse_args()
    global VARIANT, PRECISION
    VARIANT = args.variant
    PRECISION = args.precision
    if args.impl == "reference":
        return run_reference(args)
    if args.workload.startswith("sweep"):
        return run_sweep(args)
    run_ours(args)


if __name__ == "__main__":
    main()
