"""Buffer ownership and call sequencing for one privatisation step.

Nothing is computed here: these classes allocate device tensors with PyTorch and issue the
C-ABI calls of ``binding`` in the order of the paper's section 2 (per-example gradients ->
norms -> clip -> sum over the chunk, repeated per accumulation chunk -> noise -> average) or,
for per-layer clipping (section 3.5), with the clip fused into the weight-gradient call.
"""
from __future__ import annotations

import math
import torch

from . import binding as b
from .synth import Layer

_KIND = {"conv": b.DP_LAYER_CONV2D, "dense": b.DP_LAYER_DENSE, "norm": b.DP_LAYER_NORM_AFFINE}


_DTYPE = {"f32": b.DP_F32, "bf16": b.DP_BF16, "tf32": b.DP_TF32}   # "tf32": fp32 in memory, one tf32 pass on tensor cores


def layer_desc(layer: Layer, B: int, dtype: str, impl=b.DP_IMPL_AUTO, bias_separate=1):
    return b.make_desc(_KIND[layer.kind], _DTYPE[dtype], B, layer.Cin, layer.Kout,
                       layer.H, layer.W, layer.R, layer.S, layer.stride, layer.pad, int(layer.bias), bias_separate, impl)


def _tensors_of(layers):
    """[(layer index, 'w' | 'b', size)] in parameter order: weight then bias-like tensor of each layer."""
    out = []
    for li, l in enumerate(layers):
        out.append((li, "w", l.n_weight))
        if l.n_bias:
            out.append((li, "b", l.n_bias))
    return out


def _workspaces(nbytes, lanes, device):
    """One initialised dp_per_example_wgrad workspace per lane (calls that may overlap need one each)."""
    out = []
    for _ in range(lanes):
        w = torch.empty(nbytes, dtype=torch.uint8, device=device)
        b.check(b.dp_workspace_init(w), "dp_workspace_init")
        out.append(w)
    torch.cuda.synchronize()
    return out


class _NoiseKey:
    """Where the noise enters: once per step in finish() (default), or per example inside every chunk call, in which
    case the chunk calls need the step's total batch and key and finish() only divides."""

    def __init__(self, per_example, total_batch, seed, step, example0):
        if per_example and not total_batch:
            raise ValueError("per-example noise needs begin(total_batch=...)")
        self.per_example, self.total_batch, self.seed, self.step, self.example0 = per_example, total_batch, seed, step, example0

    def finish_sigma(self, sigma, total):
        if not self.per_example:
            return sigma
        if total != self.total_batch:
            raise ValueError(f"step saw {total} examples but its noise was scaled for {self.total_batch}")
        return 0.0


class GlobalClipStep:
    """Whole-model clipping.  A layer's per-example gradients are either materialised (STORE+NORM epilogue, consumed by
    the clipped sum over memory) or, when `recompute` names the layer, never written: its norms come from a NORM_ONLY
    call and its clipped sum from dp_per_example_wgrad_scaled once every layer's norm is known.  "auto" recomputes the
    dense layers whose gradients are larger than the inputs they come from; a list of layer indices names any layers."""

    def __init__(self, layers, B, dtype, C, sigma, impl=b.DP_IMPL_AUTO, device="cuda", per_example_noise=False, lanes=1,
                 recompute="none"):
        """lanes > 1: chunk() spreads the layers' calls over that many CUDA streams (a workspace each) and joins them
        around the factor computation: the calls write disjoint buffers, so they may overlap."""
        self.layers, self.B, self.dtype, self.C, self.sigma = list(layers), B, dtype, float(C), float(sigma)
        self.per_example_noise = bool(per_example_noise)
        self.tensors = _tensors_of(self.layers)
        self.L = len(self.tensors)
        self.P_l = [t[2] for t in self.tensors]
        self.P = sum(self.P_l)
        self.descs = [layer_desc(l, B, dtype, impl, 1) for l in self.layers]
        self.sq = torch.zeros((B, self.L), dtype=torch.float32, device=device)
        self.acc = torch.zeros(self.P, dtype=torch.float32, device=device)
        self.out = torch.empty(self.P, dtype=torch.float32, device=device)
        offs, o = [], 0
        for p in self.P_l:
            offs.append(o)
            o += p
        self.offsets = offs
        self.acc_views = [self.acc[o:o + p] for o, p in zip(offs, self.P_l)]
        # column of each layer's first tensor in the [B, L] norm table
        self._col, col = [], 0
        for l in self.layers:
            self._col.append(col)
            col += 2 if l.n_bias else 1
        self.recompute = self._recompute_set(recompute)
        if self.recompute and self.per_example_noise:
            raise ValueError("per-example noise is added by the clipped sum over materialised gradients")
        kept = [t[0] not in self.recompute for t in self.tensors]
        self.G = [torch.empty((B, p), dtype=torch.float32, device=device) if k else None for p, k in zip(self.P_l, kept)]
        self._kept = [i for i, k in enumerate(kept) if k]
        self.norms = torch.empty(B, dtype=torch.float32, device=device)
        self.clip = torch.empty(B, dtype=torch.float32, device=device)
        ws = max([b.dp_workspace_bytes(d, e) for d in self.descs for e in (b.DP_EPI_STORE_NORM, b.DP_EPI_NORM_ONLY, b.DP_EPI_CLIP_ACCUM)] + [256])
        self.lanes = max(1, min(int(lanes), len(self.layers)))
        self.ws_lane = _workspaces(ws, self.lanes, device)
        self.ws = self.ws_lane[0]
        self._side = [torch.cuda.Stream(device=device) for _ in range(self.lanes - 1)] if self.lanes > 1 else []
        self.clip_ws = torch.empty(max(b.dp_clip_workspace_bytes(B, self.P_l), 256), dtype=torch.uint8, device=device)
        self.chunks_done = 0

    def _recompute_set(self, recompute):
        if recompute == "none" or not recompute:
            return set()
        if recompute != "auto":
            return set(int(i) for i in recompute)
        out = set()
        esize = 2 if self.dtype == "bf16" else 4
        for li, (l, d) in enumerate(zip(self.layers, self.descs)):
            if l.kind == "norm":
                continue
            inputs = (math.prod(l.x_shape(self.B)) + math.prod(l.dy_shape(self.B))) * esize
            grads = (l.n_weight + l.n_bias) * self.B * 4
            # a dense layer's gradient is a rank-1 product: its second pass costs next to nothing.  A convolution's
            # second pass runs the whole contraction again, which only pays when the layer is bound by its stores.
            fast = l.kind == "dense"
            col = self._col[li]
            views = self.acc_views[col:col + (2 if l.n_bias else 1)]
            if grads > inputs and fast and all(v.data_ptr() % 16 == 0 for v in views):
                out.add(li)
        return out

    def begin(self, total_batch=None, seed=0, step=0, example0=0):
        """Per-example noise needs the step's total batch, its (seed, step) and this rank's first example index up front."""
        self.acc.zero_()
        self.chunks_done = 0
        self._noise = _NoiseKey(self.per_example_noise, total_batch, seed, step, example0)

    def wgrad(self, li, X, dY, lane=0, stream=None):
        """First pass of layer li: its norms, and its per-example gradients unless the layer is recomputed."""
        col = self._col[li]
        keep = li not in self.recompute
        G_w = self.G[col]
        G_b = self.G[col + 1] if self.layers[li].n_bias else None
        b.check(b.dp_per_example_wgrad(self.descs[li], X, dY, G_w, G_b, self.sq.data_ptr() + 4 * col, self.L,
                                       b.DP_EPI_STORE_NORM if keep else b.DP_EPI_NORM_ONLY, 0.0, None, None, None,
                                       self.ws_lane[lane], stream=stream), "dp_per_example_wgrad")

    def wgrad_scaled(self, li, X, dY, lane=0, stream=None):
        """Second pass of a recomputed layer: its clipped sum with the factors in self.clip."""
        col = self._col[li]
        acc_b = self.acc_views[col + 1] if self.layers[li].n_bias else None
        b.check(b.dp_per_example_wgrad_scaled(self.descs[li], X, dY, self.clip, None, 1, self.acc_views[col], acc_b,
                                              self.ws_lane[lane], stream=stream), "dp_per_example_wgrad_scaled")

    def clip_factors(self):
        """One factor per example from the norm table every layer's first pass has filled."""
        b.check(b.dp_clip_factors(b.DP_CLIP_GLOBAL, self.B, self.L, self.sq, self.C, self.norms, self.clip), "dp_clip_factors")

    def scale_kept(self, stream=None):
        """Clipped sum of the tensors whose per-example gradients are in memory, with the factors in self.clip."""
        b.check(b.dp_scale_accumulate(self.B, [self.G[i] for i in self._kept], [self.P_l[i] for i in self._kept], self.clip, 0,
                                      [self.acc_views[i] for i in self._kept], stream=stream), "dp_scale_accumulate")

    def _forked(self, calls):
        """Runs calls[k](lane, stream) spread over the lanes, joined again on the current stream."""
        if self.lanes == 1 or len(calls) <= 1:
            for c in calls:
                c(0, None)
            return
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(main)
        streams = [main] + self._side
        used = min(self.lanes, len(calls))
        for s in streams[1:used]:
            s.wait_event(fork)
        for i, c in enumerate(calls):
            c(i % used, streams[i % used])
        for s in streams[1:used]:
            done = torch.cuda.Event()
            done.record(s)
            main.wait_event(done)

    def wgrad_all(self, inputs):
        """Every layer's first-pass call: in order on the current stream, or forked over the lanes and joined."""
        self._forked([(lambda lane, stream, li=li, X=X, dY=dY: self.wgrad(li, X, dY, lane, stream))
                      for li, (X, dY) in enumerate(inputs)])

    def clip_accumulate(self, use_epilogue_norms=True, inputs=None):
        """Factors from the norm table, then the clipped sums: over memory for the kept tensors, by a second pass over
        `inputs` for the recomputed layers."""
        sq = self.sq if use_epilogue_norms else None
        if self.per_example_noise:
            k = self._noise
            b.check(b.dp_clip_accumulate_noised(b.DP_CLIP_GLOBAL, self.B, self.G, self.P_l, self.offsets, sq, self.C,
                                                self.sigma, k.total_batch, k.seed, k.step,
                                                k.example0 + self.B * self.chunks_done, self.acc_views, self.norms,
                                                self.clip, self.clip_ws), "dp_clip_accumulate_noised")
        elif not self.recompute:
            b.check(b.dp_clip_accumulate(b.DP_CLIP_GLOBAL, self.B, self.G, self.P_l, sq, self.C, self.acc_views, self.norms,
                                         self.clip, self.clip_ws), "dp_clip_accumulate")
        else:
            if inputs is None:
                raise ValueError("recomputed layers need the chunk's inputs for their second pass")
            self.clip_factors()
            calls = []
            if self._kept:
                calls.append(lambda lane, stream: self.scale_kept(stream))
            for li in sorted(self.recompute):
                X, dY = inputs[li]
                calls.append(lambda lane, stream, li=li, X=X, dY=dY: self.wgrad_scaled(li, X, dY, lane, stream))
            self._forked(calls)
        self.chunks_done += 1

    def chunk(self, inputs):
        """inputs: list of (X, dY) device tensors, one pair per layer."""
        self.wgrad_all(inputs)
        self.clip_accumulate(inputs=inputs)

    def check(self):
        """Status words of the tensor-core launches of every lane (synchronises)."""
        for w in self.ws_lane:
            b.check(b.dp_wgrad_check(w), "dp_wgrad_check")

    def finish(self, seed=0, step=0, total_batch=None):
        """total_batch: |B| of the whole step.  Left out, it is what this object saw (one process).  With several
        ranks `acc` already holds the sum over all of them (sharding.allreduce_accumulator) and the caller passes the
        global count (sharding.global_batch): ranks may have run different numbers of chunks."""
        total = self.B * self.chunks_done if total_batch is None else int(total_batch)
        sigma = self._noise.finish_sigma(self.sigma, total)
        b.check(b.dp_noise_average(self.acc, self.P, 0, sigma, self.C, total, seed, step, self.out), "dp_noise_average")
        return self.out


class FlatClipStep:
    """Flattened per-example gradients [B, P] handed in directly (no weight-gradient stage)."""

    def __init__(self, P, B, C, sigma, device="cuda", per_example_noise=False, micro=1):
        """micro > 1: runs of `micro` consecutive examples are averaged before clipping (the clipped unit is the run)."""
        self.P, self.B, self.C, self.sigma = P, B, float(C), float(sigma)
        self.per_example_noise = bool(per_example_noise)
        self.micro = int(micro)
        if self.micro < 1 or B % self.micro or (self.micro > 1 and per_example_noise):
            raise ValueError("micro must divide B, and per-example noise is defined for single examples")
        self.acc = torch.zeros(P, dtype=torch.float32, device=device)
        self.out = torch.empty(P, dtype=torch.float32, device=device)
        self.norms = torch.empty(B, dtype=torch.float32, device=device)
        self.clip = torch.empty(B, dtype=torch.float32, device=device)
        self.ws = torch.empty(max(b.dp_clip_workspace_bytes(B, [P]), 256), dtype=torch.uint8, device=device)
        self.chunks_done = 0

    def begin(self, total_batch=None, seed=0, step=0, example0=0):
        self.acc.zero_()
        self.chunks_done = 0
        self._noise = _NoiseKey(self.per_example_noise, total_batch, seed, step, example0)

    def chunk(self, G, sqnorm=None):
        if self.micro > 1:
            b.check(b.dp_clip_accumulate_micro(self.B, self.micro, [G], [self.P], self.C, [self.acc], self.norms, self.clip,
                                               self.ws), "dp_clip_accumulate_micro")
        elif self.per_example_noise:
            k = self._noise
            b.check(b.dp_clip_accumulate_noised(b.DP_CLIP_GLOBAL, self.B, [G], [self.P], [0], sqnorm, self.C, self.sigma,
                                                k.total_batch, k.seed, k.step, k.example0 + self.B * self.chunks_done,
                                                [self.acc], self.norms, self.clip, self.ws), "dp_clip_accumulate_noised")
        else:
            b.check(b.dp_clip_accumulate(b.DP_CLIP_GLOBAL, self.B, [G], [self.P], sqnorm, self.C, [self.acc], self.norms,
                                         self.clip, self.ws), "dp_clip_accumulate")
        self.chunks_done += 1

    def finish(self, seed=0, step=0, total_batch=None):
        """total_batch as for GlobalClipStep.finish (examples, not micro-batches)."""
        total = self.B * self.chunks_done if total_batch is None else int(total_batch)
        sigma = self._noise.finish_sigma(self.sigma, total)
        b.check(b.dp_noise_average(self.acc, self.P, 0, sigma, self.C, total // self.micro, seed, step, self.out),
                "dp_noise_average")
        return self.out


class PerLayerClipStep:
    """Per-layer clipping (threshold C/sqrt(L) per parameter tensor) fused into the weight-gradient call:
    no per-example gradient is written to memory."""

    def __init__(self, layers, B, dtype, C, sigma, impl=b.DP_IMPL_AUTO, device="cuda", lanes=1):
        """lanes > 1: chunk() spreads the layer calls over that many CUDA streams (each with a workspace of its own).
        The calls of one chunk touch disjoint outputs, so they may overlap; a chunk of few examples leaves most of
        the GPU idle inside any single call."""
        self.layers, self.B, self.dtype, self.C, self.sigma = list(layers), B, dtype, float(C), float(sigma)
        self.tensors = _tensors_of(self.layers)
        self.L = len(self.tensors)
        self.C_l = self.C / math.sqrt(self.L)
        self.descs = [layer_desc(l, B, dtype, impl, 1) for l in self.layers]
        # one accumulator in parameter order (weight, then bias-like tensor, of each layer); the layer calls get views.
        # A tensor that would start off a 16-byte boundary is padded forward (`self.offsets` keeps the true indices).
        self.P = sum(t[2] for t in self.tensors)
        starts, self.offsets, cur, true = [], [], 0, 0
        for _, _, size in self.tensors:
            cur = (cur + 3) // 4 * 4
            starts.append(cur)
            self.offsets.append(true)
            cur += size
            true += size
        self.acc = torch.zeros(cur, dtype=torch.float32, device=device)
        self.contiguous = cur == self.P                     # no padding: the accumulator IS the parameter vector
        views = {(li, which): self.acc[s0:s0 + size] for (li, which, size), s0 in zip(self.tensors, starts)}
        self.acc_w = [views[(li, "w")] for li in range(len(self.layers))]
        self.acc_b = [views.get((li, "b")) for li in range(len(self.layers))]
        self.sq = torch.zeros((B, self.L), dtype=torch.float32, device=device)
        ws = max([b.dp_workspace_bytes(d, b.DP_EPI_CLIP_ACCUM) for d in self.descs] + [256])
        self.lanes = max(1, int(lanes))
        self.ws_lane = _workspaces(ws, self.lanes, device)
        self.ws = self.ws_lane[0]
        self._col, col = [], 0
        for l in self.layers:
            self._col.append(col)
            col += 2 if l.n_bias else 1
        self.chunks_done = 0
        self._side = [torch.cuda.Stream(device=device) for _ in range(self.lanes - 1)] if self.lanes > 1 else []
        # layer -> lane: each call goes to the lane with the least work so far (a rough per-call cost is enough)
        load, self._lane_of = [0.0] * self.lanes, []
        for l in self.layers:
            cost = 12.0 + (l.flops() * B / 2.0e8 if l.kind == "conv" else 6.0)
            k = min(range(self.lanes), key=lambda q: load[q])
            load[k] += cost
            self._lane_of.append(k)

    def begin(self):
        self.acc.zero_()
        self.chunks_done = 0

    def wgrad(self, li, X, dY, lane=0, stream=None):
        b.check(b.dp_per_example_wgrad(self.descs[li], X, dY, None, None, self.sq.data_ptr() + 4 * self._col[li], self.L,
                                       b.DP_EPI_CLIP_ACCUM, self.C_l, self.acc_w[li], self.acc_b[li], None,
                                       self.ws_lane[lane], stream=stream), "dp_per_example_wgrad")

    def chunk_calls(self, inputs, only=None):
        """The layer calls of one chunk: in order on the current stream, or forked over the lanes and joined again.
        only: a set of layer indices to restrict the chunk to (measurements of one kind of layer)."""
        if self.lanes == 1:
            for li, (X, dY) in enumerate(inputs):
                if only is None or li in only:
                    self.wgrad(li, X, dY)
            return
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(main)
        streams = [main] + self._side
        for s in self._side:
            s.wait_event(fork)
        for li, (X, dY) in enumerate(inputs):
            if only is not None and li not in only:
                continue
            k = self._lane_of[li]
            self.wgrad(li, X, dY, lane=k, stream=streams[k])
        for s in self._side:
            done = torch.cuda.Event()
            done.record(s)
            main.wait_event(done)

    def chunk(self, inputs):
        self.chunk_calls(inputs)
        self.chunks_done += 1

    def check(self):
        """Status words of the tensor-core launches of every lane (synchronises)."""
        for w in self.ws_lane:
            b.check(b.dp_wgrad_check(w), "dp_wgrad_check")

    def finish(self, seed=0, step=0, total_batch=None):
        """Noise uses the whole-gradient bound C (the per-tensor thresholds keep the sensitivity at C).
        total_batch as for GlobalClipStep.finish."""
        total = self.B * self.chunks_done if total_batch is None else int(total_batch)
        if self.contiguous:
            b.check(b.dp_noise_average(self.acc, self.P, 0, self.sigma, self.C, total, seed, step, self.acc), "dp_noise_average")
            return self.acc_w, self.acc_b
        views = [a for pair in zip(self.acc_w, self.acc_b) for a in pair if a is not None]
        for a, off in zip(views, self.offsets):
            b.check(b.dp_noise_average(a, a.numel(), off, self.sigma, self.C, total, seed, step, a), "dp_noise_average")
        return self.acc_w, self.acc_b
