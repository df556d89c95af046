"""Seeded synthetic inputs and workload shapes.

This module holds no arithmetic of the privatisation step: it only draws random
tensors and lists layer shapes.  The same bytes are handed to the CUDA library and
to the CPU oracle by the tests and the benchmark.

The shapes stand in for the paper's workloads: 32x32x3 images (CIFAR-10 scale) and
224x224x3 images through a ResNet-50 whose batch norms are replaced by group norm
with 32 groups (section 1 and section 3 of the paper).  No dataset is read.
"""
from __future__ import annotations

from dataclasses import dataclass
import numpy as np


def generator(*key: int) -> np.random.Generator:
    """PCG64 stream addressed by a tuple of small integers, e.g. (config, layer, chunk)."""
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence(list(key))))


def normal_f32(shape, *key: int, scale: float = 1.0) -> np.ndarray:
    a = generator(*key).standard_normal(shape, dtype=np.float32)
    if scale != 1.0:
        a *= np.float32(scale)
    return a


def round_to_bf16(a: np.ndarray):
    """Round float32 to bfloat16 (nearest, ties to even).

    Returns (bits uint16, widened float32 holding exactly the rounded values)."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    r = ((u + bias) >> 16).astype(np.uint16)
    wide = (r.astype(np.uint32) << 16).view(np.float32)
    return r, wide


@dataclass(frozen=True)
class Layer:
    """One parameterised layer of a workload (channels-last tensors).

    kind: "conv" (X [B,H,W,Cin], dY [B,OH,OW,Kout]), "dense" (X [B,Cin], dY [B,Kout])
    or "norm" (xhat, dY [B,H,W,Cin]; Kout == Cin)."""
    kind: str
    Cin: int
    Kout: int
    R: int = 1
    S: int = 1
    stride: int = 1
    pad: int = 0
    H: int = 1
    W: int = 1
    bias: bool = False
    name: str = ""

    @property
    def OH(self):
        return (self.H + 2 * self.pad - self.R) // self.stride + 1 if self.kind == "conv" else self.H

    @property
    def OW(self):
        return (self.W + 2 * self.pad - self.S) // self.stride + 1 if self.kind == "conv" else self.W

    @property
    def n_weight(self):
        return self.Cin if self.kind == "norm" else self.Kout * self.R * self.S * self.Cin

    @property
    def n_bias(self):
        if self.kind == "norm":
            return self.Cin
        return self.Kout if self.bias else 0

    def x_shape(self, B):
        return (B, self.Cin) if self.kind == "dense" else (B, self.H, self.W, self.Cin)

    def dy_shape(self, B):
        if self.kind == "dense":
            return (B, self.Kout)
        if self.kind == "norm":
            return (B, self.H, self.W, self.Cin)
        return (B, self.OH, self.OW, self.Kout)

    def flops(self):
        """Multiply-adds x2 of the per-example weight gradient."""
        if self.kind == "norm":
            return 2 * 2 * self.H * self.W * self.Cin
        return 2 * self.Kout * self.R * self.S * self.Cin * self.OH * self.OW


def conv(Cin, Kout, R, stride, pad, H, bias=False, name=""):
    return Layer("conv", Cin, Kout, R, R, stride, pad, H, H, bias, name)


def dense(Cin, Kout, bias=False, name=""):
    return Layer("dense", Cin, Kout, bias=bias, name=name)


def norm(C, H, name=""):
    return Layer("norm", C, C, H=H, W=H, name=name)


# --- the five measured workloads -------------------------------------------------
def single_dense():
    """Dense 256->64 with bias, B=8, fp32; C=1.0, sigma=1.1, seed 0."""
    return dict(layers=[dense(256, 64, bias=True, name="fc")], B=8, G=1, dtype="f32",
                C=1.0, sigma=1.1, seed=0, step=0, mode="global")


def small_cnn():
    """Three 3x3 convs and a classifier on 32x32x3 inputs, B=256, fp32; every layer has a bias."""
    layers = [conv(3, 32, 3, 1, 1, 32, True, "conv1"), conv(32, 64, 3, 2, 1, 32, True, "conv2"),
              conv(64, 128, 3, 2, 1, 16, True, "conv3"), dense(8192, 10, True, "fc")]
    return dict(layers=layers, B=256, G=1, dtype="f32", C=1.5, sigma=1.0, seed=0, step=0, mode="global")


def resnet50_sweep():
    """Eight representative ResNet-50 layers at 224x224 input, B=32, bf16 inputs."""
    layers = [conv(3, 64, 7, 2, 3, 224, name="stem 7x7 3->64 s2"),
              conv(256, 64, 1, 1, 0, 56, name="1x1 256->64 @56"),
              conv(64, 64, 3, 1, 1, 56, name="3x3 64->64 @56"),
              conv(128, 128, 3, 1, 1, 28, name="3x3 128->128 @28"),
              conv(256, 256, 3, 1, 1, 14, name="3x3 256->256 @14"),
              conv(512, 512, 3, 1, 1, 7, name="3x3 512->512 @7"),
              conv(512, 2048, 1, 1, 0, 7, name="1x1 512->2048 @7"),
              dense(2048, 1000, name="dense 2048->1000")]
    return dict(layers=layers, B=32, G=1, dtype="bf16", C=1.0, sigma=1.0, seed=0, step=0, mode="global")


def resnet_gn_layers(blocks):
    """All parameter tensors of a bottleneck ResNet with `blocks` blocks per stage and a group norm after every
    convolution, stride on the 3x3 of the first block of stages 2-4 and a 1x1 projection shortcut."""
    layers = [conv(3, 64, 7, 2, 3, 224, name="stem"), norm(64, 112, "stem.gn")]
    H, inpl = 56, 64
    for si, (w, nb) in enumerate(zip([64, 128, 256, 512], blocks)):
        for b in range(nb):
            s = 2 if (b == 0 and si > 0) else 1
            Ho = (H + 2 - 3) // s + 1
            p = f"s{si}b{b}"
            layers += [conv(inpl, w, 1, 1, 0, H, name=p + ".c1"), norm(w, H, p + ".gn1"),
                       conv(w, w, 3, s, 1, H, name=p + ".c2"), norm(w, Ho, p + ".gn2"),
                       conv(w, 4 * w, 1, 1, 0, Ho, name=p + ".c3"), norm(4 * w, Ho, p + ".gn3")]
            if b == 0:
                layers += [conv(inpl, 4 * w, 1, s, 0, H, name=p + ".ds"), norm(4 * w, Ho, p + ".gnds")]
            inpl, H = 4 * w, Ho
    layers.append(dense(2048, 1000, bias=True, name="fc"))
    return layers


def resnet50_gn_layers():
    """ResNet-50 [3,4,6,3]: 53 convs + 53 norm layers (scale and shift) + classifier."""
    return resnet_gn_layers([3, 4, 6, 3])


def resnet101_gn_layers():
    """ResNet-101 [3,4,23,3], the second model of the paper's throughput comparison: 104 convs + 104 norm layers +
    classifier.  Its layer shapes are those of ResNet-50; only the third stage is longer."""
    return resnet_gn_layers([3, 4, 23, 3])


RESNET50_GN_PARAMS = 25_557_032   # sum of n_weight + n_bias over resnet50_gn_layers()
RESNET50_GN_TENSORS = 161         # 53 conv weights + 53*2 norm tensors + fc weight + fc bias
RESNET101_GN_PARAMS = 44_549_160
RESNET101_GN_TENSORS = 314        # 104 conv weights + 104*2 norm tensors + fc weight + fc bias


def resnet50_flat():
    """Flattened per-example gradients of the whole model, B=64 per chunk, 16 chunks."""
    return dict(P=RESNET50_GN_PARAMS, B=64, G=16, dtype="f32", grad_std=1e-3,
                C=1.0, sigma=1.0, seed=0, step=0, mode="global")


def resnet50_per_layer():
    """Per-layer clipping over all 161 tensors, B=32 per chunk, 32 chunks, bf16 inputs."""
    return dict(layers=resnet50_gn_layers(), B=32, G=32, dtype="bf16", C=1.0, sigma=1.0,
                seed=0, step=0, mode="per_layer", L=RESNET50_GN_TENSORS)


def resnet101_per_layer():
    """Per-layer clipping over all 314 tensors of ResNet-101, B=32 per chunk, 32 chunks, bf16 inputs."""
    return dict(layers=resnet101_gn_layers(), B=32, G=32, dtype="bf16", C=1.0, sigma=1.0,
                seed=0, step=0, mode="per_layer", L=RESNET101_GN_TENSORS)


def layer_inputs(layer: Layer, B: int, dtype: str, *key: int):
    """Draw X and dY ~ N(0,1) for one layer.  Returns dict with
    'X','dY': float32 arrays holding the exact values the GPU sees, and for bf16
    also 'X_bits','dY_bits' (uint16)."""
    X = normal_f32(layer.x_shape(B), *key, 0)
    dY = normal_f32(layer.dy_shape(B), *key, 1)
    out = {}
    if dtype == "bf16":
        out["X_bits"], X = round_to_bf16(X)
        out["dY_bits"], dY = round_to_bf16(dY)
    out["X"], out["dY"] = X, dY
    return out
