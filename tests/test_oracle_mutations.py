"""Do the oracle's pins bite?  Each case plants one plausible mistake in a copy of dp_oracle.c (a dropped term, a
wrong sign or index, a swapped operand, a wrong constant), builds it with gcc and runs a compact set of the pins
against it: every planted mistake must make at least one pin fail, and the unmodified source must pass them all.
Everything here runs on the CPU; nothing of the CUDA library is involved."""
import ctypes
import math
import os
import subprocess

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from paper_2109_12191_b200 import synth

SRC = os.path.join(os.path.dirname(oracle.__file__), "dp_oracle.c")

MUTATIONS = {
    "conv: padding sign": ("const int ih = oh * stride + r - pad;", "const int ih = oh * stride + r + pad;"),
    "conv: wrong tap index": ("const int iw = ow * stride + s - pad;", "const int iw = ow * stride + r - pad;"),
    "conv: stride dropped": ("const int iw = ow * stride + s - pad;", "const int iw = ow + s - pad;"),
    "conv: bias sum dropped": ("                    bsum += g;\n", ""),
    "dense: sum instead of product": ("= g * (double)X[(size_t)n * Cin + i];", "= g + (double)X[(size_t)n * Cin + i];"),
    "norm affine: xhat dropped": ("sg += (double)dY[idx] * (double)xhat[idx];", "sg += (double)dY[idx];"),
    "norm: abs instead of square": ("            a += v * v;\n", "            a += fabs(v);\n"),
    "clip: no square root": ("1.0 : C / sqrt(sq[j]);", "1.0 : C / sq[j];"),
    "clip: branch reversed": ("(sq[j] <= C * C) ? 1.0", "(sq[j] >= C * C) ? 1.0"),
    "accumulate: factor dropped": ("a += factor[n] * (double)G[(size_t)n * P + i];", "a += (double)G[(size_t)n * P + i];"),
    "philox: multipliers swapped": ("const uint64_t p0 = 0xD2511F53ull * c0;", "const uint64_t p0 = 0xCD9E8D57ull * c0;"),
    "philox: nine rounds": ("for (int round = 0; round < 10; ++round) {", "for (int round = 0; round < 9; ++round) {"),
    "uniform: wrong shift": ("(double)(ra >> 9) + 0.5", "(double)(ra >> 8) + 0.5"),
    "box-muller: sine and cosine swapped": ("(lane & 1) ? radius * sin(two_pi * u2) : radius * cos(two_pi * u2)",
                                            "(lane & 1) ? radius * cos(two_pi * u2) : radius * sin(two_pi * u2)"),
    "average: division dropped": ("out[i] = (acc[i] + noise) / total_batch;", "out[i] = (acc[i] + noise);"),
    "noise: C dropped from the scale": ("0.0 : sigma * C * noise_z_one(", "0.0 : sigma * noise_z_one("),
}


def _build(tmp_path, name, old=None, new=None):
    text = open(SRC).read()
    if old is not None:
        assert text.count(old) >= 1, f"mutation anchor not found: {old!r}"
        text = text.replace(old, new, 1)
    c = tmp_path / f"{name}.c"
    so = tmp_path / f"{name}.so"
    c.write_text(text)
    subprocess.run(["gcc", "-O1", "-fopenmp", "-shared", "-fPIC", "-o", str(so), str(c), "-lm"], check=True)
    return ctypes.CDLL(str(so))


def _pins():
    """A compact subset of the pins of test_oracle_*.py; raises AssertionError when the oracle is wrong."""
    # convolution against PyTorch float64 autograd, one example at a time (non-square, stride 2, padding 1, bias)
    B, H, W, Cin, Kout, R, st, pad = 2, 7, 9, 3, 4, 3, 2, 1
    OH, OW = (H + 2 * pad - R) // st + 1, (W + 2 * pad - R) // st + 1
    X = synth.normal_f32((B, H, W, Cin), 970, 0)
    dY = synth.normal_f32((B, OH, OW, Kout), 970, 1)
    dW, db = oracle.conv_wgrad(X, dY, R, R, st, pad, bias=True)
    for n in range(B):
        x = torch.from_numpy(X[n:n + 1].astype(np.float64)).permute(0, 3, 1, 2)
        g = torch.from_numpy(dY[n:n + 1].astype(np.float64)).permute(0, 3, 1, 2)
        w = torch.zeros(Kout, Cin, R, R, dtype=torch.float64, requires_grad=True)
        b = torch.zeros(Kout, dtype=torch.float64, requires_grad=True)
        (F.conv2d(x, w, b, stride=st, padding=pad) * g).sum().backward()
        np.testing.assert_allclose(dW[n], w.grad.permute(0, 2, 3, 1).numpy(), rtol=1e-11, atol=1e-11)
        np.testing.assert_allclose(db[n], b.grad.numpy(), rtol=1e-11, atol=1e-11)
    # dense: outer product; norm affine: two dot products per channel
    Xd, Yd = synth.normal_f32((3, 5), 971, 0), synth.normal_f32((3, 4), 971, 1)
    dWd, _ = oracle.dense_wgrad(Xd, Yd)
    np.testing.assert_allclose(dWd, np.einsum("no,ni->noi", Yd.astype(np.float64), Xd.astype(np.float64)), rtol=1e-13)
    xh, gy = synth.normal_f32((2, 3, 4, 5), 972, 0), synth.normal_f32((2, 3, 4, 5), 972, 1)
    dg, dbeta = oracle.norm_affine_wgrad(xh, gy)
    np.testing.assert_allclose(dg, (xh.astype(np.float64) * gy).sum(axis=(1, 2)), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(dbeta, gy.astype(np.float64).sum(axis=(1, 2)), rtol=1e-12, atol=1e-12)
    # norm, clip, accumulate
    G = synth.normal_f32((6, 50), 973) * np.logspace(-1.5, 0.5, 6).astype(np.float32)[:, None]
    s = oracle.sqnorm(G)
    np.testing.assert_allclose(s, (G.astype(np.float64) ** 2).sum(1), rtol=1e-13)
    f = oracle.clip_factor(s, 1.0)
    norms = np.sqrt(s)
    assert np.all(f[norms <= 1.0] == 1.0) and np.all(f[norms > 1.0] < 1.0) and (norms <= 1.0).any() and (norms > 1.0).any()
    assert np.all(f * norms <= 1.0 + 1e-12)
    np.testing.assert_allclose(f[norms > 1.0], 1.0 / norms[norms > 1.0], rtol=1e-13)
    acc = oracle.clip_accumulate(G, f, np.zeros(50))
    np.testing.assert_allclose(acc, np.einsum("n,np->p", f, G.astype(np.float64)), rtol=1e-12, atol=1e-14)
    # Philox known answer (all-zero counter and key), uniforms and Box-Muller from its words, noise + average
    assert oracle.philox4x32_10([0, 0, 0, 0], [0, 0]) == [0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8]
    u1, u2 = ((0x6627E8D5 >> 9) + 0.5) / 2 ** 23, (0xE169C58D >> 8) / 2 ** 24
    z = oracle.noise_z(0, 0, 0, 2)
    r = math.sqrt(-2 * math.log(u1))
    assert abs(z[0] - r * math.cos(2 * math.pi * u2)) < 1e-13 and abs(z[1] - r * math.sin(2 * math.pi * u2)) < 1e-13
    out = oracle.noise_average(np.array([1.0, 2.0]), 0, 0.5, 3.0, 4, 0, 0)
    np.testing.assert_allclose(out, (np.array([1.0, 2.0]) + 0.5 * 3.0 * z) / 4.0, rtol=1e-14)


@pytest.fixture
def swap_oracle(monkeypatch):
    def use(lib):
        monkeypatch.setattr(oracle, "_lib", lib)
    return use


def test_unmodified_oracle_passes_the_compact_pins(tmp_path, swap_oracle):
    swap_oracle(_build(tmp_path, "pristine"))
    _pins()


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name, tmp_path, swap_oracle):
    old, new = MUTATIONS[name]
    swap_oracle(_build(tmp_path, "mutant", old, new))
    with pytest.raises(AssertionError):
        _pins()
