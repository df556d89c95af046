"""The launch configuration the benchmark times: the step captured into a CUDA graph and replayed.
A replay must give the bits of the plain stream launches, and full-size per-layer calls must match the oracle."""
import math
import numpy as np
import pytest
import torch

import oracle
from paper_2109_12191_b200 import synth
from paper_2109_12191_b200.step import GlobalClipStep, PerLayerClipStep
from gpu_util import dev_inputs, oracle_layer, rel_l2, TOL_NORM, TOL_ACC_BF16, TOL_ACC_F32

pytestmark = pytest.mark.gpu


def test_graph_replay_equals_stream_launches():
    layers = [synth.conv(3, 32, 3, 1, 1, 16, True, "c1"), synth.conv(32, 64, 3, 2, 1, 16, True, "c2"),
              synth.dense(64 * 64, 10, True, "fc")]
    Bn = 16
    st = GlobalClipStep(layers, Bn, "f32", 0.5, 1.0)
    ins = [dev_inputs(synth.layer_inputs(l, Bn, "f32", 960, li), "f32") for li, l in enumerate(layers)]

    def step():
        st.begin()
        st.chunk(ins)
        return st.finish(seed=2, step=5)

    direct = step().clone()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        out = step()
    for _ in range(2):
        g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, direct)


def test_small_cnn_step_as_benchmarked_matches_the_oracle():
    """The composite the small-CNN benchmark times -- 256 examples, fp32 inputs taken as tf32, four streams, an SM target
    of half the SMs, the classifier's clipped sum recomputed instead of materialised, the whole step replayed from a
    CUDA graph -- against the oracle's privatisation step on the same inputs."""
    from paper_2109_12191_b200 import binding
    cfg = synth.small_cnn()
    layers, Bn = cfg["layers"], cfg["B"]
    # as in the benchmark: the convolutions run side by side, each told to take half of the SMs
    binding.check(binding.dp_set_sm_target(torch.cuda.get_device_properties(0).multi_processor_count // 2))
    try:
        _small_cnn_as_benchmarked(cfg, layers, Bn)
    finally:
        binding.check(binding.dp_set_sm_target(0))


def _small_cnn_as_benchmarked(cfg, layers, Bn):
    st = GlobalClipStep(layers, Bn, "tf32", cfg["C"], cfg["sigma"], lanes=4, recompute="auto")
    assert st.recompute                                    # the classifier is not materialised
    host = [synth.layer_inputs(l, Bn, "f32", 1, li, 0) for li, l in enumerate(layers)]
    # N(0,1) inputs give whole-model norms near 3200, so every example would be clipped: spread them over the threshold
    scale = (np.logspace(-0.8, 0.8, Bn) * cfg["C"] / 3200.0).astype(np.float32)
    for h in host:
        h["dY"] *= scale.reshape((Bn,) + (1,) * (h["dY"].ndim - 1))
    ins = [dev_inputs(h, "f32") for h in host]

    def step():
        st.begin()
        st.wgrad_all(ins)
        st.clip_accumulate(inputs=ins)
        return st.finish(seed=0, step=3)

    step()                                                 # warm-up outside the capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        out = step()
    g.replay(); g.replay()
    torch.cuda.synchronize()
    st.check()
    groups = []
    for l, h in zip(layers, host):
        dW, db = oracle_layer(l, h)
        groups += [dW, db]
    ref, ref_sq, ref_f = oracle.privatise([groups], cfg["C"], cfg["sigma"], "global", 0, 3)
    ref_sq, ref_f = ref_sq[0], ref_f[0]                    # [B, L] squared norms and [B] factors of the one chunk
    assert (ref_f == 1.0).any() and (ref_f < 1.0).any()
    np.testing.assert_allclose(st.norms.cpu().numpy(), np.sqrt(ref_sq.sum(1)), rtol=TOL_NORM)
    np.testing.assert_allclose(st.clip.cpu().numpy(), ref_f, rtol=TOL_NORM)
    ref = np.concatenate(ref)
    signal, _, _ = oracle.clipped_sum(groups, cfg["C"], "global")
    signal = np.concatenate(signal) / Bn
    got = out.cpu().numpy()
    # the output is signal + noise; the noise is reproduced to 1e-5 of its scale, the signal to the tf32 bound
    assert np.max(np.abs(got - ref)) <= 1e-5 * cfg["sigma"] * cfg["C"] / Bn + TOL_ACC_F32 * np.max(np.abs(signal))
    assert rel_l2(got - (ref - signal), signal) <= TOL_ACC_F32


def _distinct_resnet50_layers():
    """One layer of every distinct shape of the per-layer ResNet-50 workload: 23 convolutions, the distinct
    normalisation shapes and the classifier."""
    seen, out = set(), []
    for l in synth.resnet50_gn_layers():
        key = (l.kind, l.Cin, l.Kout, l.R, l.stride, l.H)
        if key not in seen:
            seen.add(key)
            out.append(l)
    return out


_DISTINCT = _distinct_resnet50_layers()


@pytest.mark.parametrize("layer", _DISTINCT, ids=[f"{l.name}:{l.kind}{l.R}x{l.R}_{l.Cin}to{l.Kout}_s{l.stride}_at{l.H}" for l in _DISTINCT])
def test_per_layer_workload_full_size_layers(layer):
    """Every distinct layer shape of the per-layer ResNet-50 workload at full size (B = 32, threshold C/sqrt(161),
    clip fused into the weight-gradient call), run from a replayed CUDA graph under an SM target as the benchmark does; the oracle
    checks every example's squared norm and factor and the whole clipped sum."""
    Bn, C_l = 32, 1.0 / math.sqrt(synth.RESNET50_GN_TENSORS)
    inp = synth.layer_inputs(layer, Bn, "bf16", 4, 7, 0)
    # norms of N(0,1) inputs are far above the threshold; scale so that they straddle it
    s = (np.logspace(-0.5, 0.5, Bn) * C_l / math.sqrt(layer.flops() / 2)).astype(np.float32)
    dY = inp["dY"] * s.reshape((Bn,) + (1,) * (inp["dY"].ndim - 1))
    inp["dY_bits"], inp["dY"] = synth.round_to_bf16(dY)
    # the benchmark sets an SM target (its calls run side by side), which changes how a call splits the batch over
    # thread blocks: the same setting here, queried before the workspace is sized
    from paper_2109_12191_b200 import binding
    binding.check(binding.dp_set_sm_target(torch.cuda.get_device_properties(0).multi_processor_count))
    try:
        st = PerLayerClipStep([layer], Bn, "bf16", 1.0, 1.0)
        st.C_l = C_l                                       # the threshold of the 161-tensor model, not of this one layer
        X, dYd = dev_inputs(inp, "bf16")
        st.begin()
        st.wgrad(0, X, dYd)                                # warm-up launch (sets kernel attributes before capture)
        torch.cuda.synchronize()
        st.begin()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            st.wgrad(0, X, dYd)
        g.replay()
        torch.cuda.synchronize()
        st.check()
    finally:
        binding.check(binding.dp_set_sm_target(0))
    dW, db = oracle_layer(layer, inp)
    groups = [dW] + ([db] if db is not None else [])
    sq = st.sq.cpu().numpy()
    factors = []
    for gi, grad in enumerate(groups):
        ref_sq = oracle.sqnorm(grad)
        np.testing.assert_allclose(sq[:, gi], ref_sq, rtol=TOL_NORM)
        f = oracle.clip_factor(ref_sq, C_l)
        factors.append(f)
        got = (st.acc_w[0] if gi == 0 else st.acc_b[0]).cpu().numpy()
        # capturing records without running: the accumulator holds the single replay's contribution
        assert rel_l2(got, np.einsum("n,np->p", f, grad)) <= TOL_ACC_BF16
    f = np.concatenate(factors)                            # (a classifier's bias gradient is small: never clipped)
    assert (f == 1.0).any() and (f < 1.0).any()


def test_layer_calls_spread_over_streams_give_the_same_bits():
    """The per-layer step may fork its layer calls over several streams (one workspace each) and join them again; the
    calls write disjoint outputs, so the result must equal the single-stream one bit for bit, also from a replayed graph."""
    layers = [synth.conv(64, 64, 3, 1, 1, 14, name="a"), synth.norm(64, 14, "gn_a"), synth.conv(64, 128, 1, 1, 0, 14, name="b"),
              synth.norm(128, 14, "gn_b"), synth.conv(128, 128, 3, 2, 1, 14, name="c"), synth.norm(128, 7, "gn_c"),
              synth.dense(128, 10, True, "fc")]
    Bn = 8
    ins = [dev_inputs(synth.layer_inputs(l, Bn, "bf16", 961, li), "bf16") for li, l in enumerate(layers)]

    def result(st):
        return torch.cat([t for pair in zip(st.acc_w, st.acc_b) for t in pair if t is not None]).clone()

    one = PerLayerClipStep(layers, Bn, "bf16", 50.0, 1.0)
    one.begin(); one.chunk(ins); one.chunk(ins)
    torch.cuda.synchronize()
    many = PerLayerClipStep(layers, Bn, "bf16", 50.0, 1.0, lanes=3)
    assert len(set(many._lane_of)) == 3
    many.begin(); many.chunk(ins); many.chunk(ins)
    torch.cuda.synchronize()
    many.check()
    assert torch.equal(result(many), result(one))
    assert torch.equal(many.sq, one.sq)
    many.begin()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        many.chunk_calls(ins)
    g.replay(); g.replay()
    torch.cuda.synchronize()
    assert torch.equal(result(many), result(one))


def test_full_resnet50_chunk_in_the_benchmarks_launch_configuration():
    """One whole 32-example chunk of the per-layer ResNet-50 workload (all 107 layer calls, 2.8 GB of inputs) the way the
    benchmark times it -- four streams, replayed from a CUDA graph -- against plain launches on one stream: the 161
    accumulators and the norm table must agree bit for bit.  (Single layers at this size are checked against the oracle
    above; the oracle cannot run the whole chunk in a test's time.)"""
    cfg = synth.resnet50_per_layer()
    layers, Bn = cfg["layers"], cfg["B"]
    g = torch.Generator(device="cuda"); g.manual_seed(77)
    ins = [(torch.empty(l.x_shape(Bn), device="cuda", dtype=torch.bfloat16).normal_(generator=g),
            (torch.empty(l.dy_shape(Bn), device="cuda", dtype=torch.bfloat16).normal_(generator=g) * 1e-3).contiguous())
           for l in layers]

    def result(st):
        return torch.cat([t for pair in zip(st.acc_w, st.acc_b) for t in pair if t is not None]).clone()

    one = PerLayerClipStep(layers, Bn, "bf16", cfg["C"], cfg["sigma"])
    one.begin(); one.chunk(ins)
    torch.cuda.synchronize()
    one.check()
    ref, ref_sq = result(one), one.sq.clone()
    assert ref.numel() == synth.RESNET50_GN_PARAMS and torch.isfinite(ref).all() and ref.abs().max() > 0
    f = torch.clamp((cfg["C"] / math.sqrt(one.L)) / ref_sq.sqrt(), max=1.0)
    assert (f == 1.0).any() and (f < 1.0).any()            # the scaled dY puts examples on both sides of the thresholds
    del one
    many = PerLayerClipStep(layers, Bn, "bf16", cfg["C"], cfg["sigma"], lanes=4)
    many.begin(); many.chunk(ins)                           # warm-up outside the capture
    torch.cuda.synchronize()
    many.begin()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        many.chunk_calls(ins)
    graph.replay()
    torch.cuda.synchronize()
    many.check()
    assert torch.equal(result(many), ref)
    assert torch.equal(many.sq, ref_sq)
