"""The measured workloads end to end on the GPU (C ABI) against the oracle."""
import math
import numpy as np
import pytest
import torch

import oracle
from paper_2109_12191_b200 import synth
from gpu_util import B, dev, rel_l2, gpu_layer, oracle_layer, dev_inputs, make_desc, TOL_NORM, TOL_FMA, TOL_ACC_BF16, TOL_ACC_F32

pytestmark = pytest.mark.gpu


def run_global_step(cfg, Bn=None, key0=0):
    """wgrad (STORE+NORM) per layer -> clip_accumulate(GLOBAL, norms supplied) -> noise_average."""
    b = B()
    layers, Bn = cfg["layers"], Bn or cfg["B"]
    tensors = []                                             # (layer index, "w"/"b", size)
    for li, l in enumerate(layers):
        tensors.append((li, "w", l.n_weight))
        if l.n_bias:
            tensors.append((li, "b", l.n_bias))
    L = len(tensors)
    P_l = [t[2] for t in tensors]
    sq = torch.zeros((Bn, L), device="cuda")
    G, ref_groups, col, any_tc = [], [], 0, False
    for li, l in enumerate(layers):
        inp = synth.layer_inputs(l, Bn, cfg["dtype"], key0, li, 0)
        out = gpu_layer(l, inp, cfg["dtype"], b.DP_EPI_STORE_NORM, bias_separate=1, sq=sq, sq_stride=L, sq_col=col)
        any_tc |= out["uses_tc"]
        dW, db = oracle_layer(l, inp)
        G.append(torch.from_numpy(out["G_w"]).cuda()); ref_groups.append(dW); col += 1
        if db is not None:
            G.append(torch.from_numpy(out["G_b"]).cuda()); ref_groups.append(db); col += 1
    acc = [torch.zeros(p, device="cuda") for p in P_l]
    norms = torch.empty(Bn, device="cuda")
    clip = torch.empty(Bn, device="cuda")
    ws = torch.empty(b.dp_clip_workspace_bytes(Bn, P_l), dtype=torch.uint8, device="cuda")
    b.check(b.dp_clip_accumulate(b.DP_CLIP_GLOBAL, Bn, G, P_l, sq, cfg["C"], acc, norms, clip, ws))
    ref_acc, ref_sq, ref_f = oracle.clipped_sum(ref_groups, cfg["C"], "global")
    np.testing.assert_allclose(norms.cpu().numpy(), np.sqrt(ref_sq.sum(1)), rtol=TOL_NORM)
    np.testing.assert_allclose(clip.cpu().numpy(), ref_f, rtol=TOL_NORM)
    tol = (TOL_ACC_BF16 if cfg["dtype"] == "bf16" else TOL_ACC_F32) if any_tc else TOL_FMA
    got_acc = np.concatenate([a.cpu().numpy() for a in acc])
    assert rel_l2(got_acc, np.concatenate(ref_acc)) <= tol
    off, outs = 0, []
    for a, p in zip(acc, P_l):
        b.check(b.dp_noise_average(a, p, off, cfg["sigma"], cfg["C"], Bn, cfg["seed"], cfg["step"], a))
        outs.append(a.cpu().numpy()); off += p
    ref_out = np.concatenate([oracle.noise_average(r, o, cfg["sigma"], cfg["C"], Bn, cfg["seed"], cfg["step"])
                              for r, o in zip(ref_acc, np.cumsum([0] + P_l[:-1]))])
    got = np.concatenate(outs)
    # the noise term dominates; compare the whole output and the signal part separately
    assert np.max(np.abs(got - ref_out)) <= 1e-5 * cfg["sigma"] * cfg["C"] / Bn + tol * np.max(np.abs(np.concatenate(ref_acc))) / Bn
    return ref_f


def test_single_dense_layer_workload():
    f = run_global_step(synth.single_dense())
    assert np.all(f < 1.0)                                   # norms are about 128, every example is clipped


@pytest.mark.parametrize("dtype", ["f32", "tf32"])
def test_small_cnn_workload_full_batch(dtype):
    """fp32 inputs as three split-tf32 products, and in the benchmark's mode: rounded to tf32, one product."""
    cfg = dict(synth.small_cnn()); cfg["dtype"] = dtype
    f = run_global_step(cfg)
    assert np.all(f < 1.0)


def test_small_cnn_with_unclipped_examples():
    cfg = dict(synth.small_cnn()); cfg["C"] = 1e9
    f = run_global_step(cfg, Bn=16)
    assert np.all(f == 1.0)


@pytest.mark.parametrize("li", range(8))
def test_resnet50_sweep_layer(li):
    """Every layer of the sweep at full size; the oracle runs on a subset of the examples."""
    b = B()
    cfg = synth.resnet50_sweep()
    layer = cfg["layers"][li]
    Bn = cfg["B"]
    inp = synth.layer_inputs(layer, Bn, "bf16", 2, li, 0)
    out = gpu_layer(layer, inp, "bf16", b.DP_EPI_STORE_NORM)
    out_n = gpu_layer(layer, inp, "bf16", b.DP_EPI_NORM_ONLY)
    tol = TOL_ACC_BF16 if out["uses_tc"] else TOL_FMA
    sample = [0, 13, Bn - 1]
    sub = {k: v[sample] for k, v in inp.items()}
    dW, _ = oracle_layer(layer, sub)
    for i, n in enumerate(sample):
        assert rel_l2(out["G_w"][n], dW[i]) <= tol
    np.testing.assert_allclose(out["sq"][sample, 0], oracle.sqnorm(dW), rtol=TOL_NORM)
    np.testing.assert_allclose(out_n["sq"][sample, 0], oracle.sqnorm(dW), rtol=TOL_NORM)
    # properties that hold for all examples: the stored gradient's own norm equals the reported one
    own = (out["G_w"].astype(np.float64) ** 2).sum(1)
    np.testing.assert_allclose(out["sq"][:, 0], own, rtol=TOL_NORM)
    np.testing.assert_allclose(out_n["sq"][:, 0], own, rtol=TOL_NORM)


def test_flat_gradient_workload_one_full_size_chunk():
    """P = 25,557,032, B = 64: one chunk at full size, norms computed by the library; the oracle checks all
    64 norms and factors and a sample of accumulator entries."""
    b = B()
    cfg = synth.resnet50_flat()
    P, Bn = cfg["P"], cfg["B"]
    Gh = synth.normal_f32((Bn, P), 3, 0, 0, scale=cfg["grad_std"])
    G = torch.from_numpy(Gh).cuda()
    acc = torch.zeros(P, device="cuda")
    norms = torch.empty(Bn, device="cuda"); clip = torch.empty(Bn, device="cuda")
    ws = torch.empty(b.dp_clip_workspace_bytes(Bn, [P]), dtype=torch.uint8, device="cuda")
    b.check(b.dp_clip_accumulate(b.DP_CLIP_GLOBAL, Bn, [G], [P], None, cfg["C"], [acc], norms, clip, ws))
    s = oracle.sqnorm(Gh)
    f = oracle.clip_factor(s, cfg["C"])
    np.testing.assert_allclose(norms.cpu().numpy(), np.sqrt(s), rtol=TOL_NORM)
    np.testing.assert_allclose(clip.cpu().numpy(), f, rtol=TOL_NORM)
    np.testing.assert_allclose(np.sqrt(s), 1e-3 * math.sqrt(P), rtol=1e-3)        # closed form of the recipe
    idx = np.concatenate([np.arange(0, 4096), np.arange(P - 4096, P), np.random.default_rng(1).integers(0, P, 20000)])
    ref = (Gh[:, idx].astype(np.float64) * f[:, None]).sum(0)
    assert rel_l2(acc.cpu().numpy()[idx], ref) <= TOL_FMA


def _per_layer_reduced(layers, Bn, Gn, C, sigma, key0):
    """Per-layer fused path over a list of layers: CLIP_ACCUM per layer and chunk, then noise_average."""
    b = B()
    L = sum(1 + (1 if l.n_bias else 0) for l in layers)
    C_l = C / math.sqrt(L)
    accs = [(torch.zeros(l.n_weight, device="cuda"), torch.zeros(l.n_bias, device="cuda") if l.n_bias else None) for l in layers]
    ref = [(np.zeros(l.n_weight), np.zeros(l.n_bias) if l.n_bias else None) for l in layers]
    any_tc = False
    for c in range(Gn):
        for li, l in enumerate(layers):
            inp = synth.layer_inputs(l, Bn, "bf16", key0, li, c)
            # scale so that norms straddle the per-layer threshold
            s = np.logspace(-0.7, 0.7, Bn).astype(np.float32) * np.float32(C_l) / np.float32(math.sqrt(max(l.flops() / 2, 1.0)))
            dY = inp["dY"] * s.reshape((Bn,) + (1,) * (inp["dY"].ndim - 1))
            inp["dY_bits"], inp["dY"] = synth.round_to_bf16(dY)
            out = gpu_layer(l, inp, "bf16", b.DP_EPI_CLIP_ACCUM, bias_separate=1, C_l=C_l, acc_w=accs[li][0], acc_b=accs[li][1])
            any_tc |= out["uses_tc"]
            dW, db = oracle_layer(l, inp)
            fw = oracle.clip_factor(oracle.sqnorm(dW), C_l)
            np.testing.assert_allclose(out["clip"][:, 0], fw, rtol=TOL_NORM)
            ref[li][0][:] += np.einsum("n,np->p", fw, dW)
            if db is not None:
                fb = oracle.clip_factor(oracle.sqnorm(db), C_l)
                np.testing.assert_allclose(out["clip"][:, 1], fb, rtol=TOL_NORM)
                ref[li][1][:] += np.einsum("n,np->p", fb, db)
    tol = TOL_ACC_BF16 if any_tc else TOL_FMA
    off = 0
    for (aw, ab), (rw, rb) in zip(accs, ref):
        for a, r in ((aw, rw), (ab, rb)):
            if a is None:
                continue
            assert rel_l2(a.cpu().numpy(), r) <= tol
            b.check(b.dp_noise_average(a, a.numel(), off, sigma, C, Bn * Gn, 0, 0, a))
            want = oracle.noise_average(r, off, sigma, C, Bn * Gn, 0, 0)
            assert np.max(np.abs(a.cpu().numpy() - want)) <= (1e-5 * sigma * C + tol * np.max(np.abs(r))) / (Bn * Gn)
            off += a.numel()


def test_per_layer_fused_path_on_a_reduced_resnet_block():
    """Per-layer clipping fused into the weight-gradient call: one bottleneck's worth of layer kinds at
    reduced spatial size, two chunks."""
    layers = [synth.conv(64, 64, 1, 1, 0, 14, name="c1"), synth.norm(64, 14, "gn1"),
              synth.conv(64, 64, 3, 1, 1, 14, name="c2"), synth.norm(64, 14, "gn2"),
              synth.conv(64, 256, 1, 1, 0, 14, name="c3"), synth.norm(256, 14, "gn3"),
              synth.conv(64, 128, 3, 2, 1, 14, name="c2s"), synth.conv(64, 256, 1, 2, 0, 14, name="ds"),
              synth.dense(256, 100, bias=True, name="fc")]
    _per_layer_reduced(layers, 6, 2, 1.0, 1.0, 4)
