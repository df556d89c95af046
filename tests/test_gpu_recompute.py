"""Whole-model clipping without materialising every layer: norms from a NORM_ONLY pass, factors from the norm table
(dp_clip_factors), clipped sums either over memory (dp_scale_accumulate) or by a second pass over the layer's inputs
(dp_per_example_wgrad_scaled).  Every piece and the assembled step are checked against the oracle."""
import math
import numpy as np
import pytest
import torch

import oracle
from paper_2109_12191_b200 import synth
from paper_2109_12191_b200.step import GlobalClipStep
from gpu_util import B, dev, dev_inputs, make_desc, oracle_layer, rel_l2, scaled_inputs, TOL_NORM, TOL_FMA, TOL_ACC_F32, TOL_ACC_BF16

pytestmark = pytest.mark.gpu

CASES = [
    ("f32", synth.conv(32, 64, 3, 2, 1, 16, True, "tf32 conv"), 0),
    ("bf16", synth.conv(64, 128, 3, 1, 1, 14, True, "bf16 conv"), 0),
    ("bf16", synth.conv(64, 64, 1, 1, 0, 9, False, "1x1 no bias"), 0),
    ("f32", synth.conv(3, 16, 3, 1, 1, 12, True, "cuda-core conv"), 1),
    ("f32", synth.dense(512, 10, True, "dense"), 0),
    ("bf16", synth.dense(256, 24, False, "dense bf16"), 0),
    ("bf16", synth.norm(64, 10, "norm"), 0),
]


@pytest.mark.parametrize("dtype,layer,impl", CASES, ids=[c[1].name for c in CASES])
def test_scaled_wgrad_matches_the_oracle(dtype, layer, impl):
    b = B()
    Bn = 7
    inp = scaled_inputs(layer, Bn, dtype, 970, len(layer.name))
    dW, db = oracle_layer(layer, inp)
    rng = np.random.default_rng(5)
    fw = rng.uniform(0.05, 1.0, Bn).astype(np.float32)
    fb = rng.uniform(0.05, 1.0, Bn).astype(np.float32)
    X, dY = dev_inputs(inp, dtype)
    d = make_desc(layer, Bn, dtype, impl, 1)
    ws_bytes = b.dp_workspace_bytes(d, b.DP_EPI_CLIP_ACCUM)
    tol = TOL_FMA if (impl == 1 or layer.kind != "conv") else (TOL_ACC_BF16 if dtype == "bf16" else TOL_ACC_F32)
    for separate in (False, True):
        ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
        ws.fill_(0xAB)
        guard = ws[ws_bytes:].clone()
        b.check(b.dp_workspace_init(ws, ws_bytes))
        table = torch.full((Bn, 3), float("nan"), device="cuda")          # factors at a stride, as in a [B, L] table
        table[:, 0] = dev(fw)
        table[:, 1] = dev(fb)
        acc_w0 = np.linspace(-1, 1, layer.n_weight).astype(np.float32)   # read-modify-write: start from something
        acc_w = dev(acc_w0)
        acc_b = torch.zeros(layer.n_bias, device="cuda") if layer.n_bias else None
        f_b = (table.data_ptr() + 4) if separate else None
        b.check(b.dp_per_example_wgrad_scaled(d, X, dY, table, f_b, 3, acc_w, acc_b, ws, ws_bytes))
        b.check(b.dp_wgrad_check(ws))
        torch.cuda.synchronize()
        assert torch.equal(ws[ws_bytes:], guard)
        want_w = acc_w0.astype(np.float64) + np.einsum("n,np->p", fw.astype(np.float64), dW)
        assert rel_l2(acc_w.cpu().numpy() - acc_w0, want_w - acc_w0) <= tol
        if db is not None:
            want_b = np.einsum("n,np->p", (fb if separate else fw).astype(np.float64), db)
            assert rel_l2(acc_b.cpu().numpy(), want_b) <= tol


def test_factors_and_scale_accumulate_alone():
    b = B()
    Bn, sizes, C = 10, [640, 33, 4100], 0.4
    s = np.logspace(-1.5, 1.0, Bn).astype(np.float32)
    groups = [synth.normal_f32((Bn, p), 923, 1, l) * s[:, None] / np.float32(70) for l, p in enumerate(sizes)]
    sq = np.stack([oracle.sqnorm(g) for g in groups], axis=1)
    for mode, per_tensor in (("global", 0), ("per_layer", 1)):
        ref, _, f = oracle.clipped_sum(groups, C, mode)
        shape = (Bn, len(sizes)) if per_tensor else (Bn,)
        fac = torch.full(shape, float("nan"), device="cuda")
        norms = torch.full(shape, float("nan"), device="cuda")
        b.check(b.dp_clip_factors(b.DP_CLIP_PER_LAYER if per_tensor else b.DP_CLIP_GLOBAL, Bn, len(sizes), dev(sq.astype(np.float32)),
                                  C, norms, fac))
        np.testing.assert_allclose(fac.cpu().numpy(), f, rtol=TOL_NORM)
        np.testing.assert_allclose(norms.cpu().numpy(), np.sqrt(sq) if per_tensor else np.sqrt(sq.sum(1)), rtol=TOL_NORM)
        assert (f == 1.0).any() and (f < 1.0).any()
        acc = [torch.zeros(p, device="cuda") for p in sizes]
        b.check(b.dp_scale_accumulate(Bn, [dev(g) for g in groups], sizes, fac, per_tensor, acc))
        torch.cuda.synchronize()
        for a, r in zip(acc, ref):
            assert rel_l2(a.cpu().numpy(), r) <= TOL_FMA


@pytest.mark.parametrize("recompute,lanes", [("auto", 1), ("auto", 3), ([0, 1, 2], 2)])
def test_step_with_recomputed_layers_matches_the_oracle(recompute, lanes):
    """A small CNN whose classifier's gradients outweigh its inputs: 'auto' recomputes that dense layer; the explicit list
    recomputes every layer.  Two chunks, noise, average, against the oracle's whole step."""
    layers = [synth.conv(3, 32, 3, 1, 1, 16, True, "c1"), synth.conv(32, 128, 3, 2, 1, 16, True, "c2"),
              synth.dense(128 * 64, 10, True, "fc")]
    Bn, C, sigma = 12, 0.6, 0.9
    st = GlobalClipStep(layers, Bn, "f32", C, sigma, lanes=lanes, recompute=recompute)
    if recompute == "auto":
        assert st.recompute == {2}
    st.begin()
    chunks = []
    for c in range(2):
        ins = [scaled_inputs(l, Bn, "f32", 971, li, c) for li, l in enumerate(layers)]
        for i in ins:
            i["dY"] = i["dY"] * np.float32(0.01)
        st.chunk([dev_inputs(i, "f32") for i in ins])
        groups = []
        for l, i in zip(layers, ins):
            dW, db = oracle_layer(l, i)
            groups += [dW, db]
        chunks.append(groups)
    torch.cuda.synchronize()
    st.check()
    got = st.finish(seed=4, step=2).cpu().numpy()
    ref, norms, factors = oracle.privatise(chunks, C, sigma, "global", 4, 2)
    ref = np.concatenate(ref)
    assert rel_l2(got, ref) <= TOL_ACC_F32
    np.testing.assert_allclose(st.clip.cpu().numpy(), factors[-1], rtol=TOL_NORM)
    f = factors[-1]
    assert (f == 1.0).any() and (f < 1.0).any()


def test_argument_errors():
    b = B()
    layer = synth.dense(16, 4, True, "d")
    d = make_desc(layer, 2, "f32", 0, 1)
    t = lambda *shape: torch.zeros(shape, device="cuda")
    ws = torch.empty(b.dp_workspace_bytes(d, b.DP_EPI_CLIP_ACCUM), dtype=torch.uint8, device="cuda")
    b.check(b.dp_workspace_init(ws))
    ok = dict(desc=d, X=t(2, 16), dY=t(2, 4), factor_w=t(2), factor_b=None, factor_stride=1, acc_w=t(64), acc_b=t(4), workspace=ws)
    assert b.dp_per_example_wgrad_scaled(**ok) == b.DP_OK
    for bad in (dict(factor_w=None), dict(factor_stride=0), dict(acc_w=None), dict(acc_b=None), dict(X=None)):
        assert b.dp_per_example_wgrad_scaled(**{**ok, **bad}) == b.DP_ERR_INVALID_ARG, bad
    assert b.dp_per_example_wgrad_scaled(**{**ok, "workspace": None}) == b.DP_ERR_WORKSPACE
    assert b.dp_clip_factors(0, 2, 1, None, 1.0, None, t(2)) == b.DP_ERR_INVALID_ARG
    assert b.dp_clip_factors(0, 2, 1, t(2, 1), 0.0, None, t(2)) == b.DP_ERR_INVALID_ARG
    assert b.dp_scale_accumulate(2, [t(2, 8)], [8], None, 0, [t(8)]) == b.DP_ERR_INVALID_ARG
    assert b.dp_scale_accumulate(2, [t(2, 8)], [8], t(2), 2, [t(8)]) == b.DP_ERR_INVALID_ARG
    torch.cuda.synchronize()
