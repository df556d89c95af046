"""GPU parity of dp_clip_accumulate against the oracle's clipped sum (global and per-layer)."""
import math
import numpy as np
import pytest
import torch

import oracle
from paper_2109_12191_b200 import synth
from gpu_util import B, dev, rel_l2, TOL_NORM, TOL_FMA

pytestmark = pytest.mark.gpu


def _run(mode, groups, C, give_norms=False, acc0=None, want_out=True):
    b = B()
    L, Bn = len(groups), groups[0].shape[0]
    P_l = [int(np.prod(g.shape[1:])) for g in groups]
    G = [dev(g.reshape(Bn, -1)) for g in groups]
    acc = [dev(a) for a in acc0] if acc0 is not None else [torch.zeros(p, device="cuda") for p in P_l]
    per_layer = mode == "per_layer"
    shape = (Bn, L) if per_layer else (Bn,)
    norms = torch.full(shape, float("nan"), device="cuda") if want_out else None
    clip = torch.full(shape, float("nan"), device="cuda") if want_out else None
    sq = None
    if give_norms:
        sq = dev(np.stack([oracle.sqnorm(g) for g in groups], axis=1).astype(np.float32))
    wsb = b.dp_clip_workspace_bytes(Bn, P_l)
    ws = torch.empty(wsb + 256, dtype=torch.uint8, device="cuda")
    ws.fill_(0xCD)
    guard = ws[wsb:].clone()
    b.check(b.dp_clip_accumulate(b.DP_CLIP_PER_LAYER if per_layer else b.DP_CLIP_GLOBAL, Bn, G, P_l, sq, C, acc, norms,
                                 clip, ws, wsb))
    torch.cuda.synchronize()
    assert torch.equal(ws[wsb:], guard)
    return [a.cpu().numpy() for a in acc], (norms.cpu().numpy() if want_out else None), (clip.cpu().numpy() if want_out else None)


def _check(mode, groups, C, **kw):
    acc, norms, clip = _run(mode, groups, C, **kw)
    ref_acc, ref_sq, ref_f = oracle.clipped_sum(groups, C, mode)
    ref_norm = np.sqrt(ref_sq.sum(1)) if mode == "global" else np.sqrt(ref_sq)
    np.testing.assert_allclose(norms, ref_norm, rtol=TOL_NORM)
    np.testing.assert_allclose(clip, ref_f, rtol=TOL_NORM)
    for a, r in zip(acc, ref_acc):
        assert rel_l2(a, r) <= TOL_FMA
    return ref_f


def _spread(Bn, sizes, seed, lo=-1.5, hi=1.0):
    s = np.logspace(lo, hi, Bn).astype(np.float32)
    return [synth.normal_f32((Bn, p), 920, seed, l) * s[:, None] / np.float32(math.sqrt(sum(sizes))) for l, p in enumerate(sizes)]


@pytest.mark.parametrize("give_norms", [False, True])
@pytest.mark.parametrize("sizes", [[4096], [1000, 24], [1001, 7, 12288 + 4], [8192 * 3 + 5], [3], [1024, 1024, 2048]])
def test_global_mode(sizes, give_norms):
    groups = _spread(16, sizes, len(sizes))
    f = _check("global", groups, 0.3, give_norms=give_norms)
    assert (f == 1.0).any() and (f < 1.0).any()              # both branches exercised


@pytest.mark.parametrize("give_norms", [False, True])
def test_per_layer_mode(give_norms):
    sizes = [640, 33, 4096, 10]
    groups = _spread(12, sizes, 7)
    f = _check("per_layer", groups, 0.4, give_norms=give_norms)
    assert (f == 1.0).any() and (f < 1.0).any()


def test_more_tensors_than_one_launch_table_holds():
    sizes = [64 + 3 * l for l in range(97)]                  # 97 tensors, odd sizes: several tables, scalar path
    groups = _spread(5, sizes, 8)
    _check("global", groups, 0.2)
    _check("per_layer", groups, 0.2)


def test_161_tensors_like_resnet50():
    layers = synth.resnet50_gn_layers()
    sizes = []
    for l in layers:
        sizes.append(min(l.n_weight, 4096 + l.n_weight % 13))   # shrunk weights, true tensor count
        if l.n_bias:
            sizes.append(l.n_bias)
    assert len(sizes) == synth.RESNET50_GN_TENSORS
    groups = _spread(4, sizes, 9)
    _check("per_layer", groups, 1.0)


def test_batch_larger_than_the_factor_tile_and_single_example():
    _check("global", _spread(300, [512, 5], 10, lo=-1, hi=0.5), 0.5)
    _check("global", _spread(1, [257], 11), 1e-3)


def test_infinite_C_never_clips_and_zero_gradient_is_safe():
    groups = _spread(6, [300, 20], 12)
    groups[0][2] = 0.0
    groups[1][2] = 0.0
    acc, norms, clip = _run("global", groups, float("inf"))
    assert np.all(clip == 1.0) and norms[2] == 0.0
    ref = [g.astype(np.float64).sum(0) for g in groups]
    for a, r in zip(acc, ref):
        assert rel_l2(a, r) <= TOL_FMA
    acc, norms, clip = _run("per_layer", groups, 0.01)
    assert np.all(clip[2] == 1.0) and np.all(np.isfinite(clip))


def test_accumulates_over_chunks_and_is_reproducible():
    sizes, C = [2048 + 4, 17], 0.25
    chunks = [_spread(8, sizes, 30 + c) for c in range(4)]
    acc = [np.zeros(p, dtype=np.float32) for p in sizes]
    for ch in chunks:
        acc, _, _ = _run("global", ch, C, acc0=acc)
    ref = None
    for ch in chunks:
        ref, _, _ = oracle.clipped_sum(ch, C, "global", ref)
    for a, r in zip(acc, ref):
        assert rel_l2(a, r) <= TOL_FMA
    again = [np.zeros(p, dtype=np.float32) for p in sizes]
    for ch in chunks:
        again, _, _ = _run("global", ch, C, acc0=again)
    for a, a2 in zip(acc, again):
        np.testing.assert_array_equal(a, a2)                   # fixed reduction order: same bits every run


def test_clipped_examples_respect_the_bound_on_device_results():
    """Section 2 invariant on the GPU's own outputs: factor * norm <= C."""
    groups = _spread(32, [5000, 100], 13)
    _, norms, clip = _run("global", groups, 0.1)
    assert np.all(norms * clip <= 0.1 * (1 + 1e-5))


def test_flat_gradient_workload_shape_reduced():
    """The flattened-gradient workload with P reduced (odd size, several norm chunks), all 16 chunks."""
    P, Bn, Gn = 300_007, 64, 16
    acc = [np.zeros(P, dtype=np.float32)]
    ref = None
    for c in range(Gn):
        g = [synth.normal_f32((Bn, P), 3, 0, c, scale=1e-3)]
        acc, norms, clip = _run("global", g, 0.2, acc0=acc)
        ref, sq, f = oracle.clipped_sum(g, 0.2, "global", ref)
        np.testing.assert_allclose(norms, np.sqrt(sq[:, 0]), rtol=TOL_NORM)
        np.testing.assert_allclose(clip, f, rtol=TOL_NORM)
    assert rel_l2(acc[0], ref[0]) <= TOL_FMA
