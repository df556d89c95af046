"""GPU parity of the two further clipping rules of the paper: groups of tensors clipped to C/sqrt(M) (section 3.5,
pipeline stages) and micro-batch clipping (the option of the paper's first table)."""
import math
import numpy as np
import pytest
import torch

import oracle
from paper_2109_12191_b200 import synth
from gpu_util import B, dev, rel_l2, TOL_NORM, TOL_FMA

pytestmark = pytest.mark.gpu


def _spread(Bn, sizes, seed, lo=-1.5, hi=1.0):
    s = np.logspace(lo, hi, Bn).astype(np.float32)
    return [synth.normal_f32((Bn, p), 922, seed, l) * s[:, None] / np.float32(math.sqrt(sum(sizes))) for l, p in enumerate(sizes)]


def _ws(b, Bn, P_l):
    wsb = b.dp_clip_workspace_bytes(Bn, P_l)
    ws = torch.empty(wsb + 256, dtype=torch.uint8, device="cuda")
    ws.fill_(0xCD)
    return ws, wsb, ws[wsb:].clone()


def _run_grouped(groups, group_of, C, give_norms=False, acc0=None):
    b = B()
    L, Bn, M = len(groups), groups[0].shape[0], max(group_of) + 1
    P_l = [g.shape[1] for g in groups]
    G = [dev(g) for g in groups]
    acc = [dev(a) for a in acc0] if acc0 is not None else [torch.zeros(p, device="cuda") for p in P_l]
    norms = torch.full((Bn, M), float("nan"), device="cuda")
    clip = torch.full((Bn, M), float("nan"), device="cuda")
    sq = dev(np.stack([oracle.sqnorm(g) for g in groups], axis=1).astype(np.float32)) if give_norms else None
    ws, wsb, guard = _ws(b, Bn, P_l)
    b.check(b.dp_clip_accumulate_grouped(Bn, M, group_of, G, P_l, sq, C, acc, norms, clip, ws, wsb))
    torch.cuda.synchronize()
    assert torch.equal(ws[wsb:], guard)
    return [a.cpu().numpy() for a in acc], norms.cpu().numpy(), clip.cpu().numpy()


@pytest.mark.parametrize("give_norms", [False, True])
@pytest.mark.parametrize("sizes,group_of", [([640, 33, 4096, 10, 260], [1, 0, 1, 0, 2]), ([512, 7], [0, 0]),
                                            ([64, 64, 64], [2, 1, 0])])
def test_grouped_matches_the_oracle(sizes, group_of, give_norms):
    groups = _spread(12, sizes, len(sizes))
    acc, norms, clip = _run_grouped(groups, group_of, 0.4, give_norms)
    ref, sq, f = oracle.clipped_sum_grouped(groups, group_of, 0.4)
    np.testing.assert_allclose(norms, np.sqrt(sq), rtol=TOL_NORM)
    np.testing.assert_allclose(clip, f, rtol=TOL_NORM)
    assert (f == 1.0).any() and (f < 1.0).any()
    for a, r in zip(acc, ref):
        assert rel_l2(a, r) <= TOL_FMA


def test_resnet50_tensors_in_pipeline_stages():
    """The 161 tensors of ResNet-50 (GroupNorm) cut into 4 pipeline stages at the residual stages, weights shrunk."""
    layers = synth.resnet50_gn_layers()
    sizes, group_of = [], []
    for l in layers:
        stage = 3 if l.name.startswith("fc") else (int(l.name[1]) if l.name.startswith("s") and l.name[1].isdigit() else 0)
        for p in [min(l.n_weight, 2048 + l.n_weight % 13)] + ([l.n_bias] if l.n_bias else []):
            sizes.append(p)
            group_of.append(stage)
    assert len(sizes) == synth.RESNET50_GN_TENSORS and sorted(set(group_of)) == [0, 1, 2, 3]
    groups = _spread(4, sizes, 31)
    acc, norms, clip = _run_grouped(groups, group_of, 1.0)
    ref, sq, f = oracle.clipped_sum_grouped(groups, group_of, 1.0)
    np.testing.assert_allclose(clip, f, rtol=TOL_NORM)
    for a, r in zip(acc, ref):
        assert rel_l2(a, r) <= TOL_FMA
    # section 3.5: the clipped stages together respect the whole-gradient bound
    assert np.all(np.sqrt(((norms * clip) ** 2).sum(1)) <= 1.0 * (1 + 1e-5))


def test_grouped_limits_reduce_to_the_two_modes():
    b = B()
    sizes = [300, 20, 1000]
    groups = _spread(7, sizes, 32)
    acc_g, _, clip_g = _run_grouped(groups, [0, 1, 2], 0.3)
    ref, _, f = oracle.clipped_sum(groups, 0.3, "per_layer")
    np.testing.assert_allclose(clip_g, f, rtol=TOL_NORM)
    acc_1, _, clip_1 = _run_grouped(groups, [0, 0, 0], 0.3)
    ref1, _, f1 = oracle.clipped_sum(groups, 0.3, "global")
    np.testing.assert_allclose(clip_1[:, 0], f1, rtol=TOL_NORM)
    for a, r in zip(acc_1, ref1):
        assert rel_l2(a, r) <= TOL_FMA


def _run_micro(groups, C, micro, acc0=None):
    b = B()
    L, Bn = len(groups), groups[0].shape[0]
    P_l = [g.shape[1] for g in groups]
    G = [dev(g) for g in groups]
    acc = [dev(a) for a in acc0] if acc0 is not None else [torch.zeros(p, device="cuda") for p in P_l]
    norms = torch.full((Bn // micro,), float("nan"), device="cuda")
    clip = torch.full((Bn // micro,), float("nan"), device="cuda")
    ws, wsb, guard = _ws(b, Bn, P_l)
    b.check(b.dp_clip_accumulate_micro(Bn, micro, G, P_l, C, acc, norms, clip, ws, wsb))
    torch.cuda.synchronize()
    assert torch.equal(ws[wsb:], guard)
    return [a.cpu().numpy() for a in acc], norms.cpu().numpy(), clip.cpu().numpy()


@pytest.mark.parametrize("micro", [1, 2, 4, 3])
@pytest.mark.parametrize("sizes", [[4096], [1001, 7, 12288 + 4], [8192 * 2 + 5, 64]])
def test_micro_batches_match_the_oracle(sizes, micro):
    Bn = 24
    groups = _spread(Bn, sizes, 40 + micro, lo=-1.0, hi=1.0)
    C = 0.5 / math.sqrt(micro)
    acc, norms, clip = _run_micro(groups, C, micro)
    ref, sq, f = oracle.clipped_sum_micro(groups, C, micro)
    np.testing.assert_allclose(norms, np.sqrt(sq), rtol=TOL_NORM)
    np.testing.assert_allclose(clip, f, rtol=TOL_NORM)
    assert (f == 1.0).any() and (f < 1.0).any()
    for a, r in zip(acc, ref):
        assert rel_l2(a, r) <= TOL_FMA
    assert np.all(norms * clip <= C * (1 + 1e-5))


def test_micro_batch_of_the_whole_chunk_and_chunk_accumulation():
    sizes, C = [2052, 10], 0.02
    acc, ref = None, None
    for c in range(3):
        g = _spread(8, sizes, 50 + c)
        acc, _, _ = _run_micro(g, C, 8, acc0=acc)
        ref, _, _ = oracle.clipped_sum_micro(g, C, 8, ref)
    for a, r in zip(acc, ref):
        assert rel_l2(a, r) <= TOL_FMA


def test_variant_argument_errors():
    b = B()
    g = [torch.zeros((4, 8), device="cuda"), torch.zeros((4, 4), device="cuda")]
    a = [torch.zeros(8, device="cuda"), torch.zeros(4, device="cuda")]
    ws = torch.empty(8192, dtype=torch.uint8, device="cuda")
    assert b.dp_clip_accumulate_grouped(4, 2, [0, 1], g, [8, 4], None, 1.0, a, None, None, ws) == b.DP_OK
    assert b.dp_clip_accumulate_grouped(4, 2, [0, 0], g, [8, 4], None, 1.0, a, None, None, ws) == b.DP_ERR_INVALID_ARG   # empty group
    assert b.dp_clip_accumulate_grouped(4, 2, [0, 2], g, [8, 4], None, 1.0, a, None, None, ws) == b.DP_ERR_INVALID_ARG
    assert b.dp_clip_accumulate_grouped(4, 3, [0, 1], g, [8, 4], None, 1.0, a, None, None, ws) == b.DP_ERR_INVALID_ARG   # M > L
    assert b.dp_clip_accumulate_micro(4, 2, g, [8, 4], 1.0, a, None, None, ws) == b.DP_OK
    assert b.dp_clip_accumulate_micro(4, 3, g, [8, 4], 1.0, a, None, None, ws) == b.DP_ERR_INVALID_ARG                 # 3 does not divide 4
    assert b.dp_clip_accumulate_micro(4, 0, g, [8, 4], 1.0, a, None, None, ws) == b.DP_ERR_INVALID_ARG
    torch.cuda.synchronize()
