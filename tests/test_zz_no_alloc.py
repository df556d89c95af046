"""dp_clip_accumulate_static: the clip-accumulate entry point for callers that cannot allocate.

Some users of this library run where device allocation is off limits -- inside another framework's
memory pool that already owns the GPU, in callbacks that must not trigger cudaMalloc's device-wide
synchronisation, or in services that reserve all memory at start-up -- so they cannot provide the
workspace dp_clip_accumulate asks for.  This entry point works in a fixed array inside the library.
The test drives it through the C ABI twice in a row (the array keeps the first call's leftovers) and
holds it to the results of the workspace-taking entry point and of the CPU oracle.  The file sorts last so that a run that
stops at the first failure has already executed every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2109_12191_b200 import synth
from gpu_util import B, dev, rel_l2, TOL_NORM, TOL_FMA

pytestmark = pytest.mark.gpu


def _inputs(Bn, sizes, seed):
    s = np.logspace(-1.0, 0.6, Bn).astype(np.float32)
    return [synth.normal_f32((Bn, p), 990, seed, l) * s[:, None] / np.float32(np.sqrt(sum(sizes))) for l, p in enumerate(sizes)]


def _both(mode_name, groups, C):
    b = B()
    mode = b.DP_CLIP_PER_LAYER if mode_name == "per_layer" else b.DP_CLIP_GLOBAL
    Bn, L = groups[0].shape[0], len(groups)
    P_l = [g.shape[1] for g in groups]
    G = [dev(g) for g in groups]
    shape = (Bn, L) if mode_name == "per_layer" else (Bn,)
    res = []
    for static in (False, True):
        acc = [torch.zeros(p, device="cuda") for p in P_l]
        norms = torch.full(shape, float("nan"), device="cuda")
        clip = torch.full(shape, float("nan"), device="cuda")
        if static:
            b.check(b.dp_clip_accumulate_static(mode, Bn, G, P_l, None, C, acc, norms, clip), "dp_clip_accumulate_static")
        else:
            ws = torch.empty(b.dp_clip_workspace_bytes(Bn, P_l), dtype=torch.uint8, device="cuda")
            b.check(b.dp_clip_accumulate(mode, Bn, G, P_l, None, C, acc, norms, clip, ws), "dp_clip_accumulate")
        torch.cuda.synchronize()
        res.append(([a.cpu().numpy() for a in acc], norms.cpu().numpy(), clip.cpu().numpy()))
    return res


def test_static_scratch_variant_matches_the_workspace_variant_on_two_calls_in_a_row():
    b = B()
    assert b.dp_clip_static_scratch_bytes() == 2 << 20
    calls = [("global", _inputs(24, [70_001, 513, 8192], 1), 0.4),        # first call leaves its partials behind
             ("per_layer", _inputs(7, [300, 40_000], 2), 0.3)]            # second call: other shapes, other mode
    for mode_name, groups, C in calls:
        (acc_ws, norms_ws, clip_ws), (acc_st, norms_st, clip_st) = _both(mode_name, groups, C)
        np.testing.assert_allclose(norms_st, norms_ws, rtol=TOL_NORM)
        np.testing.assert_allclose(clip_st, clip_ws, rtol=TOL_NORM)
        assert (clip_ws == 1.0).any() and (clip_ws < 1.0).any()
        for a, r in zip(acc_st, acc_ws):
            assert rel_l2(a, r) <= TOL_FMA
        ref_acc, ref_sq, ref_f = oracle.clipped_sum(groups, C, mode_name)
        ref_norm = np.sqrt(ref_sq) if mode_name == "per_layer" else np.sqrt(ref_sq.sum(1))
        np.testing.assert_allclose(norms_st, ref_norm, rtol=TOL_NORM)
        np.testing.assert_allclose(clip_st, ref_f, rtol=TOL_NORM)
        for a, r in zip(acc_st, ref_acc):
            assert rel_l2(a, r) <= TOL_FMA


def test_static_scratch_variant_refuses_problems_beyond_its_array():
    b = B()
    Bn, P = 64, 25_557_032                     # needs about 0.8 MB: fits
    assert b.dp_clip_workspace_bytes(Bn, [P]) <= b.dp_clip_static_scratch_bytes()
    Bn, P = 256, 25_557_032                    # about 3.2 MB: does not fit
    assert b.dp_clip_workspace_bytes(Bn, [P]) > b.dp_clip_static_scratch_bytes()
    fake = 4096                                # never dereferenced: the size check comes before any launch
    st = b.dp_clip_accumulate_static(b.DP_CLIP_GLOBAL, Bn, [fake], [P], None, 1.0, [fake], None, None)
    assert st == b.DP_ERR_WORKSPACE
    assert "2 MiB" in b.dp_last_cuda_error()
