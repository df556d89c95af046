"""GPU parity of the per-example noise form (paper section 2, the block after the equation for g_t): each clipped
example receives its own draw of variance sigma^2 C^2 / |B| before the sum.  The stream is deterministic, so parity
with the oracle is element by element; that the form is equal in distribution to one draw on the sum is checked on
the device's own output."""
import math
import numpy as np
import pytest
import torch

import oracle
from paper_2109_12191_b200 import synth
from gpu_util import B, dev, rel_l2, TOL_NORM

pytestmark = pytest.mark.gpu

TOL_Z = 1e-5   # |z_gpu - z_oracle|, fp32 logf / sincospif against float64


def _offsets(sizes, first=0):
    out, o = [], first
    for p in sizes:
        out.append(o)
        o += p
    return out


def _run(mode, groups, offs, C, sigma, total, seed, step, example0, acc0=None, give_norms=False):
    b = B()
    L, Bn = len(groups), groups[0].shape[0]
    P_l = [int(np.prod(g.shape[1:])) for g in groups]
    G = [dev(g.reshape(Bn, -1)) for g in groups]
    acc = [dev(a) for a in acc0] if acc0 is not None else [torch.zeros(p, device="cuda") for p in P_l]
    per_layer = mode == "per_layer"
    shape = (Bn, L) if per_layer else (Bn,)
    norms = torch.full(shape, float("nan"), device="cuda")
    clip = torch.full(shape, float("nan"), device="cuda")
    sq = dev(np.stack([oracle.sqnorm(g) for g in groups], axis=1).astype(np.float32)) if give_norms else None
    wsb = b.dp_clip_workspace_bytes(Bn, P_l)
    ws = torch.empty(wsb + 256, dtype=torch.uint8, device="cuda")
    ws.fill_(0xCD)
    guard = ws[wsb:].clone()
    b.check(b.dp_clip_accumulate_noised(b.DP_CLIP_PER_LAYER if per_layer else b.DP_CLIP_GLOBAL, Bn, G, P_l, offs, sq, C,
                                        sigma, total, seed, step, example0, acc, norms, clip, ws, wsb))
    torch.cuda.synchronize()
    assert torch.equal(ws[wsb:], guard)
    return [a.cpu().numpy() for a in acc], norms.cpu().numpy(), clip.cpu().numpy()


def _oracle(mode, groups, offs, C, sigma, total, seed, step, example0, acc0=None):
    _, sq, f = oracle.clipped_sum(groups, C, mode)
    sd = sigma * C / math.sqrt(total) if sigma > 0 else 0.0
    out = []
    for l, g in enumerate(groups):
        a = np.zeros(g.shape[1], dtype=np.float64) if acc0 is None else acc0[l].astype(np.float64).copy()
        fl = f[:, l] if mode == "per_layer" else f
        oracle.clip_accumulate_noised(g, fl, a, sd, seed, step, example0, offs[l])
        out.append(a)
    return out, sq, f


def _spread(Bn, sizes, seed, lo=-1.5, hi=1.0):
    s = np.logspace(lo, hi, Bn).astype(np.float32)
    return [synth.normal_f32((Bn, p), 921, seed, l) * s[:, None] / np.float32(math.sqrt(sum(sizes))) for l, p in enumerate(sizes)]


def test_example_stream_matches_the_oracle():
    b = B()
    for example, first, count in [(0, 0, 4099), (5, 3, 1001), (2**31 - 1, 2**33 + 1, 515)]:
        z = torch.empty(count, device="cuda")
        b.check(b.dp_debug_example_noise_z(z, count, first, example, 11, 7))
        ref = oracle.example_noise_z(11, 7, example, first, count)
        assert np.max(np.abs(z.cpu().numpy() - ref)) <= TOL_Z


def test_example_stream_differs_from_the_parameter_stream_and_between_examples():
    b = B()
    n = 1 << 16
    zp, z0, z1 = (torch.empty(n, device="cuda") for _ in range(3))
    b.check(b.dp_debug_noise_z(zp, n, 0, 3, 1))
    b.check(b.dp_debug_example_noise_z(z0, n, 0, 0, 3, 1))
    b.check(b.dp_debug_example_noise_z(z1, n, 0, 1, 3, 1))
    zp, z0, z1 = (t.cpu().numpy().astype(np.float64) for t in (zp, z0, z1))
    for a, c in [(zp, z0), (z0, z1), (zp, z1)]:
        assert abs(np.corrcoef(a, c)[0, 1]) < 5 / math.sqrt(n)


@pytest.mark.parametrize("mode", ["global", "per_layer"])
@pytest.mark.parametrize("sizes,first", [([4096], 0), ([1000, 24, 2052], 8), ([1001, 7, 12288 + 4], 0), ([516, 260], 2)])
def test_noised_accumulate_matches_the_oracle(mode, sizes, first):
    """Aligned tensors (one Philox block per thread) and unaligned ones (one lane per parameter), with examples on both
    sides of the threshold."""
    groups = _spread(12, sizes, len(sizes) + first)
    offs = _offsets(sizes, first)
    C, sigma, total = 0.3, 1.3, 48
    acc, norms, clip = _run(mode, groups, offs, C, sigma, total, 21, 4, 12)
    ref, sq, f = _oracle(mode, groups, offs, C, sigma, total, 21, 4, 12)
    np.testing.assert_allclose(clip, f, rtol=TOL_NORM)
    assert (f == 1.0).any() and (f < 1.0).any()
    sd = sigma * C / math.sqrt(total)
    for a, r in zip(acc, ref):
        # B normals of error <= TOL_Z each, scaled by sd, plus fp32 rounding of the running sum
        assert np.max(np.abs(a - r)) <= 12 * sd * TOL_Z + 2e-6 * np.max(np.abs(r))


def test_chunks_use_their_own_example_ranges_and_accumulate():
    sizes, C, sigma, total = [2048 + 4, 20], 0.25, 0.8, 24
    offs = _offsets(sizes)
    acc, ref = None, None
    for c in range(3):
        g = _spread(8, sizes, 40 + c)
        acc, _, _ = _run("global", g, offs, C, sigma, total, 9, 2, 8 * c, acc0=acc, give_norms=bool(c & 1))
        ref, _, _ = _oracle("global", g, offs, C, sigma, total, 9, 2, 8 * c, acc0=ref)
    for a, r in zip(acc, ref):
        assert rel_l2(a, r) <= 2e-5
    # the same chunk under another example range draws other noise
    other, _, _ = _run("global", _spread(8, sizes, 40), offs, C, sigma, total, 9, 2, 8)
    first, _, _ = _run("global", _spread(8, sizes, 40), offs, C, sigma, total, 9, 2, 0)
    assert rel_l2(other[0], first[0]) > 0.1


def test_sigma_zero_is_the_plain_clipped_sum():
    sizes = [777, 12]
    groups = _spread(9, sizes, 50)
    acc, _, _ = _run("global", groups, _offsets(sizes), 0.2, 0.0, 9, 1, 1, 0)
    ref, _, _ = oracle.clipped_sum(groups, 0.2, "global")
    for a, r in zip(acc, ref):
        assert rel_l2(a, r) <= 2e-5


def test_sum_of_per_example_draws_has_the_variance_of_one_draw_on_the_sum():
    """Section 2: B draws of variance sigma^2 C^2 / |B| add up to variance sigma^2 C^2 (zero gradients isolate the noise)."""
    Bn, P, sigma, C = 64, 1 << 18, 1.1, 0.7
    G = [np.zeros((Bn, P), dtype=np.float32)]
    acc, _, _ = _run("global", G, [0], C, sigma, Bn, 5, 0, 0)
    x = acc[0].astype(np.float64) / (sigma * C)
    assert abs(x.mean()) < 5 / math.sqrt(P)
    assert abs(x.var() - 1.0) < 5 * math.sqrt(2.0 / P)
    # fourth moment of a normal: a sum of B independent normals is normal again
    assert abs((x ** 4).mean() - 3.0) < 5 * math.sqrt(96.0 / P)


def test_argument_errors():
    b = B()
    g = torch.zeros((2, 8), device="cuda")
    a = torch.zeros(8, device="cuda")
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    ok = dict(mode=b.DP_CLIP_GLOBAL, B=2, G=[g], P_l=[8], param_offset_l=[0], sqnorm=None, C=1.0, sigma=1.0,
              total_batch=2, seed=0, step=0, example0=0, acc=[a], norms_out=None, clip_out=None, workspace=ws)
    assert b.dp_clip_accumulate_noised(**ok) == b.DP_OK
    for bad in [dict(param_offset_l=None), dict(param_offset_l=[-4]), dict(sigma=-1.0), dict(total_batch=0),
                dict(example0=-1), dict(example0=2**31 - 1), dict(C=float("inf")), dict(sigma=float("inf"))]:
        assert b.dp_clip_accumulate_noised(**{**ok, **bad}) == b.DP_ERR_INVALID_ARG, bad
    assert b.dp_clip_accumulate_noised(**{**ok, "param_offset_l": [2**34]}) == b.DP_ERR_UNSUPPORTED
    torch.cuda.synchronize()
