"""Pins for the oracle's norm / clip / accumulate / average chain.

What fixes the expected values: the invariants of the paper's section 2 (every clipped
example has norm <= C; C = inf and sigma = 0 give the plain average) and section 3.5
(per-group bound C/sqrt(M) keeps the whole-vector norm <= C), closed forms for the
synthetic inputs, and a second routine written differently (numpy einsum / a torch
float64 batch gradient).
"""
import math
import numpy as np
import torch
import torch.nn.functional as F

import oracle
from paper_2109_12191_b200 import synth


def _groups(B, sizes, seed, scale=1.0):
    return [synth.normal_f32((B, p), 910, seed, l, scale=scale) for l, p in enumerate(sizes)]


def test_clip_factor_branches_and_edges():
    sq = np.array([0.0, 0.25, 1.0, 1.0 + 1e-12, 4.0, 1e300])
    f = oracle.clip_factor(sq, 1.0)
    assert f[0] == 1.0 and f[1] == 1.0 and f[2] == 1.0       # ||g|| <= C -> exactly 1
    assert f[3] < 1.0
    assert f[4] == 0.5
    assert f[5] == 1e-150
    assert np.all(oracle.clip_factor(sq, math.inf) == 1.0)    # C = inf never clips


def test_clipped_norm_never_exceeds_C_global():
    B, sizes, C = 16, [37, 5, 128], 1.5
    groups = _groups(B, sizes, 1)
    scale = np.logspace(-2, 1.3, B).astype(np.float32)        # both branches and near the boundary
    groups = [g * scale[:, None] for g in groups]
    _, sq, f = oracle.clipped_sum(groups, C, "global")
    flat = np.concatenate([g.astype(np.float64) for g in groups], axis=1)
    norms = np.linalg.norm(flat, axis=1)
    np.testing.assert_allclose(np.sqrt(sq.sum(1)), norms, rtol=1e-13)
    clipped = np.linalg.norm(flat * f[:, None], axis=1)
    assert np.all(clipped <= C * (1 + 1e-14))
    assert np.all(f[norms <= C] == 1.0) and np.all(f[norms > C] < 1.0)
    assert (norms <= C).any() and (norms > C).any()
    np.testing.assert_allclose(f, np.minimum(1.0, C / norms), rtol=1e-14)


def test_clipped_sum_equals_einsum():
    B, sizes, C = 9, [33, 64], 0.7
    groups = _groups(B, sizes, 2, scale=0.1)
    acc, sq, f = oracle.clipped_sum(groups, C, "global")
    for g, a in zip(groups, acc):
        np.testing.assert_allclose(a, np.einsum("n,np->p", f, g.astype(np.float64)), rtol=1e-13, atol=1e-15)


def test_per_layer_bound_and_whole_vector_bound():
    B, sizes, C = 12, [10, 200, 3, 64], 1.0
    L = len(sizes)
    groups = _groups(B, sizes, 3)
    scale = np.logspace(-2.5, 0.5, B).astype(np.float32)
    groups = [g * scale[:, None] for g in groups]
    _, sq, f = oracle.clipped_sum(groups, C, "per_layer")
    assert f.shape == (B, L)
    total = np.zeros(B)
    for l, g in enumerate(groups):
        cn = np.linalg.norm(g.astype(np.float64) * f[:, l:l + 1], axis=1)
        assert np.all(cn <= C / math.sqrt(L) * (1 + 1e-14))
        total += cn ** 2
    assert np.all(total <= C * C * (1 + 1e-13))               # sum_j ||g_j||^2 <= C^2
    assert (f == 1.0).any() and (f < 1.0).any()


def test_per_layer_with_one_layer_is_global():
    B, C = 7, 0.9
    groups = _groups(B, [257], 4, scale=0.08)
    a1, s1, f1 = oracle.clipped_sum(groups, C, "global")
    a2, s2, f2 = oracle.clipped_sum(groups, C, "per_layer")
    np.testing.assert_array_equal(a1[0], a2[0])
    np.testing.assert_array_equal(f1, f2[:, 0])


def test_no_clip_no_noise_is_the_plain_average_of_the_batch_gradient():
    """C = inf, sigma = 0: the step returns the ordinary mini-batch gradient / |B| (brute force by torch)."""
    Cin, Kout, R, stride, pad, H = 3, 4, 3, 1, 1, 6
    B, G = 4, 3
    chunks, xs, gs = [], [], []
    for c in range(G):
        X = synth.normal_f32((B, H, H, Cin), 911, c, 0)
        dY = synth.normal_f32((B, H, H, Kout), 911, c, 1)
        dW, db = oracle.conv_wgrad(X, dY, R, R, stride, pad)
        chunks.append([dW, db])
        xs.append(X)
        gs.append(dY)
    out, _, factors = oracle.privatise(chunks, math.inf, 0.0, "global", seed=1, step=2)
    assert all(np.all(f == 1.0) for f in factors)
    x = torch.from_numpy(np.concatenate(xs).astype(np.float64)).permute(0, 3, 1, 2)
    g = torch.from_numpy(np.concatenate(gs).astype(np.float64)).permute(0, 3, 1, 2)
    w = torch.zeros(Kout, Cin, R, R, dtype=torch.float64, requires_grad=True)
    b = torch.zeros(Kout, dtype=torch.float64, requires_grad=True)
    (F.conv2d(x, w, b, stride=stride, padding=pad) * g).sum().backward()
    np.testing.assert_allclose(out[0].reshape(Kout, R, R, Cin), w.grad.permute(0, 2, 3, 1).numpy() / (B * G), rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(out[1], b.grad.numpy() / (B * G), rtol=1e-11, atol=1e-13)


def test_accumulation_over_chunks_equals_one_big_batch():
    B, G, sizes, C = 5, 4, [40, 9], 0.5
    chunks = [_groups(B, sizes, 20 + c, scale=0.2) for c in range(G)]
    acc = None
    for ch in chunks:
        acc, _, _ = oracle.clipped_sum(ch, C, "global", acc)
    big = [np.concatenate([ch[l] for ch in chunks]) for l in range(len(sizes))]
    acc_big, _, _ = oracle.clipped_sum(big, C, "global")
    for a, b in zip(acc, acc_big):
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-14)


def test_closed_form_norms_of_the_flat_gradient_workload():
    """Entries N(0, 1e-6): ||g_n|| = 1e-3 sqrt(P) up to sampling spread, so the factor is C/(1e-3 sqrt(P))."""
    P, B = 200_000, 4
    G = synth.normal_f32((B, P), 912, scale=1e-3)
    s = oracle.sqnorm(G)
    np.testing.assert_allclose(np.sqrt(s), 1e-3 * math.sqrt(P), rtol=5 / math.sqrt(2 * P))
    f = oracle.clip_factor(s, 0.1)
    np.testing.assert_allclose(f, 0.1 / (1e-3 * math.sqrt(P)), rtol=5 / math.sqrt(2 * P))
    # the full-size workload's value: P = 25,557,032 gives norm 5.0554 and factor 0.19781
    assert abs(1e-3 * math.sqrt(synth.RESNET50_GN_PARAMS) - 5.05540) < 1e-4


def test_noise_average_arithmetic():
    P = 64
    acc = np.arange(P, dtype=np.float64)
    z = oracle.noise_z(7, 3, 100, P)
    out = oracle.noise_average(acc, 100, 1.1, 2.0, 8, 7, 3)
    np.testing.assert_allclose(out, (acc + 1.1 * 2.0 * z) / 8.0, rtol=1e-15)
    # sigma = 0 -> plain division
    np.testing.assert_array_equal(oracle.noise_average(acc, 0, 0.0, 1.0, 4, 0, 0), acc / 4.0)


def test_noise_std_uses_the_global_C_in_per_layer_mode():
    sizes = [6, 10]
    chunks = [[np.zeros((2, p), dtype=np.float32) for p in sizes]]
    out, _, _ = oracle.privatise(chunks, 2.0, 0.5, "per_layer", seed=9, step=1)
    z = oracle.noise_z(9, 1, 0, 16)
    np.testing.assert_allclose(np.concatenate(out), 0.5 * 2.0 * z / 2.0, rtol=1e-15)


def test_sgd_update_plain_and_momentum_closed_form():
    """theta after k steps of a constant gradient g: theta_0 - lr*g*sum_{j=1..k} (1-mu^j)/(1-mu)."""
    P, lr, mu, k = 7, 0.1, 0.9, 5
    g = np.linspace(-1.0, 2.0, P)
    theta = np.ones(P)
    oracle.sgd_update(g, lr, 0.0, theta)                      # no momentum buffer: theta - lr*g
    np.testing.assert_allclose(theta, 1.0 - lr * g, rtol=1e-15)
    theta, m = np.zeros(P), np.zeros(P)
    for _ in range(k):
        oracle.sgd_update(g, lr, mu, theta, m)
    np.testing.assert_allclose(m, g * (1 - mu ** k) / (1 - mu), rtol=1e-13)
    np.testing.assert_allclose(theta, -lr * g * sum((1 - mu ** j) / (1 - mu) for j in range(1, k + 1)), rtol=1e-13)
    # against torch.optim.SGD (momentum, no dampening, no Nesterov)
    w = torch.zeros(P, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([w], lr=lr, momentum=mu)
    for _ in range(k):
        w.grad = torch.from_numpy(g.copy())
        opt.step()
    np.testing.assert_allclose(theta, w.detach().numpy(), rtol=1e-13)


def test_grouped_clipping_special_cases_and_bound():
    """Section 3.5 with M groups of tensors: one tensor per group is per-layer clipping, one group is whole-model
    clipping, and in between every group keeps norm <= C/sqrt(M), hence the whole vector norm <= C."""
    B, sizes, C = 10, [10, 200, 3, 64, 17], 0.8
    groups = _groups(B, sizes, 20)
    scale = np.logspace(-2.5, 0.5, B).astype(np.float32)
    groups = [g * scale[:, None] for g in groups]
    acc_a, _, f_a = oracle.clipped_sum_grouped(groups, [0, 1, 2, 3, 4], C)
    acc_b, _, f_b = oracle.clipped_sum(groups, C, "per_layer")
    np.testing.assert_array_equal(f_a, f_b)
    for a, b in zip(acc_a, acc_b):
        np.testing.assert_array_equal(a, b)
    acc_a, _, f_a = oracle.clipped_sum_grouped(groups, [0] * 5, C)
    acc_b, _, f_b = oracle.clipped_sum(groups, C, "global")
    np.testing.assert_array_equal(f_a[:, 0], f_b)
    for a, b in zip(acc_a, acc_b):
        np.testing.assert_array_equal(a, b)
    # two stages, tensors interleaved; brute force with numpy on the concatenated stage vectors
    group_of = [1, 0, 1, 0, 0]
    acc, sq, f = oracle.clipped_sum_grouped(groups, group_of, C)
    thr = C / math.sqrt(2)
    total = np.zeros(B)
    for m in range(2):
        flat = np.concatenate([g.astype(np.float64) for g, mm in zip(groups, group_of) if mm == m], axis=1)
        norms = np.linalg.norm(flat, axis=1)
        np.testing.assert_allclose(np.sqrt(sq[:, m]), norms, rtol=1e-13)
        np.testing.assert_allclose(f[:, m], np.minimum(1.0, thr / norms), rtol=1e-14)
        clipped = np.linalg.norm(flat * f[:, m:m + 1], axis=1)
        assert np.all(clipped <= thr * (1 + 1e-14))
        total += clipped ** 2
    assert np.all(np.sqrt(total) <= C * (1 + 1e-14))
    assert (f == 1.0).any() and (f < 1.0).any()
    for g, m, a in zip(groups, group_of, acc):
        np.testing.assert_allclose(a, np.einsum("n,np->p", f[:, m], g.astype(np.float64)), rtol=1e-13, atol=1e-18)


def test_micro_batch_clipping_special_cases_and_brute_force():
    """Clipping the mean of each run of `micro` examples: micro = 1 is per-example clipping; with C = inf the sum of the
    micro-batch means times micro is the plain sum; otherwise a Python loop over micro-batches gives the same."""
    B, sizes, C = 12, [33, 7], 0.05
    groups = _groups(B, sizes, 21, scale=0.02)
    scale = np.logspace(-1.5, 1.0, B).astype(np.float32)
    groups = [g * scale[:, None] for g in groups]
    acc_a, sq_a, f_a = oracle.clipped_sum_micro(groups, C, 1)
    acc_b, sq_b, f_b = oracle.clipped_sum(groups, C, "global")
    np.testing.assert_allclose(f_a, f_b, rtol=1e-15)
    for a, b in zip(acc_a, acc_b):
        np.testing.assert_allclose(a, b, rtol=1e-13, atol=1e-18)
    acc, _, f = oracle.clipped_sum_micro(groups, math.inf, 4)
    assert np.all(f == 1.0)
    for a, g in zip(acc, groups):
        np.testing.assert_allclose(4 * a, g.astype(np.float64).sum(0), rtol=1e-12, atol=1e-15)
    mu = 3
    acc, sq, f = oracle.clipped_sum_micro(groups, C, mu)
    want = [np.zeros(p) for p in sizes]
    for j in range(B // mu):
        mean = [sum(g[j * mu + i].astype(np.float64) for i in range(mu)) / mu for g in groups]
        norm = math.sqrt(sum(float(np.dot(m, m)) for m in mean))
        fac = 1.0 if norm <= C else C / norm
        assert abs(f[j] - fac) <= 1e-15 and abs(math.sqrt(sq[j]) - norm) <= 1e-13 * norm
        assert norm * fac <= C * (1 + 1e-14)
        for w, m in zip(want, mean):
            w += fac * m
    assert (f == 1.0).any() and (f < 1.0).any()
    for a, w in zip(acc, want):
        np.testing.assert_allclose(a, w, rtol=1e-12, atol=1e-18)


def test_synthetic_model_inventories():
    """Tensor and parameter counts of the two ResNets whose layer shapes the workloads use (the counts of the public
    architectures: 25,557,032 and 44,549,160 parameters)."""
    for layers, tensors, params in ((synth.resnet50_gn_layers(), synth.RESNET50_GN_TENSORS, synth.RESNET50_GN_PARAMS),
                                    (synth.resnet101_gn_layers(), synth.RESNET101_GN_TENSORS, synth.RESNET101_GN_PARAMS)):
        assert sum(1 + (l.n_bias > 0) for l in layers) == tensors
        assert sum(l.n_weight + l.n_bias for l in layers) == params
    assert synth.RESNET50_GN_PARAMS == 25_557_032 and synth.RESNET101_GN_PARAMS == 44_549_160
