"""GPU parity of the noise stream and of dp_noise_average against the oracle (through the C ABI)."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import B, dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed,step,first,n", [(0, 0, 0, 1000), (42, 3, 5, 777), (2 ** 63 + 11, 2 ** 40 + 9, 2 ** 33 + 1, 513),
                                               (1, 2 ** 32, 2 ** 32 - 3, 9)])
def test_philox_words_bit_exact(seed, step, first, n):
    b = B()
    out = torch.zeros((n, 4), dtype=torch.int32, device="cuda")
    b.check(b.dp_debug_philox_raw(out, n, first, seed, step))
    got = out.cpu().numpy().view(np.uint32)
    np.testing.assert_array_equal(got, oracle.philox_blocks(seed, step, first, n))


@pytest.mark.parametrize("seed,step,first,n", [(0, 0, 0, 200_003), (7, 1, 3, 10_001), (9, 9, 2 ** 35 + 2, 4099), (5, 0, 1, 1)])
def test_normals_match_oracle(seed, step, first, n):
    b = B()
    z = torch.full((n + 8,), float("nan"), device="cuda")
    b.check(b.dp_debug_noise_z(z, n, first, seed, step))
    got = z.cpu().numpy()
    assert np.all(np.isnan(got[n:]))                        # nothing written past the end
    ref = oracle.noise_z(seed, step, first, n)
    assert np.max(np.abs(got[:n] - ref)) <= 1e-5
    assert np.max(np.abs(got[:n])) <= 5.768 + 1e-3


@pytest.mark.parametrize("P,off", [(4096, 0), (1000, 4), (1001, 0), (37, 1), (5003, 2), (3, 3), (1, 0), (262_147, 8)])
def test_noise_average_parity(P, off):
    b = B()
    sigma, C, total = 1.1, 0.8, 24
    acc = np.random.default_rng(P + off).standard_normal(P).astype(np.float32) * 3
    a = dev(acc)
    out = torch.full((P + 4,), float("nan"), device="cuda")
    b.check(b.dp_noise_average(a, P, off, sigma, C, total, 11, 5, out))
    got = out.cpu().numpy()
    assert np.all(np.isnan(got[P:]))
    ref = oracle.noise_average(acc.astype(np.float64), off, sigma, C, total, 11, 5)
    scale = sigma * C / total
    assert np.max(np.abs(got[:P] - ref)) <= 1e-5 * scale + 1e-6 * np.max(np.abs(ref))
    # in place gives the same bits
    b.check(b.dp_noise_average(a, P, off, sigma, C, total, 11, 5, a))
    np.testing.assert_array_equal(a.cpu().numpy(), got[:P])


def test_sigma_zero_is_a_plain_division_even_with_infinite_C():
    b = B()
    acc = np.arange(1, 1025, dtype=np.float32)
    out = torch.empty(1024, device="cuda")
    b.check(b.dp_noise_average(dev(acc), 1024, 0, 0.0, float("inf"), 8, 0, 0, out))
    np.testing.assert_array_equal(out.cpu().numpy(), acc / 8)


def test_result_is_independent_of_how_the_parameters_are_split():
    b = B()
    P = 10_007
    acc = dev(np.zeros(P, dtype=np.float32))
    whole = torch.empty(P, device="cuda")
    b.check(b.dp_noise_average(acc, P, 0, 1.0, 1.0, 1, 3, 4, whole))
    parts = torch.empty(P + 3, device="cuda")
    cuts = [0, 12, 4001, 4003, P]                            # pieces start at 16-byte aligned addresses or not
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        pad = (-lo) % 4                                      # keep device pointers 16-byte aligned
        tmp_in = torch.zeros(hi - lo, device="cuda")
        tmp_out = torch.empty(hi - lo, device="cuda")
        b.check(b.dp_noise_average(tmp_in, hi - lo, lo, 1.0, 1.0, 1, 3, 4, tmp_out))
        parts[lo:hi] = tmp_out
    np.testing.assert_array_equal(parts[:P].cpu().numpy(), whole.cpu().numpy())


def test_statistics_at_full_model_size():
    """25.56 M draws (one per ResNet-50 parameter): mean, variance and range of the GPU stream itself."""
    b = B()
    P = 25_557_032
    acc = torch.zeros(P, device="cuda")
    b.check(b.dp_noise_average(acc, P, 0, 1.0, 1.0, 1, 0, 0, acc))
    z = acc.double()
    assert abs(z.mean().item()) < 5 / P ** 0.5
    assert abs(z.var().item() - 1.0) < 5 * (2.0 / P) ** 0.5
    assert z.abs().max().item() <= 5.768 + 1e-3
    idx = np.random.default_rng(0).integers(0, P, 2000)
    ref = np.array([oracle.noise_z(0, 0, int(i), 1)[0] for i in idx])
    assert np.max(np.abs(acc[torch.from_numpy(idx).cuda()].cpu().numpy() - ref)) <= 1e-5


@pytest.mark.parametrize("P,off,mu", [(4099, 0, 0.9), (1000, 3, 0.0), (37, 6, 0.5)])
def test_fused_sgd_update_matches_oracle_over_several_steps(P, off, mu):
    """noise + average + (momentum) SGD in one pass against the oracle's noise_average followed by sgd_update."""
    b = B()
    sigma, C, total, lr = 0.8, 1.2, 16, 0.05
    rng = np.random.default_rng(P)
    theta0 = rng.standard_normal(P).astype(np.float32)
    theta, mom = dev(theta0), torch.zeros(P, device="cuda")
    g_out = torch.full((P,), float("nan"), device="cuda")
    ref_theta, ref_m = theta0.astype(np.float64), np.zeros(P)
    for step in range(3):
        acc = (rng.standard_normal(P) * 4).astype(np.float32)
        b.check(b.dp_noise_average_sgd(dev(acc), P, off, sigma, C, total, 21, step, lr, mu, theta,
                                       mom if mu > 0 else None, g_out))
        g = oracle.noise_average(acc.astype(np.float64), off, sigma, C, total, 21, step)
        oracle.sgd_update(g, lr, mu, ref_theta, ref_m if mu > 0 else None)
        assert np.max(np.abs(g_out.cpu().numpy() - g)) <= 1e-5 * sigma * C / total + 1e-6 * np.max(np.abs(g))
    assert np.max(np.abs(theta.cpu().numpy() - ref_theta)) <= 1e-5
    if mu > 0:
        assert np.max(np.abs(mom.cpu().numpy() - ref_m)) <= 1e-5
    # the same gradient as the unfused entry point, bit for bit
    out = torch.empty(P, device="cuda")
    b.check(b.dp_noise_average(dev(acc), P, off, sigma, C, total, 21, 2, out))
    np.testing.assert_array_equal(out.cpu().numpy(), g_out.cpu().numpy())
