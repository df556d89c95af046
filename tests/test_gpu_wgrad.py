"""GPU parity of dp_per_example_wgrad (every layer kind, epilogue and implementation) against the oracle."""
import math
import numpy as np
import pytest
import torch

import oracle
from paper_2109_12191_b200 import synth
from gpu_util import (B, rel_l2, gpu_layer, oracle_layer, scaled_inputs, make_desc, dev_inputs, TOL_NORM, TOL_FMA, TOL_ACC_BF16,
                      TOL_ACC_F32)

pytestmark = pytest.mark.gpu

STORE, NORM, CLIP = 0, 1, 2
AUTO, CUDA_CORE, TENSOR_CORE = 0, 1, 2


def tol_for(out, dtype):
    """Accumulated / stored gradient tolerance: plain fp32 rounding on the CUDA-core path and for bf16
    inputs (their products are exact in fp32); the TF32-class bound for fp32 inputs on tensor cores."""
    # bf16 products are exact in fp32 and fp32 inputs run as split tf32, so both implementations are held
    # to plain fp32 rounding here -- far inside the 1e-2 / 2e-3 bounds the workload tests apply.  "tf32" is the
    # single-pass mode: inputs rounded to 11 significant bits, held to the TF32 bound
    return TOL_ACC_F32 if (dtype == "tf32" and out["uses_tc"]) else TOL_FMA


def check_layer(layer, Bn, dtype, impl, key, bias_separate=0, spread=False, clip_impl=None):
    inp = scaled_inputs(layer, Bn, dtype, *key, spread=spread)
    dW, db = oracle_layer(layer, inp)
    sq_w = oracle.sqnorm(dW)
    sq_b = oracle.sqnorm(db) if db is not None else np.zeros(Bn)
    groups = 2 if (bias_separate and db is not None) else 1
    ref_sq = np.stack([sq_w, sq_b], 1) if groups == 2 else (sq_w + sq_b)[:, None]

    out = gpu_layer(layer, inp, dtype, STORE, impl, bias_separate)
    tol = tol_for(out, dtype)
    for n in range(Bn):
        assert rel_l2(out["G_w"][n], dW[n]) <= tol, (layer.name, n)
    if db is not None:
        for n in range(Bn):
            assert rel_l2(out["G_b"][n], db[n]) <= tol
    np.testing.assert_allclose(out["sq"], ref_sq, rtol=TOL_NORM)

    out_n = gpu_layer(layer, inp, dtype, NORM, impl, bias_separate)
    np.testing.assert_allclose(out_n["sq"], ref_sq, rtol=TOL_NORM)

    # per-layer clip + accumulate, threshold at the median norm so both branches occur when norms spread
    C_l = float(np.sqrt(np.median(ref_sq)))
    f = oracle.clip_factor(ref_sq, C_l).reshape(Bn, groups)
    ref_acc_w = np.einsum("n,np->p", f[:, 0], dW)
    out_c = gpu_layer(layer, inp, dtype, CLIP, clip_impl if clip_impl is not None else impl, bias_separate, C_l=C_l)
    np.testing.assert_allclose(out_c["clip"], f, rtol=TOL_NORM)
    np.testing.assert_allclose(out_c["sq"], ref_sq, rtol=TOL_NORM)
    assert rel_l2(out_c["acc_w"], ref_acc_w) <= tol_for(out_c, dtype)
    if db is not None:
        ref_acc_b = np.einsum("n,np->p", f[:, groups - 1], db)
        assert rel_l2(out_c["acc_b"], ref_acc_b) <= tol_for(out_c, dtype)
    if out_c["uses_tc"] and db is None:
        # the tensor-core clip has a single-pass form (taken when the layer qualifies) and a two-pass form: check the other too
        b = B()
        b.dp_debug_set_single_pass(0)
        try:
            out_2 = gpu_layer(layer, inp, dtype, CLIP, clip_impl if clip_impl is not None else impl, bias_separate, C_l=C_l)
        finally:
            b.dp_debug_set_single_pass(1)
        np.testing.assert_allclose(out_2["clip"], f, rtol=TOL_NORM)
        np.testing.assert_allclose(out_2["sq"], ref_sq, rtol=TOL_NORM)
        assert rel_l2(out_2["acc_w"], ref_acc_w) <= tol_for(out_2, dtype)
    return out


FMA_CONVS = [
    # Cin, Kout, R, stride, pad, H, bias
    (3, 32, 3, 1, 1, 32, True),      # first conv of the small CNN: 27 columns
    (32, 64, 3, 2, 1, 32, True),
    (64, 128, 3, 2, 1, 16, True),
    (3, 64, 7, 2, 3, 30, False),     # stem-like: 147 columns (not a multiple of 4), stride 2, pad 3
    (5, 7, 3, 1, 0, 9, True),        # nothing aligned
    (16, 8, 1, 2, 0, 8, False),      # strided 1x1
    (8, 70, 5, 1, 2, 7, True),       # K = 49 pixels, ragged tile rows
    (2, 3, 3, 1, 1, 1, False),       # 1x1 image with padding: only the centre tap sees data
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("case", FMA_CONVS)
def test_conv_cuda_core(case, dtype):
    Cin, Kout, R, stride, pad, H, bias = case
    layer = synth.conv(Cin, Kout, R, stride, pad, H, bias, name=str(case))
    check_layer(layer, 5, dtype, CUDA_CORE, (930, sum(case[:6])), spread=True)


THIN_CONVS = [(3, 32, 3, 1, 1, 32, True), (3, 64, 3, 2, 1, 17, False), (2, 32, 3, 1, 0, 9, True), (1, 32, 5, 1, 2, 12, True),
              (3, 32, 3, 1, 1, 3, False), (3, 64, 3, 1, 1, 13, True)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("case", THIN_CONVS)
def test_conv_thin_inputs_default_route(case, dtype):
    """Few-column convolutions (RGB inputs) under DP_IMPL_AUTO: the one-block-per-example kernel for
    STORE / NORM, the general kernels for the fused clip."""
    Cin, Kout, R, stride, pad, H, bias = case
    layer = synth.conv(Cin, Kout, R, stride, pad, H, bias, name=str(case))
    check_layer(layer, 6, dtype, AUTO, (945, sum(case[:6])), spread=True)
    check_layer(layer, 3, dtype, AUTO, (946, sum(case[:6])), bias_separate=1, spread=True)


def test_conv_non_square_image_and_filter():
    layer = synth.Layer("conv", 6, 9, R=3, S=5, stride=2, pad=1, H=11, W=14, bias=True, name="3x5")
    check_layer(layer, 3, "f32", CUDA_CORE, (931,), spread=True)


@pytest.mark.parametrize("bias_separate", [0, 1])
def test_bias_group_handling(bias_separate):
    layer = synth.conv(8, 16, 3, 1, 1, 10, True, "bias groups")
    check_layer(layer, 6, "f32", CUDA_CORE, (932,), bias_separate=bias_separate, spread=True)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("Cin,Kout,bias", [(256, 64, True), (8192, 10, True), (13, 7, False), (2048, 1000, False)])
def test_dense(Cin, Kout, bias, dtype):
    layer = synth.dense(Cin, Kout, bias, "dense")
    Bn = 8 if Cin * Kout < 1_000_000 else 3
    check_layer(layer, Bn, dtype, AUTO, (933, Cin), spread=True)
    check_layer(layer, Bn, dtype, AUTO, (933, Cin), bias_separate=1, spread=True)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("C,H", [(64, 12), (256, 7), (2048, 3), (24, 20), (5, 6), (512, 17)])
def test_norm_affine(C, H, dtype):
    layer = synth.norm(C, H, "gn")
    check_layer(layer, 4, dtype, AUTO, (934, C), bias_separate=1, spread=True)
    check_layer(layer, 4, dtype, AUTO, (934, C), bias_separate=0, spread=True)


def test_rerun_gives_identical_bits():
    layer = synth.conv(32, 64, 3, 2, 1, 32, True)
    inp = synth.layer_inputs(layer, 6, "f32", 935)
    a = gpu_layer(layer, inp, "f32", STORE, CUDA_CORE)
    b = gpu_layer(layer, inp, "f32", STORE, CUDA_CORE)
    np.testing.assert_array_equal(a["G_w"], b["G_w"])
    np.testing.assert_array_equal(a["sq"], b["sq"])


def test_sqnorm_stride_writes_one_column_of_a_table():
    layer = synth.conv(8, 16, 3, 1, 1, 10, True)
    inp = synth.layer_inputs(layer, 4, "f32", 936)
    table = torch.full((4, 5), -1.0, device="cuda")
    gpu_layer(layer, inp, "f32", NORM, CUDA_CORE, bias_separate=1, sq=table, sq_stride=5, sq_col=2)
    t = table.cpu().numpy()
    dW, db = oracle_layer(layer, inp)
    np.testing.assert_allclose(t[:, 2], oracle.sqnorm(dW), rtol=TOL_NORM)
    np.testing.assert_allclose(t[:, 3], oracle.sqnorm(db), rtol=TOL_NORM)
    assert np.all(t[:, [0, 1, 4]] == -1.0)


def test_dense_norm_is_the_rank1_closed_form():
    layer = synth.dense(300, 40, True)
    inp = synth.layer_inputs(layer, 7, "f32", 937)
    out = gpu_layer(layer, inp, "f32", NORM)
    x2 = (inp["X"].astype(np.float64) ** 2).sum(1)
    y2 = (inp["dY"].astype(np.float64) ** 2).sum(1)
    np.testing.assert_allclose(out["sq"][:, 0], y2 * x2 + y2, rtol=1e-6)


# ------------------------------------------------------------------ tcgen05 path
TC_CONVS = [
    # dtype, Cin, Kout, R, stride, pad, H, bias        (bf16: channels in multiples of 64; fp32 runs as tf32: multiples of 32)
    ("bf16", 64, 64, 1, 1, 0, 8, False),       # both extents 64: half of the 128-row tile is unused
    ("bf16", 64, 64, 3, 1, 1, 8, True),        # 576 columns: ragged last tile
    ("bf16", 128, 128, 3, 1, 1, 8, False),
    ("bf16", 64, 256, 1, 1, 0, 14, False),     # 14x14: pixel tiles hang over the image edge (zero filled)
    ("bf16", 256, 64, 1, 1, 0, 14, False),
    ("bf16", 128, 192, 3, 1, 1, 12, True),
    ("bf16", 64, 64, 3, 1, 1, 7, False),       # 49 pixels
    ("bf16", 64, 128, 3, 1, 0, 10, False),     # no padding: 8x8 outputs from a 10x10 input
    ("bf16", 320, 64, 1, 1, 0, 6, False),      # extent 320 = 2.5 row tiles
    ("bf16", 64, 64, 5, 1, 2, 9, False),       # 5x5 taps
    ("bf16", 128, 128, 3, 2, 1, 14, False),    # stride 2 through the tensor map's element stride
    ("bf16", 64, 128, 1, 2, 0, 14, False),     # strided 1x1 (projection shortcut)
    ("bf16", 64, 64, 3, 2, 1, 15, True),       # odd input size with stride 2
    ("f32", 32, 64, 3, 2, 1, 32, True),        # second conv of the small CNN
    ("f32", 64, 128, 3, 2, 1, 16, True),       # third conv of the small CNN
    ("f32", 32, 32, 1, 1, 0, 8, False),
    ("f32", 96, 160, 3, 1, 1, 9, False),       # extents that are multiples of 32 but not of 64 or 128
    ("bf16", 3, 64, 7, 2, 3, 30, False),       # stem: 3 input channels are unfolded to 147 (+45 zero) columns first;
                                               # its fused clip regroups 2 x 2 pixel blocks into channels instead
    ("bf16", 4, 64, 5, 2, 2, 21, False),       # ... 16 regrouped channels exactly, three of the four window taps exist
    ("bf16", 3, 128, 3, 2, 1, 17, False),      # ... two taps a row, odd input size
    ("bf16", 1, 64, 7, 4, 3, 29, False),       # ... stride 4: 4 x 4 blocks of a single channel
    ("f32", 3, 32, 3, 1, 1, 32, True),         # first conv of the small CNN: 27 (+5 zero) columns
    ("bf16", 4, 128, 3, 1, 1, 9, True),        # 36 columns, rows of the gradient not 16-byte aligned
    ("f32", 1, 64, 5, 2, 2, 13, False),        # single input channel
    ("tf32", 32, 64, 3, 2, 1, 32, True),       # single-pass tf32: the small CNN's convs ...
    ("tf32", 64, 128, 3, 2, 1, 16, True),
    ("tf32", 96, 160, 3, 1, 1, 9, False),      # ... ragged extents ...
    ("tf32", 3, 32, 3, 1, 1, 32, True),        # ... and the unfolded small-channel form
]


@pytest.mark.parametrize("case", TC_CONVS)
def test_conv_tensor_core(case):
    dtype, Cin, Kout, R, stride, pad, H, bias = case
    layer = synth.conv(Cin, Kout, R, stride, pad, H, bias, name=str(case))
    out = check_layer(layer, 5, dtype, TENSOR_CORE, (940, sum(case[1:7])), spread=True)
    assert out["uses_tc"]


@pytest.mark.parametrize("Bn", [1, 37])
def test_clipped_sum_example_ranges(Bn):
    """Fused clip + accumulate cuts the batch into example ranges (ragged for 37) whose partial sums are folded
    in order; both implementations, accumulating on top of a non-zero accumulator."""
    b = B()
    for impl, dtype, layer in ((TENSOR_CORE, "bf16", synth.conv(64, 64, 3, 1, 1, 8, name="tc ranges")),
                               (TENSOR_CORE, "f32", synth.conv(32, 64, 3, 2, 1, 16, name="tf32 ranges")),
                               (TENSOR_CORE, "tf32", synth.conv(32, 64, 3, 2, 1, 16, name="single-pass tf32 ranges")),
                               (CUDA_CORE, "f32", synth.conv(3, 16, 3, 1, 1, 12, True, name="fma ranges"))):
        inp = scaled_inputs(layer, Bn, dtype, 943, Bn, spread=Bn > 1)
        dW, db = oracle_layer(layer, inp)
        sq = oracle.sqnorm(dW) + (oracle.sqnorm(db) if db is not None else 0.0)
        C_l = float(np.sqrt(np.median(sq)))
        f = oracle.clip_factor(sq, C_l)
        start_w = synth.normal_f32((layer.n_weight,), 944)
        acc_w = torch.from_numpy(start_w.copy()).cuda()
        acc_b = torch.zeros(layer.n_bias, device="cuda") if layer.n_bias else None
        out = gpu_layer(layer, inp, dtype, CLIP, impl, 0, C_l=C_l, acc_w=acc_w, acc_b=acc_b)
        np.testing.assert_allclose(out["clip"][:, 0], f, rtol=TOL_NORM)
        assert rel_l2(out["acc_w"], start_w + np.einsum("n,np->p", f, dW)) <= (TOL_ACC_F32 if dtype == "tf32" else TOL_FMA)
        if db is not None:
            assert rel_l2(out["acc_b"], np.einsum("n,np->p", f, db)) <= TOL_FMA


def test_tensor_core_matches_cuda_core_bitwise_norm_inputs():
    """Same layer through both implementations: bf16 products are exact in fp32, so the two differ by
    accumulation order only."""
    layer = synth.conv(128, 128, 3, 1, 1, 14, name="tc vs fma")
    inp = synth.layer_inputs(layer, 4, "bf16", 941)
    a = gpu_layer(layer, inp, "bf16", STORE, TENSOR_CORE)
    b = gpu_layer(layer, inp, "bf16", STORE, CUDA_CORE)
    assert rel_l2(a["G_w"], b["G_w"]) <= 1e-5
    np.testing.assert_allclose(a["sq"], b["sq"], rtol=1e-5)


def test_tensor_core_rerun_is_bit_identical():
    layer = synth.conv(64, 128, 3, 1, 1, 14, name="tc rerun")
    inp = synth.layer_inputs(layer, 6, "bf16", 942)
    a = gpu_layer(layer, inp, "bf16", STORE, TENSOR_CORE)
    b = gpu_layer(layer, inp, "bf16", STORE, TENSOR_CORE)
    np.testing.assert_array_equal(a["G_w"], b["G_w"])
    np.testing.assert_array_equal(a["sq"], b["sq"])


def test_a_wait_that_runs_out_is_reported_and_later_calls_do_not_hide_it():
    """Every wait of the tensor-core kernel is bounded.  With the poll limit at zero each role gives up before it
    copies or multiplies anything, the kernel returns, and the workspace's status word says so; the word is sticky,
    so a good call on the same workspace afterwards must not hide it, and reading it clears it."""
    b = B()
    layer = synth.conv(64, 64, 3, 1, 1, 14, name="c")
    Bn = 4
    inp = synth.layer_inputs(layer, Bn, "bf16", 955, 0)
    X, dY = dev_inputs(inp, "bf16")
    d = make_desc(layer, Bn, "bf16", b.DP_IMPL_TENSOR_CORE, 0)
    ws = torch.empty(b.dp_workspace_bytes(d, b.DP_EPI_NORM_ONLY), dtype=torch.uint8, device="cuda")
    b.check(b.dp_workspace_init(ws))
    sq = torch.zeros((Bn, 1), device="cuda")
    call = lambda: b.dp_per_example_wgrad(d, X, dY, None, None, sq, 1, b.DP_EPI_NORM_ONLY, 0.0, None, None, None, ws)
    b.dp_debug_set_wait_polls(0)
    try:
        assert call() == b.DP_OK                           # the launch itself succeeds; the kernel gives up on the device
        torch.cuda.synchronize()
    finally:
        b.dp_debug_set_wait_polls(-1)
    assert call() == b.DP_OK                               # a good call on the same workspace ...
    assert b.dp_wgrad_check(ws) == b.DP_ERR_TIMEOUT        # ... does not hide the earlier time-out
    assert b.dp_wgrad_check(ws) == b.DP_OK                 # reported once, then the header starts over
    assert call() == b.DP_OK
    assert b.dp_wgrad_check(ws) == b.DP_OK
    dW, _ = oracle_layer(layer, inp)
    np.testing.assert_allclose(sq.cpu().numpy()[:, 0], oracle.sqnorm(dW), rtol=TOL_NORM)


def test_fused_clip_runs_one_contraction_where_the_gradient_fits_a_cluster():
    """bf16 layers whose per-example gradient fits the tensor memory of one thread-block cluster take the single-pass
    form of the fused clip: fewer launches than the two-pass form, same results (checked layer by layer above)."""
    b = B()
    layer = synth.conv(64, 128, 3, 1, 1, 14, name="c")
    inp = scaled_inputs(layer, 6, "bf16", 956, 0, spread=True)
    counts = []
    for on in (1, 0):
        b.dp_debug_set_single_pass(on)
        try:
            c0 = b.dp_debug_launch_count()
            gpu_layer(layer, inp, "bf16", CLIP, AUTO, 0, C_l=1.0)
            counts.append(b.dp_debug_launch_count() - c0)
        finally:
            b.dp_debug_set_single_pass(1)
    assert counts[0] < counts[1]


GRAM_CONVS = [
    # Cin, Kout, R, stride, pad, H: gradients too large for a cluster, output planes of at most 256 pixels
    (128, 256, 3, 1, 1, 14),      # 196 pixels in a 16 x 14 box: two row tiles, the second with 96 rows
    (128, 256, 3, 1, 1, 10),      # 100 pixels in a 12 x 12 box: second row tile of 16 rows
    (128, 256, 3, 1, 1, 5),       # 25 pixels in a 48-row box: one row tile, mostly zero rows
    (128, 256, 3, 2, 1, 14),      # strided taps, 7 x 7 output in an 8 x 8 box
    (512, 1024, 1, 2, 0, 14),     # strided 1 x 1
    (1024, 512, 1, 1, 0, 14),     # 1 x 1 with flattened pixels: 196 -> 208 rows
    (256, 1152, 1, 1, 0, 16),     # exactly 256 pixels: two full row tiles
]


def gram_plan(b, layer, Bn):
    plan = b.dp_debug_wgrad_plan(make_desc(layer, Bn, "bf16", b.DP_IMPL_AUTO, 0), epilogue=5)
    return None if plan is None else list(plan.values())


@pytest.mark.parametrize("case", GRAM_CONVS)
def test_conv_norms_from_pixel_gram_matrices(case):
    """Large layers over small planes take their norms from the Gram matrices of dY and of the unfolded input over
    the pixels; norms, factors and the clipped sum are held to the same bounds as every other route, and
    check_layer also runs the route that forms the gradients."""
    Cin, Kout, R, stride, pad, H = case
    b = B()
    layer = synth.conv(Cin, Kout, R, stride, pad, H, False, name=str(case))
    plan = gram_plan(b, layer, 5)
    assert plan is not None and plan[1] % 16 == 0 and plan[1] <= 256
    c0 = b.dp_debug_launch_count()
    out = check_layer(layer, 5, "bf16", AUTO, (960, sum(case)), spread=True)
    assert out["uses_tc"]
    assert b.dp_debug_launch_count() > c0


def test_gram_norm_waits_are_bounded():
    """The Gram-matrix kernel's waits give up like the others: poll limit zero, the kernels return, the status word says so."""
    b = B()
    layer = synth.conv(128, 256, 3, 1, 1, 14, name="c")
    Bn = 3
    assert gram_plan(b, layer, Bn) is not None
    inp = synth.layer_inputs(layer, Bn, "bf16", 961, 0)
    X, dY = dev_inputs(inp, "bf16")
    d = make_desc(layer, Bn, "bf16", b.DP_IMPL_AUTO, 0)
    ws = torch.empty(b.dp_workspace_bytes(d, b.DP_EPI_CLIP_ACCUM), dtype=torch.uint8, device="cuda")
    b.check(b.dp_workspace_init(ws))
    sq = torch.zeros((Bn, 1), device="cuda")
    acc = torch.zeros(layer.n_weight, device="cuda")
    call = lambda: b.dp_per_example_wgrad(d, X, dY, None, None, sq, 1, b.DP_EPI_CLIP_ACCUM, 1.0, acc, None, None, ws)
    b.dp_debug_set_wait_polls(0)
    try:
        assert call() == b.DP_OK
        torch.cuda.synchronize()
    finally:
        b.dp_debug_set_wait_polls(-1)
    assert b.dp_wgrad_check(ws) == b.DP_ERR_TIMEOUT
    assert b.dp_wgrad_check(ws) == b.DP_OK


@pytest.mark.parametrize("case", [(64, 128, 3, 1, 1, 14), (128, 256, 3, 1, 1, 14), (3, 64, 7, 2, 3, 30), (256, 64, 1, 1, 0, 28)])
def test_fused_clip_under_an_sm_target_with_a_ragged_batch(case):
    """With an SM target set (calls meant to run side by side) a cluster walks through up to thirty-two examples and the
    one-product clipped sum takes fewer example ranges: 37 examples leave a ragged last range in both."""
    Cin, Kout, R, stride, pad, H = case
    b = B()
    layer = synth.conv(Cin, Kout, R, stride, pad, H, False, name=str(case))
    b.check(b.dp_set_sm_target(torch.cuda.get_device_properties(0).multi_processor_count))
    try:
        out = check_layer(layer, 37, "bf16", AUTO, (962, sum(case)), spread=True)
    finally:
        b.check(b.dp_set_sm_target(0))
    assert out["uses_tc"]


@pytest.mark.parametrize("case", [(128, 256, 3, 1, 1, 14), (512, 512, 3, 1, 1, 7), (256, 1024, 1, 1, 0, 14), (3, 64, 7, 2, 3, 30)])
@pytest.mark.parametrize("target", [0, 1])
def test_fused_clip_rerun_is_bit_identical(case, target):
    """Norms from Gram matrices, the known-factor and one-product clipped sums, the cluster exchange and the
    space-to-depth stem add in a fixed order: a second run gives the same bits, with and without an SM target."""
    Cin, Kout, R, stride, pad, H = case
    b = B()
    layer = synth.conv(Cin, Kout, R, stride, pad, H, False, name=str(case))
    inp = scaled_inputs(layer, 9, "bf16", 963, sum(case), spread=True)
    b.check(b.dp_set_sm_target(torch.cuda.get_device_properties(0).multi_processor_count if target else 0))
    try:
        one = gpu_layer(layer, inp, "bf16", CLIP, AUTO, 0, C_l=0.7)
        two = gpu_layer(layer, inp, "bf16", CLIP, AUTO, 0, C_l=0.7)
    finally:
        b.check(b.dp_set_sm_target(0))
    np.testing.assert_array_equal(one["acc_w"], two["acc_w"])
    np.testing.assert_array_equal(one["sq"], two["sq"])
    np.testing.assert_array_equal(one["clip"], two["clip"])
