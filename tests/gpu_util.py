"""Shared helpers of the GPU parity tests: run one layer through the C ABI, run it through the oracle."""
import math
import numpy as np
import torch

import oracle
from paper_2109_12191_b200 import synth

TOL_NORM = 1e-4        # per-example norms and clip factors, relative
TOL_ACC_F32 = 2e-3     # accumulated gradients, relative L2, fp32 inputs (TF32-class tensor-core path)
TOL_ACC_BF16 = 1e-2    # accumulated gradients, relative L2, bf16 inputs
TOL_FMA = 2e-5         # CUDA-core fp32 path: plain fp32 rounding only


def B():
    from paper_2109_12191_b200 import binding
    return binding


def rel_l2(a, ref):
    a = np.asarray(a, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    d = np.linalg.norm(a - ref)
    n = np.linalg.norm(ref)
    return d / n if n > 0 else d


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t if dtype is None else t.to(dtype)


def dev_inputs(inp, dtype):
    """Device tensors of a synth.layer_inputs() draw in the layer's dtype."""
    if dtype == "bf16":
        X = torch.from_numpy(inp["X_bits"].view(np.int16)).cuda().view(torch.bfloat16)
        dY = torch.from_numpy(inp["dY_bits"].view(np.int16)).cuda().view(torch.bfloat16)
    else:
        X, dY = dev(inp["X"]), dev(inp["dY"])
    return X, dY


def make_desc(layer, Bn, dtype, impl=0, bias_separate=0):
    b = B()
    kind = {"conv": b.DP_LAYER_CONV2D, "dense": b.DP_LAYER_DENSE, "norm": b.DP_LAYER_NORM_AFFINE}[layer.kind]
    code = {"f32": b.DP_F32, "bf16": b.DP_BF16, "tf32": b.DP_TF32}[dtype]
    return b.make_desc(kind, code, Bn, layer.Cin, layer.Kout, layer.H, layer.W,
                       layer.R, layer.S, layer.stride, layer.pad, int(layer.bias), bias_separate, impl)


def oracle_layer(layer, inp):
    """(dW [B,P_w] float64, db [B,P_b] float64 or None) from the oracle."""
    Bn = inp["X"].shape[0]
    if layer.kind == "conv":
        dW, db = oracle.conv_wgrad(inp["X"], inp["dY"], layer.R, layer.S, layer.stride, layer.pad, bias=layer.bias)
    elif layer.kind == "dense":
        dW, db = oracle.dense_wgrad(inp["X"], inp["dY"], bias=layer.bias)
    else:
        dW, db = oracle.norm_affine_wgrad(inp["X"], inp["dY"])
    return dW.reshape(Bn, -1), (db.reshape(Bn, -1) if db is not None else None)


def gpu_layer(layer, inp, dtype, epilogue, impl=0, bias_separate=0, C_l=1.0, acc_w=None, acc_b=None, sq=None,
              sq_stride=None, sq_col=0, check_status=True):
    """Runs dp_per_example_wgrad. Returns dict(G_w, G_b, sq [B,groups], clip, acc_w, acc_b) as numpy."""
    b = B()
    Bn = inp["X"].shape[0]
    X, dY = dev_inputs(inp, dtype)
    d = make_desc(layer, Bn, dtype, impl, bias_separate)
    groups = b.dp_layer_groups(d)
    has_b = layer.n_bias > 0
    G_w = torch.full((Bn, layer.n_weight), float("nan"), device="cuda") if epilogue == b.DP_EPI_STORE_NORM else None
    G_b = torch.full((Bn, layer.n_bias), float("nan"), device="cuda") if (epilogue == b.DP_EPI_STORE_NORM and has_b) else None
    own_sq = sq is None
    if own_sq:
        sq = torch.full((Bn, groups), float("nan"), device="cuda")
        sq_stride, sq_col = groups, 0
    clip = torch.full((Bn, groups), float("nan"), device="cuda") if epilogue == b.DP_EPI_CLIP_ACCUM else None
    if epilogue == b.DP_EPI_CLIP_ACCUM:
        if acc_w is None:
            acc_w = torch.zeros(layer.n_weight, device="cuda")
        if acc_b is None and has_b:
            acc_b = torch.zeros(layer.n_bias, device="cuda")
    ws_bytes = b.dp_workspace_bytes(d, epilogue)
    assert ws_bytes > 0
    ws = torch.empty(ws_bytes + 256, dtype=torch.uint8, device="cuda")
    ws.fill_(0xAB)                                   # beyond the header dp_workspace_init clears, nothing may be assumed
    guard = ws[ws_bytes:].clone()
    b.check(b.dp_workspace_init(ws, ws_bytes), "dp_workspace_init")
    sq_ptr = sq.data_ptr() + 4 * sq_col
    st = b.dp_per_example_wgrad(d, X, dY, G_w, G_b, sq_ptr, sq_stride, epilogue, C_l, acc_w, acc_b, clip, ws, ws_bytes)
    if check_status:
        b.check(st, "dp_per_example_wgrad")
        b.check(b.dp_wgrad_check(ws), "dp_wgrad_check")
    torch.cuda.synchronize()
    assert torch.equal(ws[ws_bytes:], guard), "workspace overrun"
    out = dict(status=st, sq=sq.cpu().numpy() if own_sq else None, desc=d,
               uses_tc=bool(b.dp_wgrad_uses_tensor_cores(d, epilogue)))
    for k, v in dict(G_w=G_w, G_b=G_b, clip=clip, acc_w=acc_w, acc_b=acc_b).items():
        out[k] = v.cpu().numpy() if v is not None else None
    return out


def scaled_inputs(layer, Bn, dtype, *key, spread=True):
    """Layer inputs whose per-example gradient norms spread over ~3 decades, so that clipping
    thresholds can be placed with examples on both sides."""
    inp = synth.layer_inputs(layer, Bn, dtype, *key)
    if spread:
        s = np.logspace(-1.5, 1.0, Bn).astype(np.float32)
        shape = (Bn,) + (1,) * (inp["dY"].ndim - 1)
        dY = inp["dY"] * s.reshape(shape)
        if dtype == "bf16":
            inp["dY_bits"], dY = synth.round_to_bf16(dY)
        inp["dY"] = dY
    return inp
