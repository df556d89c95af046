"""ctypes binding of libdpstep.so: the same entry points as include/dpstep.h, argument
marshalling only.  Tensors are torch CUDA tensors (or raw device addresses as int); every
step of the computation runs inside the library's kernels.  There is no fallback: if the
compiled library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdpstep.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2109_12191_b200.build` "
                      "(there is no CPU or PyTorch fallback)")
_lib = ctypes.CDLL(LIB_PATH)

# enums of dpstep.h
DP_OK, DP_ERR_INVALID_ARG, DP_ERR_UNSUPPORTED, DP_ERR_WORKSPACE, DP_ERR_CUDA, DP_ERR_TIMEOUT = range(6)
DP_F32, DP_BF16, DP_TF32 = 0, 1, 2
DP_LAYER_DENSE, DP_LAYER_CONV2D, DP_LAYER_NORM_AFFINE = 0, 1, 2
DP_CLIP_GLOBAL, DP_CLIP_PER_LAYER = 0, 1
DP_EPI_STORE_NORM, DP_EPI_NORM_ONLY, DP_EPI_CLIP_ACCUM = 0, 1, 2
DP_IMPL_AUTO, DP_IMPL_CUDA_CORE, DP_IMPL_TENSOR_CORE = 0, 1, 2

EXPORTS = ["dp_layer_groups", "dp_workspace_bytes", "dp_per_example_wgrad", "dp_clip_workspace_bytes",
           "dp_clip_accumulate", "dp_noise_average", "dp_debug_philox_raw", "dp_debug_noise_z",
           "dp_wgrad_check", "dp_wgrad_uses_tensor_cores", "dp_status_string", "dp_last_cuda_error",
           "dp_debug_launch_count", "dp_debug_wgrad_plan", "dp_clip_accumulate_static",
           "dp_clip_static_scratch_bytes", "dp_noise_average_sgd", "dp_clip_accumulate_noised",
           "dp_debug_example_noise_z", "dp_clip_accumulate_grouped", "dp_clip_accumulate_micro",
           "dp_per_example_wgrad_scaled", "dp_clip_factors", "dp_scale_accumulate", "dp_workspace_init",
           "dp_debug_set_wait_polls", "dp_set_sm_target", "dp_debug_set_single_pass"]


class dp_layer_desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("kind", "dtype", "B", "C_in", "H", "W", "K_out", "R", "S",
                                            "stride", "pad", "has_bias", "bias_separate", "impl")]


class DpError(RuntimeError):
    def __init__(self, status, where=""):
        self.status = status
        extra = dp_last_cuda_error() if status == DP_ERR_CUDA else ""
        super().__init__(f"{where}: {dp_status_string(status)} ({status}) {extra}".strip())


def check(status, where="dpstep"):
    if status != DP_OK:
        raise DpError(status, where)


_vp, _ll, _ull, _f, _i, _sz = (ctypes.c_void_p, ctypes.c_longlong, ctypes.c_ulonglong, ctypes.c_float,
                               ctypes.c_int, ctypes.c_size_t)
_dp = ctypes.POINTER(dp_layer_desc)
_lib.dp_layer_groups.argtypes = [_dp]; _lib.dp_layer_groups.restype = _i
_lib.dp_workspace_bytes.argtypes = [_dp, _i]; _lib.dp_workspace_bytes.restype = _sz
_lib.dp_wgrad_uses_tensor_cores.argtypes = [_dp, _i]; _lib.dp_wgrad_uses_tensor_cores.restype = _i
_lib.dp_per_example_wgrad.argtypes = [_dp, _vp, _vp, _vp, _vp, _vp, _ll, _i, _f, _vp, _vp, _vp, _vp, _sz, _vp]
_lib.dp_per_example_wgrad.restype = _i
_lib.dp_per_example_wgrad_scaled.argtypes = [_dp, _vp, _vp, _vp, _vp, _ll, _vp, _vp, _vp, _sz, _vp]
_lib.dp_per_example_wgrad_scaled.restype = _i
_lib.dp_clip_factors.argtypes = [_i, _i, _i, _vp, _f, _vp, _vp, _vp]; _lib.dp_clip_factors.restype = _i
_lib.dp_scale_accumulate.argtypes = [_i, _i, ctypes.POINTER(_vp), ctypes.POINTER(_ll), _vp, _i, ctypes.POINTER(_vp), _vp]
_lib.dp_scale_accumulate.restype = _i
_lib.dp_clip_workspace_bytes.argtypes = [_i, _i, ctypes.POINTER(_ll)]; _lib.dp_clip_workspace_bytes.restype = _sz
_lib.dp_clip_accumulate.argtypes = [_i, _i, _i, ctypes.POINTER(_vp), ctypes.POINTER(_ll), _vp, _f,
                                    ctypes.POINTER(_vp), _vp, _vp, _vp, _sz, _vp]
_lib.dp_clip_accumulate.restype = _i
_lib.dp_clip_accumulate_noised.argtypes = [_i, _i, _i, ctypes.POINTER(_vp), ctypes.POINTER(_ll), ctypes.POINTER(_ll), _vp,
                                           _f, _f, _ll, _ull, _ull, _ll, ctypes.POINTER(_vp), _vp, _vp, _vp, _sz, _vp]
_lib.dp_clip_accumulate_noised.restype = _i
_lib.dp_debug_example_noise_z.argtypes = [_vp, _ll, _ll, _ll, _ull, _ull, _vp]; _lib.dp_debug_example_noise_z.restype = _i
_lib.dp_clip_accumulate_grouped.argtypes = [_i, _i, _i, ctypes.POINTER(_i), ctypes.POINTER(_vp), ctypes.POINTER(_ll), _vp, _f,
                                            ctypes.POINTER(_vp), _vp, _vp, _vp, _sz, _vp]
_lib.dp_clip_accumulate_grouped.restype = _i
_lib.dp_clip_accumulate_micro.argtypes = [_i, _i, _i, ctypes.POINTER(_vp), ctypes.POINTER(_ll), _f, ctypes.POINTER(_vp), _vp,
                                          _vp, _vp, _sz, _vp]
_lib.dp_clip_accumulate_micro.restype = _i
_lib.dp_clip_accumulate_static.argtypes = [_i, _i, _i, ctypes.POINTER(_vp), ctypes.POINTER(_ll), _vp, _f,
                                           ctypes.POINTER(_vp), _vp, _vp, _vp]
_lib.dp_clip_accumulate_static.restype = _i
_lib.dp_clip_static_scratch_bytes.argtypes = []; _lib.dp_clip_static_scratch_bytes.restype = _sz
_lib.dp_noise_average.argtypes = [_vp, _ll, _ll, _f, _f, _ll, _ull, _ull, _vp, _vp]; _lib.dp_noise_average.restype = _i
_lib.dp_noise_average_sgd.argtypes = [_vp, _ll, _ll, _f, _f, _ll, _ull, _ull, _f, _f, _vp, _vp, _vp, _vp]
_lib.dp_noise_average_sgd.restype = _i
_lib.dp_debug_philox_raw.argtypes = [_vp, _ll, _ll, _ull, _ull, _vp]; _lib.dp_debug_philox_raw.restype = _i
_lib.dp_debug_noise_z.argtypes = [_vp, _ll, _ll, _ull, _ull, _vp]; _lib.dp_debug_noise_z.restype = _i
_lib.dp_wgrad_check.argtypes = [_vp, _vp]; _lib.dp_wgrad_check.restype = _i
_lib.dp_workspace_init.argtypes = [_vp, _sz, _vp]; _lib.dp_workspace_init.restype = _i
_lib.dp_debug_set_wait_polls.argtypes = [_ll]; _lib.dp_debug_set_wait_polls.restype = None
_lib.dp_set_sm_target.argtypes = [_i]; _lib.dp_set_sm_target.restype = _i
_lib.dp_debug_set_single_pass.argtypes = [_i]; _lib.dp_debug_set_single_pass.restype = None
_lib.dp_status_string.argtypes = [_i]; _lib.dp_status_string.restype = ctypes.c_char_p
_lib.dp_last_cuda_error.argtypes = []; _lib.dp_last_cuda_error.restype = ctypes.c_char_p
_lib.dp_debug_launch_count.argtypes = []; _lib.dp_debug_launch_count.restype = _ull
_lib.dp_debug_wgrad_plan.argtypes = [_dp, _i, ctypes.POINTER(_i), _i]; _lib.dp_debug_wgrad_plan.restype = _i


def _ptr(t):
    """Device address of a torch tensor (must be contiguous), an int address, or None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def _nbytes(t):
    return t.numel() * t.element_size()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


def make_desc(kind, dtype, B, C_in, K_out, H=1, W=1, R=1, S=1, stride=1, pad=0, has_bias=0,
              bias_separate=0, impl=DP_IMPL_AUTO):
    return dp_layer_desc(kind, dtype, B, C_in, H, W, K_out, R, S, stride, pad, int(has_bias), int(bias_separate), impl)


def dp_layer_groups(desc):
    return _lib.dp_layer_groups(ctypes.byref(desc))


def dp_workspace_bytes(desc, epilogue):
    return _lib.dp_workspace_bytes(ctypes.byref(desc), epilogue)


def dp_wgrad_uses_tensor_cores(desc, epilogue):
    return _lib.dp_wgrad_uses_tensor_cores(ctypes.byref(desc), epilogue)


def dp_per_example_wgrad(desc, X, dY, G_w, G_b, sqnorm, sqnorm_stride, epilogue, C_l, acc_w, acc_b, clip_out,
                         workspace, workspace_bytes=None, stream=None):
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None or isinstance(workspace, int) else _nbytes(workspace)
    return _lib.dp_per_example_wgrad(ctypes.byref(desc) if desc is not None else None, _ptr(X), _ptr(dY), _ptr(G_w),
                                     _ptr(G_b), _ptr(sqnorm), sqnorm_stride, epilogue, C_l, _ptr(acc_w), _ptr(acc_b),
                                     _ptr(clip_out), _ptr(workspace), workspace_bytes, _stream(stream))


def dp_per_example_wgrad_scaled(desc, X, dY, factor_w, factor_b, factor_stride, acc_w, acc_b, workspace, workspace_bytes=None,
                                stream=None):
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None or isinstance(workspace, int) else _nbytes(workspace)
    return _lib.dp_per_example_wgrad_scaled(ctypes.byref(desc) if desc is not None else None, _ptr(X), _ptr(dY), _ptr(factor_w),
                                            _ptr(factor_b), factor_stride, _ptr(acc_w), _ptr(acc_b), _ptr(workspace),
                                            workspace_bytes, _stream(stream))


def dp_clip_factors(mode, B, L, sqnorm, C, norms_out, factors_out, stream=None):
    return _lib.dp_clip_factors(mode, B, L, _ptr(sqnorm), C, _ptr(norms_out), _ptr(factors_out), _stream(stream))


def dp_scale_accumulate(B, G, P_l, factor, per_tensor, acc, stream=None):
    L = len(P_l)
    Gp = (_vp * L)(*[_ptr(g) for g in G]) if G is not None else None
    Ap = (_vp * L)(*[_ptr(a) for a in acc]) if acc is not None else None
    return _lib.dp_scale_accumulate(B, L, Gp, (_ll * L)(*P_l), _ptr(factor), per_tensor, Ap, _stream(stream))


def dp_clip_workspace_bytes(B, P_l):
    L = len(P_l)
    return _lib.dp_clip_workspace_bytes(B, L, (_ll * L)(*P_l))


def dp_clip_accumulate(mode, B, G, P_l, sqnorm, C, acc, norms_out, clip_out, workspace, workspace_bytes=None,
                       stream=None):
    L = len(P_l)
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None or isinstance(workspace, int) else _nbytes(workspace)
    Gp = (_vp * L)(*[_ptr(g) for g in G]) if G is not None else None
    Ap = (_vp * L)(*[_ptr(a) for a in acc]) if acc is not None else None
    return _lib.dp_clip_accumulate(mode, B, L, Gp, (_ll * L)(*P_l), _ptr(sqnorm), C, Ap, _ptr(norms_out),
                                   _ptr(clip_out), _ptr(workspace), workspace_bytes, _stream(stream))


def dp_clip_accumulate_noised(mode, B, G, P_l, param_offset_l, sqnorm, C, sigma, total_batch, seed, step, example0, acc,
                              norms_out, clip_out, workspace, workspace_bytes=None, stream=None):
    """dp_clip_accumulate with each example's own noise draw added before the sum."""
    L = len(P_l)
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None or isinstance(workspace, int) else _nbytes(workspace)
    Gp = (_vp * L)(*[_ptr(g) for g in G]) if G is not None else None
    Ap = (_vp * L)(*[_ptr(a) for a in acc]) if acc is not None else None
    Op = (_ll * L)(*param_offset_l) if param_offset_l is not None else None
    return _lib.dp_clip_accumulate_noised(mode, B, L, Gp, (_ll * L)(*P_l), Op, _ptr(sqnorm), C, sigma, total_batch, seed,
                                          step, example0, Ap, _ptr(norms_out), _ptr(clip_out), _ptr(workspace),
                                          workspace_bytes, _stream(stream))


def dp_debug_example_noise_z(z, count, first_index, example, seed, step, stream=None):
    return _lib.dp_debug_example_noise_z(_ptr(z), count, first_index, example, seed, step, _stream(stream))


def dp_clip_accumulate_grouped(B, M, group_of, G, P_l, sqnorm, C, acc, norms_out, clip_out, workspace, workspace_bytes=None,
                               stream=None):
    """dp_clip_accumulate over M groups of tensors, each clipped to C/sqrt(M)."""
    L = len(P_l)
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None or isinstance(workspace, int) else _nbytes(workspace)
    Gp = (_vp * L)(*[_ptr(g) for g in G]) if G is not None else None
    Ap = (_vp * L)(*[_ptr(a) for a in acc]) if acc is not None else None
    go = (_i * L)(*group_of) if group_of is not None else None
    return _lib.dp_clip_accumulate_grouped(B, L, M, go, Gp, (_ll * L)(*P_l), _ptr(sqnorm), C, Ap, _ptr(norms_out),
                                           _ptr(clip_out), _ptr(workspace), workspace_bytes, _stream(stream))


def dp_clip_accumulate_micro(B, micro, G, P_l, C, acc, norms_out, clip_out, workspace, workspace_bytes=None, stream=None):
    """Whole-model clipping of the means of runs of `micro` consecutive examples."""
    L = len(P_l)
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None or isinstance(workspace, int) else _nbytes(workspace)
    Gp = (_vp * L)(*[_ptr(g) for g in G]) if G is not None else None
    Ap = (_vp * L)(*[_ptr(a) for a in acc]) if acc is not None else None
    return _lib.dp_clip_accumulate_micro(B, L, micro, Gp, (_ll * L)(*P_l), C, Ap, _ptr(norms_out), _ptr(clip_out),
                                         _ptr(workspace), workspace_bytes, _stream(stream))


def dp_clip_accumulate_static(mode, B, G, P_l, sqnorm, C, acc, norms_out, clip_out, stream=None):
    """dp_clip_accumulate with the library's built-in scratch array instead of a caller workspace."""
    L = len(P_l)
    Gp = (_vp * L)(*[_ptr(g) for g in G]) if G is not None else None
    Ap = (_vp * L)(*[_ptr(a) for a in acc]) if acc is not None else None
    return _lib.dp_clip_accumulate_static(mode, B, L, Gp, (_ll * L)(*P_l), _ptr(sqnorm), C, Ap, _ptr(norms_out),
                                          _ptr(clip_out), _stream(stream))


def dp_clip_static_scratch_bytes():
    return _lib.dp_clip_static_scratch_bytes()


def dp_noise_average(acc, P, param_offset, sigma, C, total_batch, seed, step, out, stream=None):
    return _lib.dp_noise_average(_ptr(acc), P, param_offset, sigma, C, total_batch, seed, step, _ptr(out), _stream(stream))


def dp_noise_average_sgd(acc, P, param_offset, sigma, C, total_batch, seed, step, lr, momentum, theta, momentum_buf=None,
                         g_out=None, stream=None):
    return _lib.dp_noise_average_sgd(_ptr(acc), P, param_offset, sigma, C, total_batch, seed, step, lr, momentum,
                                     _ptr(theta), _ptr(momentum_buf), _ptr(g_out), _stream(stream))


def dp_debug_philox_raw(out4, n_blocks, first_block, seed, step, stream=None):
    return _lib.dp_debug_philox_raw(_ptr(out4), n_blocks, first_block, seed, step, _stream(stream))


def dp_debug_noise_z(z, count, first_index, seed, step, stream=None):
    return _lib.dp_debug_noise_z(_ptr(z), count, first_index, seed, step, _stream(stream))


def dp_workspace_init(workspace, workspace_bytes=None, stream=None):
    if workspace_bytes is None:
        workspace_bytes = 0 if workspace is None or isinstance(workspace, int) else _nbytes(workspace)
    return _lib.dp_workspace_init(_ptr(workspace), workspace_bytes, _stream(stream))


def dp_set_sm_target(sms):
    return _lib.dp_set_sm_target(sms)


def dp_debug_set_single_pass(on):
    _lib.dp_debug_set_single_pass(int(on))


def dp_debug_set_wait_polls(polls):
    _lib.dp_debug_set_wait_polls(polls)


def dp_wgrad_check(workspace, stream=None):
    return _lib.dp_wgrad_check(_ptr(workspace), _stream(stream))


def dp_status_string(status):
    return _lib.dp_status_string(status).decode()


def dp_last_cuda_error():
    return _lib.dp_last_cuda_error().decode()


def dp_debug_launch_count():
    return _lib.dp_debug_launch_count()


PLAN_FIELDS = ("a_is_x", "a_ext", "b_ext", "m_tiles", "n_tiles", "NT", "OWt", "OHt", "Kt", "k_tiles", "stages", "stage_bytes")


def dp_debug_wgrad_plan(desc, epilogue=DP_EPI_STORE_NORM):
    out = (_i * 12)()
    n = _lib.dp_debug_wgrad_plan(ctypes.byref(desc), epilogue, out, 12)
    return dict(zip(PLAN_FIELDS, list(out)[:n])) if n else None
