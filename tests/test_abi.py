"""Host-side checks that need no GPU: the library loads, exports what the header declares, and
rejects bad arguments before launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def b():
    from paper_2109_12191_b200 import build
    build.build()
    from paper_2109_12191_b200 import binding
    return binding


def _declared():
    text = open(os.path.join(ROOT, "include", "dpstep.h")).read()
    return re.findall(r"^DP_API\s+[\w\s\*]+?\b(dp_\w+)\s*\(", text, flags=re.M)


def test_every_declared_symbol_is_exported(b):
    names = _declared()
    assert len(names) >= 12
    lib = ctypes.CDLL(b.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(names) == sorted(b.EXPORTS)


def test_status_strings(b):
    assert b.dp_status_string(b.DP_OK) == "ok"
    assert "workspace" in b.dp_status_string(b.DP_ERR_WORKSPACE)
    assert b.dp_status_string(99) == "unknown status"


def test_descriptor_validation_and_workspace_query(b):
    good = b.make_desc(b.DP_LAYER_CONV2D, b.DP_F32, 4, 8, 16, 10, 10, 3, 3, 1, 1, 1, 0)
    assert b.dp_workspace_bytes(good, b.DP_EPI_STORE_NORM) > 0
    assert b.dp_layer_groups(good) == 1
    sep = b.make_desc(b.DP_LAYER_CONV2D, b.DP_F32, 4, 8, 16, 10, 10, 3, 3, 1, 1, 1, 1)
    assert b.dp_layer_groups(sep) == 2
    nobias = b.make_desc(b.DP_LAYER_CONV2D, b.DP_F32, 4, 8, 16, 10, 10, 3, 3, 1, 1, 0, 1)
    assert b.dp_layer_groups(nobias) == 1
    norm = b.make_desc(b.DP_LAYER_NORM_AFFINE, b.DP_BF16, 4, 8, 8, 10, 10, bias_separate=1)
    assert b.dp_layer_groups(norm) == 2
    bad = [
        b.make_desc(7, b.DP_F32, 4, 8, 16, 10, 10, 3, 3, 1, 1),               # kind
        b.make_desc(b.DP_LAYER_CONV2D, 5, 4, 8, 16, 10, 10, 3, 3, 1, 1),      # dtype
        b.make_desc(b.DP_LAYER_CONV2D, b.DP_F32, 0, 8, 16, 10, 10, 3, 3, 1, 1),   # B = 0
        b.make_desc(b.DP_LAYER_CONV2D, b.DP_F32, 4, 8, 16, 10, 10, 3, 3, 0, 1),   # stride 0
        b.make_desc(b.DP_LAYER_CONV2D, b.DP_F32, 4, 8, 16, 2, 2, 7, 7, 1, 0),     # filter larger than padded input
        b.make_desc(b.DP_LAYER_DENSE, b.DP_F32, 4, 8, 16, 2, 2),                  # dense with H != 1
        b.make_desc(b.DP_LAYER_NORM_AFFINE, b.DP_F32, 4, 8, 16, 4, 4),            # norm with K_out != C_in
        b.make_desc(b.DP_LAYER_CONV2D, b.DP_F32, 4, 8, 16, 10, 10, 3, 3, 1, 1, impl=9),
    ]
    for d in bad:
        assert b.dp_workspace_bytes(d, 0) == 0
        assert b.dp_layer_groups(d) == 0
        assert b.dp_per_example_wgrad(d, 256, 256, 256, 256, 256, 1, 0, 1.0, None, None, None, 256, 1 << 20, stream=0) == b.DP_ERR_INVALID_ARG
    assert b.dp_workspace_bytes(good, 3) == 0


def test_wgrad_rejects_bad_arguments_without_launching(b):
    d = b.make_desc(b.DP_LAYER_CONV2D, b.DP_F32, 4, 8, 16, 10, 10, 3, 3, 1, 1, 1, 0)
    ws = b.dp_workspace_bytes(d, 0)
    A = 4096   # fake, aligned "device address"; nothing is dereferenced on the error paths
    call = lambda **kw: b.dp_per_example_wgrad(
        kw.get("d", d), kw.get("X", A), kw.get("dY", A), kw.get("G_w", A), kw.get("G_b", A), kw.get("sq", A),
        kw.get("stride", 1), kw.get("epi", 0), kw.get("C_l", 1.0), kw.get("acc_w", A), kw.get("acc_b", A), None,
        kw.get("ws", A), kw.get("ws_bytes", ws), stream=0)
    assert call(d=None) == b.DP_ERR_INVALID_ARG
    assert call(X=None) == b.DP_ERR_INVALID_ARG
    assert call(dY=A + 4) == b.DP_ERR_INVALID_ARG            # misaligned
    assert call(sq=None) == b.DP_ERR_INVALID_ARG
    assert call(stride=0) == b.DP_ERR_INVALID_ARG
    assert call(G_w=None) == b.DP_ERR_INVALID_ARG            # STORE needs G_w
    assert call(G_b=None) == b.DP_ERR_INVALID_ARG            # ... and G_b when the layer has a bias
    assert call(epi=5) == b.DP_ERR_INVALID_ARG
    assert call(epi=2, C_l=0.0) == b.DP_ERR_INVALID_ARG
    assert call(epi=2, C_l=float("nan")) == b.DP_ERR_INVALID_ARG
    assert call(epi=2, acc_w=None) == b.DP_ERR_INVALID_ARG
    assert call(ws=None) == b.DP_ERR_WORKSPACE
    assert call(ws=A + 16) == b.DP_ERR_WORKSPACE             # not 256-byte aligned
    assert call(ws_bytes=ws - 1) == b.DP_ERR_WORKSPACE
    forced = b.make_desc(b.DP_LAYER_CONV2D, b.DP_F32, 4, 3, 16, 10, 10, 3, 3, 1, 1, 1, 0, impl=b.DP_IMPL_TENSOR_CORE)
    assert b.dp_per_example_wgrad(forced, A, A, A, A, A, 1, 0, 1.0, None, None, None, A, 1 << 24, stream=0) == b.DP_ERR_UNSUPPORTED


def test_workspace_init_rejects_bad_arguments(b):
    A = 4096
    assert b.dp_workspace_init(None, 1 << 20, stream=0) == b.DP_ERR_WORKSPACE
    assert b.dp_workspace_init(A + 16, 1 << 20, stream=0) == b.DP_ERR_WORKSPACE     # not 256-byte aligned
    assert b.dp_workspace_init(A, 1024, stream=0) == b.DP_ERR_WORKSPACE             # smaller than the header it clears
    d = b.make_desc(b.DP_LAYER_DENSE, b.DP_F32, 1, 4, 4)
    assert b.dp_workspace_bytes(d, b.DP_EPI_NORM_ONLY) >= 16384                     # every workspace holds the header


def test_clip_rejects_bad_arguments(b):
    A = 4096
    P = [100, 7]
    ws = b.dp_clip_workspace_bytes(4, P)
    assert ws > 0
    assert b.dp_clip_workspace_bytes(0, P) == 0
    assert b.dp_clip_workspace_bytes(4, [10, 0]) == 0
    ok = dict(mode=0, B=4, G=[A, A], P_l=P, sqnorm=None, C=1.0, acc=[A, A], norms_out=None, clip_out=None,
              workspace=A, workspace_bytes=ws)
    def call(**kw):
        a = dict(ok); a.update(kw)
        return b.dp_clip_accumulate(a["mode"], a["B"], a["G"], a["P_l"], a["sqnorm"], a["C"], a["acc"], a["norms_out"],
                                    a["clip_out"], a["workspace"], a["workspace_bytes"], stream=0)
    assert call(mode=3) == b.DP_ERR_INVALID_ARG
    assert call(B=0) == b.DP_ERR_INVALID_ARG
    assert call(C=0.0) == b.DP_ERR_INVALID_ARG
    assert call(C=-1.0) == b.DP_ERR_INVALID_ARG
    assert call(C=float("nan")) == b.DP_ERR_INVALID_ARG
    assert call(G=[A, None]) == b.DP_ERR_INVALID_ARG
    assert call(acc=[None, A]) == b.DP_ERR_INVALID_ARG
    assert call(P_l=[100, -1]) == b.DP_ERR_INVALID_ARG
    assert call(G=[A + 2, A]) == b.DP_ERR_INVALID_ARG
    assert call(workspace=None) == b.DP_ERR_WORKSPACE
    assert call(workspace_bytes=ws - 1) == b.DP_ERR_WORKSPACE


def test_noised_clip_rejects_bad_arguments(b):
    A = 4096
    P = [100, 8]
    ws = b.dp_clip_workspace_bytes(4, P)
    ok = dict(mode=0, B=4, G=[A, A], P_l=P, param_offset_l=[0, 100], sqnorm=None, C=1.0, sigma=1.0, total_batch=16, seed=1,
              step=2, example0=4, acc=[A, A], norms_out=None, clip_out=None, workspace=A, workspace_bytes=ws, stream=0)
    call = lambda **kw: b.dp_clip_accumulate_noised(**{**ok, **kw})
    assert call(param_offset_l=None) == b.DP_ERR_INVALID_ARG
    assert call(param_offset_l=[0, -1]) == b.DP_ERR_INVALID_ARG
    assert call(param_offset_l=[0, 2**34]) == b.DP_ERR_UNSUPPORTED     # global index beyond the stream's counter word
    assert call(sigma=-1.0) == b.DP_ERR_INVALID_ARG
    assert call(sigma=float("nan")) == b.DP_ERR_INVALID_ARG
    assert call(C=float("inf")) == b.DP_ERR_INVALID_ARG                # no finite noise scale
    assert call(total_batch=0) == b.DP_ERR_INVALID_ARG
    assert call(example0=-1) == b.DP_ERR_INVALID_ARG
    assert call(example0=2**31 - 3) == b.DP_ERR_INVALID_ARG            # example index leaves its 31 bits
    assert call(G=[A, None]) == b.DP_ERR_INVALID_ARG                   # the shared checks of dp_clip_accumulate
    assert call(workspace=None) == b.DP_ERR_WORKSPACE
    assert b.dp_debug_example_noise_z(None, 4, 0, 0, 0, 0, stream=0) == b.DP_ERR_INVALID_ARG
    assert b.dp_debug_example_noise_z(A, 4, 0, 2**31, 0, 0, stream=0) == b.DP_ERR_INVALID_ARG


def test_grouped_and_micro_clip_reject_bad_arguments(b):
    A = 4096
    P = [100, 8, 16]
    ws = b.dp_clip_workspace_bytes(4, P)
    grouped = lambda **kw: b.dp_clip_accumulate_grouped(**{**dict(B=4, M=2, group_of=[0, 1, 1], G=[A, A, A], P_l=P, sqnorm=None,
                                                                  C=1.0, acc=[A, A, A], norms_out=None, clip_out=None,
                                                                  workspace=A, workspace_bytes=ws, stream=0), **kw})
    assert grouped(group_of=None) == b.DP_ERR_INVALID_ARG
    assert grouped(group_of=[0, 0, 0]) == b.DP_ERR_INVALID_ARG          # group 1 owns no tensor
    assert grouped(group_of=[0, 1, 2]) == b.DP_ERR_INVALID_ARG          # index outside [0, M)
    assert grouped(M=0) == b.DP_ERR_INVALID_ARG
    assert grouped(M=4, group_of=[0, 1, 2]) == b.DP_ERR_INVALID_ARG     # more groups than tensors
    assert grouped(C=0.0) == b.DP_ERR_INVALID_ARG
    assert grouped(workspace=None) == b.DP_ERR_WORKSPACE
    micro = lambda **kw: b.dp_clip_accumulate_micro(**{**dict(B=4, micro=2, G=[A, A, A], P_l=P, C=1.0, acc=[A, A, A],
                                                              norms_out=None, clip_out=None, workspace=A, workspace_bytes=ws,
                                                              stream=0), **kw})
    assert micro(micro=0) == b.DP_ERR_INVALID_ARG
    assert micro(micro=3) == b.DP_ERR_INVALID_ARG                       # does not divide B
    assert micro(G=[A, None, A]) == b.DP_ERR_INVALID_ARG
    assert micro(workspace_bytes=ws - 1) == b.DP_ERR_WORKSPACE


def test_noise_rejects_bad_arguments(b):
    A = 4096
    call = lambda acc=A, P=16, off=0, sigma=1.0, C=1.0, tb=8, out=A: b.dp_noise_average(acc, P, off, sigma, C, tb, 0, 0, out, stream=0)
    assert call(acc=None) == b.DP_ERR_INVALID_ARG
    assert call(out=None) == b.DP_ERR_INVALID_ARG
    assert call(P=0) == b.DP_ERR_INVALID_ARG
    assert call(off=-1) == b.DP_ERR_INVALID_ARG
    assert call(sigma=-0.1) == b.DP_ERR_INVALID_ARG
    assert call(sigma=float("nan")) == b.DP_ERR_INVALID_ARG
    assert call(C=0.0) == b.DP_ERR_INVALID_ARG
    assert call(C=float("inf")) == b.DP_ERR_INVALID_ARG       # infinite C with sigma > 0 has no finite noise scale
    assert call(tb=0) == b.DP_ERR_INVALID_ARG
    assert call(acc=A + 4) == b.DP_ERR_INVALID_ARG
    sgd = lambda acc=A, theta=A, lr=0.1, mu=0.9, sigma=1.0, C=1.0: b.dp_noise_average_sgd(acc, 16, 0, sigma, C, 8, 0, 0, lr, mu, theta, None, None, stream=0)
    assert sgd(acc=None) == b.DP_ERR_INVALID_ARG
    assert sgd(theta=None) == b.DP_ERR_INVALID_ARG
    assert sgd(lr=float("nan")) == b.DP_ERR_INVALID_ARG
    assert sgd(mu=-0.1) == b.DP_ERR_INVALID_ARG
    assert sgd(C=float("inf")) == b.DP_ERR_INVALID_ARG
    assert b.dp_debug_philox_raw(None, 4, 0, 0, 0, stream=0) == b.DP_ERR_INVALID_ARG
    assert b.dp_debug_philox_raw(A, 0, 0, 0, 0, stream=0) == b.DP_ERR_INVALID_ARG
    assert b.dp_debug_noise_z(None, 4, 0, 0, 0, stream=0) == b.DP_ERR_INVALID_ARG


def test_binding_has_no_fallback():
    src = open(os.path.join(ROOT, "paper_2109_12191_b200", "binding.py")).read()
    assert "oracle" not in src.replace("no CPU or PyTorch fallback", "")
    for path in ("paper_2109_12191_b200/build.py", "paper_2109_12191_b200/synth.py"):
        assert "import oracle" not in open(os.path.join(ROOT, path)).read()
