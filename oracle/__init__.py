"""Float64 CPU oracle of the DPSGD gradient-privatisation step -- TEST INFRASTRUCTURE.

This package wraps ``dp_oracle.c`` (plain C loops, double arithmetic) with ctypes and
adds the few lines of glue that chain its pieces in the order of the paper's section 2
(per-example gradient -> L2 norm -> clip to C -> sum over the batch and over
accumulation chunks -> + N(0, sigma^2 C^2) -> / |B|) and of section 3.5 (each of M
groups clipped to C/sqrt(M)).

Only tests, the smoke check and the CPU-baseline leg of the benchmark may import this
package.  It imports nothing from the CUDA library and the CUDA library imports nothing
from it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dp_oracle.c")
_SO = os.path.join(_HERE, "libdp_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile dp_oracle.c with gcc (OpenMP) into libdp_oracle.so next to the source."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.run(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _SO)
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def threads() -> int:
    """Number of OpenMP threads the C loops will use."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        return int(env.split(",")[0])
    return len(os.sched_getaffinity(0))


_f32p = ctypes.POINTER(ctypes.c_float)
_f64p = ctypes.POINTER(ctypes.c_double)
_u32p = ctypes.POINTER(ctypes.c_uint32)


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(_f32p)


def _f64(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(_f64p)


def conv_out_size(H, R, stride, pad):
    return (H + 2 * pad - R) // stride + 1


# ----------------------------------------------------------------------------- layers
def conv_wgrad(X, dY, R, S, stride, pad, bias=True):
    """X [B,H,W,Cin], dY [B,OH,OW,Kout] (float32 containers) -> dW [B,Kout,R,S,Cin], db [B,Kout] | None."""
    lib = _load()
    X, xp = _f32(X)
    dY, yp = _f32(dY)
    B, H, W, Cin = X.shape
    B2, OH, OW, Kout = dY.shape
    assert B == B2 and OH == conv_out_size(H, R, stride, pad) and OW == conv_out_size(W, S, stride, pad)
    dW = np.empty((B, Kout, R, S, Cin), dtype=np.float64)
    db = np.empty((B, Kout), dtype=np.float64) if bias else None
    lib.oracle_conv_wgrad(xp, yp, B, H, W, Cin, Kout, R, S, stride, pad,
                          dW.ctypes.data_as(_f64p), db.ctypes.data_as(_f64p) if bias else None)
    return dW, db


def dense_wgrad(X, dY, bias=True):
    """X [B,Cin], dY [B,Kout] -> dW [B,Kout,Cin], db [B,Kout] | None."""
    lib = _load()
    X, xp = _f32(X)
    dY, yp = _f32(dY)
    B, Cin = X.shape
    Kout = dY.shape[1]
    dW = np.empty((B, Kout, Cin), dtype=np.float64)
    db = np.empty((B, Kout), dtype=np.float64) if bias else None
    lib.oracle_dense_wgrad(xp, yp, B, Cin, Kout, dW.ctypes.data_as(_f64p),
                           db.ctypes.data_as(_f64p) if bias else None)
    return dW, db


def norm_affine_wgrad(xhat, dY):
    """xhat, dY [B,H,W,C] (or [B,HW,C]) -> dgamma [B,C], dbeta [B,C]."""
    lib = _load()
    xhat, xp = _f32(xhat)
    dY, yp = _f32(dY)
    B, C = xhat.shape[0], xhat.shape[-1]
    HW = int(np.prod(xhat.shape[1:-1]))
    dg = np.empty((B, C), dtype=np.float64)
    dbeta = np.empty((B, C), dtype=np.float64)
    lib.oracle_norm_affine_wgrad(xp, yp, B, HW, C, dg.ctypes.data_as(_f64p), dbeta.ctypes.data_as(_f64p))
    return dg, dbeta


# ----------------------------------------------------------------- norm / clip / sum
def sqnorm(G):
    """G [B, ...] float32 or float64 -> per-example sum of squares [B] (float64)."""
    lib = _load()
    B = G.shape[0]
    P = int(np.prod(G.shape[1:]))
    s = np.zeros(B, dtype=np.float64)
    if G.dtype == np.float32:
        G, gp = _f32(G)
        lib.oracle_sqnorm_add_f32(gp, B, ctypes.c_size_t(P), s.ctypes.data_as(_f64p))
    else:
        G, gp = _f64(G)
        lib.oracle_sqnorm_add_f64(gp, B, ctypes.c_size_t(P), s.ctypes.data_as(_f64p))
    return s


def clip_factor(sq, C):
    """min(1, C/sqrt(sq)) elementwise, as a branch (sq <= C^2 -> exactly 1)."""
    lib = _load()
    sq, sp = _f64(sq)
    out = np.empty_like(sq)
    lib.oracle_clip_factor(sp, ctypes.c_size_t(sq.size), ctypes.c_double(C), out.ctypes.data_as(_f64p))
    return out


def clip_accumulate(G, factor, acc):
    """acc[P] += sum_n factor[n] * G[n, :]; acc is float64 and updated in place."""
    lib = _load()
    B = G.shape[0]
    P = int(np.prod(G.shape[1:]))
    assert acc.dtype == np.float64 and acc.size == P and acc.flags.c_contiguous
    factor, fp = _f64(factor)
    assert factor.size == B
    if G.dtype == np.float32:
        G, gp = _f32(G)
        lib.oracle_clip_accumulate_f32(gp, B, ctypes.c_size_t(P), fp, acc.ctypes.data_as(_f64p))
    else:
        G, gp = _f64(G)
        lib.oracle_clip_accumulate_f64(gp, B, ctypes.c_size_t(P), fp, acc.ctypes.data_as(_f64p))
    return acc


def clipped_sum(groups, C, mode, acc=None):
    """One chunk of the clipped sum.

    groups : list of L arrays [B, ...], the per-example gradients of L parameter tensors.
    mode   : "global"    -- one factor per example from the whole-model norm (section 2);
             "per_layer" -- one factor per (example, tensor) with threshold C/sqrt(L) (section 3.5).
    acc    : list of L float64 arrays to add into (created as zeros when None).
    Returns (acc, sq [B,L], factor [B] or [B,L]).
    """
    L = len(groups)
    B = groups[0].shape[0]
    sq = np.stack([sqnorm(g) for g in groups], axis=1)              # [B, L]
    if mode == "global":
        factor = clip_factor(sq.sum(axis=1), C)                     # [B]
        per_group = [factor] * L
    elif mode == "per_layer":
        factor = clip_factor(sq, C / np.sqrt(L)).reshape(B, L)      # [B, L]
        per_group = [np.ascontiguousarray(factor[:, l]) for l in range(L)]
    else:
        raise ValueError(mode)
    if acc is None:
        acc = [np.zeros(int(np.prod(g.shape[1:])), dtype=np.float64) for g in groups]
    for g, f, a in zip(groups, per_group, acc):
        clip_accumulate(g, f, a)
    return acc, sq, factor


def clipped_sum_grouped(groups, group_of, C, acc=None):
    """Section 3.5 with M groups of parameter tensors (the paper's pipeline stages): group m holds the tensors l with
    group_of[l] == m, its per-example norm is taken over all of them, and it is clipped to C/sqrt(M).
    Returns (acc, sq [B, M], factor [B, M])."""
    L, B = len(groups), groups[0].shape[0]
    group_of = [int(m) for m in group_of]
    M = max(group_of) + 1
    assert len(group_of) == L and sorted(set(group_of)) == list(range(M))
    sq = np.zeros((B, M), dtype=np.float64)
    for g, m in zip(groups, group_of):
        sq[:, m] += sqnorm(g)
    factor = clip_factor(sq, C / np.sqrt(M)).reshape(B, M)
    if acc is None:
        acc = [np.zeros(int(np.prod(g.shape[1:])), dtype=np.float64) for g in groups]
    for g, m, a in zip(groups, group_of, acc):
        clip_accumulate(g, np.ascontiguousarray(factor[:, m]), a)
    return acc, sq, factor


def clipped_sum_micro(groups, C, micro, acc=None):
    """Micro-batch clipping (the TFDP option of the paper's Table 1): consecutive runs of `micro` examples are
    averaged first, the average is clipped to C over the whole model, and the clipped averages are summed.
    Returns (acc, sq [B/micro] of the averages, factor [B/micro])."""
    B = groups[0].shape[0]
    assert micro >= 1 and B % micro == 0
    means = [g.reshape(B // micro, micro, -1).astype(np.float64).mean(axis=1) for g in groups]
    acc, sq, factor = clipped_sum(means, C, "global", acc)
    return acc, sq.sum(axis=1), factor


# ----------------------------------------------------------------------------- noise
def philox4x32_10(ctr, key):
    """Raw Philox4x32-10: 4 counter words, 2 key words -> 4 output words."""
    lib = _load()
    c = (ctypes.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    o = (ctypes.c_uint32 * 4)()
    lib.oracle_philox4x32_10(c, k, o)
    return [int(v) for v in o]


def philox_blocks(seed, step, first_block, n_blocks):
    """Raw words [n_blocks,4] of blocks first_block.. for the (seed, step) stream."""
    lib = _load()
    out = np.empty((n_blocks, 4), dtype=np.uint32)
    o = (ctypes.c_uint32 * 4)()
    for j in range(n_blocks):
        lib.oracle_philox_block(ctypes.c_uint64(seed), ctypes.c_uint64(step), ctypes.c_uint64(first_block + j), o)
        out[j] = o[:]
    return out


def noise_z(seed, step, first_index, count):
    """Standard normals z_i for global parameter indices first_index .. +count-1."""
    lib = _load()
    z = np.empty(count, dtype=np.float64)
    lib.oracle_noise_z(ctypes.c_uint64(seed), ctypes.c_uint64(step), ctypes.c_uint64(first_index),
                       ctypes.c_size_t(count), z.ctypes.data_as(_f64p))
    return z


def noise_average(acc, param_offset, sigma, C, total_batch, seed, step):
    """(acc + sigma*C*z) / |B| (section 2, equation for g_t).  C here is always the global C."""
    lib = _load()
    acc, ap = _f64(acc)
    out = np.empty_like(acc)
    lib.oracle_noise_average(ap, ctypes.c_size_t(acc.size), ctypes.c_uint64(param_offset),
                             ctypes.c_double(sigma), ctypes.c_double(C), ctypes.c_double(total_batch),
                             ctypes.c_uint64(seed), ctypes.c_uint64(step), out.ctypes.data_as(_f64p))
    return out


def example_noise_z(seed, step, example, first_index, count):
    """Standard normals of example `example`'s own stream for global parameter indices first_index .. +count-1."""
    lib = _load()
    z = np.empty(count, dtype=np.float64)
    lib.oracle_example_noise_z(ctypes.c_uint64(seed), ctypes.c_uint64(step), ctypes.c_uint32(example),
                               ctypes.c_uint64(first_index), ctypes.c_size_t(count), z.ctypes.data_as(_f64p))
    return z


def clip_accumulate_noised(G, factor, acc, sd, seed, step, example0, param_offset):
    """acc[P] += sum_n (factor[n]*G[n,:] + sd*z_{example0+n}); G float32 [B, P], acc float64 updated in place."""
    lib = _load()
    G, gp = _f32(G)
    B, P = G.shape[0], int(np.prod(G.shape[1:]))
    factor, fp = _f64(factor)
    assert acc.dtype == np.float64 and acc.size == P and acc.flags.c_contiguous and factor.size == B
    lib.oracle_clip_accumulate_noised_f32(gp, B, ctypes.c_size_t(P), fp, ctypes.c_double(sd), ctypes.c_uint64(seed),
                                          ctypes.c_uint64(step), ctypes.c_uint32(example0), ctypes.c_uint64(param_offset),
                                          acc.ctypes.data_as(_f64p))
    return acc


def sgd_update(g, lr, mu, theta, m=None):
    """theta, m (float64, updated in place): m <- mu*m + g; theta <- theta - lr*m.  m=None is plain SGD."""
    lib = _load()
    g, gp = _f64(g)
    assert theta.dtype == np.float64 and theta.flags.c_contiguous and theta.size == g.size
    mp = None
    if m is not None:
        assert m.dtype == np.float64 and m.flags.c_contiguous and m.size == g.size
        mp = m.ctypes.data_as(_f64p)
    lib.oracle_sgd_update(gp, ctypes.c_size_t(g.size), ctypes.c_double(lr), ctypes.c_double(mu),
                          theta.ctypes.data_as(_f64p), mp)
    return theta


def privatise(chunks, C, sigma, mode, seed, step):
    """The whole step.  chunks: iterable of lists of L per-example gradient arrays [B, ...].

    Returns (out list of L arrays, sq list per chunk, factor list per chunk); parameter
    indices for the noise stream run over the tensors in list order.
    """
    acc, sqs, factors, total = None, [], [], 0
    for groups in chunks:
        acc, sq, f = clipped_sum(groups, C, mode, acc)
        sqs.append(sq)
        factors.append(f)
        total += groups[0].shape[0]
    out, off = [], 0
    for a in acc:
        out.append(noise_average(a, off, sigma, C, total, seed, step))
        off += a.size
    return out, sqs, factors
