"""Python face of the CPU oracle (oracle/rocket_oracle.c).

TEST INFRASTRUCTURE ONLY: importable from tests/, from the smoke check and from the
benchmark's CPU-baseline leg.  The product package never imports it, and it never
imports the product package.  Functions take a rocket_inputs.KernelParams (plain numpy
arrays) and numpy inputs, and return numpy float64 / integer arrays.
"""
import ctypes
import os
import subprocess
from types import SimpleNamespace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rocket_oracle.c")
_SRC_MINI = os.path.join(_HERE, "minirocket_oracle.c")
_SRC_F16 = os.path.join(_HERE, "rocket_f16_oracle.c")
_LIB = os.path.join(_HERE, "_build", "librocket_oracle.so")
_lib = None


def build(force=False):
    """Compile the oracle with gcc (-O2, OpenMP).  Returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_SRC_MINI), os.path.getmtime(_SRC_F16)):
        os.makedirs(os.path.dirname(_LIB), exist_ok=True)
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-ffp-contract=off", "-o", tmp, _SRC, _SRC_MINI, _SRC_F16, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _CParams(ctypes.Structure):
    _fields_ = [("K", ctypes.c_int), ("C", ctypes.c_int), ("L", ctypes.c_int),
                ("length", ctypes.c_void_p), ("dilation", ctypes.c_void_p),
                ("padding", ctypes.c_void_p), ("num_channels", ctypes.c_void_p),
                ("channel_idx", ctypes.c_void_p), ("weights", ctypes.c_void_p),
                ("bias", ctypes.c_void_p), ("channel_offset", ctypes.c_void_p),
                ("weight_offset", ctypes.c_void_p)]


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.rocket_oracle_conv.restype = ctypes.c_int64
        lib.minirocket_oracle_conv.restype = ctypes.c_int64
        lib.rocket_oracle_num_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def _cparams(p):
    """Pack a KernelParams into the C struct; returns (struct, keepalive list)."""
    arrs = dict(
        length=np.ascontiguousarray(p.length, np.int32), dilation=np.ascontiguousarray(p.dilation, np.int32),
        padding=np.ascontiguousarray(p.padding, np.int32),
        num_channels=np.ascontiguousarray(p.num_channels, np.int32),
        channel_idx=np.ascontiguousarray(p.channel_idx, np.int32),
        weights=np.ascontiguousarray(p.weights, np.float32), bias=np.ascontiguousarray(p.bias, np.float32),
        channel_offset=np.ascontiguousarray(p.channel_offset, np.int64),
        weight_offset=np.ascontiguousarray(p.weight_offset, np.int64))
    s = _CParams(K=p.K, C=p.C, L=p.L, **{k: v.ctypes.data for k, v in arrs.items()})
    return s, arrs


def _check_x(p, X):
    X = np.ascontiguousarray(X, dtype=np.float32)
    if X.ndim != 3 or X.shape[1] != p.C or X.shape[2] != p.L:
        raise ValueError("X must be [N, %d, %d]" % (p.C, p.L))
    return X


def num_threads():
    return int(_load().rocket_oracle_num_threads())


def set_threads(t):
    _load().rocket_oracle_set_threads(ctypes.c_int(int(t)))


def conv(p, X, n, k):
    """z[0..L_out) of kernel k on example n, float64."""
    lib = _load()
    X = _check_x(p, X)
    s, keep = _cparams(p)
    nout = lib.rocket_oracle_conv(ctypes.byref(s), _ptr(X), ctypes.c_int(n), ctypes.c_int(k), None)
    z = np.empty(max(int(nout), 0), dtype=np.float64)
    lib.rocket_oracle_conv(ctypes.byref(s), _ptr(X), ctypes.c_int(n), ctypes.c_int(k), _ptr(z))
    return z


def scale_u8(X_u8, mean, inv_std):
    """Per-channel feature scaling of raw 8-bit intensities (Sections 4.1 and 4.3):
    x[n, c, i] = (X_u8[n, c, i] - mean[c]) * inv_std[c], evaluated in float64 and rounded once to
    the float32 input of the transform."""
    v = np.asarray(X_u8)
    if v.dtype != np.uint8 or v.ndim != 3:
        raise ValueError("X_u8 must be a uint8 array [N, C, L]")
    mean = np.asarray(mean, dtype=np.float64).reshape(1, -1, 1)
    inv_std = np.asarray(inv_std, dtype=np.float64).reshape(1, -1, 1)
    if mean.shape[1] != v.shape[1] or inv_std.shape[1] != v.shape[1]:
        raise ValueError("one mean and one inv_std per channel")
    return ((v.astype(np.float64) - mean) * inv_std).astype(np.float32)


def ridge_fit(F, y, alpha):
    """Ridge regressor of Section 3.3 on features F [N, P] with targets y [N], float64 throughout:
    the weights w minimise |Fc w - yc|^2 + alpha |w|^2 over the column-centred Fc, yc (the intercept
    is not penalised), written out as the normal equations (Fc^T Fc + alpha I) w = Fc^T yc, and
    b = mean(y) - mean(F) . w.  Returns (w [P], b)."""
    F = np.asarray(F, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    if F.ndim != 2 or y.shape != (F.shape[0],):
        raise ValueError("F must be [N, P] and y [N]")
    mu, ybar = F.mean(axis=0), y.mean()
    Fc, yc = F - mu, y - ybar
    P = F.shape[1]
    w = np.linalg.solve(Fc.T @ Fc + float(alpha) * np.eye(P), Fc.T @ yc)
    return w, float(ybar - mu @ w)


def ridge_predict(F, w, b):
    """yhat = b + F w (Section 3 step (3)), float64."""
    return np.asarray(F, dtype=np.float64) @ np.asarray(w, dtype=np.float64) + float(b)


def forward_pairs(p, X, pair_n, pair_k, lam=1.0, shift=3.0, amb_eps=1e-5):
    """Pooled features for explicit (example, kernel) pairs.

    Returns a namespace of 1-D arrays: ppv, max, soft (float64), argmax (int32),
    pos_eps, amb (int64), gap (float64), out_len (int64).
    """
    lib = _load()
    X = _check_x(p, X)
    pn = np.ascontiguousarray(pair_n, np.int32)
    pk = np.ascontiguousarray(pair_k, np.int32)
    if pn.shape != pk.shape or pn.ndim != 1:
        raise ValueError("pair_n and pair_k must be 1-D and of equal length")
    if len(pn) and (pn.min() < 0 or pn.max() >= X.shape[0] or pk.min() < 0 or pk.max() >= p.K):
        raise ValueError("pair index out of range")
    P = len(pn)
    out = SimpleNamespace(ppv=np.empty(P), max=np.empty(P), soft=np.empty(P), argmax=np.empty(P, np.int32),
                          pos_eps=np.empty(P, np.int64), amb=np.empty(P, np.int64), gap=np.empty(P))
    s, keep = _cparams(p)
    lib.rocket_oracle_forward_pairs(ctypes.byref(s), _ptr(X), ctypes.c_int64(P), _ptr(pn), _ptr(pk),
                                    ctypes.c_double(lam), ctypes.c_double(shift), ctypes.c_double(amb_eps),
                                    _ptr(out.ppv), _ptr(out.max), _ptr(out.soft), _ptr(out.argmax),
                                    _ptr(out.pos_eps), _ptr(out.amb), _ptr(out.gap))
    out.out_len = p.out_len[pk]
    return out


def forward(p, X, lam=1.0, shift=3.0, amb_eps=1e-5):
    """Pooled features for every (example, kernel): each field reshaped to [N, K]."""
    N = np.asarray(X).shape[0]
    pn = np.repeat(np.arange(N, dtype=np.int32), p.K)
    pk = np.tile(np.arange(p.K, dtype=np.int32), N)
    out = forward_pairs(p, X, pn, pk, lam, shift, amb_eps)
    for name, v in vars(out).items():
        setattr(out, name, v.reshape(N, p.K))
    return out


def features_hard(out):
    """Interleave (PPV_k, MAX_k) into [N, 2K], the layout of the library's feature matrix."""
    return np.stack([out.ppv, out.max], axis=-1).reshape(out.ppv.shape[0], -1)


def features_soft(out):
    return np.stack([out.soft, out.max], axis=-1).reshape(out.soft.shape[0], -1)


def backward(p, X, g, argmax, lam=1.0, shift=3.0, examples=None, kernels=None):
    """Gradients (dW ragged float64, db float64[K]) of sum(g * features_soft).

    g: [N, 2K] float32 interleaved (gP, gM); argmax: [N, K] int32.  examples / kernels
    restrict the sum over n and the kernels computed (others are left at zero).
    """
    lib = _load()
    X = _check_x(p, X)
    N = X.shape[0]
    g = np.ascontiguousarray(g, np.float32)
    argmax = np.ascontiguousarray(argmax, np.int32)
    if g.shape != (N, 2 * p.K) or argmax.shape != (N, p.K):
        raise ValueError("g must be [N, 2K] and argmax [N, K]")
    ex = np.arange(N, dtype=np.int32) if examples is None else np.ascontiguousarray(examples, np.int32)
    ks = np.arange(p.K, dtype=np.int32) if kernels is None else np.ascontiguousarray(kernels, np.int32)
    dW = np.zeros(len(p.weights), dtype=np.float64)
    db = np.zeros(p.K, dtype=np.float64)
    s, keep = _cparams(p)
    lib.rocket_oracle_backward(ctypes.byref(s), _ptr(X), ctypes.c_int(len(ex)), _ptr(ex), ctypes.c_int(len(ks)),
                               _ptr(ks), ctypes.c_double(lam), ctypes.c_double(shift), _ptr(g), _ptr(argmax),
                               _ptr(dW), _ptr(db))
    return dW, db


# ---- half-precision transform (oracle/rocket_f16_oracle.c) ---------------------------------------------------

def round_f16(a):
    """The binary16 numbers nearest to a (ties to even), as float32."""
    with np.errstate(over="raise"):
        return np.asarray(a, np.float32).astype(np.float16).astype(np.float32)


def forward_f16_pairs(p, X, pair_n, pair_k, return_z=False):
    """Half-precision hard transform for explicit (example, kernel) pairs: samples, weights and biases are rounded
    to binary16 here, every multiply-add of the convolution rounds once to binary16 (bias first, then the channels
    in the kernel's order, taps 0 .. len - 1).  Returns a namespace of 1-D arrays: count (int64), ppv, max
    (float64), argmax (int32), out_len; with return_z also z (the outputs of the first pair)."""
    import copy
    lib = _load()
    X16 = round_f16(_check_x(p, X))
    p16 = copy.copy(p)
    p16.weights = round_f16(p.weights)
    p16.bias = round_f16(p.bias)
    pn = np.ascontiguousarray(pair_n, np.int32)
    pk = np.ascontiguousarray(pair_k, np.int32)
    if pn.shape != pk.shape or pn.ndim != 1:
        raise ValueError("pair_n and pair_k must be 1-D and of equal length")
    P = len(pn)
    out = SimpleNamespace(count=np.empty(P, np.int64), ppv=np.empty(P), max=np.empty(P), argmax=np.empty(P, np.int32))
    z = np.empty(int(p.out_len[pk[0]]) if (return_z and P) else 0)
    s, keep = _cparams(p16)
    lib.rocket_oracle_f16_forward_pairs.restype = ctypes.c_int
    rc = lib.rocket_oracle_f16_forward_pairs(ctypes.byref(s), _ptr(X16), ctypes.c_int64(P), _ptr(pn), _ptr(pk), _ptr(out.count),
                                             _ptr(out.ppv), _ptr(out.max), _ptr(out.argmax), _ptr(z) if return_z and P else None)
    if rc != 0:
        raise FloatingPointError("an input is no binary16 number or an intermediate result overflows binary16")
    out.out_len = p.out_len[pk]
    if return_z:
        out.z = z
    return out


def forward_f16(p, X):
    """forward_f16_pairs for every (example, kernel): each field reshaped to [N, K]."""
    N = np.asarray(X).shape[0]
    pn = np.repeat(np.arange(N, dtype=np.int32), p.K)
    pk = np.tile(np.arange(p.K, dtype=np.int32), N)
    out = forward_f16_pairs(p, X, pn, pk)
    for name, v in vars(out).items():
        setattr(out, name, v.reshape(N, p.K))
    return out


# ---- MINIROCKET (oracle/minirocket_oracle.c) ---------------------------------------------------------------

class _CMini(ctypes.Structure):
    _fields_ = [("C", ctypes.c_int), ("L", ctypes.c_int), ("F", ctypes.c_int), ("n_combos", ctypes.c_int),
                ("taps", ctypes.c_void_p), ("dilation", ctypes.c_void_p), ("kernel_index", ctypes.c_void_p),
                ("padded", ctypes.c_void_p), ("num_channels", ctypes.c_void_p), ("channel_idx", ctypes.c_void_p),
                ("channel_offset", ctypes.c_void_p), ("feature_offset", ctypes.c_void_p)]


def _cmini(p):
    arrs = dict(taps=np.ascontiguousarray(p.taps, np.int32), dilation=np.ascontiguousarray(p.dilation, np.int32),
                kernel_index=np.ascontiguousarray(p.kernel_index, np.int32), padded=np.ascontiguousarray(p.padded, np.int32),
                num_channels=np.ascontiguousarray(p.num_channels, np.int32),
                channel_idx=np.ascontiguousarray(p.channel_idx, np.int32),
                channel_offset=np.ascontiguousarray(p.channel_offset, np.int64),
                feature_offset=np.ascontiguousarray(p.feature_offset, np.int32))
    s = _CMini(C=p.C, L=p.L, F=p.F, n_combos=p.n_combos, **{k: v.ctypes.data for k, v in arrs.items()})
    return s, arrs


def minirocket_conv(p, X, n, c):
    """Convolution outputs of combination c on example n over the combination's output range, float64."""
    lib = _load()
    X = _check_x(p, X)
    s, keep = _cmini(p)
    nout = lib.minirocket_oracle_conv(ctypes.byref(s), _ptr(X), ctypes.c_int(n), ctypes.c_int(c), None)
    z = np.empty(int(nout), dtype=np.float64)
    lib.minirocket_oracle_conv(ctypes.byref(s), _ptr(X), ctypes.c_int(n), ctypes.c_int(c), _ptr(z))
    return z


def minirocket_example_index(p, N):
    """Which of N training examples every combination reads its biases from."""
    return np.minimum((p.example_draw * N).astype(np.int64), N - 1).astype(np.int32)


def minirocket_fit(p, X):
    """Biases [F] (float64) from the quantiles of the training examples' convolution outputs."""
    lib = _load()
    X = _check_x(p, X)
    s, keep = _cmini(p)
    ex = minirocket_example_index(p, X.shape[0])
    q = np.ascontiguousarray(p.quantile, np.float64)
    bias = np.empty(p.F, dtype=np.float64)
    lib.minirocket_oracle_fit(ctypes.byref(s), _ptr(X), _ptr(ex), _ptr(q), _ptr(bias))
    return bias


def minirocket_transform(p, X, bias, eps=1e-5):
    """PPV features [N, F] against the biases, and the counts that bound what fp32 arithmetic may decide
    differently: pos_eps = #{z > bias + eps}, amb = #{|z - bias| <= eps}, n_out [F] = outputs per feature."""
    lib = _load()
    X = _check_x(p, X)
    s, keep = _cmini(p)
    N = X.shape[0]
    bias = np.ascontiguousarray(bias, np.float64)
    out = SimpleNamespace(ppv=np.empty((N, p.F)), pos_eps=np.empty((N, p.F), np.int64), amb=np.empty((N, p.F), np.int64))
    lib.minirocket_oracle_transform(ctypes.byref(s), _ptr(X), ctypes.c_int(N), _ptr(bias), ctypes.c_double(eps),
                                    _ptr(out.ppv), _ptr(out.pos_eps), _ptr(out.amb))
    n_out = np.empty(p.F, np.int64)
    for c in range(p.n_combos):
        first, last = p.out_range(c)
        n_out[p.feature_offset[c]:p.feature_offset[c + 1]] = last - first
    out.n_out = n_out
    return out
