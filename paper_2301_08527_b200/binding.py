"""ctypes binding of include/rocket.h.  Same names as the C entry points; marshalling only.

torch is used for device memory and streams; tensors are passed to the library as raw device
pointers together with the current CUDA stream.
"""
import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "librocket_b200.so")
_lib = None

c_int32_p = ctypes.POINTER(ctypes.c_int32)
c_float_p = ctypes.POINTER(ctypes.c_float)

# name -> (restype, argtypes); every symbol include/rocket.h declares
SIGNATURES = {
    "rocket_strerror": (ctypes.c_char_p, [ctypes.c_int]),
    "rocket_params_generate": (ctypes.c_int, [ctypes.c_uint64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                              ctypes.POINTER(ctypes.c_void_p)]),
    "rocket_params_from_arrays": (ctypes.c_int, [ctypes.c_int, ctypes.c_int, ctypes.c_int] + [ctypes.c_void_p] * 7 +
                                  [ctypes.POINTER(ctypes.c_void_p)]),
    "rocket_params_counts": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int),
                                            ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_int64),
                                            ctypes.POINTER(ctypes.c_int64)]),
    "rocket_params_host_view": (ctypes.c_int, [ctypes.c_void_p] + [ctypes.POINTER(ctypes.c_void_p)] * 7),
    "rocket_params_work": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_double),
                                          ctypes.POINTER(ctypes.c_double)]),
    "rocket_params_destroy": (None, [ctypes.c_void_p]),
    "rocket_params_set_path": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int]),
    "rocket_params_set_weights": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "rocket_params_bind_device": (ctypes.c_int, [ctypes.c_void_p]),
    "rocket_params_device_status": (ctypes.c_int, [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int)]),
    "rocket_transform_soft_backward_noalloc": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                                              ctypes.c_int, ctypes.c_int, ctypes.c_float,
                                                              ctypes.c_float, ctypes.c_void_p, ctypes.c_void_p,
                                                              ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "rocket_kernel_launch_count": (ctypes.c_int64, []),
    "rocket_device_alloc_count": (ctypes.c_int64, []),
    "rocket_params_reserve": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.c_int]),
    "rocket_params_set_profiling": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int]),
    "rocket_params_last_profile": (ctypes.c_int, [ctypes.c_void_p] + [ctypes.POINTER(ctypes.c_double)] * 4),
    "rocket_mini_create": (ctypes.c_int, [ctypes.c_uint64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                          ctypes.POINTER(ctypes.c_void_p)]),
    "rocket_mini_counts": (ctypes.c_int, [ctypes.c_void_p] + [ctypes.POINTER(ctypes.c_int)] * 4 + [ctypes.POINTER(ctypes.c_int64)]),
    "rocket_mini_host_view": (ctypes.c_int, [ctypes.c_void_p] + [ctypes.POINTER(ctypes.c_void_p)] * 10),
    "rocket_mini_fit": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]),
    "rocket_mini_set_biases": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p]),
    "rocket_mini_transform": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                             ctypes.c_void_p, ctypes.c_void_p]),
    "rocket_mini_destroy": (None, [ctypes.c_void_p]),
    "rocket_transform": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                        ctypes.c_void_p, ctypes.c_void_p]),
    "rocket_transform_f16": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                            ctypes.c_void_p, ctypes.c_void_p]),
    "rocket_transform_soft": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                             ctypes.c_int, ctypes.c_float, ctypes.c_float, ctypes.c_void_p,
                                             ctypes.c_void_p, ctypes.c_void_p]),
    "rocket_transform_soft_backward": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                                      ctypes.c_int, ctypes.c_float, ctypes.c_float, ctypes.c_void_p,
                                                      ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                                      ctypes.c_void_p]),
    "rocket_transform_u8": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "rocket_transform_soft_u8": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                                ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float,
                                                ctypes.c_float, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "rocket_transform_u8_host": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                                ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "rocket_ridge_fit": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_float,
                                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]),
    "rocket_ridge_predict": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                            ctypes.c_void_p, ctypes.c_void_p]),
    "rocket_transform_host": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                             ctypes.c_int, ctypes.c_void_p]),
    "rocket_transform_soft_host": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                                  ctypes.c_int, ctypes.c_float, ctypes.c_float, ctypes.c_void_p,
                                                  ctypes.c_void_p]),
    "rocket_transform_soft_backward_host": (ctypes.c_int, [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                                           ctypes.c_int, ctypes.c_int, ctypes.c_float, ctypes.c_float,
                                                           ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                                           ctypes.c_void_p]),
}


class RocketError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        msg = load_library().rocket_strerror(self.status).decode()
        super().__init__("%s failed: %s (status %d)" % (where, msg, self.status))


def library_path():
    return _LIB_PATH


def load_library():
    """Loads librocket_b200.so; raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError("%s is missing: run `python -m paper_2301_08527_b200.build` "
                               "(or __graft_entry__.build()) first; there is no CPU fallback" % _LIB_PATH)
        lib = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _lib = lib
    return _lib


def _check(status, where):
    if status != 0:
        raise RocketError(status, where)


PASS_HARD, PASS_SOFT, PASS_BACKWARD, PASS_U8_INPUT = 1, 2, 4, 8


def device_alloc_count():
    return int(load_library().rocket_device_alloc_count())


def kernel_launch_count():
    return int(load_library().rocket_kernel_launch_count())


def _np_ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


class RocketParams:
    """Owner of a rocket_params_t handle (kernel parameters on host and device)."""

    def __init__(self, handle):
        self._h = ctypes.c_void_p(handle)
        lib = load_library()
        K, C, L = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
        nch, nw = ctypes.c_int64(), ctypes.c_int64()
        _check(lib.rocket_params_counts(self._h, K, C, L, nch, nw), "rocket_params_counts")
        self.K, self.C, self.L = K.value, C.value, L.value
        self.n_channel_idx, self.n_weights = nch.value, nw.value

    @classmethod
    def generate(cls, seed, K, C, L):
        """rocket_params_generate: draw K kernels from one seed (Section 3.1)."""
        h = ctypes.c_void_p()
        _check(load_library().rocket_params_generate(ctypes.c_uint64(seed), K, C, L, ctypes.byref(h)),
               "rocket_params_generate")
        return cls(h.value)

    @classmethod
    def from_arrays(cls, K, C, L, length, dilation, padding, num_channels, channel_idx, weights, bias):
        """rocket_params_from_arrays: adopt explicit kernels (numpy arrays are copied)."""
        arrs = [np.ascontiguousarray(a, np.int32) for a in (length, dilation, padding, num_channels, channel_idx)]
        arrs += [np.ascontiguousarray(a, np.float32) for a in (weights, bias)]
        h = ctypes.c_void_p()
        _check(load_library().rocket_params_from_arrays(K, C, L, *[_np_ptr(a) for a in arrs], ctypes.byref(h)),
               "rocket_params_from_arrays")
        return cls(h.value)

    @classmethod
    def from_kernel_params(cls, kp):
        """Adopt any object with the fields of rocket_inputs.KernelParams."""
        return cls.from_arrays(kp.K, kp.C, kp.L, kp.length, kp.dilation, kp.padding, kp.num_channels,
                               kp.channel_idx, kp.weights, kp.bias)

    def host_arrays(self):
        """Copies of the handle's host arrays (rocket_params_host_view) as a dict of numpy arrays."""
        ptrs = [ctypes.c_void_p() for _ in range(7)]
        _check(load_library().rocket_params_host_view(self._h, *[ctypes.byref(p) for p in ptrs]),
               "rocket_params_host_view")
        names = ["length", "dilation", "padding", "num_channels", "channel_idx", "weights", "bias"]
        sizes = [self.K, self.K, self.K, self.K, self.n_channel_idx, self.n_weights, self.K]
        out = {}
        for name, p, n in zip(names, ptrs, sizes):
            ctype = ctypes.c_float if name in ("weights", "bias") else ctypes.c_int32
            buf = (ctype * n).from_address(p.value) if n else (ctype * 0)()
            out[name] = np.array(buf, copy=True)
        return out

    def work(self):
        """(conv flop per example, conv outputs per example) under the count 2*len*channels*L_out."""
        f, o = ctypes.c_double(), ctypes.c_double()
        _check(load_library().rocket_params_work(self._h, f, o), "rocket_params_work")
        return f.value, o.value

    def bind_device(self):
        """rocket_params_bind_device: upload the parameters to the current device now."""
        _check(load_library().rocket_params_bind_device(self._h), "rocket_params_bind_device")

    def reserve(self, max_N, passes=PASS_HARD):
        _check(load_library().rocket_params_reserve(self._h, ctypes.c_int(int(max_N)), ctypes.c_int(int(passes))),
               "rocket_params_reserve")

    def device_status(self):
        """rocket_params_device_status: number of bounded waits that gave up (0 = healthy)."""
        flag = ctypes.c_int()
        _check(load_library().rocket_params_device_status(self._h, flag), "rocket_params_device_status")
        return flag.value

    def set_profiling(self, enable):
        """rocket_params_set_profiling: record events around the two fused kernels of the hard transform."""
        _check(load_library().rocket_params_set_profiling(self._h, int(bool(enable))), "rocket_params_set_profiling")

    def last_profile(self):
        """rocket_params_last_profile: dict with the last call's kernel times (ms) and the per-example
        conv flop of the two kernels."""
        v = [ctypes.c_double() for _ in range(4)]
        _check(load_library().rocket_params_last_profile(self._h, *v), "rocket_params_last_profile")
        return {"ms_small_dilations": v[0].value, "ms_large_dilations": v[1].value,
                "flops_small_dilations": v[2].value, "flops_large_dilations": v[3].value}

    def set_weights(self, weights, bias):
        """rocket_params_set_weights: install new weights (ragged, n_weights floats) and biases (K floats)."""
        w = np.ascontiguousarray(weights, dtype=np.float32).reshape(-1)
        b = np.ascontiguousarray(bias, dtype=np.float32).reshape(-1)
        if w.shape[0] != self.n_weights or b.shape[0] != self.K:
            raise ValueError("weights must hold n_weights values and bias K values")
        _check(load_library().rocket_params_set_weights(self._h, _np_ptr(w), _np_ptr(b)), "rocket_params_set_weights")

    def set_path(self, path):
        _check(load_library().rocket_params_set_path(self._h, int(path)), "rocket_params_set_path")

    @property
    def handle(self):
        return self._h

    def close(self):
        if self._h is not None and self._h.value:
            load_library().rocket_params_destroy(self._h)
        self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _dev_ptr(t, dtype, name):
    import torch
    if not isinstance(t, torch.Tensor) or not t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError("%s must be a contiguous CUDA tensor of dtype %s" % (name, dtype))
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    import torch
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check_x(params, X):
    if X.dim() != 3:
        raise ValueError("X must be [N, C, L]")
    return int(X.shape[0]), int(X.shape[1]), int(X.shape[2])


def rocket_transform(params, X, out=None):
    """Hard PPV + max.  X: CUDA fp32 [N, C, L] -> features CUDA fp32 [N, 2K] on the current stream."""
    import torch
    N, C, L = _check_x(params, X)
    feat = out if out is not None else torch.empty((N, 2 * params.K), dtype=torch.float32, device=X.device)
    _check(load_library().rocket_transform(params.handle, _dev_ptr(X, torch.float32, "X"), N, C, L,
                                           _dev_ptr(feat, torch.float32, "out"), _stream()), "rocket_transform")
    return feat


def rocket_transform_f16(params, X, out=None):
    """Hard PPV + max in half precision (binary16 samples, weights and biases; one rounding per multiply-add)."""
    import torch
    N, C, L = _check_x(params, X)
    feat = out if out is not None else torch.empty((N, 2 * params.K), dtype=torch.float32, device=X.device)
    _check(load_library().rocket_transform_f16(params.handle, _dev_ptr(X, torch.float32, "X"), N, C, L,
                                               _dev_ptr(feat, torch.float32, "out"), _stream()), "rocket_transform_f16")
    return feat


def rocket_transform_soft(params, X, lam, shift=3.0, out=None, argmax_out=None, want_argmax=True):
    """softPPV + max (Eq. 3-4).  Returns (features [N, 2K], argmax [N, K] int32 or None)."""
    import torch
    N, C, L = _check_x(params, X)
    feat = out if out is not None else torch.empty((N, 2 * params.K), dtype=torch.float32, device=X.device)
    arg = argmax_out
    if arg is None and want_argmax:
        arg = torch.empty((N, params.K), dtype=torch.int32, device=X.device)
    _check(load_library().rocket_transform_soft(
        params.handle, _dev_ptr(X, torch.float32, "X"), N, C, L, ctypes.c_float(lam), ctypes.c_float(shift),
        _dev_ptr(feat, torch.float32, "out"),
        _dev_ptr(arg, torch.int32, "argmax_out") if arg is not None else None, _stream()), "rocket_transform_soft")
    return feat, arg


def _stats(params, mean, inv_std):
    m = np.ascontiguousarray(mean, dtype=np.float32)
    s = np.ascontiguousarray(inv_std, dtype=np.float32)
    if m.shape != (params.C,) or s.shape != (params.C,):
        raise ValueError("mean and inv_std must hold one value per channel")
    return m, s


def rocket_transform_u8(params, X_u8, mean, inv_std, out=None):
    """Hard PPV + max of raw 8-bit intensities scaled per channel: x = (v - mean[c]) * inv_std[c].
    X_u8: CUDA uint8 [N, C, L]; mean, inv_std: host arrays of C floats."""
    import torch
    N, C, L = _check_x(params, X_u8)
    m, s = _stats(params, mean, inv_std)
    feat = out if out is not None else torch.empty((N, 2 * params.K), dtype=torch.float32, device=X_u8.device)
    _check(load_library().rocket_transform_u8(params.handle, _dev_ptr(X_u8, torch.uint8, "X_u8"), N, C, L, _np_ptr(m),
                                              _np_ptr(s), _dev_ptr(feat, torch.float32, "out"), _stream()),
           "rocket_transform_u8")
    return feat


def rocket_transform_soft_u8(params, X_u8, mean, inv_std, lam, shift=3.0, out=None, argmax_out=None, want_argmax=True):
    """softPPV + max of raw 8-bit intensities scaled per channel.  Returns (features, argmax or None)."""
    import torch
    N, C, L = _check_x(params, X_u8)
    m, s = _stats(params, mean, inv_std)
    feat = out if out is not None else torch.empty((N, 2 * params.K), dtype=torch.float32, device=X_u8.device)
    arg = argmax_out
    if arg is None and want_argmax:
        arg = torch.empty((N, params.K), dtype=torch.int32, device=X_u8.device)
    _check(load_library().rocket_transform_soft_u8(
        params.handle, _dev_ptr(X_u8, torch.uint8, "X_u8"), N, C, L, _np_ptr(m), _np_ptr(s), ctypes.c_float(lam),
        ctypes.c_float(shift), _dev_ptr(feat, torch.float32, "out"),
        _dev_ptr(arg, torch.int32, "argmax_out") if arg is not None else None, _stream()), "rocket_transform_soft_u8")
    return feat, arg


def rocket_transform_soft_backward(params, X, lam, shift, dfeat, argmax, dW_out=None, db_out=None):
    """Gradients of sum(dfeat * soft features) for weights (ragged like the weights) and biases."""
    import torch
    N, C, L = _check_x(params, X)
    dW = dW_out if dW_out is not None else torch.empty((params.n_weights,), dtype=torch.float32, device=X.device)
    db = db_out if db_out is not None else torch.empty((params.K,), dtype=torch.float32, device=X.device)
    _check(load_library().rocket_transform_soft_backward(
        params.handle, _dev_ptr(X, torch.float32, "X"), N, C, L, ctypes.c_float(lam), ctypes.c_float(shift),
        _dev_ptr(dfeat, torch.float32, "dfeat"), _dev_ptr(argmax, torch.int32, "argmax"),
        _dev_ptr(dW, torch.float32, "dW_out"), _dev_ptr(db, torch.float32, "db_out"), _stream()),
        "rocket_transform_soft_backward")
    return dW, db


def rocket_transform_soft_backward_noalloc(params, X, lam, shift, dfeat, argmax, dW_out, db_out):
    """Allocation-free backward: same results as rocket_transform_soft_backward, scratch in a fixed
    library-owned array (see include/rocket.h for its size limit and sharing rules).  The caller
    supplies the outputs, and the handle must already be bound to the device."""
    import torch
    N, C, L = _check_x(params, X)
    _check(load_library().rocket_transform_soft_backward_noalloc(
        params.handle, _dev_ptr(X, torch.float32, "X"), N, C, L, ctypes.c_float(lam), ctypes.c_float(shift),
        _dev_ptr(dfeat, torch.float32, "dfeat"), _dev_ptr(argmax, torch.int32, "argmax"),
        _dev_ptr(dW_out, torch.float32, "dW_out"), _dev_ptr(db_out, torch.float32, "db_out"), _stream()),
        "rocket_transform_soft_backward_noalloc")
    return dW_out, db_out


def rocket_ridge_fit(feat, y, alpha):
    """Ridge regressor on pooled features (Section 3.3): feat CUDA fp32 [N, P], y CUDA fp32 [N].
    Returns (w [P], b [1]) on the device; the intercept is fitted and not penalised."""
    import torch
    if feat.dim() != 2 or y.dim() != 1 or y.shape[0] != feat.shape[0]:
        raise ValueError("feat must be [N, P] and y [N]")
    N, Pn = int(feat.shape[0]), int(feat.shape[1])
    w = torch.empty((Pn,), dtype=torch.float32, device=feat.device)
    b = torch.empty((1,), dtype=torch.float32, device=feat.device)
    _check(load_library().rocket_ridge_fit(_dev_ptr(feat, torch.float32, "feat"), N, Pn, _dev_ptr(y, torch.float32, "y"),
                                           ctypes.c_float(alpha), _dev_ptr(w, torch.float32, "w"),
                                           _dev_ptr(b, torch.float32, "b"), _stream()), "rocket_ridge_fit")
    return w, b


def rocket_ridge_predict(feat, w, b, out=None):
    """yhat[n] = b + feat[n] . w on the device (current stream)."""
    import torch
    if feat.dim() != 2 or w.dim() != 1 or w.shape[0] != feat.shape[1]:
        raise ValueError("feat must be [N, P] and w [P]")
    N, Pn = int(feat.shape[0]), int(feat.shape[1])
    yhat = out if out is not None else torch.empty((N,), dtype=torch.float32, device=feat.device)
    _check(load_library().rocket_ridge_predict(_dev_ptr(feat, torch.float32, "feat"), N, Pn, _dev_ptr(w, torch.float32, "w"),
                                               _dev_ptr(b, torch.float32, "b"), _dev_ptr(yhat, torch.float32, "out"),
                                               _stream()), "rocket_ridge_predict")
    return yhat


def _host_ptr(t, dtype, name):
    import torch
    if isinstance(t, np.ndarray):
        t = torch.from_numpy(t)
    if t.is_cuda or t.dtype != dtype or not t.is_contiguous():
        raise TypeError("%s must be a contiguous host tensor of dtype %s" % (name, dtype))
    return ctypes.c_void_p(t.data_ptr())


def rocket_transform_host(params, X_host, feat_host):
    """Host-buffer form: X_host / feat_host are host tensors (pinned for asynchronous copies)."""
    import torch
    N, C, L = _check_x(params, X_host)
    _check(load_library().rocket_transform_host(params.handle, _host_ptr(X_host, torch.float32, "X_host"), N, C, L,
                                                _host_ptr(feat_host, torch.float32, "feat_host")),
           "rocket_transform_host")
    return feat_host


def rocket_transform_u8_host(params, X_u8_host, mean, inv_std, feat_host):
    """Host-buffer form of rocket_transform_u8 (the bytes travel to the device inside the call)."""
    import torch
    N, C, L = _check_x(params, X_u8_host)
    m, s = _stats(params, mean, inv_std)
    _check(load_library().rocket_transform_u8_host(params.handle, _host_ptr(X_u8_host, torch.uint8, "X_u8_host"), N, C, L,
                                                   _np_ptr(m), _np_ptr(s), _host_ptr(feat_host, torch.float32, "feat_host")),
           "rocket_transform_u8_host")
    return feat_host


def rocket_transform_soft_host(params, X_host, lam, shift, feat_host, argmax_host=None):
    import torch
    N, C, L = _check_x(params, X_host)
    _check(load_library().rocket_transform_soft_host(
        params.handle, _host_ptr(X_host, torch.float32, "X_host"), N, C, L, ctypes.c_float(lam),
        ctypes.c_float(shift), _host_ptr(feat_host, torch.float32, "feat_host"),
        _host_ptr(argmax_host, torch.int32, "argmax_host") if argmax_host is not None else None),
        "rocket_transform_soft_host")
    return feat_host, argmax_host


def rocket_transform_soft_backward_host(params, X_host, lam, shift, dfeat_host, argmax_host, dW_host, db_host):
    import torch
    N, C, L = _check_x(params, X_host)
    _check(load_library().rocket_transform_soft_backward_host(
        params.handle, _host_ptr(X_host, torch.float32, "X_host"), N, C, L, ctypes.c_float(lam),
        ctypes.c_float(shift), _host_ptr(dfeat_host, torch.float32, "dfeat_host"),
        _host_ptr(argmax_host, torch.int32, "argmax_host"), _host_ptr(dW_host, torch.float32, "dW_host"),
        _host_ptr(db_host, torch.float32, "db_host")), "rocket_transform_soft_backward_host")
    return dW_host, db_host


class MiniRocket:
    """Owner of a rocket_mini_t handle (MINIROCKET parameters on host and device)."""

    def __init__(self, handle):
        self._h = handle
        lib = load_library()
        C, L, F, nc = ctypes.c_int(), ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
        nch = ctypes.c_int64()
        _check(lib.rocket_mini_counts(self._h, ctypes.byref(C), ctypes.byref(L), ctypes.byref(F), ctypes.byref(nc),
                                      ctypes.byref(nch)), "rocket_mini_counts")
        self.C, self.L, self.F, self.n_combos, self.n_channel_idx = C.value, L.value, F.value, nc.value, nch.value

    @classmethod
    def create(cls, seed, C, L, num_features=10000):
        h = ctypes.c_void_p()
        _check(load_library().rocket_mini_create(ctypes.c_uint64(seed), C, L, num_features, ctypes.byref(h)), "rocket_mini_create")
        return cls(h)

    def host_arrays(self):
        """Copies of the handle's host arrays as a dict of numpy arrays."""
        ptrs = [ctypes.c_void_p() for _ in range(10)]
        _check(load_library().rocket_mini_host_view(self._h, *[ctypes.byref(q) for q in ptrs]), "rocket_mini_host_view")
        names = ["taps", "dilation", "kernel_index", "padded", "num_channels", "channel_idx", "feature_offset",
                 "example_draw", "quantile", "bias"]
        sizes = [84 * 3, self.n_combos, self.n_combos, self.n_combos, self.n_combos, self.n_channel_idx, self.n_combos + 1,
                 self.n_combos, self.F, self.F]
        types = [np.int32] * 7 + [np.float64, np.float64, np.float32]
        out = {}
        for name, q, n, t in zip(names, ptrs, sizes, types):
            ct = {np.int32: ctypes.c_int32, np.float64: ctypes.c_double, np.float32: ctypes.c_float}[t]
            out[name] = np.ctypeslib.as_array(ctypes.cast(q, ctypes.POINTER(ct)), shape=(n,)).copy() if n else np.zeros(0, t)
        out["taps"] = out["taps"].reshape(84, 3)
        return out

    def fit(self, X_host):
        """Biases from the training examples X_host [N, C, L] (numpy float32, host)."""
        X = np.ascontiguousarray(X_host, dtype=np.float32)
        if X.ndim != 3 or X.shape[1] != self.C or X.shape[2] != self.L:
            raise ValueError("X must be [N, %d, %d]" % (self.C, self.L))
        _check(load_library().rocket_mini_fit(self._h, _np_ptr(X), X.shape[0]), "rocket_mini_fit")

    def set_biases(self, bias):
        b = np.ascontiguousarray(bias, dtype=np.float32)
        if b.shape != (self.F,):
            raise ValueError("one bias per feature")
        _check(load_library().rocket_mini_set_biases(self._h, _np_ptr(b)), "rocket_mini_set_biases")

    def transform(self, X, out=None):
        """PPV features [N, F] of a CUDA float32 tensor X [N, C, L]."""
        import torch
        _check_x(self, X)
        N = X.shape[0]
        if out is None:
            out = torch.empty((N, self.F), dtype=torch.float32, device=X.device)
        _check(load_library().rocket_mini_transform(self._h, _dev_ptr(X, torch.float32, "X"), N, self.C, self.L,
                                                    _dev_ptr(out, torch.float32, "out"), _stream()), "rocket_mini_transform")
        return out

    @property
    def handle(self):
        return self._h

    def close(self):
        if self._h:
            load_library().rocket_mini_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
