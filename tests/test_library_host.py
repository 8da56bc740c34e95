"""Host-side checks of the C-ABI library that need no GPU: exported symbols, parameter
generation equal to the reference generator, argument validation."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2301_08527_b200 as rk
from paper_2301_08527_b200 import binding
from rocket_inputs import generate_kernels, kernels_from_lists

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2301_08527_b200.build import build
    build()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "rocket.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rocket_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(rk.library_path())
    names = _declared_symbols()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(binding.SIGNATURES), "binding and header disagree"


def test_generate_matches_reference_generator_bit_for_bit_on_integers():
    for (seed, K, C, L) in [(8527, 1000, 1, 512), (8527, 3000, 20, 5000), (7, 500, 5, 50000), (1, 64, 3, 11)]:
        p = rk.RocketParams.generate(seed, K, C, L)
        h = p.host_arrays()
        q = generate_kernels(seed, K, C, L)
        for f in ("length", "dilation", "padding", "num_channels", "channel_idx"):
            assert np.array_equal(h[f], getattr(q, f)), f
        np.testing.assert_allclose(h["bias"], q.bias, rtol=0, atol=1e-7)
        np.testing.assert_allclose(h["weights"], q.weights, rtol=0, atol=1e-6)
        flops, outs = p.work()
        assert flops == pytest.approx(q.conv_flops_per_example(), rel=1e-12)
        assert outs == pytest.approx(float(q.out_len.sum()), rel=1e-12)
        p.close()


def test_from_arrays_roundtrip():
    q = generate_kernels(3, 200, 6, 400)
    p = rk.RocketParams.from_kernel_params(q)
    h = p.host_arrays()
    for f in ("length", "dilation", "padding", "num_channels", "channel_idx", "weights", "bias"):
        assert h[f].tobytes() == getattr(q, f).tobytes()
    assert (p.K, p.C, p.L, p.n_weights) == (200, 6, 400, len(q.weights))


def _make(C, L, **kd):
    q = kernels_from_lists(C, L, [kd])
    return rk.RocketParams.from_kernel_params(q)


def test_set_weights_replaces_values_and_rejects_bad_input():
    kp = generate_kernels(4, 50, 3, 200)
    p = binding.RocketParams.from_kernel_params(kp)
    w = (np.arange(p.n_weights, dtype=np.float32) * 0.01 - 1.0)
    b = np.linspace(-0.5, 0.5, p.K).astype(np.float32)
    p.set_weights(w, b)
    arrs = p.host_arrays()
    assert np.array_equal(arrs["weights"], w) and np.array_equal(arrs["bias"], b)
    assert np.array_equal(arrs["dilation"], kp.dilation) and np.array_equal(arrs["channel_idx"], kp.channel_idx)
    bad = w.copy(); bad[3] = np.inf
    with pytest.raises(binding.RocketError):
        p.set_weights(bad, b)
    with pytest.raises(ValueError):
        p.set_weights(w[:-1], b)
    assert np.array_equal(p.host_arrays()["weights"], w)
    p.close()


def test_validation_rejects_bad_kernels():
    ok = dict(dilation=2, padding=0, channels=[0, 1], weights=np.ones((2, 7)), bias=0.0)
    _make(3, 100, **ok).close()
    bad = [
        dict(ok, dilation=0),
        dict(ok, padding=-1),
        dict(ok, dilation=17),                       # span 6*17+1 > 100 -> L_out < 1
        dict(ok, channels=[0, 3]),                   # channel out of range
        dict(ok, channels=[1, 1]),                   # duplicate channel
        dict(ok, weights=np.ones((2, 12))),          # length > 11
        dict(dilation=1, padding=0, channels=[0, 1, 2, 0], weights=np.ones((4, 7)), bias=0.0),
    ]
    for kd in bad:
        with pytest.raises(rk.RocketError) as ei:
            _make(3, 100, **kd)
        assert ei.value.status == -1
    with pytest.raises(rk.RocketError):
        rk.RocketParams.generate(1, 0, 2, 100)
    with pytest.raises(rk.RocketError):
        rk.RocketParams.generate(1, 10, 2, 10)
    with pytest.raises(rk.RocketError):
        rk.RocketParams.generate(1, 10, 0, 100)


def test_device_calls_fail_loudly_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("this check is for GPU-less machines")
    lib = rk.load_library()
    p = rk.RocketParams.generate(1, 4, 1, 64)
    x = np.zeros((1, 1, 64), np.float32)
    f = np.zeros((1, 8), np.float32)
    st = lib.rocket_transform_host(p.handle, x.ctypes.data_as(ctypes.c_void_p), 1, 1, 64,
                                   f.ctypes.data_as(ctypes.c_void_p))
    assert st == -5  # ROCKET_ECUDA, not a silent CPU result
    assert lib.rocket_transform(p.handle, None, 1, 1, 64, None, None) == -1
    assert lib.rocket_transform(p.handle, ctypes.c_void_p(16), 1, 2, 64, ctypes.c_void_p(16), None) == -2
    assert lib.rocket_transform(None, None, 0, 1, 64, None, None) == -1
    assert lib.rocket_strerror(-3) == b"unsupported size or configuration"
    assert lib.rocket_params_set_path(p.handle, 7) == -1


def test_product_package_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2301_08527_b200")
    for dirpath, _, files in os.walk(pkg):
        if "_build" in dirpath:
            continue
        for fn in files:
            if fn.endswith((".py", ".cu", ".cpp", ".h", ".cuh")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "oracle" not in text.lower(), fn
    for fn in os.listdir(os.path.join(ROOT, "oracle")):
        if fn.endswith((".py", ".c")):
            assert "paper_2301_08527_b200" not in open(os.path.join(ROOT, "oracle", fn)).read()
